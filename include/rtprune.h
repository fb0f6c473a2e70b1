/*
 * rtprune.h -- C ABI of the B200 (sm_100a) implementation of RTPrune's visual-token pruning
 * module: the computation that shrinks a vision-language model's visual token set before LLM
 * prefill (RTPrune, Section 3.3 and Algorithm 1).
 *
 * For every image i of a ragged batch X[sum N_i, d] the library computes, entirely on the GPU:
 *   1. the selection criterion C_k = ||T_v^k||_2 of every token                     (Eq. 1)
 *   2. the mean inter-token cosine similarity phi                                    (Eq. 8)
 *   3. the pruning ratio r: fixed, or r_dyn = f_normalize(phi) (1 - rho)             (Eq. 10)
 *   4. T_kept = the M = N (1 - r) tokens of largest norm, T_prop = the other B       (Sec. 3.3.1)
 *   5. the cosine scores S [M x B] between kept and proposed-to-prune tokens        (Sec. 3.3.2)
 *   6. the dustbin-augmented transport plan P-bar by Sinkhorn iterations            (Eq. 5, App. C)
 *   7. the merged tokens T_k + alpha P T_p                                           (Eq. 7)
 * and writes the merged kept tokens of all images packed back to back (Algorithm 1, output).
 *
 * Conventions
 *   - All pointers marked DEVICE are device-global addresses valid on the current CUDA device;
 *     pointers marked HOST are ordinary host addresses.  The library never allocates or frees
 *     device memory and never frees or keeps caller memory; the only object it owns is the plan.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Every function returns an rtprune_status_t; nothing throws or aborts across this boundary.
 *     Errors the host can detect are returned before anything is launched.  Conditions only the
 *     device can see (a non-finite input) are recorded in a status word inside the workspace and
 *     read back with rtprune_query_status.
 *   - One plan may be used by one stream at a time.  Runs that share a workspace must not overlap.
 *   - Token indices are image-local (0 .. N_i-1).  Ties in any ranking go to the lower index.
 */
#ifndef RTPRUNE_H_
#define RTPRUNE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rtprune_plan_s rtprune_plan_t; /* opaque, host memory, library-owned */

typedef enum {
    RTPRUNE_OK = 0,
    RTPRUNE_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, parameter out of range      */
    RTPRUNE_ERR_UNSUPPORTED = 2, /* shape outside what the kernels handle (see rtprune_plan) */
    RTPRUNE_ERR_WORKSPACE = 3,   /* workspace / arena smaller than the plan requires         */
    RTPRUNE_ERR_CUDA = 4,        /* a CUDA runtime call failed; see rtprune_last_cuda_error  */
    RTPRUNE_ERR_NONFINITE = 5,   /* device saw a non-finite token norm (query_status only)   */
    RTPRUNE_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (query_status only); the
                                    outputs of that run are not to be used                    */
    RTPRUNE_ERR_BAD_OFFSETS = 7  /* device saw offsets outside the contract (query_status only) */
} rtprune_status_t;

typedef enum { RTPRUNE_BF16 = 0, RTPRUNE_FP32 = 1 } rtprune_dtype_t;

/* How the Sinkhorn iterations of Appendix C are carried out.  Both forms run the same iteration
 * (u from v, then v from u, `iters` times, starting from u = v = 0 in the log domain) and give the
 * same plan up to rounding.
 *   LOG     u, v are the log-domain duals and every sweep is a max-shifted log-sum-exp, as printed.
 *   SCALING the duals are carried as e^u, e^v against the kernel K = exp((S-bar - c)/eps), c = max(1, z):
 *           every sweep is a matrix-vector product and nothing is subtracted, so the plan is as accurate in
 *           fp32 as the log form's (more so at small eps).  Allowed while every factor stays inside fp32's
 *           range: (2 max(1, z) - min(-1, z)) / eps <= 62, i.e. eps >= 0.05 at z = 0.2 and eps >= 0.25 for
 *           any |z| <= 4; otherwise RTPRUNE_ERR_INVALID_ARG.
 *   AUTO    SCALING when that condition holds, else LOG.
 *   EXACT   no iterations: the linear program of Eq. 2-6 itself is solved (the limit eps -> 0 of the
 *           entropic problem).  With the dustbins of Eq. 5 it is a maximum-weight partial matching in
 *           which pairing kept token i with pruned token j gains S_ij - z over leaving both in the
 *           dustbins; the solver finds a vertex by shortest augmenting paths in fp32.  The plan then
 *           holds ones at the pairs and zeros elsewhere, Eq. 7 adds alpha T_p^j to the partner of every
 *           paired token, merge_partner is the kept position or -1 (unpaired: the token is dropped),
 *           merge_weight is 1 or 0, stats[5] counts path-search steps and stats[6] the rows paired before any search.  eps, iters,
 *           stop_at_fixed_point, tol and schedule are ignored.  Where several matchings reach the optimum
 *           any one of them may be returned. */
typedef enum {
    RTPRUNE_SINKHORN_AUTO = 0,
    RTPRUNE_SINKHORN_LOG = 1,
    RTPRUNE_SINKHORN_SCALING = 2,
    RTPRUNE_SINKHORN_EXACT = 3
} rtprune_sinkhorn_form_t;

/* Criterion C_k by which stage 1 ranks the tokens of an image (the M largest are kept).  The paper's
 * method uses the l2 norm (Eq. 1); its ablation on the selection metric also ranks by variance and by
 * entropy.  Only the ranking changes: the cosine scores divide by the l2 norms whatever the criterion.
 *   L2NORM   C_k = ||T_v^k||_2                                                          (Eq. 1)
 *   VARIANCE C_k = (1/d) sum_c (T_kc - mean_k)^2, the population variance over the d features
 *   ENTROPY  C_k = - sum_c p_c log p_c with p = softmax of the token's d features.  The paper names
 *            this metric without a formula: this is the library's reading of it. */
typedef enum { RTPRUNE_CRITERION_L2NORM = 0, RTPRUNE_CRITERION_VARIANCE = 1, RTPRUNE_CRITERION_ENTROPY = 2 }
    rtprune_criterion_t;

/* How stage 2 (scores, Sinkhorn, merge: Sec. 3.3.2, App. C, Eq. 7) is scheduled on the device.  The results are
 * the same up to fp32 rounding; only the kernels differ.
 *   AUTO     the library chooses by batch shape
 *   SEPARATE one kernel per step, handing images to one another through the workspace
 *   FUSED    one kernel, a cluster of two CTAs per image, nothing through global memory between the steps;
 *            taken only when every image the run can hold fits it (bf16, width a multiple of 64, at most 512
 *            tokens and 256 pruned tokens per image, scaling form), else SEPARATE is used */
typedef enum { RTPRUNE_SCHEDULE_AUTO = 0, RTPRUNE_SCHEDULE_SEPARATE = 1, RTPRUNE_SCHEDULE_FUSED = 2 } rtprune_schedule_t;

/* Parameters of one run (Algorithm 1 inputs; Appendix C for `iters`). */
typedef struct {
    int32_t dynamic;      /* 0: use r_fixed.  1: r = min(r_max, f_normalize(phi) (1 - rho)), Eq. 10 */
    float r_fixed;        /* pruning ratio r in [0, 1); retention is 1 - r (Sec. 3.3.1)             */
    const float *rho;     /* DEVICE [batch] textual density of each image (Eq. 9); NULL means 0     */
    float phi_lo, phi_hi; /* f_normalize(phi) = clamp((phi - phi_lo) / (phi_hi - phi_lo), 0, 1);
                             the paper leaves f_normalize open; phi_lo = 0, phi_hi = 1 is identity   */
    float r_max;          /* cap on the dynamic ratio, in (0, 1]                                     */
    float z;              /* dustbin score, Eq. 5 (paper: 0.2)                                       */
    float alpha;          /* merge strength, Eq. 7 (paper: 0.1)                                      */
    float eps;            /* entropic regularisation: Z = S-bar / eps; > 0 (1 uses S-bar itself)     */
    int32_t iters;        /* Sinkhorn iterations T, >= 0 (paper: 100)                                */
    int32_t form;         /* rtprune_sinkhorn_form_t                                                 */
    int32_t stop_at_fixed_point; /* 1: leave the loop once an iteration reproduces its input: the duals
                             of the scaling form all within one unit in the last place of their
                             previous values (bit-identical log-domain duals in the LOG form) -- later
                             iterations could only move them within rounding, so the result is that
                             of all `iters` iterations to fp32 accuracy.  (Images with more than 640
                             pruned tokens: within four units, the rounding noise of their long sums.)
                             0: always run `iters`.                                                  */
    float tol;            /* > 0: also stop once no dual moved by more than tol (log units) in an
                             iteration.  0 (default): never stop on a tolerance.                    */
    int32_t criterion;    /* rtprune_criterion_t: what stage 1 ranks by (default L2NORM, Eq. 1)     */
    int32_t schedule;     /* rtprune_schedule_t: which kernels carry out stage 2 (same results)     */
} rtprune_params_t;

/* Number of floats per image in the `stats` output. */
#define RTPRUNE_STATS_STRIDE 8
/* stats[i*8 + ..]: 0 phi, 1 rho, 2 r, 3 M (kept), 4 B (pruned), 5 Sinkhorn iterations executed,
 *                  6 largest dual change of the last executed iteration (log units), 7 reserved */

/* Bits of the device status word (rtprune_query_status). */
#define RTPRUNE_DEV_NONFINITE 1u
#define RTPRUNE_DEV_TIMEOUT 2u
#define RTPRUNE_DEV_BAD_OFFSETS 4u /* an image had N_i < 1 or N_i > max_tokens_per_image */

/* Fills *params with the paper's defaults: fixed r = 0.25, z = 0.2, alpha = 0.1, eps = 1,
 * iters = 100, identity f_normalize, r_max = 1, form AUTO, stop_at_fixed_point = 1, tol = 0,
 * criterion L2NORM, schedule AUTO. */
rtprune_status_t rtprune_default_params(rtprune_params_t *params);

/*
 * Creates a plan for batches of at most `max_batch` images, `max_total_tokens` tokens in total and
 * `max_tokens_per_image` tokens per image, of width d and storage type dtype, on the current CUDA
 * device, and reports the workspace a run needs (Algorithm 1; sizes are worst case over every
 * pruning ratio).  HOST pointers.  No device memory is allocated.
 * Unsupported: d not a multiple of 8 (bf16) or 4 (fp32); d > 4096 (bf16) or 2048 (fp32);
 * max_tokens_per_image > 8192.
 */
rtprune_status_t rtprune_plan(rtprune_plan_t **plan, int32_t d, rtprune_dtype_t dtype,
                              int32_t max_batch, int64_t max_total_tokens,
                              int32_t max_tokens_per_image, size_t *workspace_bytes);

/*
 * Runs Algorithm 1 on a ragged batch, asynchronously on `cuda_stream`: no allocation, no host
 * synchronisation.  Inputs are not modified.  The kernels of a run hand images to one another through
 * the workspace and tell this run's entries from the last run's by a run number that the first kernel
 * counts up in the workspace itself, so the call may be captured into a CUDA graph and the graph
 * replayed (the pointers and sizes of the capture are then fixed; keep per-kernel profiling off while
 * capturing).  One workspace serves one run at a time.
 *
 *   X        DEVICE [total_tokens, d] row-major, dtype of the plan, 16-byte aligned
 *   offsets  DEVICE int32 [batch+1]: offsets[0] = 0, offsets[batch] = total_tokens, image i owns
 *            rows offsets[i] .. offsets[i+1]-1, with 1 <= N_i <= max_tokens_per_image.  The host
 *            cannot see these values: a batch that breaks the rule gives undefined output rows for
 *            the offending image, never an out-of-bounds access beyond the stated capacities.
 *   params   HOST; copied before return
 *   workspace DEVICE, 256-byte aligned, workspace_bytes >= what rtprune_plan reported.  Its first
 *            run must be preceded by rtprune_workspace_init on the same stream.
 * Outputs, all DEVICE, caller-allocated at the stated worst-case capacity:
 *   Y             [total_tokens, d], dtype of the plan: the merged kept tokens, images back to back,
 *                 each image's rows in ascending original index; rows >= out_offsets[batch] untouched
 *   out_offsets   int32 [batch+1]: exclusive prefix sum of counts
 *   counts        int32 [batch]: M_i
 *   kept_idx      int32 [total_tokens]: kept_idx[out_offsets[i] + p] = image-local index of Y's row
 *   merged_idx    int32 [total_tokens]: image i's B_i pruned tokens, ascending, starting at
 *                 offsets[i] - out_offsets[i]
 *   merge_partner int32, parallel to merged_idx: position p in image i's kept list of
 *                 argmax_p P[p][j] (the pair the pruned token is merged into most strongly)
 *   merge_weight  float, parallel: P at that cell
 *   stats         float [batch, RTPRUNE_STATS_STRIDE]
 */
rtprune_status_t rtprune_run(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                             const int32_t *offsets, int32_t batch, int64_t total_tokens,
                             const rtprune_params_t *params, void *workspace,
                             size_t workspace_bytes, void *Y, int32_t *out_offsets,
                             int32_t *counts, int32_t *kept_idx, int32_t *merged_idx,
                             int32_t *merge_partner, float *merge_weight, float *stats);

/* Clears the workspace header (status word, inter-block counters).  Asynchronous on the stream.
 * Needed once per workspace before its first run; runs leave the header ready for the next. */
rtprune_status_t rtprune_workspace_init(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                        size_t workspace_bytes);

/*
 * Stage 1 alone (Eq. 1, Eq. 8, Eq. 10, top-M selection): fills counts, out_offsets, stats[0..4]
 * and, in the workspace, the per-image selection the later stages use.  norms_out (DEVICE float
 * [total_tokens], may be NULL) receives the criterion C_k the run ranks by (the l2 norms unless
 * params->criterion says otherwise); order_out (DEVICE int32 [total_tokens], may be NULL)
 * receives, for image i at offsets[i], its kept indices (ascending) followed by its pruned indices
 * (ascending).  Same argument rules as rtprune_run.
 */
rtprune_status_t rtprune_select(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                                const int32_t *offsets, int32_t batch, int64_t total_tokens,
                                const rtprune_params_t *params, void *workspace,
                                size_t workspace_bytes, int32_t *out_offsets, int32_t *counts,
                                float *stats, float *norms_out, int32_t *order_out);

/*
 * Stage 1 for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * convenience of the library).  Some hosts of this code own no allocator at the point where they
 * call it: a plug-in running inside another framework's memory pool that must not be disturbed, a
 * real-time loop in which cudaMalloc's implicit synchronisation is forbidden, a process whose
 * memory budget was fixed at start-up.  For them this entry point does what rtprune_select does,
 * with the same arguments minus the workspace: its scratch is a fixed array of
 * RTPRUNE_STATIC_SCRATCH_BYTES that is part of the library's device image (every GPU that loads the
 * library holds it until the process exits).  It calls no cudaMalloc / cudaFree and no allocating
 * library routine; inputs and outputs are still the caller's buffers.
 *
 *   - Limit: the plan's stage-1 scratch must fit the array, else RTPRUNE_ERR_WORKSPACE is returned and
 *     nothing is launched.  rtprune_static_scratch_needed reports it for a plan; with a(x) = x rounded
 *     up to a multiple of 256 it is
 *         256 + 4 a(4 max_batch) + 4 a(4 max_total_tokens)
 *             + a(4 max_batch ceil(max_tokens_per_image / 32) d)   bytes,
 *     the last term (partial sums of the unit tokens, Eq. 8) being the large one: a 64-image x 400-token
 *     x 1280 plan needs 4,670,720 bytes (4.45 MiB), and 114 such images are the most the array holds.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - Every call on a device shares the one array, which keeps the previous call's contents; the
 *     call clears the words that must start at zero itself.  Two calls that overlap on the same
 *     GPU (different streams, or threads) race on it: serialise them.
 *   - The device status word lives in the array too: read it with rtprune_query_status_static (a
 *     non-finite token norm, an image outside the offsets contract, whose count is then 0).
 */
#define RTPRUNE_STATIC_SCRATCH_BYTES (8u << 20)
rtprune_status_t rtprune_select_static(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                                       const int32_t *offsets, int32_t batch, int64_t total_tokens,
                                       const rtprune_params_t *params, int32_t *out_offsets,
                                       int32_t *counts, float *stats, float *norms_out,
                                       int32_t *order_out);

/* Bytes of the built-in array rtprune_select_static uses for this plan (it runs iff they are at most
 * RTPRUNE_STATIC_SCRATCH_BYTES).  HOST pointers. */
rtprune_status_t rtprune_static_scratch_needed(const rtprune_plan_t *plan, size_t *bytes);

/* rtprune_query_status for the built-in array of the current device: synchronises the stream, reads the
 * status word the last rtprune_select_static call on this device left there and clears it.  Allocates
 * nothing.  Before any rtprune_select_static call on the device it reports RTPRUNE_OK and no bits. */
rtprune_status_t rtprune_query_status_static(rtprune_plan_t *plan, void *cuda_stream, uint32_t *flags_out);

/*
 * The same run, from and to HOST buffers (pinned memory recommended): copies X, offsets and rho to
 * the device arena, runs, and copies every output back, all asynchronously on the stream; the
 * caller synchronises the stream before reading.  `rho_host` may be NULL (params->rho is ignored
 * here).  Y_host has room for total_tokens rows; the first out_offsets[batch] are written when the ratio is
 * fixed (the kept counts are then known on the host before the launch), all total_tokens rows when it is
 * dynamic (only the first out_offsets[batch] are meaningful).
 * `arena` is DEVICE memory, 256-byte aligned, of at least rtprune_host_arena_bytes bytes; it holds
 * the device copies and the workspace (initialised by this call).
 */
rtprune_status_t rtprune_run_host(rtprune_plan_t *plan, void *cuda_stream, const void *X_host,
                                  const int32_t *offsets_host, const float *rho_host,
                                  int32_t batch, int64_t total_tokens,
                                  const rtprune_params_t *params, void *arena, size_t arena_bytes,
                                  void *Y_host, int32_t *out_offsets_host, int32_t *counts_host,
                                  int32_t *kept_idx_host, int32_t *merged_idx_host,
                                  int32_t *merge_partner_host, float *merge_weight_host,
                                  float *stats_host);

/* Device bytes rtprune_run_host needs for a batch of the plan's maximum size.  HOST pointers. */
rtprune_status_t rtprune_host_arena_bytes(const rtprune_plan_t *plan, size_t *arena_bytes);

/* Synchronises the stream, reads the workspace's device status word and clears it.  Returns
 * RTPRUNE_ERR_NONFINITE / RTPRUNE_ERR_TIMEOUT if the corresponding bit was set, else RTPRUNE_OK.
 * `flags_out` (HOST, may be NULL) receives the raw bits. */
rtprune_status_t rtprune_query_status(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                      uint32_t *flags_out);

/*
 * Per-kernel timing of a run (measurement aid; Algorithm 1's steps map to the kernels named).
 * With profiling enabled the library records a CUDA event on the launching stream before the first
 * kernel of rtprune_run / rtprune_run_host and after every kernel.  rtprune_profile_read waits for
 * the last event and returns, for the most recent run, the number of kernels (*n, at most
 * RTPRUNE_PROFILE_MAX), each one's duration in milliseconds and a static name.  Enabling creates
 * the events (plan-owned), disabling destroys them.  HOST pointers.
 */
#define RTPRUNE_PROFILE_MAX 8
rtprune_status_t rtprune_profile_enable(rtprune_plan_t *plan, int32_t enable);
rtprune_status_t rtprune_profile_read(rtprune_plan_t *plan, int32_t *n, float *ms,
                                      const char **names);

/*
 * Textual density rho of page images (Eq. 9; Appendix B), the input `rho` of the dynamic ratio
 * (Eq. 10): BT.601 grayscale of the 8-bit channels on the [0, 1] scale, the two 3 x 3 Sobel kernels,
 * E = [sqrt(Gx^2 + Gy^2) >= tau], rho_k = mean of E over the patch x patch pixels of token patch k,
 * rho = mean of rho_k.  Pixels outside the image take the value of the nearest pixel inside (the paper
 * does not say).  The decision G >= tau is taken in exact integer arithmetic.  No plan is needed.
 *
 *   images       DEVICE [batch][height][width][3] uint8, R, G, B interleaved, 16-byte aligned; read only
 *   patch        16, 32 or 64; height and width are multiples of it (else RTPRUNE_ERR_UNSUPPORTED)
 *   tau          threshold on the gradient magnitude, >= 0 (Algorithm 1: 0.2)
 *   rho          DEVICE [batch] float, written
 *   image_counts DEVICE [batch] uint32 scratch of the caller, written: edge pixels of each image
 *   edge_counts  DEVICE [batch][height/patch][width/patch] int32, written: edge pixels of each patch
 *                (rho_k = edge_counts / patch^2); may be NULL
 * Asynchronous on the stream (one memset, two kernels), allocates nothing.  Host-detectable errors
 * are returned before any launch.
 */
rtprune_status_t rtprune_density(void *cuda_stream, const uint8_t *images, int32_t batch, int32_t height,
                                 int32_t width, int32_t patch, float tau, float *rho,
                                 uint32_t *image_counts, int32_t *edge_counts);

/*
 * Test aid: makes the library's bounded device-side waits run out without any fault.  Launches one small
 * kernel on the stream that waits, with the same wait routines the kernels of a run use but only
 * `poll_limit` polls (1 .. 65536), first for a run number that no run ever has (the flag in the workspace
 * header the second-stage kernels wait on) and then on a shared-memory barrier nobody arrives at.  Each wait
 * that gives up sets RTPRUNE_DEV_TIMEOUT in the workspace's status word, exactly as a kernel of a run does;
 * the kernel then returns normally, so the context and the workspace stay usable and the next
 * rtprune_query_status reports RTPRUNE_ERR_TIMEOUT.  `expired_out` (DEVICE int32, may be NULL) receives the
 * number of waits that gave up (2).  The workspace must have been initialised.
 */
rtprune_status_t rtprune_test_expire_waits(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                           size_t workspace_bytes, uint32_t poll_limit, int32_t *expired_out);

/*
 * Test aid for the give-up path of stage 1 (Eq. 1 / Eq. 8 pass): sets how many polls its waits on the copies
 * that stream X into shared memory make before they give up (default 2^20; negative restores the default; 0
 * makes every wait give up at once although its copy is on its way).  A CTA whose wait gave up reports
 * RTPRUNE_DEV_TIMEOUT, waits once more, with the default limit, for the copies still in flight into its
 * shared memory, and marks its image, which then passes through unpruned (M = N, Y rows = X rows): nothing
 * faults, nothing is read that never arrived, and the next run with the default limit is clean.
 */
rtprune_status_t rtprune_test_set_poll_limit(rtprune_plan_t *plan, int64_t polls);

/* Kernels launched by the most recent run / select / run_host call on this plan. */
int32_t rtprune_last_launch_count(const rtprune_plan_t *plan);

/* Host time, in nanoseconds, that the most recent rtprune_run call on this plan spent launching (argument
 * checks excluded; measurement aid). */
int64_t rtprune_last_host_ns(const rtprune_plan_t *plan);

/* cudaError_t value of the most recent failed CUDA call on this plan (0 if none). */
int32_t rtprune_last_cuda_error(const rtprune_plan_t *plan);

/* Frees the plan (host memory only).  NULL is allowed. */
void rtprune_destroy(rtprune_plan_t *plan);

/* Static, NUL-terminated name of a status code. */
const char *rtprune_status_string(rtprune_status_t status);

/* Library version, major * 10000 + minor * 100 + patch. */
int32_t rtprune_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RTPRUNE_H_ */
