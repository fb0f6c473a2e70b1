// C ABI of the RTPrune pruning path: plan, argument checks, workspace layout and kernel launches.
// Every step of the path runs in the kernels included below; this file only marshals.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>

#include "common.cuh"
#include "exact.cuh"
#include "fused.cuh"
#include "gemm_simt.cuh"
#include "merge_umma.cuh"
#include "scores_umma.cuh"
#include "sinkhorn.cuh"
#include "sinkhorn_cluster.cuh"
#include "sinkhorn_reg.cuh"
#include "sinkhorn_tall.cuh"
#include "stage1.cuh"

using namespace rtp;

static_assert(sizeof(rtprune_params_t) == 64, "rtprune_params_t layout is part of the ABI");

struct rtprune_plan_s {
    int d;
    rtprune_dtype_t dtype;
    int max_batch;
    int64_t max_total;
    int max_tokens;
    WsLayout ws;
    int device;
    int sm_count;
    int smem_optin;       // bytes of opt-in shared memory per CTA
    int sink_smem_bytes;  // dynamic shared memory of the general Sinkhorn kernel
    int fast_smem_bytes;  // dynamic shared memory of the one-pass Sinkhorn kernel
    void *encode_tiled;   // cuTensorMapEncodeTiled, resolved through the runtime (no libcuda link)
    int last_launches;
    int last_cuda_error;
    bool profiling;
    cudaEvent_t ev[RTPRUNE_PROFILE_MAX + 1];
    const char *ev_name[RTPRUNE_PROFILE_MAX];
    int ev_count;  // kernels recorded by the most recent run
    int tall_c16_clusters;  // clusters of 16 CTAs of the wide-tile Sinkhorn kernel the device runs at once (0: none)
    int fused_clusters;     // clusters of 2 CTAs of the fused stage-2 kernel the device runs at once (0: none)
    int exact_smem_bytes;   // dynamic shared memory of the exact-pairing kernel
    // Tensor maps of the tensor-core kernels, kept from run to run: a map depends only on the buffers' addresses
    // and extents, which a caller cycling over a few buffer sets repeats.
    struct MapSet {
        const void *X;
        const void *ws;
        int total, batch, pbuf_pitch;
        bool valid;
        CUtensorMap scX, scXp, mgX, mgXp, mgP;
    };
    static constexpr int kMapSets = 8;
    MapSet maps[kMapSets];
    int map_next;           // entry the next miss replaces
    int64_t last_host_ns;   // host time the most recent rtprune_run call spent inside the library
    uint32_t poll_limit;    // polls after which stage 1's waits on its copies give up (ptx::kSpinLimit; tests lower it)
};

// Scratch of rtprune_select_static: lives in the library's device image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[RTPRUNE_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WsLayout make_layout(int d, rtprune_dtype_t dtype, int max_batch, int64_t max_total, int max_tokens)
{
    WsLayout L;
    L.chunks = (max_tokens + kChunkTokens - 1) / kChunkTokens;
    L.kmat_stride = 4 * ((max_tokens + 8 + 15) / 16);
    size_t off = 0;
    L.header = off;
    off = align_up(off + sizeof(WsHeader), 256);
    L.img_done = off;
    off = align_up(off + sizeof(uint32_t) * (size_t)max_batch, 256);
    L.sink_done = off;
    off = align_up(off + sizeof(uint32_t) * (size_t)max_batch, 256);
    L.ready_list = off;
    off = align_up(off + sizeof(int32_t) * (size_t)max_batch, 256);
    L.scores_done = off;
    off = align_up(off + sizeof(uint32_t) * (size_t)max_batch, 256);
    L.clear_bytes = off;
    L.norms = off;
    off = align_up(off + sizeof(float) * (size_t)max_total, 256);
    L.crit = off;
    off = align_up(off + sizeof(float) * (size_t)max_total, 256);
    L.spart = off;
    off = align_up(off + sizeof(float) * (size_t)max_batch * L.chunks * d, 256);
    L.order = off;
    off = align_up(off + sizeof(int32_t) * (size_t)max_total, 256);
    L.kpos = off;
    off = align_up(off + sizeof(int32_t) * (size_t)max_total, 256);
    L.kmat = off;
    off = align_up(off + sizeof(float) * (size_t)L.kmat_stride * (size_t)(max_total + 8 * (int64_t)max_batch), 256);
    L.xp = off;
    if (dtype == RTPRUNE_BF16)
        off = align_up(off + sizeof(__nv_bfloat16) * (size_t)(max_total + 64 * (int64_t)max_batch) * d, 256);
    L.pbuf = off;
    L.pbuf_pitch_max = (max_tokens + 63) / 64 * 64;
    if (dtype == RTPRUNE_BF16)
        off = align_up(off + sizeof(__nv_bfloat16) * (size_t)max_total * L.pbuf_pitch_max, 256);
    L.total = off;
    return L;
}

struct Checked {
    rtprune_plan_t *plan;
    bool ok(cudaError_t e)
    {
        if (e == cudaSuccess) return true;
        plan->last_cuda_error = (int)e;
        return false;
    }
};

// Profiling: event 0 before the first kernel, event k after the k-th.
void prof_begin(rtprune_plan_t *plan, cudaStream_t st)
{
    plan->ev_count = 0;
    if (plan->profiling) cudaEventRecord(plan->ev[0], st);
}

void launched(rtprune_plan_t *plan, cudaStream_t st, const char *name)
{
    ++plan->last_launches;
    if (plan->profiling && plan->ev_count < RTPRUNE_PROFILE_MAX) {
        plan->ev_name[plan->ev_count] = name;
        cudaEventRecord(plan->ev[++plan->ev_count], st);
    }
}

// Launch with programmatic stream serialization (the kernel may begin while the one ahead of it in the
// stream drains; it calls grid_dep_wait() before touching anything that kernel produced), optionally
// as thread-block clusters of `cluster` CTAs.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       unsigned cluster, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Test aid (rtprune_test_expire_waits): two waits that nothing ends, with a short poll limit.
__global__ void expire_waits_kernel(WsHeader *hdr, uint32_t poll_limit, int32_t *expired_out)
{
    __shared__ uint64_t bar;
    if (threadIdx.x != 0) return;
    int expired = 0;
    // run numbers count up from 1 on every workspace: -1 is not stored before 2^32 - 1 runs on it
    if (!ptx::wait_equal_gpu(&hdr->run_tag, -1, poll_limit)) {
        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
        ++expired;
    }
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait(&bar, 0, poll_limit)) {     // phase 0 never completes: nobody arrives
        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
        ++expired;
    }
    if (expired_out) *expired_out = expired;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 tensor map over a row-major [rows, cols] matrix with the given row pitch, boxes of
// box_cols x box_rows elements, 128-byte swizzle, out-of-range elements read as zero.
bool make_tmap_bf16(rtprune_plan_t *plan, CUtensorMap *map, const void *base, uint64_t rows,
                    uint64_t cols, uint64_t pitch_bytes, uint32_t box_cols, uint32_t box_rows)
{
    if (!plan->encode_tiled) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = ((EncodeTiledFn)plan->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        plan->last_cuda_error = (int)cudaErrorInvalidValue;
        return false;
    }
    return true;
}

// The scaling form carries e^u, e^v and K = exp((S-bar - c)/eps), c = max(1, z), in fp32.  With lo = min(-1, z)
// the exponents of K span (c - lo)/eps, the duals stay within that span plus log N of their start, and V starts
// at e^{c/eps}: every factor and product stays inside fp32's range while (2c - lo)/eps <= 62 (eps >= 0.05 at the
// paper's z = 0.2; eps >= 0.25 for any |z| <= 4).
bool scaling_in_range(const rtprune_params_t *p)
{
    const float c = std::fmax(1.f, p->z), lo = std::fmin(-1.f, p->z);
    return (2.f * c - lo) / p->eps <= 62.f;
}

// The five tensor maps of a bf16 run over (X, workspace): from the plan's cache, or encoded into it.
const rtprune_plan_s::MapSet *tensor_maps(rtprune_plan_t *plan, const void *X, char *ws, int total, int batch,
                                          int pbuf_pitch)
{
    for (int i = 0; i < rtprune_plan_s::kMapSets; ++i) {
        const rtprune_plan_s::MapSet &m = plan->maps[i];
        if (m.valid && m.X == X && m.ws == ws && m.total == total && m.batch == batch && m.pbuf_pitch == pbuf_pitch)
            return &m;
    }
    rtprune_plan_s::MapSet &m = plan->maps[plan->map_next];
    plan->map_next = (plan->map_next + 1) % rtprune_plan_s::kMapSets;
    m.valid = false;
    const WsLayout &L = plan->ws;
    const uint64_t d = (uint64_t)plan->d, rows_xp = (uint64_t)total + 64 * (uint64_t)batch;
    if (!make_tmap_bf16(plan, &m.scX, X, (uint64_t)total, d, d * 2, kScBK, kScTileM) ||
        !make_tmap_bf16(plan, &m.scXp, ws + L.xp, rows_xp, d, d * 2, kScBK, kScBBoxRows) ||
        !make_tmap_bf16(plan, &m.mgX, X, (uint64_t)total, d, d * 2, 64, kMgBK) ||
        !make_tmap_bf16(plan, &m.mgXp, ws + L.xp, rows_xp, d, d * 2, 64, kMgBK) ||
        !make_tmap_bf16(plan, &m.mgP, ws + L.pbuf, (uint64_t)total, (uint64_t)pbuf_pitch, (uint64_t)pbuf_pitch * 2,
                        kMgBK, kMgTileM))
        return nullptr;
    m.X = X;
    m.ws = ws;
    m.total = total;
    m.batch = batch;
    m.pbuf_pitch = pbuf_pitch;
    m.valid = true;
    return &m;
}

rtprune_status_t check_params(const rtprune_params_t *p)
{
    if (!p) return RTPRUNE_ERR_INVALID_ARG;
    if (p->dynamic != 0 && p->dynamic != 1) return RTPRUNE_ERR_INVALID_ARG;
    if (!p->dynamic && !(p->r_fixed >= 0.f && p->r_fixed < 1.f)) return RTPRUNE_ERR_INVALID_ARG;
    if (p->dynamic) {
        if (!(p->phi_hi > p->phi_lo)) return RTPRUNE_ERR_INVALID_ARG;
        if (!(p->r_max > 0.f && p->r_max <= 1.f)) return RTPRUNE_ERR_INVALID_ARG;
    }
    if (!(p->eps > 0.f) || !std::isfinite(p->eps)) return RTPRUNE_ERR_INVALID_ARG;
    if (!std::isfinite(p->z) || !std::isfinite(p->alpha)) return RTPRUNE_ERR_INVALID_ARG;
    if (p->iters < 0) return RTPRUNE_ERR_INVALID_ARG;
    if (p->form < RTPRUNE_SINKHORN_AUTO || p->form > RTPRUNE_SINKHORN_EXACT)
        return RTPRUNE_ERR_INVALID_ARG;
    if (!(p->tol >= 0.f)) return RTPRUNE_ERR_INVALID_ARG;
    if (p->criterion < RTPRUNE_CRITERION_L2NORM || p->criterion > RTPRUNE_CRITERION_ENTROPY)
        return RTPRUNE_ERR_INVALID_ARG;
    if (p->schedule < RTPRUNE_SCHEDULE_AUTO || p->schedule > RTPRUNE_SCHEDULE_FUSED) return RTPRUNE_ERR_INVALID_ARG;
    if (p->form == RTPRUNE_SINKHORN_SCALING && !scaling_in_range(p)) return RTPRUNE_ERR_INVALID_ARG;
    return RTPRUNE_OK;
}

bool use_log_form(const rtprune_params_t *p)
{
    if (p->form == RTPRUNE_SINKHORN_LOG) return true;
    if (p->form == RTPRUNE_SINKHORN_SCALING) return false;
    return !scaling_in_range(p);
}

// Largest B any image of at most max_tokens tokens can get under these parameters.
int max_pruned(const rtprune_params_t *p, int max_tokens)
{
    const float r = p->dynamic ? std::fmin(p->r_max, 1.f) : p->r_fixed;
    if (r <= 0.f) return 0;  // nothing can be pruned: stage 2 is not launched
    long b = (long)std::floor((double)r * max_tokens + 0.5) + 1;  // +1: fp32 vs fp64 rounding slack
    if (b > max_tokens - 1) b = max_tokens - 1;
    if (b < 0) b = 0;
    return (int)b;
}

template <typename T>
cudaError_t launch_stage1_kernel(const rtprune_plan_t *pl, cudaStream_t st, const void *X,
                                 const int32_t *offsets, int batch, int total, const RatioParams &rp,
                                 const float *rho, char *ws, int32_t *out_offsets, int32_t *counts,
                                 float *stats, float *norms_out, int32_t *order_out, int scan_here,
                                 int attr_only = 0)
{
    // attr_only > 0: no launch; give the plan's instance of the kernel that much dynamic shared memory (the
    // attribute belongs to the function: rtprune_plan sets it once, to what the device allows)
    constexpr int EPV = Elem<T>::kPerVec;
    const WsLayout &L = pl->ws;
    const int d = pl->d;
    const int vpl = (d / EPV + 31) / 32;
    // tokens per CTA: about one wave of CTAs (two per SM) for small batches, never fewer than
    // kChunkTokens (the partial-sum region is sized for that) nor more than 512 (on 1024 images of 400 tokens a
    // CTA per image streams at 4.4 TB/s, four CTAs of 128 tokens each at 3.8 TB/s)
    const int slots = 2 * pl->sm_count;
    const int per_image = std::max(1, slots / std::max(batch, 1));
    int chunk_tokens = (pl->max_tokens + per_image - 1) / per_image;
    chunk_tokens = std::min(512, std::max(kChunkTokens, (chunk_tokens + 7) / 8 * 8));
    const int chunks_run = (pl->max_tokens + chunk_tokens - 1) / chunk_tokens;   // <= L.chunks
    dim3 grid(chunks_run, batch);
    const size_t smem = sizeof(float) * stage1_smem_floats(d, pl->max_tokens, sizeof(T));
#define RTP_CASE(V)                                                                              \
    case V: {                                                                                    \
        auto k = stage1_kernel<T, V>;                                                            \
        if (attr_only) return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, attr_only); \
        cudaError_t e = launch_pdl(k, grid, dim3(kS1Threads), smem, st, 1u,                      \
            (const T *)X, offsets, batch, d, L.chunks, chunk_tokens, pl->max_tokens, total, rp, rho, \
            (float *)(ws + L.norms), (float *)(ws + (rp.criterion ? L.crit : L.norms)),          \
            (float *)(ws + L.spart), (uint32_t *)(ws + L.img_done),                              \
            (int32_t *)(ws + L.order), (int32_t *)(ws + L.kpos), counts, out_offsets, stats,     \
            norms_out, order_out, (WsHeader *)(ws + L.header), scan_here, pl->poll_limit);       \
        if (e != cudaSuccess) return e;                                                          \
        break;                                                                                   \
    }
    switch (vpl) {
        RTP_CASE(1) RTP_CASE(2) RTP_CASE(3) RTP_CASE(4) RTP_CASE(5) RTP_CASE(6) RTP_CASE(7)
        RTP_CASE(8) RTP_CASE(9) RTP_CASE(10) RTP_CASE(11) RTP_CASE(12) RTP_CASE(13) RTP_CASE(14)
        RTP_CASE(15) RTP_CASE(16)
    default: return cudaErrorInvalidValue;
    }
#undef RTP_CASE
    return cudaGetLastError();
}

struct DevOut {
    void *Y;
    int32_t *out_offsets, *counts, *kept_idx, *merged_idx, *merge_partner;
    float *merge_weight, *stats;
};

// The plan's SM count, shared-memory limits and function attributes are those of the device it was made on.
bool on_plan_device(const rtprune_plan_t *plan)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == plan->device;
}

rtprune_status_t check_common(rtprune_plan_t *plan, const void *X, const int32_t *offsets,
                              int32_t batch, int64_t total, const rtprune_params_t *params,
                              void *workspace, size_t workspace_bytes)
{
    if (!plan || !params) return RTPRUNE_ERR_INVALID_ARG;
    if (!on_plan_device(plan)) return RTPRUNE_ERR_INVALID_ARG;
    if (batch < 0 || total < 0) return RTPRUNE_ERR_INVALID_ARG;
    if (batch > plan->max_batch || total > plan->max_total) return RTPRUNE_ERR_INVALID_ARG;
    if (total < batch) return RTPRUNE_ERR_INVALID_ARG;  // every image has at least one token
    if (batch > 0 && (!X || !offsets)) return RTPRUNE_ERR_INVALID_ARG;
    if (!workspace) return RTPRUNE_ERR_INVALID_ARG;
    if (((uintptr_t)X & 15u) || ((uintptr_t)workspace & 255u)) return RTPRUNE_ERR_INVALID_ARG;
    if (workspace_bytes < plan->ws.total) return RTPRUNE_ERR_WORKSPACE;
    return check_params(params);
}

// Stage 1: norms, statistics, ratio and selection in one kernel.
rtprune_status_t launch_stage1(rtprune_plan_t *plan, cudaStream_t st, const void *X,
                               const int32_t *offsets, int32_t batch, int total,
                               const rtprune_params_t *params, char *ws, int32_t *out_offsets,
                               int32_t *counts, float *stats, float *norms_out,
                               int32_t *order_out, bool scan_here)
{
    Checked c{plan};
    RatioParams rp{params->dynamic, params->r_fixed, params->phi_lo, params->phi_hi, params->r_max,
                   params->criterion};
    cudaError_t e = (plan->dtype == RTPRUNE_BF16)
                        ? launch_stage1_kernel<__nv_bfloat16>(plan, st, X, offsets, batch, total, rp, params->rho,
                                                              ws, out_offsets, counts, stats, norms_out, order_out,
                                                              scan_here ? 1 : 0)
                        : launch_stage1_kernel<float>(plan, st, X, offsets, batch, total, rp, params->rho, ws,
                                                      out_offsets, counts, stats, norms_out, order_out,
                                                      scan_here ? 1 : 0);
    if (!c.ok(e)) return RTPRUNE_ERR_CUDA;
    launched(plan, st, "stage1");
    return RTPRUNE_OK;
}

// The fused kernel takes the run's second stage: bf16 storage, scaling form, every possible tile fits.
bool fused_stage2_ok(const rtprune_plan_t *plan, const rtprune_params_t *params)
{
    const int maxB = max_pruned(params, plan->max_tokens);
    if (params->schedule == RTPRUNE_SCHEDULE_SEPARATE || params->form == RTPRUNE_SINKHORN_EXACT) return false;
    // AUTO: the separate kernels overlap one another across the images of a batch and are ahead on the batches
    // measured so far; the fused kernel is taken on request
    if (params->schedule == RTPRUNE_SCHEDULE_AUTO) return false;
    return plan->dtype == RTPRUNE_BF16 && maxB > 0 && plan->fused_clusters > 0 && !use_log_form(params) &&
           fused_eligible(plan->d, plan->max_tokens, maxB);
}
template <typename T>
rtprune_status_t launch_stage2(rtprune_plan_t *plan, cudaStream_t st, const void *X,
                               const int32_t *offsets, int32_t batch, int total,
                               const rtprune_params_t *params, char *ws, const DevOut &o)
{
    Checked c{plan};
    const WsLayout &L = plan->ws;
    float *norms = (float *)(ws + L.norms);
    int32_t *order = (int32_t *)(ws + L.order);
    float *kmat = (float *)(ws + L.kmat);
    const int maxN = plan->max_tokens;
    const int maxB = max_pruned(params, maxN);
    const int mtiles = (maxN + kSimtTile - 1) / kSimtTile;
    constexpr bool kTensor = std::is_same<T, __nv_bfloat16>::value;
    __nv_bfloat16 *pbuf = kTensor ? (__nv_bfloat16 *)(ws + L.pbuf) : nullptr;
    const int pbuf_pitch = (std::max(maxB, 1) + 63) / 64 * 64;   // <= L.pbuf_pitch_max
    int32_t *ready_list = nullptr;   // images in the order their plans are finished, when the merge follows it
    uint32_t *scores_done = nullptr; // per-image counts of finished score tiles, when the scores kernel keeps them
    const bool iterate = params->form != RTPRUNE_SINKHORN_EXACT;   // Sinkhorn iterations, else the exact pairing

    if constexpr (kTensor) {
        // One kernel for the whole second stage when every image the run can hold fits it
        if (fused_stage2_ok(plan, params)) {
            OtParams op{params->z, params->alpha, params->eps, params->iters, params->stop_at_fixed_point,
                        params->tol};
            const int clusters = std::min(batch, plan->fused_clusters);
            if (!c.ok(launch_pdl(stage2_fused_kernel, dim3((unsigned)(2 * clusters)), dim3(kFuThreads),
                                 (size_t)kFuSmemBytes, st, 2u, (const __nv_bfloat16 *)X, offsets, plan->d, batch,
                                 (const int32_t *)o.counts, (const int32_t *)order, (const float *)norms, maxN, total, op,
                                 (__nv_bfloat16 *)o.Y, o.out_offsets, o.kept_idx, o.merged_idx, o.merge_partner,
                                 o.merge_weight, o.stats, (WsHeader *)(ws + L.header))))
                return RTPRUNE_ERR_CUDA;
            launched(plan, st, "stage2_fused");
            return RTPRUNE_OK;
        }
    }
    if (maxB > 0) {
        if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            // compact copy of the pruned rows for the tensor-core kernels
            {
                const int rows_max = (maxB + 63) & ~63;
                dim3 ggrid((rows_max + kGpRows - 1) / kGpRows, batch);
                if (!c.ok(launch_pdl(gather_prop_kernel, ggrid, dim3(128), 0, st, 1u,
                                     (const __nv_bfloat16 *)X, offsets, o.counts, order, plan->d, maxN, total,
                                     (__nv_bfloat16 *)(ws + L.xp), (uint32_t *)(ws + L.sink_done),
                                     (int32_t *)(ws + L.ready_list), (WsHeader *)(ws + L.header), batch,
                                     o.out_offsets, (uint32_t *)(ws + L.scores_done))))
                    return RTPRUNE_ERR_CUDA;
                launched(plan, st, "gather");
            }
            // scores: one CTA per (128 consecutive tokens, image)
            const rtprune_plan_s::MapSet *ms = tensor_maps(plan, X, ws, total, batch, pbuf_pitch);
            if (!ms) return RTPRUNE_ERR_CUDA;
            const CUtensorMap &tmapX = ms->scX, &tmapXp = ms->scXp;
            dim3 grid((maxN + kScTileM - 1) / kScTileM, batch);
            // The Sinkhorn kernel can start on an image as soon as that image's score tiles are in.  That
            // costs each scores CTA a release (its stores made visible before it counts itself), which
            // pays when the grid is one wave of CTAs and its end is a tail of a few slow CTAs, not when
            // CTAs queue for the SMs.
            if (iterate && (long long)grid.x * grid.y <= 2LL * plan->sm_count)
                scores_done = (uint32_t *)(ws + L.scores_done);
            if (!c.ok(launch_pdl(scores_umma_kernel, grid, dim3(kScThreads), kScSmemBytes, st, 1u, tmapX, tmapXp,
                                 offsets, plan->d, o.counts, order, (const int32_t *)(ws + L.kpos), norms, kmat,
                                 L.kmat_stride, maxN, total, (WsHeader *)(ws + L.header), scores_done)))
                return RTPRUNE_ERR_CUDA;
        } else {
            const int btiles = (maxB + kSimtTile - 1) / kSimtTile;
            dim3 grid(mtiles * btiles, batch);
            scores_simt_kernel<T><<<grid, 256, 0, st>>>((const T *)X, offsets, plan->d, btiles,
                                                       o.counts, order, norms, kmat,
                                                       L.kmat_stride, maxN, total);
        }
        if (!c.ok(cudaGetLastError())) return RTPRUNE_ERR_CUDA;
        launched(plan, st, "scores");

        OtParams op{params->z, params->alpha, params->eps, params->iters,
                    params->stop_at_fixed_point, params->tol};
        const int smem_floats = plan->sink_smem_bytes / (int)sizeof(float);
        // Scaling form: the cluster kernel takes every tile of up to 32 * kSfMaxNc columns; the general
        // kernel then takes what is left (it skips the images already solved).
        int fast_c = 0;
        const int fast_floats = plan->fast_smem_bytes / (int)sizeof(float);
        bool all_fast = false;
        // Scaling form, every possible tile small enough for a thread's K values to stay in registers: clusters
        // of two CTAs per image, in one wave when the batch allows (else the cluster kernels below)
        if (!iterate) {
            // Eq. 2-6 solved exactly, one CTA per image (an ordinary launch: it starts when the scores are complete)
            exact_pairing_kernel<<<batch, kExThreads, plan->exact_smem_bytes, st>>>(
                offsets, o.counts, o.out_offsets, order, kmat, L.kmat_stride, maxN, total, op,
                plan->exact_smem_bytes / (int)sizeof(float), pbuf, pbuf_pitch, o.merged_idx, o.merge_partner,
                o.merge_weight, o.stats, (WsHeader *)(ws + L.header));
            if (!c.ok(cudaGetLastError())) return RTPRUNE_ERR_CUDA;
            launched(plan, st, "exact_pairing");
        }
        const bool use_reg = iterate && kTensor && !use_log_form(params) && plan->fused_clusters > 0 &&
                             sinkhorn_reg_eligible(maxN, maxB) && batch <= plan->fused_clusters;
        if (use_reg) {
            ready_list = (int32_t *)(ws + L.ready_list);
            if (!c.ok(launch_pdl(sinkhorn_reg_kernel, dim3((unsigned)(2 * batch)), dim3(kFuThreads), (size_t)kFuSmemBytes,
                                 st, 2u, offsets, (const int32_t *)o.counts, (const int32_t *)o.out_offsets,
                                 (const int32_t *)order, (const float *)kmat, L.kmat_stride, maxN, total, op, pbuf,
                                 pbuf_pitch, o.merged_idx, o.merge_partner, o.merge_weight, o.stats,
                                 (uint32_t *)(ws + L.sink_done), ready_list, (WsHeader *)(ws + L.header),
                                 (const uint32_t *)scores_done)))
                return RTPRUNE_ERR_CUDA;
            launched(plan, st, "sinkhorn_reg");
            all_fast = true;
        }
        if (iterate && !use_log_form(params) && !use_reg) {
            // CTAs per image: as many as keep the whole batch on the chip at once, and more if the largest
            // possible tile needs them to keep K in their shared memory; 8 at most (tiles larger than the
            // cluster's shared memory iterate on K in the workspace)
            fast_c = 1;
            while (fast_c < 8 && (long long)batch * fast_c * 2 <= plan->sm_count) fast_c *= 2;
            auto all_tiles = [&](int cc, bool in_smem) {
                bool ok = maxB <= 32 * kSfMaxNc;
                for (int b = 1; b <= maxB && ok; ++b) {
                    const int m = std::max(maxN - b, 1);
                    ok = in_smem ? sinkhorn_cluster_fits(m, b, cc, fast_floats)
                                 : sinkhorn_cluster_handles(m, b, cc, fast_floats);
                }
                return ok;
            };
            // Larger clusters so that every K stays in shared memory only while the grid still fits the chip
            // at once.  Beyond that the tiles that do not fit iterate on K in the workspace: with 2 CTAs per
            // image when they are far larger than one CTA's shared memory (128 ragged images of up to 1156
            // tokens: clusters of 8 take seven waves and 287 us, clusters of 2 take 199 us, single CTAs 311 us),
            // with 1 when only the very largest exceed it (1024 images of 400 tokens: 272 us against 379 us).
            while (fast_c < 8 && !all_tiles(fast_c, true) && (long long)batch * fast_c * 2 <= plan->sm_count)
                fast_c *= 2;
            if (fast_c < 2 && !all_tiles(2, true)) fast_c = 2;
            all_fast = all_tiles(fast_c, false);
            // tiles wider than 256 columns, or too tall for the cluster's shared memory, are possible
            const bool wide = maxB > 256 || !all_tiles(fast_c, true);
            // When one instance solves every image, it hands them to the merge kernel one by one
            ready_list = (kTensor && all_fast) ? (int32_t *)(ws + L.ready_list) : nullptr;
            const uint32_t *sd = ready_list ? (const uint32_t *)scores_done : (const uint32_t *)nullptr;
            if (!wide) {
                if (!c.ok(launch_pdl(sinkhorn_cluster_kernel<false>, dim3((unsigned)(batch * fast_c)),
                                     dim3(kSfThreads), (size_t)plan->fast_smem_bytes, st, (unsigned)fast_c, offsets,
                                     o.counts, o.out_offsets, order, kmat, L.kmat_stride, maxN, total, op,
                                     fast_floats, pbuf, pbuf_pitch, o.merged_idx, o.merge_partner, o.merge_weight,
                                     o.stats, (uint32_t *)(ws + L.sink_done), ready_list,
                                     (WsHeader *)(ws + L.header), sd, 0)))
                    return RTPRUNE_ERR_CUDA;
                launched(plan, st, "sinkhorn_cluster");
            } else {
                // the instance for wide or tall tiles takes the narrow ones of the same run too
                if (!c.ok(launch_pdl(sinkhorn_cluster_kernel<true>, dim3((unsigned)(batch * fast_c)),
                                     dim3(kSfThreads), (size_t)plan->fast_smem_bytes, st, (unsigned)fast_c,
                                     offsets, o.counts, o.out_offsets, order, kmat, L.kmat_stride, maxN, total,
                                     op, fast_floats, pbuf, pbuf_pitch, o.merged_idx, o.merge_partner,
                                     o.merge_weight, o.stats, (uint32_t *)(ws + L.sink_done), ready_list,
                                     (WsHeader *)(ws + L.header), sd, 1)))
                    return RTPRUNE_ERR_CUDA;
                launched(plan, st, "sinkhorn_wide");
            }
        }
        // Scaling form, tiles the cluster kernels left (more than 32 * kSfMaxNc columns): clusters of 8
        // CTAs iterate on K in the workspace tile; the general kernel keeps only what is wider still.
        // It takes all the shared memory a CTA can have: what its fixed regions leave is the ring of row blocks.
        const size_t tall_smem = (size_t)std::max(plan->smem_optin - 1024, 0);
        const bool tall = iterate && !use_log_form(params) && !all_fast &&
                          sizeof(float) * (sinkhorn_tall_smem_floats(std::min(maxB, kTallMaxB), maxN) +
                                           kTallStageFloatsMax) <= tall_smem;
        if (tall) {      // (rtprune_plan gave the kernel its shared memory)
            // 16 CTAs per image when all the images' clusters then still run at once, else 8
            // (a CTA owns a slice of at most 512 columns, one per thread: 8 CTAs cover every pitch, 4 cover
            // pitches of up to 2048 floats).  Batches whose clusters of 8 need several waves get clusters of 4
            // when their tiles are narrow (pitch <= 1024 floats): 64 images of 2137 tokens 0.63 -> 0.54 ms in
            // this kernel; wider tiles lose (32 images of 4512 tokens: 1.6 -> 4.2 ms, too many tiles in flight
            // for L2).
            int tall_c = (batch <= plan->tall_c16_clusters) ? kTallCMax : kTallC;
            if ((long long)batch * kTallC > plan->sm_count && score_pitch(std::min(maxB, kTallMaxB)) <= 1024)
                tall_c = 4;
            if (!c.ok(launch_pdl(sinkhorn_tall_kernel, dim3((unsigned)(batch * tall_c)), dim3(kTallThreads),
                                 tall_smem, st, (unsigned)tall_c, offsets, o.counts, o.out_offsets, order, kmat,
                                 L.kmat_stride, maxN, total, op, pbuf, pbuf_pitch, o.merged_idx, o.merge_partner,
                                 o.merge_weight, o.stats, fast_c, fast_floats, (int)(tall_smem / sizeof(float)),
                                 (WsHeader *)(ws + L.header))))
                return RTPRUNE_ERR_CUDA;
            launched(plan, st, "sinkhorn_tall");
            if (maxB <= kTallMaxB) all_fast = true;       // nothing is left for the general kernel
        }
        if (!iterate) {
        } else if (use_log_form(params))
            sinkhorn_kernel<true><<<batch, kSinkThreads, plan->sink_smem_bytes, st>>>(
                offsets, o.counts, o.out_offsets, order, kmat, L.kmat_stride, maxN, total, op,
                smem_floats, pbuf, pbuf_pitch, o.merged_idx, o.merge_partner, o.merge_weight,
                o.stats, 0, 0, 0);
        else if (!all_fast)
            sinkhorn_kernel<false><<<batch, kSinkThreads, plan->sink_smem_bytes, st>>>(
                offsets, o.counts, o.out_offsets, order, kmat, L.kmat_stride, maxN, total, op,
                smem_floats, pbuf, pbuf_pitch, o.merged_idx, o.merge_partner, o.merge_weight,
                o.stats, fast_c, fast_floats, tall ? kTallMaxB : 0);
        if (!c.ok(cudaGetLastError())) return RTPRUNE_ERR_CUDA;
        if (iterate && (use_log_form(params) || !all_fast)) launched(plan, st, "sinkhorn");
    }

    if constexpr (kTensor) {
        // every operand by tiled TMA: X rows (token tiles), the compact copy of pruned rows, the plan
        const rtprune_plan_s::MapSet *ms = tensor_maps(plan, X, ws, total, batch, pbuf_pitch);
        if (!ms) return RTPRUNE_ERR_CUDA;
        const CUtensorMap &tmapXm = ms->mgX, &tmapXpm = ms->mgXp, &tmapP = ms->mgP;
        const int mtiles_m = (maxN + kMgTileM - 1) / kMgTileM;
        const int nct = (plan->d + kMgTileN - 1) / kMgTileN;
        const long long nunits = (long long)batch * mtiles_m * nct;
        const int grid = (int)std::min<long long>(nunits, plan->sm_count);
        if (!c.ok(launch_pdl(merge_umma_kernel, dim3((unsigned)grid), dim3(kMgThreads), kMgSmemBytes, st, 1u,
                             tmapXm, tmapXpm, tmapP, offsets, plan->d, batch, mtiles_m, o.counts, o.out_offsets,
                             (const int32_t *)(ws + L.kpos), maxN, total, (__nv_bfloat16 *)o.Y, o.kept_idx,
                             (WsHeader *)(ws + L.header), (const int32_t *)ready_list)))
            return RTPRUNE_ERR_CUDA;
    } else {
        const int dtiles = (plan->d + kSimtTile - 1) / kSimtTile;
        dim3 grid(mtiles * dtiles, batch);
        merge_simt_kernel<T><<<grid, 256, 0, st>>>((const T *)X, offsets, plan->d, dtiles, o.counts,
                                                  o.out_offsets, order, kmat, L.kmat_stride, maxN,
                                                  total, params->alpha, (T *)o.Y, o.kept_idx);
    }
    if (!c.ok(cudaGetLastError())) return RTPRUNE_ERR_CUDA;
    launched(plan, st, "merge");
    return RTPRUNE_OK;
}

rtprune_status_t run_device(rtprune_plan_t *plan, cudaStream_t st, const void *X,
                            const int32_t *offsets, int32_t batch, int total,
                            const rtprune_params_t *params, char *ws, const DevOut &o)
{
    if (batch == 0) {
        Checked c{plan};
        if (!c.ok(cudaMemsetAsync(o.out_offsets, 0, sizeof(int32_t), st))) return RTPRUNE_ERR_CUDA;
        return RTPRUNE_OK;
    }
    prof_begin(plan, st);
    // with bf16 storage and anything to prune, the kernel that copies the pruned rows also turns the counts
    // into out_offsets, so that stage 1 ends with the last image's selection
    const bool scan_later = plan->dtype == RTPRUNE_BF16 && max_pruned(params, plan->max_tokens) > 0;
    rtprune_status_t s = launch_stage1(plan, st, X, offsets, batch, total, params, ws, o.out_offsets,
                                       o.counts, o.stats, nullptr, nullptr, !scan_later);
    if (s != RTPRUNE_OK) return s;
    return (plan->dtype == RTPRUNE_BF16)
               ? launch_stage2<__nv_bfloat16>(plan, st, X, offsets, batch, total, params, ws, o)
               : launch_stage2<float>(plan, st, X, offsets, batch, total, params, ws, o);
}

// Device arena of rtprune_run_host: device copies of the inputs and outputs, then the workspace.
struct Arena {
    size_t X, offsets, rho, Y, out_offsets, counts, kept_idx, merged_idx, partner, weight, stats,
        ws, total;
};

Arena make_arena(const rtprune_plan_t *p)
{
    Arena a;
    const size_t esz = p->dtype == RTPRUNE_BF16 ? 2 : 4;
    const size_t tot = (size_t)p->max_total, nb = (size_t)p->max_batch;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    a.X = take(tot * p->d * esz);
    a.offsets = take((nb + 1) * 4);
    a.rho = take(nb * 4);
    a.Y = take(tot * p->d * esz);
    a.out_offsets = take((nb + 1) * 4);
    a.counts = take(nb * 4);
    a.kept_idx = take(tot * 4);
    a.merged_idx = take(tot * 4);
    a.partner = take(tot * 4);
    a.weight = take(tot * 4);
    a.stats = take(nb * kStats * 4);
    a.ws = take(p->ws.total);
    a.total = off;
    return a;
}

}  // namespace

extern "C" {

rtprune_status_t rtprune_default_params(rtprune_params_t *p)
{
    if (!p) return RTPRUNE_ERR_INVALID_ARG;
    std::memset(p, 0, sizeof(*p));
    p->dynamic = 0;
    p->r_fixed = 0.25f;
    p->rho = nullptr;
    p->phi_lo = 0.f;
    p->phi_hi = 1.f;
    p->r_max = 1.f;
    p->z = 0.2f;
    p->alpha = 0.1f;
    p->eps = 1.f;
    p->iters = 100;
    p->form = RTPRUNE_SINKHORN_AUTO;
    p->stop_at_fixed_point = 1;
    p->tol = 0.f;
    p->criterion = RTPRUNE_CRITERION_L2NORM;
    p->schedule = RTPRUNE_SCHEDULE_AUTO;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_plan(rtprune_plan_t **plan_out, int32_t d, rtprune_dtype_t dtype,
                              int32_t max_batch, int64_t max_total_tokens,
                              int32_t max_tokens_per_image, size_t *workspace_bytes)
{
    if (!plan_out || !workspace_bytes) return RTPRUNE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    if (dtype != RTPRUNE_BF16 && dtype != RTPRUNE_FP32) return RTPRUNE_ERR_INVALID_ARG;
    if (d <= 0 || max_batch <= 0 || max_total_tokens <= 0 || max_tokens_per_image <= 0)
        return RTPRUNE_ERR_INVALID_ARG;
    if (max_total_tokens > 0x7fff0000LL) return RTPRUNE_ERR_UNSUPPORTED;  // int32 offsets
    if (max_batch > 65535) return RTPRUNE_ERR_UNSUPPORTED;
    const int epv = dtype == RTPRUNE_BF16 ? 8 : 4;
    if (d % epv != 0 || d > 16 * 32 * epv) return RTPRUNE_ERR_UNSUPPORTED;
    if (max_tokens_per_image > 8192) return RTPRUNE_ERR_UNSUPPORTED;
    if (max_tokens_per_image > max_total_tokens) max_tokens_per_image = (int32_t)max_total_tokens;

    rtprune_plan_t *p = new (std::nothrow) rtprune_plan_t();
    if (!p) return RTPRUNE_ERR_INVALID_ARG;
    p->d = d;
    p->dtype = dtype;
    p->max_batch = max_batch;
    p->max_total = max_total_tokens;
    p->max_tokens = max_tokens_per_image;
    p->ws = make_layout(d, dtype, max_batch, max_total_tokens, max_tokens_per_image);
    p->last_launches = 0;
    p->last_cuda_error = 0;
    for (int i = 0; i < rtprune_plan_s::kMapSets; ++i) p->maps[i].valid = false;
    p->map_next = 0;
    p->last_host_ns = 0;
    p->poll_limit = ptx::kSpinLimit;
    p->profiling = false;
    p->ev_count = 0;

    Checked c{p};
    int dev = 0, optin = 0, sms = 0;
    if (!c.ok(cudaGetDevice(&dev)) ||
        !c.ok(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) ||
        !c.ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) {
        delete p;
        return RTPRUNE_ERR_CUDA;
    }
    p->device = dev;
    p->smem_optin = optin;
    p->sm_count = sms;

    // Sinkhorn shared memory: enough for the largest matrix an image of max_tokens can produce
    // ((N/2+1)^2 cells at r = 1/2), capped by what one CTA may have.
    const long long half = max_tokens_per_image / 2 + 2;
    long long want = (half * (half | 1) + max_tokens_per_image + 2 + 2 * kSinkThreads) * 4 + 64;
    const long long cap = (long long)optin - 1024;
    if (want > cap) want = cap;
    p->sink_smem_bytes = (int)(want / 16 * 16);
    // The attribute belongs to the function, not to the plan: every plan sets it to what the device allows,
    // so that a plan made later for smaller images does not lower it under an earlier plan's launches.
    if (!c.ok(cudaFuncSetAttribute(sinkhorn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)(cap / 16 * 16))) ||
        !c.ok(cudaFuncSetAttribute(sinkhorn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)(cap / 16 * 16)))) {
        delete p;
        return RTPRUNE_ERR_CUDA;
    }
    {
        const int s1_cap = std::max(optin - 4096, 0);       // the kernel's static shared memory is under 4 KB
        RatioParams rp0{};
        const cudaError_t e1 =
            dtype == RTPRUNE_BF16
                ? launch_stage1_kernel<__nv_bfloat16>(p, nullptr, nullptr, nullptr, 1, 1, rp0, nullptr, nullptr, nullptr,
                                                      nullptr, nullptr, nullptr, nullptr, 0, s1_cap)
                : launch_stage1_kernel<float>(p, nullptr, nullptr, nullptr, 1, 1, rp0, nullptr, nullptr, nullptr, nullptr,
                                              nullptr, nullptr, nullptr, 0, s1_cap);
        if (!c.ok(e1) ||
            sizeof(float) * stage1_smem_floats(d, max_tokens_per_image, dtype == RTPRUNE_BF16 ? 2 : 4) > (size_t)s1_cap) {
            if (!p->last_cuda_error) p->last_cuda_error = (int)cudaErrorInvalidValue;
            delete p;
            return RTPRUNE_ERR_CUDA;
        }
    }
    p->fast_smem_bytes = (int)(cap / 16 * 16);
    p->exact_smem_bytes = (int)(exact_smem_bytes(max_tokens_per_image, (size_t)std::max(optin - 4096, 0)) / 16 * 16);
    if (4 * exact_array_words(max_tokens_per_image) > (size_t)p->exact_smem_bytes ||
        !c.ok(cudaFuncSetAttribute(exact_pairing_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   std::max(optin - 4096, 0)))) {
        if (!p->last_cuda_error) p->last_cuda_error = (int)cudaErrorInvalidValue;
        delete p;
        return RTPRUNE_ERR_CUDA;
    }
    if (!c.ok(cudaFuncSetAttribute(sinkhorn_cluster_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   p->fast_smem_bytes)) ||
        !c.ok(cudaFuncSetAttribute(sinkhorn_cluster_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   p->fast_smem_bytes))) {
        delete p;
        return RTPRUNE_ERR_CUDA;
    }
    p->encode_tiled = nullptr;
    {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            p->encode_tiled = fn;
        else
            (void)cudaGetLastError();
    }
    if (dtype == RTPRUNE_BF16) {
        if (!p->encode_tiled ||
            !c.ok(cudaFuncSetAttribute(scores_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kScSmemBytes)) ||
            !c.ok(cudaFuncSetAttribute(merge_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kMgSmemBytes))) {
            if (!p->last_cuda_error) p->last_cuda_error = (int)cudaErrorNotSupported;
            delete p;
            return RTPRUNE_ERR_CUDA;
        }
    }
    // The fused stage-2 kernel: clusters of 2 CTAs with all of an SM's shared memory each; how many the
    // device runs at once is what a run's grid is capped at (its clusters then loop over the images).
    p->fused_clusters = 0;
    if (dtype == RTPRUNE_BF16 &&
        cudaFuncSetAttribute(stage2_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFuSmemBytes) ==
            cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2);
        cfg.blockDim = dim3(kFuThreads);
        cfg.dynamicSmemBytes = (size_t)kFuSmemBytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, stage2_fused_kernel, &cfg) == cudaSuccess && nclusters > 0)
            p->fused_clusters = nclusters;
    }
    (void)cudaGetLastError();
    if (dtype == RTPRUNE_BF16)
        (void)cudaFuncSetAttribute(sinkhorn_reg_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFuSmemBytes);
    (void)cudaGetLastError();
    // Clusters of 16 CTAs (beyond the portable size) for the wide-tile Sinkhorn kernel: ask the device how
    // many it can run at once; a run uses them only if all its images fit that number.
    p->tall_c16_clusters = 0;
    {
        const int tall_smem = std::max(p->smem_optin - 1024, 0);
        if (cudaFuncSetAttribute(sinkhorn_tall_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tall_smem) ==
                cudaSuccess &&
            cudaFuncSetAttribute(sinkhorn_tall_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) ==
                cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(kTallCMax);
            cfg.blockDim = dim3(kTallThreads);
            cfg.dynamicSmemBytes = (size_t)tall_smem;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = kTallCMax;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int nclusters = 0;
            if (cudaOccupancyMaxActiveClusters(&nclusters, sinkhorn_tall_kernel, &cfg) == cudaSuccess && nclusters > 0)
                p->tall_c16_clusters = nclusters;
        }
        (void)cudaGetLastError();
    }
    *workspace_bytes = p->ws.total;
    *plan_out = p;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_workspace_init(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                        size_t workspace_bytes)
{
    if (!plan || !workspace || ((uintptr_t)workspace & 255u)) return RTPRUNE_ERR_INVALID_ARG;
    if (workspace_bytes < plan->ws.total) return RTPRUNE_ERR_WORKSPACE;
    Checked c{plan};
    if (!c.ok(cudaMemsetAsync((char *)workspace + plan->ws.header, 0, plan->ws.clear_bytes,
                              (cudaStream_t)cuda_stream)))
        return RTPRUNE_ERR_CUDA;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_run(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                             const int32_t *offsets, int32_t batch, int64_t total_tokens,
                             const rtprune_params_t *params, void *workspace,
                             size_t workspace_bytes, void *Y, int32_t *out_offsets,
                             int32_t *counts, int32_t *kept_idx, int32_t *merged_idx,
                             int32_t *merge_partner, float *merge_weight, float *stats)
{
    rtprune_status_t s = check_common(plan, X, offsets, batch, total_tokens, params, workspace,
                                      workspace_bytes);
    if (s != RTPRUNE_OK) return s;
    if (!out_offsets) return RTPRUNE_ERR_INVALID_ARG;
    if (batch > 0 && (!Y || !counts || !kept_idx || !merged_idx || !merge_partner ||
                      !merge_weight || !stats))
        return RTPRUNE_ERR_INVALID_ARG;
    if ((uintptr_t)Y & 15u) return RTPRUNE_ERR_INVALID_ARG;
    plan->last_launches = 0;
    DevOut o{Y, out_offsets, counts, kept_idx, merged_idx, merge_partner, merge_weight, stats};
    const auto t0 = std::chrono::steady_clock::now();
    s = run_device(plan, (cudaStream_t)cuda_stream, X, offsets, batch, (int)total_tokens, params,
                   (char *)workspace, o);
    plan->last_host_ns = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    return s;
}

rtprune_status_t rtprune_select(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                                const int32_t *offsets, int32_t batch, int64_t total_tokens,
                                const rtprune_params_t *params, void *workspace,
                                size_t workspace_bytes, int32_t *out_offsets, int32_t *counts,
                                float *stats, float *norms_out, int32_t *order_out)
{
    rtprune_status_t s = check_common(plan, X, offsets, batch, total_tokens, params, workspace,
                                      workspace_bytes);
    if (s != RTPRUNE_OK) return s;
    if (!out_offsets || (batch > 0 && (!counts || !stats))) return RTPRUNE_ERR_INVALID_ARG;
    plan->last_launches = 0;
    if (batch == 0) {
        Checked c{plan};
        if (!c.ok(cudaMemsetAsync(out_offsets, 0, sizeof(int32_t), (cudaStream_t)cuda_stream)))
            return RTPRUNE_ERR_CUDA;
        return RTPRUNE_OK;
    }
    prof_begin(plan, (cudaStream_t)cuda_stream);
    return launch_stage1(plan, (cudaStream_t)cuda_stream, X, offsets, batch, (int)total_tokens, params,
                         (char *)workspace, out_offsets, counts, stats, norms_out, order_out, true);
}

rtprune_status_t rtprune_select_static(rtprune_plan_t *plan, void *cuda_stream, const void *X,
                                       const int32_t *offsets, int32_t batch, int64_t total_tokens,
                                       const rtprune_params_t *params, int32_t *out_offsets,
                                       int32_t *counts, float *stats, float *norms_out,
                                       int32_t *order_out)
{
    if (!plan || !params) return RTPRUNE_ERR_INVALID_ARG;
    if (!on_plan_device(plan)) return RTPRUNE_ERR_INVALID_ARG;
    if (batch < 0 || total_tokens < 0 || batch > plan->max_batch || total_tokens > plan->max_total ||
        total_tokens < batch)
        return RTPRUNE_ERR_INVALID_ARG;
    if (batch > 0 && (!X || !offsets)) return RTPRUNE_ERR_INVALID_ARG;
    if ((uintptr_t)X & 15u) return RTPRUNE_ERR_INVALID_ARG;
    if (!out_offsets || (batch > 0 && (!counts || !stats))) return RTPRUNE_ERR_INVALID_ARG;
    // Stage 1 uses the workspace regions that precede the score tiles; they must fit the array.
    if (plan->ws.kmat > (size_t)RTPRUNE_STATIC_SCRATCH_BYTES) return RTPRUNE_ERR_WORKSPACE;
    rtprune_status_t s = check_params(params);
    if (s != RTPRUNE_OK) return s;

    Checked c{plan};
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int dev = -1;
    if (!c.ok(cudaGetDevice(&dev))) return RTPRUNE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return RTPRUNE_ERR_UNSUPPORTED;
    char *scratch = nullptr;
    {
        // first call on this device: ask the runtime where this device keeps the array
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_scratch_addr[dev]) {
            void *p = nullptr;
            if (!c.ok(cudaGetSymbolAddress(&p, g_static_scratch)) || !p) return RTPRUNE_ERR_CUDA;
            g_static_scratch_addr[dev] = p;
        }
        scratch = (char *)g_static_scratch_addr[dev];
    }
    plan->last_launches = 0;
    if (batch == 0) {
        if (!c.ok(cudaMemsetAsync(out_offsets, 0, sizeof(int32_t), st))) return RTPRUNE_ERR_CUDA;
        return RTPRUNE_OK;
    }
    // the array keeps whatever the last call left: the status word and the counters must start at 0
    if (!c.ok(cudaMemsetAsync(scratch + plan->ws.header, 0, plan->ws.clear_bytes, st)))
        return RTPRUNE_ERR_CUDA;
    prof_begin(plan, st);
    return launch_stage1(plan, st, X, offsets, batch, (int)total_tokens, params, scratch, out_offsets,
                         counts, stats, norms_out, order_out, true);
}

rtprune_status_t rtprune_static_scratch_needed(const rtprune_plan_t *plan, size_t *bytes)
{
    if (!plan || !bytes) return RTPRUNE_ERR_INVALID_ARG;
    *bytes = plan->ws.kmat;      // stage 1 uses the workspace regions that precede the score tiles
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_query_status_static(rtprune_plan_t *plan, void *cuda_stream, uint32_t *flags_out)
{
    if (!plan) return RTPRUNE_ERR_INVALID_ARG;
    if (!on_plan_device(plan)) return RTPRUNE_ERR_INVALID_ARG;
    Checked c{plan};
    int dev = -1;
    if (!c.ok(cudaGetDevice(&dev))) return RTPRUNE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return RTPRUNE_ERR_UNSUPPORTED;
    char *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        scratch = (char *)g_static_scratch_addr[dev];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t flags = 0;
    if (scratch) {
        WsHeader *hdr = (WsHeader *)(scratch + plan->ws.header);
        if (!c.ok(cudaMemcpyAsync(&flags, &hdr->status, sizeof(flags), cudaMemcpyDeviceToHost, st)) ||
            !c.ok(cudaMemsetAsync(&hdr->status, 0, sizeof(uint32_t), st)) || !c.ok(cudaStreamSynchronize(st)))
            return RTPRUNE_ERR_CUDA;
    }
    if (flags_out) *flags_out = flags;
    if (flags & RTPRUNE_DEV_NONFINITE) return RTPRUNE_ERR_NONFINITE;
    if (flags & RTPRUNE_DEV_BAD_OFFSETS) return RTPRUNE_ERR_BAD_OFFSETS;
    if (flags & RTPRUNE_DEV_TIMEOUT) return RTPRUNE_ERR_TIMEOUT;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_test_expire_waits(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                           size_t workspace_bytes, uint32_t poll_limit, int32_t *expired_out)
{
    if (!plan || !workspace || ((uintptr_t)workspace & 255u)) return RTPRUNE_ERR_INVALID_ARG;
    if (!on_plan_device(plan)) return RTPRUNE_ERR_INVALID_ARG;
    if (workspace_bytes < plan->ws.total) return RTPRUNE_ERR_WORKSPACE;
    if (poll_limit < 1 || poll_limit > 65536) return RTPRUNE_ERR_INVALID_ARG;
    Checked c{plan};
    expire_waits_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>((WsHeader *)((char *)workspace + plan->ws.header),
                                                                 poll_limit, expired_out);
    if (!c.ok(cudaGetLastError())) return RTPRUNE_ERR_CUDA;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_test_set_poll_limit(rtprune_plan_t *plan, int64_t polls)
{
    if (!plan || polls > (int64_t)ptx::kSpinLimit) return RTPRUNE_ERR_INVALID_ARG;
    plan->poll_limit = polls < 0 ? ptx::kSpinLimit : (uint32_t)polls;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_host_arena_bytes(const rtprune_plan_t *plan, size_t *arena_bytes)
{
    if (!plan || !arena_bytes) return RTPRUNE_ERR_INVALID_ARG;
    *arena_bytes = make_arena(plan).total;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_run_host(rtprune_plan_t *plan, void *cuda_stream, const void *X_host,
                                  const int32_t *offsets_host, const float *rho_host,
                                  int32_t batch, int64_t total_tokens,
                                  const rtprune_params_t *params, void *arena, size_t arena_bytes,
                                  void *Y_host, int32_t *out_offsets_host, int32_t *counts_host,
                                  int32_t *kept_idx_host, int32_t *merged_idx_host,
                                  int32_t *merge_partner_host, float *merge_weight_host,
                                  float *stats_host)
{
    if (!plan || !params || !arena || ((uintptr_t)arena & 255u)) return RTPRUNE_ERR_INVALID_ARG;
    if (!on_plan_device(plan)) return RTPRUNE_ERR_INVALID_ARG;
    if (batch < 0 || total_tokens < 0 || batch > plan->max_batch ||
        total_tokens > plan->max_total || total_tokens < batch)
        return RTPRUNE_ERR_INVALID_ARG;
    if (!out_offsets_host) return RTPRUNE_ERR_INVALID_ARG;
    if (batch > 0 && (!X_host || !offsets_host || !Y_host || !counts_host || !kept_idx_host ||
                      !merged_idx_host || !merge_partner_host || !merge_weight_host || !stats_host))
        return RTPRUNE_ERR_INVALID_ARG;
    const Arena a = make_arena(plan);
    if (arena_bytes < a.total) return RTPRUNE_ERR_WORKSPACE;
    rtprune_status_t s = check_params(params);
    if (s != RTPRUNE_OK) return s;
    // the host can see the offsets here: check the contract before anything is launched
    if (batch > 0) {
        if (offsets_host[0] != 0 || offsets_host[batch] != total_tokens) return RTPRUNE_ERR_INVALID_ARG;
        for (int i = 0; i < batch; ++i) {
            const int64_t n = (int64_t)offsets_host[i + 1] - offsets_host[i];
            if (n < 1 || n > plan->max_tokens) return RTPRUNE_ERR_INVALID_ARG;
        }
    }
    plan->last_launches = 0;
    Checked c{plan};
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *base = (char *)arena;
    const size_t esz = plan->dtype == RTPRUNE_BF16 ? 2 : 4;
    const size_t row = (size_t)plan->d * esz;
    if (batch == 0) {
        out_offsets_host[0] = 0;
        return RTPRUNE_OK;
    }
    rtprune_params_t p = *params;
    p.rho = rho_host ? (const float *)(base + a.rho) : nullptr;
    if (!c.ok(cudaMemcpyAsync(base + a.X, X_host, (size_t)total_tokens * row, cudaMemcpyHostToDevice, st)) ||
        !c.ok(cudaMemcpyAsync(base + a.offsets, offsets_host, ((size_t)batch + 1) * 4, cudaMemcpyHostToDevice, st)))
        return RTPRUNE_ERR_CUDA;
    if (rho_host && !c.ok(cudaMemcpyAsync(base + a.rho, rho_host, (size_t)batch * 4, cudaMemcpyHostToDevice, st)))
        return RTPRUNE_ERR_CUDA;
    if (!c.ok(cudaMemsetAsync(base + a.ws + plan->ws.header, 0, plan->ws.clear_bytes, st)))
        return RTPRUNE_ERR_CUDA;
    DevOut o{base + a.Y,
             (int32_t *)(base + a.out_offsets),
             (int32_t *)(base + a.counts),
             (int32_t *)(base + a.kept_idx),
             (int32_t *)(base + a.merged_idx),
             (int32_t *)(base + a.partner),
             (float *)(base + a.weight),
             (float *)(base + a.stats)};
    s = run_device(plan, st, base + a.X, (const int32_t *)(base + a.offsets), batch,
                   (int)total_tokens, &p,
                   base + a.ws, o);
    if (s != RTPRUNE_OK) return s;
    // Rows of Y to bring back: with a fixed ratio every image's kept count is known here (the expression stage 1
    // evaluates, in the same arithmetic); a dynamic ratio is decided on the device, so all rows are copied.
    size_t y_rows = (size_t)total_tokens;
    if (!p.dynamic) {
        y_rows = 0;
        const float r = std::fmax(p.r_fixed, 0.f);
        for (int i = 0; i < batch; ++i) {
            const int n = offsets_host[i + 1] - offsets_host[i];
            int b = (int)std::floor(std::fmaf(r, (float)n, 0.5f));
            b = std::max(0, std::min(b, n - 1));
            y_rows += (size_t)(n - b);
        }
    }
    const size_t tot4 = (size_t)total_tokens * 4;
    if (!c.ok(cudaMemcpyAsync(out_offsets_host, o.out_offsets, ((size_t)batch + 1) * 4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(counts_host, o.counts, (size_t)batch * 4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(kept_idx_host, o.kept_idx, tot4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(merged_idx_host, o.merged_idx, tot4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(merge_partner_host, o.merge_partner, tot4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(merge_weight_host, o.merge_weight, tot4, cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemcpyAsync(stats_host, o.stats, (size_t)batch * kStats * 4, cudaMemcpyDeviceToHost, st)) ||
        (y_rows && !c.ok(cudaMemcpyAsync(Y_host, o.Y, y_rows * row, cudaMemcpyDeviceToHost, st))))
        return RTPRUNE_ERR_CUDA;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_query_status(rtprune_plan_t *plan, void *cuda_stream, void *workspace,
                                      uint32_t *flags_out)
{
    if (!plan || !workspace) return RTPRUNE_ERR_INVALID_ARG;
    Checked c{plan};
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t flags = 0;
    WsHeader *hdr = (WsHeader *)((char *)workspace + plan->ws.header);
    if (!c.ok(cudaMemcpyAsync(&flags, &hdr->status, sizeof(flags), cudaMemcpyDeviceToHost, st)) ||
        !c.ok(cudaMemsetAsync(&hdr->status, 0, sizeof(uint32_t), st)) ||
        !c.ok(cudaStreamSynchronize(st)))
        return RTPRUNE_ERR_CUDA;
    if (flags_out) *flags_out = flags;
    if (flags & RTPRUNE_DEV_NONFINITE) return RTPRUNE_ERR_NONFINITE;
    if (flags & RTPRUNE_DEV_BAD_OFFSETS) return RTPRUNE_ERR_BAD_OFFSETS;
    if (flags & RTPRUNE_DEV_TIMEOUT) return RTPRUNE_ERR_TIMEOUT;
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_profile_enable(rtprune_plan_t *plan, int32_t enable)
{
    if (!plan) return RTPRUNE_ERR_INVALID_ARG;
    Checked c{plan};
    if (enable && !plan->profiling) {
        for (int i = 0; i <= RTPRUNE_PROFILE_MAX; ++i)
            if (!c.ok(cudaEventCreate(&plan->ev[i]))) {
                for (int k = 0; k < i; ++k) cudaEventDestroy(plan->ev[k]);
                return RTPRUNE_ERR_CUDA;
            }
        plan->profiling = true;
        plan->ev_count = 0;
    } else if (!enable && plan->profiling) {
        for (int i = 0; i <= RTPRUNE_PROFILE_MAX; ++i) cudaEventDestroy(plan->ev[i]);
        plan->profiling = false;
        plan->ev_count = 0;
    }
    return RTPRUNE_OK;
}

rtprune_status_t rtprune_profile_read(rtprune_plan_t *plan, int32_t *n, float *ms,
                                      const char **names)
{
    if (!plan || !n || !ms || !names) return RTPRUNE_ERR_INVALID_ARG;
    *n = 0;
    if (!plan->profiling || plan->ev_count == 0) return RTPRUNE_OK;
    Checked c{plan};
    if (!c.ok(cudaEventSynchronize(plan->ev[plan->ev_count]))) return RTPRUNE_ERR_CUDA;
    for (int i = 0; i < plan->ev_count; ++i) {
        if (!c.ok(cudaEventElapsedTime(&ms[i], plan->ev[i], plan->ev[i + 1]))) return RTPRUNE_ERR_CUDA;
        names[i] = plan->ev_name[i];
    }
    *n = plan->ev_count;
    return RTPRUNE_OK;
}

int32_t rtprune_last_launch_count(const rtprune_plan_t *plan) { return plan ? plan->last_launches : 0; }

int32_t rtprune_last_cuda_error(const rtprune_plan_t *plan) { return plan ? plan->last_cuda_error : 0; }

int64_t rtprune_last_host_ns(const rtprune_plan_t *plan) { return plan ? plan->last_host_ns : 0; }

void rtprune_destroy(rtprune_plan_t *plan)
{
    if (!plan) return;
    if (plan->profiling) rtprune_profile_enable(plan, 0);
    delete plan;
}

const char *rtprune_status_string(rtprune_status_t s)
{
    switch (s) {
    case RTPRUNE_OK: return "RTPRUNE_OK";
    case RTPRUNE_ERR_INVALID_ARG: return "RTPRUNE_ERR_INVALID_ARG";
    case RTPRUNE_ERR_UNSUPPORTED: return "RTPRUNE_ERR_UNSUPPORTED";
    case RTPRUNE_ERR_WORKSPACE: return "RTPRUNE_ERR_WORKSPACE";
    case RTPRUNE_ERR_CUDA: return "RTPRUNE_ERR_CUDA";
    case RTPRUNE_ERR_NONFINITE: return "RTPRUNE_ERR_NONFINITE";
    case RTPRUNE_ERR_TIMEOUT: return "RTPRUNE_ERR_TIMEOUT";
    case RTPRUNE_ERR_BAD_OFFSETS: return "RTPRUNE_ERR_BAD_OFFSETS";
    }
    return "RTPRUNE_ERR_UNKNOWN";
}

int32_t rtprune_version(void) { return 100; }

}  // extern "C"
