// Stage 1 of Algorithm 1: token norms (Eq. 1), the similarity statistic phi (Eq. 8), the pruning
// ratio (Eq. 10) and the top-M selection (Section 3.3.1), in one kernel, plus the kernel that makes
// the compact copy of the pruned rows for the tensor-core kernels.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace rtp {

struct RatioParams {
    int dynamic;
    float r_fixed, phi_lo, phi_hi, r_max;
    int criterion;      // 0 l2 norm (Eq. 1), 1 variance, 2 entropy of the softmax of the features
};

constexpr int kS1Threads = 256;
constexpr int kS1Warps = kS1Threads / 32;

constexpr int kS1StageRows = kS1Warps;   // rows per stage of the streaming ring: one per warp
constexpr int kS1MaxStages = 4;

// Stages of the streaming ring for rows of row_bytes: as many as fit in 96 KB, 2 to 4.
__host__ __device__ inline int stage1_stages(size_t row_bytes)
{
    const size_t s = (96u * 1024u) / (kS1StageRows * row_bytes);
    return s < 2 ? 2 : (s > (size_t)kS1MaxStages ? kS1MaxStages : (int)s);
}

// Dynamic shared memory (floats) of stage1_kernel: the ring of row stages, reused for the 8 warps'
// partial sums of unit tokens and then for the image's norm keys of the ranking.
__host__ __device__ inline size_t stage1_smem_floats(int d, int max_tokens, size_t elem_bytes)
{
    const size_t ring = (size_t)stage1_stages((size_t)d * elem_bytes) * kS1StageRows * d * elem_bytes / 4;
    const size_t a = (size_t)kS1Warps * d, b = (size_t)max_tokens + 64;
    const size_t m = a > b ? a : b;
    return ring > m ? ring : m;
}

// Exclusive prefix sum of one int per thread over the CTA (256 threads); `scratch` holds 32 ints.
__device__ inline int block_excl_scan(int v, int *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                       // scratch may still be read from an earlier scan
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < kS1Warps) ? scratch[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;
    }
    __syncthreads();
    return scratch[warp] + incl - v;
}

// ---------------------------------------------------------------------------------------------
// Selection of one image by one CTA (256 threads): phi from the chunk partials; r and
// B = floor(r N + 1/2) clamped to [0, N-1], M = N - B; the M tokens of largest criterion (`norms`: the
// l2 norms, or the variance / entropy values of a run that ranks by those; ties to the lower
// index) are T_kept.  The M-th largest value is found by a radix select over its bits (four
// 8-bit digits, a 256-bin histogram each), tokens equal to it are admitted in index order.  Writes
// order[] = kept indices ascending, then pruned indices ascending, and its inverse kpos[]; counts,
// stats.
// ---------------------------------------------------------------------------------------------
__device__ inline void select_image(int img, int t_begin, int N, int d, int chunks, int chunk_tokens,
                                    const RatioParams &rp,
                                    const float *__restrict__ rho, const float *norms, const float *spart,
                                    int32_t *__restrict__ order, int32_t *__restrict__ kpos,
                                    int32_t *counts, float *__restrict__ stats,
                                    float *__restrict__ norms_out, int32_t *__restrict__ order_out,
                                    uint32_t *s_keys)
{
    __shared__ float s_redf[32];
    __shared__ int s_redi[32];
    __shared__ int s_hist[256];
    __shared__ int s_M;
    __shared__ uint32_t s_prefix;
    __shared__ int s_need;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nth = kS1Threads;

    // Every global read is issued before the first use of any of them (one trip to L2, not one per
    // loop iteration): rho, the norms (keys of the ranking), the chunk partials.
    const float rho_i = (tid == 0 && rho) ? __ldg(rho + img) : 0.f;
    constexpr int kKeysAhead = 4;      // norms per thread held in registers (N <= 1024), the rest in a loop
    float key_r[kKeysAhead];
#pragma unroll
    for (int q = 0; q < kKeysAhead; ++q) {
        const int k = tid + q * nth;
        key_r[q] = (k < N) ? __ldcg(norms + t_begin + k) : 0.f;
    }
    // phi (Eq. 8) via |sum of unit tokens|^2; the partials were written by other CTAs: read them from L2.
    // A thread owns groups of 4 columns (tid, tid + 256, ...) and adds them over the chunks, four chunks
    // and four groups to a batch of loads.
    const int nchunk = (N + chunk_tokens - 1) / chunk_tokens;
    const float4 *sp4 = reinterpret_cast<const float4 *>(spart + (size_t)img * chunks * d);
    const int ngroups = d >> 2, d4 = d >> 2;
    float local = 0.f;
    for (int g0 = tid; g0 < ngroups; g0 += 4 * nth) {
        float4 a4[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) a4[a] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k0 = 0; k0 < nchunk; k0 += 4) {
            float4 v[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int g = g0 + a * nth;
                    v[a][u] = (g < ngroups && k0 + u < nchunk) ? __ldcg(sp4 + (size_t)(k0 + u) * d4 + g)
                                                               : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a4[a].x += v[a][u].x;
                    a4[a].y += v[a][u].y;
                    a4[a].z += v[a][u].z;
                    a4[a].w += v[a][u].w;
                }
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            local = fmaf(a4[a].x, a4[a].x, local);
            local = fmaf(a4[a].y, a4[a].y, local);
            local = fmaf(a4[a].z, a4[a].z, local);
            local = fmaf(a4[a].w, a4[a].w, local);
        }
    }
    // norm bits: for non-negative floats the unsigned order is the float order, and a NaN still ranks.
    // The other criteria may round to just below zero: sign-aware map of the bits to unsigned order.
    const bool signed_keys = rp.criterion != 0;
    auto key_bits = [&](float c) -> uint32_t {
        const uint32_t b = __float_as_uint(c);
        if (!signed_keys) return b & 0x7fffffffu;
        return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    };
#pragma unroll
    for (int q = 0; q < kKeysAhead; ++q) {
        const int k = tid + q * nth;
        if (k < N) {
            s_keys[k] = key_bits(key_r[q]);
            if (norms_out) norms_out[t_begin + k] = key_r[q];
        }
    }
    for (int k = tid + kKeysAhead * nth; k < N; k += nth) {
        const float key = __ldcg(norms + t_begin + k);
        s_keys[k] = key_bits(key);
        if (norms_out) norms_out[t_begin + k] = key;
    }
    const float ssum = block_sum(local, s_redf);
    if (tid == 0) {
        const float Nf = (float)N;
        const float phi = (N >= 2) ? (ssum - Nf) / (Nf * (Nf - 1.f)) : 0.f;
        float r;
        if (rp.dynamic) {
            float f = (phi - rp.phi_lo) / (rp.phi_hi - rp.phi_lo);
            f = fminf(fmaxf(f, 0.f), 1.f);
            r = fminf(f * (1.f - rho_i), rp.r_max);
        } else {
            r = rp.r_fixed;
        }
        r = fmaxf(r, 0.f);
        int B = (int)floorf(fmaf(r, Nf, 0.5f));     // one rounding: the host evaluates the same expression
        B = max(0, min(B, N - 1));
        s_M = N - B;
        float *st = stats + (size_t)img * kStats;
        st[0] = phi;
        st[1] = rho_i;
        st[2] = r;
        st[3] = (float)(N - B);
        st[4] = (float)B;
        st[5] = 0.f;
        st[6] = 0.f;
        st[7] = 0.f;
        counts[img] = N - B;
    }
    __syncthreads();
    const int M = s_M;

    // radix select: after the four digits `prefix` is the M-th largest key and `need` is how many
    // tokens equal to it are kept
    uint32_t prefix = 0;
    int need = M;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        s_hist[tid] = 0;
        __syncthreads();
        for (int k = tid; k < N; k += nth) {
            const uint32_t key = s_keys[k];
            if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1);
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns the bins 255 - 8 l down to 248 - 8 l: largest digits first
            int h[8], sum8 = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                h[q] = s_hist[255 - 8 * lane - q];
                sum8 += h[q];
            }
            int incl = sum8;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            int c = incl - sum8;
            if (c < need && need <= incl) {            // exactly one lane
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (c < need && need <= c + h[q]) {
                        s_prefix = (prefix << 8) | (uint32_t)(255 - 8 * lane - q);
                        s_need = need - c;
                    }
                    c += h[q];
                }
            }
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
    }
    const uint32_t thr = prefix;

    // Each thread owns a contiguous range of tokens so that block scans give positions in ascending
    // index: first among the tokens equal to the threshold, then among the kept ones.
    const int ipt = (N + nth - 1) / nth;          // <= 32 for N <= 8192
    const int k0 = min(tid * ipt, N), k1 = min(k0 + ipt, N);
    int neq = 0;
    for (int k = k0; k < k1; ++k) neq += (s_keys[k] == thr) ? 1 : 0;
    int eq_run = block_excl_scan(neq, s_redi);
    uint32_t keptmask = 0;
    int nkept = 0;
    for (int k = k0; k < k1; ++k) {
        const uint32_t key = s_keys[k];
        bool kept = key > thr;
        if (key == thr) {
            kept = eq_run < need;
            ++eq_run;
        }
        if (kept) {
            keptmask |= 1u << (k - k0);
            ++nkept;
        }
    }
    int kpos_run = block_excl_scan(nkept, s_redi);   // kept tokens before k0
    int32_t *ord = order + t_begin;
    for (int k = k0; k < k1; ++k) {
        const bool kept = (keptmask >> (k - k0)) & 1u;
        const int pos = kept ? kpos_run : (M + (k - kpos_run));
        ord[pos] = k;
        kpos[t_begin + k] = kept ? kpos_run : -1 - (k - kpos_run);
        if (order_out) order_out[t_begin + pos] = k;
        kpos_run += kept ? 1 : 0;
    }
    __syncthreads();
}

// out_offsets = exclusive prefix sum of counts (and the total at [batch]), by one CTA of NTH threads;
// `scratch` holds 32 ints.
template <int NTH>
__device__ inline void scan_counts(const int32_t *counts, int32_t *__restrict__ out_offsets, int batch,
                                   int *scratch)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ipt2 = (batch + NTH - 1) / NTH;
    const int b0 = min(tid * ipt2, batch), b1 = min(b0 + ipt2, batch);
    int sum = 0;
    for (int b = b0; b < b1; ++b) sum += __ldcg(counts + b);
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < (NTH >> 5)) ? scratch[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;
    }
    __syncthreads();
    int run = scratch[warp] + incl - sum;
    for (int b = b0; b < b1; ++b) {
        out_offsets[b] = run;
        run += __ldcg(counts + b);
    }
    if (tid == NTH - 1) out_offsets[batch] = run;  // the last thread's running sum is the total
}

// ---------------------------------------------------------------------------------------------
// grid = (chunks of this run, batch), 256 threads; CTA (c, i) owns chunk_tokens consecutive tokens of
// image i (a multiple of 8, at least kChunkTokens, chosen by the host so that the grid is about one wave).
//   Pass over X: the chunk's rows stream through a shared-memory ring (bulk copies issued by one
//   thread); a warp takes one row of each stage: fp32 sum of squares
//   by shuffle reduction; while the row is still in registers it is added, divided by its
//   norm, into per-lane accumulators; the CTA writes the partial sum of unit tokens of its chunk to
//   spart[img][chunk][d].  phi needs only |sum_k x_k/|x_k||^2:
//       sum_{k<l} cos(x_k, x_l) = (|sum_k xhat_k|^2 - N) / 2.
//   The CTA that finishes an image last (a counter per image) runs the selection of that image; the
//   CTA that finishes the last image turns counts into out_offsets (exclusive prefix sum).
// Dynamic shared memory: stage1_smem_floats(d, max_tokens, sizeof(T)) floats.
// ---------------------------------------------------------------------------------------------
template <typename T, int VPL>  // VPL = 16-byte vectors per lane = ceil(d / (32 * kPerVec))
__global__ void __launch_bounds__(kS1Threads, 2)
stage1_kernel(const T *__restrict__ X, const int32_t *__restrict__ offsets, int batch, int d, int chunks,
              int chunk_tokens, int max_tokens, int total, RatioParams rp, const float *__restrict__ rho,
              float *norms, float *critv, float *spart, uint32_t *img_done, int32_t *__restrict__ order,
              int32_t *__restrict__ kpos, int32_t *counts, int32_t *__restrict__ out_offsets,
              float *__restrict__ stats, float *__restrict__ norms_out, int32_t *__restrict__ order_out,
              WsHeader *hdr, int scan_here, uint32_t poll_limit)
{
    constexpr int EPV = Elem<T>::kPerVec;
    extern __shared__ __align__(16) float s_dyn[];
    __shared__ bool s_last, s_unseen;
    __shared__ int s_scan[32];
    __shared__ uint64_t s_full[kS1MaxStages], s_empty[kS1MaxStages];
    const int img = blockIdx.y, chunk = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        // This CTA numbers the run: the kernels behind tell this run's counters and lists in the workspace from
        // the last run's by the number.  It is counted up here, on the device, after the run ahead in the stream
        // has ended and BEFORE this CTA lets the dependents go (they are scheduled once every CTA of this grid
        // has done so), so every kernel of the run reads the new number, also in a replayed CUDA graph.
        ptx::grid_dep_wait();
        if (tid == 0) {
            int seq = hdr->launch_seq + 1;
            if (seq == 0) seq = 1;         // 0 is what a fresh workspace holds
            ptx::st_release_gpu(&hdr->launch_seq, seq);
            __threadfence();
        }
        __syncthreads();
        ptx::grid_dep_launch();
    } else {
        ptx::grid_dep_launch();
        ptx::grid_dep_wait();     // the workspace may still be in use by the run ahead in the stream
    }
    int t_begin, n_img;
    const bool valid = image_range(offsets, img, max_tokens, total, t_begin, n_img);
    if (!valid) {
        if (chunk != 0) return;
        if (tid == 0) {   // offsets broke the contract: the image yields no output
            atomicOr(&hdr->status, RTPRUNE_DEV_BAD_OFFSETS);
            counts[img] = 0;
            float *st = stats + (size_t)img * kStats;
            for (int q = 0; q < kStats; ++q) st[q] = 0.f;
        }
    } else {
        const int t0 = t_begin + chunk * chunk_tokens;
        const int t_end = t_begin + n_img;
        if (t0 >= t_end) return;
        const int t1 = min(t0 + chunk_tokens, t_end);
        const int nvec = d / EPV;

        float acc[VPL * EPV];
#pragma unroll
        for (int i = 0; i < VPL * EPV; ++i) acc[i] = 0.f;
        bool bad = false, gave_up = false;

        // The chunk's rows are contiguous in X: thread 0 streams them through a ring of shared-memory
        // stages (8 rows each, one per warp) with bulk copies, a few stages ahead of the warps.
        const size_t row_bytes = (size_t)d * sizeof(T);
        const int nstage = stage1_stages(row_bytes);
        const uint32_t stage_bytes = (uint32_t)(kS1StageRows * row_bytes);
        const uint32_t ring_u32 = ptx::smem_u32(s_dyn);
        const int nit = (t1 - t0 + kS1StageRows - 1) / kS1StageRows;
        if (tid == 0) {
            for (int s = 0; s < kS1MaxStages; ++s) {
                ptx::mbar_init(&s_full[s], 1);
                ptx::mbar_init(&s_empty[s], kS1Warps);
            }
            s_unseen = false;
            ptx::fence_mbar_init();
        }
        __syncthreads();
        auto issue = [&](int it) {
            const int s = it % nstage;
            const int r0 = t0 + it * kS1StageRows;
            const uint32_t bytes = (uint32_t)(min(kS1StageRows, t1 - r0) * row_bytes);
            ptx::mbar_arrive_expect_tx(&s_full[s], bytes);
            ptx::bulk_load(ring_u32 + s * stage_bytes, X + (size_t)r0 * d, bytes, &s_full[s]);
        };
        int issued = 0;           // thread 0: copies issued so far
        if (tid == 0)
            for (int it = 0; it < min(nstage, nit); ++it, ++issued) issue(it);
        for (int it = 0; it < nit; ++it) {
            const int s = it % nstage;
            {   // a warp goes on or gives up as one (the row's reductions below are warp-wide)
                const bool landed = !gave_up && ptx::mbar_wait(&s_full[s], (it / nstage) & 1, poll_limit);
                if (!__all_sync(0xffffffffu, landed)) gave_up = true;
            }
            const int t = t0 + it * kS1StageRows + warp;
            if (t < t1 && !gave_up) {
                const uint4 *row = reinterpret_cast<const uint4 *>(
                    reinterpret_cast<const uint8_t *>(s_dyn) + s * stage_bytes + warp * row_bytes);
                uint4 cur[VPL];
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    const int vi = lane + 32 * j;
                    cur[j] = (vi < nvec) ? row[vi] : make_uint4(0, 0, 0, 0);
                }
                float ss = 0.f;
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    float f[EPV];
                    Elem<T>::unpack(cur[j], f);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
                }
                ss = warp_sum(ss);
                const float n = sqrtf(ss);
                if (!(ss <= 3.0e38f)) bad = true;  // inf or NaN
                const float inv = 1.f / fmaxf(n, kNormFloor);
                if (lane == 0) norms[t] = n;
                if (rp.criterion != 0) {           // uniform over the grid: the ranking of the ablation
                    float cval;
                    if (rp.criterion == 1) {
                        // variance over the d features, two passes over the row held in registers
                        float sum = 0.f;
#pragma unroll
                        for (int j = 0; j < VPL; ++j) {
                            float f[EPV];
                            Elem<T>::unpack(cur[j], f);
#pragma unroll
                            for (int e = 0; e < EPV; ++e) sum += f[e];      // lanes past the row hold zeros
                        }
                        const float mean = warp_sum(sum) / (float)d;
                        float dev2 = 0.f;
#pragma unroll
                        for (int j = 0; j < VPL; ++j) {
                            if (lane + 32 * j < nvec) {
                                float f[EPV];
                                Elem<T>::unpack(cur[j], f);
#pragma unroll
                                for (int e = 0; e < EPV; ++e) dev2 = fmaf(f[e] - mean, f[e] - mean, dev2);
                            }
                        }
                        cval = warp_sum(dev2) / (float)d;
                    } else {
                        // entropy of softmax(row): log(sum e^(x-m)) - sum (x-m) e^(x-m) / sum e^(x-m)
                        float mx = -INFINITY;
#pragma unroll
                        for (int j = 0; j < VPL; ++j) {
                            if (lane + 32 * j < nvec) {
                                float f[EPV];
                                Elem<T>::unpack(cur[j], f);
#pragma unroll
                                for (int e = 0; e < EPV; ++e) mx = fmaxf(mx, f[e]);
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                        float se = 0.f, sxe = 0.f;
#pragma unroll
                        for (int j = 0; j < VPL; ++j) {
                            if (lane + 32 * j < nvec) {
                                float f[EPV];
                                Elem<T>::unpack(cur[j], f);
#pragma unroll
                                for (int e = 0; e < EPV; ++e) {
                                    const float dx = f[e] - mx;
                                    const float ex = expf(dx);
                                    se += ex;
                                    sxe = fmaf(dx, ex, sxe);
                                }
                            }
                        }
                        se = warp_sum(se);
                        sxe = warp_sum(sxe);
                        cval = logf(se) - sxe / se;
                    }
                    if (lane == 0) critv[t] = cval;
                }
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    float f[EPV];
                    Elem<T>::unpack(cur[j], f);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc[j * EPV + e] = fmaf(f[e], inv, acc[j * EPV + e]);
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&s_empty[s]);
            if (tid == 0 && it + nstage < nit && !gave_up) {     // refill the stage once all eight warps have left it
                if (ptx::mbar_wait(&s_empty[s], (it / nstage) & 1, poll_limit)) {
                    issue(it + nstage);
                    ++issued;
                } else {
                    s_unseen = true;       // (read after the barrier below; only ever set)
                }
            }
        }
        // Did any wait of this CTA run out?  Then rows of the chunk were never seen: report it, wait once more
        // (with the full limit) for the copies still on their way into this CTA's shared memory, which is not
        // touched until then, and mark the image: it will pass through unpruned.
        const int unseen = __syncthreads_or((gave_up || (tid == 0 && s_unseen)) ? 1 : 0);
        if (bad && lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_NONFINITE);
        if (unseen) {
            if (tid == 0) {
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                for (int s = 0; s < nstage; ++s) {
                    // the last copy issued into stage s (an earlier one has completed: its barrier was waited for
                    // before the stage was refilled)
                    const int last = issued - 1 - ((issued - 1 - s) % nstage + nstage) % nstage;
                    if (issued > s && last >= 0) (void)ptx::mbar_wait(&s_full[s], (last / nstage) & 1);
                }
                atomicOr(&img_done[img], 0x80000000u);
            }
            __syncthreads();
        } else {
            // the ring is free: it now holds the warps' partial sums, reduced through shared memory
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = lane + 32 * j;
                if (vi < nvec) {
#pragma unroll
                    for (int e = 0; e < EPV; ++e) s_dyn[warp * d + vi * EPV + e] = acc[j * EPV + e];
                }
            }
            __syncthreads();
            float *out = spart + ((size_t)img * chunks + chunk) * d;
            for (int c = tid; c < d; c += kS1Threads) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kS1Warps; ++w) s += s_dyn[w * d + c];
                out[c] = s;
            }
        }

        // the CTA that completes the image selects its tokens
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const uint32_t nchunk = (uint32_t)((n_img + chunk_tokens - 1) / chunk_tokens);
            const uint32_t prev = atomicAdd(&img_done[img], 1u);      // (after this CTA's own mark, if it set one)
            s_last = ((prev & 0x7fffffffu) == nchunk - 1u);
            s_unseen = (prev & 0x80000000u) != 0u;
            if (s_last) img_done[img] = 0;       // ready for the next run
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        if (s_unseen) {
            // some chunk of the image was never read (reported above): the image passes through unpruned
            for (int k = tid; k < n_img; k += kS1Threads) {
                order[t_begin + k] = k;
                kpos[t_begin + k] = k;
                if (order_out) order_out[t_begin + k] = k;
                if (norms_out) norms_out[t_begin + k] = 0.f;
            }
            if (tid == 0) {
                counts[img] = n_img;
                float *st = stats + (size_t)img * kStats;
                for (int q = 0; q < kStats; ++q) st[q] = 0.f;
                st[3] = (float)n_img;
            }
            __syncthreads();
        } else {
            select_image(img, t_begin, n_img, d, chunks, chunk_tokens, rp, rho, critv, spart, order, kpos, counts, stats,
                         norms_out, order_out, reinterpret_cast<uint32_t *>(s_dyn));
        }
    }

    // the CTA that completes the batch: out_offsets = exclusive prefix sum of counts (unless a kernel
    // that follows does it, off the path of the last image's selection)
    if (!scan_here) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const uint32_t prev = atomicAdd(&hdr->select_done, 1u);
        s_last = (prev == (uint32_t)batch - 1u);
        if (s_last) hdr->select_done = 0;        // ready for the next run
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    scan_counts<kS1Threads>(counts, out_offsets, batch, s_scan);
}

// ---------------------------------------------------------------------------------------------
// Compact copy of T_prop for the tensor-core kernels (bf16 storage): image i's B pruned rows, in
// ascending token order, at rows xp_row0(offsets[i], i) .., then rows of zeros up to a multiple of
// 64 so that whole 64-row tiles can be fetched.  grid = (ceil(max rows / 8), batch), 128 threads:
// a warp copies two rows, all loads of a row issued before the stores.
// ---------------------------------------------------------------------------------------------
constexpr int kGpRows = 8;     // rows per CTA: four warps, two rows each
__global__ void __launch_bounds__(128)
gather_prop_kernel(const __nv_bfloat16 *__restrict__ Xb, const int32_t *__restrict__ offsets,
                   const int32_t *__restrict__ counts, const int32_t *__restrict__ order, int d,
                   int max_tokens, int total, __nv_bfloat16 *__restrict__ xp, uint32_t *__restrict__ sink_done,
                   int32_t *__restrict__ ready_list, WsHeader *__restrict__ hdr, int batch,
                   int32_t *__restrict__ out_offsets, uint32_t *__restrict__ scores_done)
{
    __shared__ int s_scan[32];
    const int img = blockIdx.y;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();     // counts and order come from the kernel ahead
    // One CTA prepares what the kernels behind this one share through the workspace, while the others
    // copy: it empties the per-image counters and the list of finished plans, then publishes the run's
    // number.  Kernels launched as programmatic dependents may already be resident and must not read
    // those words before they see that number: until then they hold what the run before left.  (That
    // run has ended: it is ahead of stage 1 in the stream.)  It also turns the counts into out_offsets.
    if (blockIdx.x == 0 && img == 0) {
        for (int i = threadIdx.x; i < batch; i += 128) {
            sink_done[i] = 0;
            scores_done[i] = 0;
            ready_list[i] = 0;
        }
        if (threadIdx.x == 0) {
            hdr->n_ready = 0;
            hdr->merge_next = 0;
        }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) ptx::st_release_gpu(&hdr->run_tag, ptx::ld_acquire_gpu(&hdr->launch_seq));
        scan_counts<128>(counts, out_offsets, batch, s_scan);
    }
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M, Bpad = (B + 63) & ~63;
    const int j0 = blockIdx.x * kGpRows + (threadIdx.x >> 5) * 2;
    if (j0 >= Bpad) return;
    const int lane = threadIdx.x & 31;
    const int nvec = d >> 3;
    uint4 *seg = reinterpret_cast<uint4 *>(xp + (size_t)xp_row0(t_begin, img) * d);
    int src_row[2];
#pragma unroll
    for (int a = 0; a < 2; ++a)
        src_row[a] = (j0 + a < B) ? t_begin + __ldg(order + t_begin + M + j0 + a) : -1;
    for (int v0 = lane; v0 < nvec; v0 += 32 * 5) {
        uint4 t[2][5];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 5; ++b) {
                const int v = v0 + 32 * b;
                t[a][b] = (src_row[a] >= 0 && v < nvec)
                              ? __ldg(reinterpret_cast<const uint4 *>(Xb + (size_t)src_row[a] * d) + v)
                              : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 5; ++b) {
                const int v = v0 + 32 * b;
                if (j0 + a < Bpad && v < nvec) seg[(size_t)(j0 + a) * nvec + v] = t[a][b];
            }
    }
}

}  // namespace rtp
