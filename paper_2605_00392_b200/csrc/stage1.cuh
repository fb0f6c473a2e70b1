// Stage 1 of Algorithm 1: token norms (Eq. 1), the similarity statistic phi (Eq. 8), the pruning
// ratio (Eq. 10) and the top-M selection (Section 3.3.1).
#pragma once
#include "common.cuh"

namespace rtp {

// ---------------------------------------------------------------------------------------------
// Kernel (a1)+(d): one streaming pass over X.  grid = (chunks, batch), 256 threads.
// A warp owns a token at a time: 128-bit loads, fp32 sum of squares, shuffle reduction.  While the
// row is still in registers it is added, divided by its norm, into per-lane accumulators; the CTA
// then writes the partial sum of unit tokens of its chunk to spart[img][chunk][d].
// phi needs only |sum_k x_k/||x_k|| |^2:  sum_{k<l} cos(x_k, x_l) = (|sum_k xhat_k|^2 - N) / 2.
// ---------------------------------------------------------------------------------------------
template <typename T, int VPL>  // VPL = 16-byte vectors per lane = ceil(d / (32 * kPerVec))
__global__ void __launch_bounds__(256)
norm_stats_kernel(const T *__restrict__ X, const int32_t *__restrict__ offsets, int d, int chunks,
                  int max_tokens, int total, float *__restrict__ norms, float *__restrict__ spart,
                  WsHeader *__restrict__ hdr)
{
    constexpr int EPV = Elem<T>::kPerVec;
    extern __shared__ float s_red[];  // [8 warps][d]
    const int img = blockIdx.y, chunk = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int t_begin, n_img;
    if (!image_range(offsets, img, max_tokens, total, t_begin, n_img)) return;
    const int t_end = t_begin + n_img;
    const int t0 = t_begin + chunk * kChunkTokens;
    if (t0 >= t_end) return;
    const int t1 = min(t0 + kChunkTokens, t_end);
    const int nvec = d / EPV;

    float acc[VPL * EPV];
#pragma unroll
    for (int i = 0; i < VPL * EPV; ++i) acc[i] = 0.f;
    bool bad = false;

    for (int t = t0 + warp; t < t1; t += 8) {
        const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)t * d);
        uint4 v[VPL];
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int vi = lane + 32 * j;
            v[j] = (vi < nvec) ? __ldg(row + vi) : make_uint4(0, 0, 0, 0);
        }
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            float f[EPV];
            Elem<T>::unpack(v[j], f);
#pragma unroll
            for (int e = 0; e < EPV; ++e) ss = fmaf(f[e], f[e], ss);
        }
        ss = warp_sum(ss);
        const float n = sqrtf(ss);
        if (!(ss <= 3.0e38f)) bad = true;  // inf or NaN
        const float inv = 1.f / fmaxf(n, kNormFloor);
        if (lane == 0) norms[t] = n;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            float f[EPV];
            Elem<T>::unpack(v[j], f);
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[j * EPV + e] = fmaf(f[e], inv, acc[j * EPV + e]);
        }
    }
    if (bad && lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_NONFINITE);

    // reduce the 8 warps' accumulators through shared memory
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int vi = lane + 32 * j;
        if (vi < nvec) {
#pragma unroll
            for (int e = 0; e < EPV; ++e) s_red[warp * d + vi * EPV + e] = acc[j * EPV + e];
        }
    }
    __syncthreads();
    float *out = spart + ((size_t)img * chunks + chunk) * d;
    for (int c = threadIdx.x; c < d; c += 256) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += s_red[w * d + c];
        out[c] = s;
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel (a2)-(a4): one CTA per image, 1024 threads.
//   phi from the chunk partials; r and B = floor(r N + 1/2) clamped to [0, N-1], M = N - B;
//   rank of every token under (norm descending, index ascending) by counting; the M best are
//   T_kept.  Writes order[] = kept indices ascending, then pruned indices ascending, and its
//   inverse kpos[]; counts, stats; for bf16 storage also the compact copy of T_prop's rows;
//   the last CTA to finish turns counts into out_offsets (exclusive prefix sum).
// Shared memory: float keys[max_tokens] (dynamic) + static scratch.
// ---------------------------------------------------------------------------------------------
struct RatioParams {
    int dynamic;
    float r_fixed, phi_lo, phi_hi, r_max;
};

__global__ void __launch_bounds__(1024)
select_kernel(const int32_t *__restrict__ offsets, int batch, int d, int chunks, int max_tokens,
              int total, RatioParams rp, const float *__restrict__ rho, const float *__restrict__ norms,
              const float *__restrict__ spart, int32_t *__restrict__ order,
              int32_t *__restrict__ kpos, int32_t *__restrict__ counts, int32_t *__restrict__ out_offsets,
              float *__restrict__ stats, float *__restrict__ norms_out,
              int32_t *__restrict__ order_out, WsHeader *__restrict__ hdr,
              const __nv_bfloat16 *__restrict__ Xb, __nv_bfloat16 *__restrict__ xp)
{
    extern __shared__ uint32_t s_keys[];  // norm bits: for non-negative floats the unsigned order
    __shared__ float s_redf[32];          // is the float order, and a NaN still ranks somewhere
    __shared__ int s_redi[32];
    __shared__ int s_M;
    __shared__ bool s_last;
    const int img = blockIdx.x, tid = threadIdx.x, nth = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5;
    int t_begin, N;
    const bool valid = image_range(offsets, img, max_tokens, total, t_begin, N);
    int M = 0;

    if (valid) {
        // phi (Eq. 8) via |sum of unit tokens|^2
        const int nchunk = (N + kChunkTokens - 1) / kChunkTokens;
        const float *sp = spart + (size_t)img * chunks * d;
        float local = 0.f;
        for (int c = tid; c < d; c += nth) {
            float s = 0.f;
            for (int k = 0; k < nchunk; ++k) s += sp[(size_t)k * d + c];
            local = fmaf(s, s, local);
        }
        const float ssum = block_sum(local, s_redf);
        if (tid == 0) {
            const float Nf = (float)N;
            const float phi = (N >= 2) ? (ssum - Nf) / (Nf * (Nf - 1.f)) : 0.f;
            const float rho_i = rho ? rho[img] : 0.f;
            float r;
            if (rp.dynamic) {
                float f = (phi - rp.phi_lo) / (rp.phi_hi - rp.phi_lo);
                f = fminf(fmaxf(f, 0.f), 1.f);
                r = fminf(f * (1.f - rho_i), rp.r_max);
            } else {
                r = rp.r_fixed;
            }
            r = fmaxf(r, 0.f);
            int B = (int)floorf(r * Nf + 0.5f);
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
        for (int k = tid; k < N; k += nth) {
            const float key = norms[t_begin + k];
            s_keys[k] = __float_as_uint(key) & 0x7fffffffu;
            if (norms_out) norms_out[t_begin + k] = key;
        }
        __syncthreads();
        M = s_M;

        // Each thread owns a contiguous range of tokens so that a block scan of its kept count
        // gives output positions in ascending index.
        const int ipt = (N + nth - 1) / nth;
        const int k0 = min(tid * ipt, N), k1 = min(k0 + ipt, N);
        uint32_t keptmask = 0;  // ipt <= 8 for N <= 8192
        int nkept = 0;
        for (int k = k0; k < k1; ++k) {
            const uint32_t my = s_keys[k];
            int rank = 0;
            for (int l = 0; l < N; ++l) {
                const uint32_t o = s_keys[l];
                rank += (o > my || (o == my && l < k)) ? 1 : 0;
            }
            if (rank < M) {
                keptmask |= 1u << (k - k0);
                ++nkept;
            }
        }
        // exclusive block scan of nkept
        int incl = nkept;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_redi[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = (lane < (nth >> 5)) ? s_redi[lane] : 0;
            int wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += t;
            }
            s_redi[lane] = wi - w;
        }
        __syncthreads();
        int kpos_run = s_redi[warp] + incl - nkept;  // kept tokens before k0
        int32_t *ord = order + t_begin;
        for (int k = k0; k < k1; ++k) {
            const bool kept = (keptmask >> (k - k0)) & 1u;
            const int pos = kept ? kpos_run : (M + (k - kpos_run));
            ord[pos] = k;
            kpos[t_begin + k] = kept ? kpos_run : -1 - (k - kpos_run);
            if (order_out) order_out[t_begin + pos] = k;
            kpos_run += kept ? 1 : 0;
        }

        // compact copy of T_prop for the tensor-core kernels (bf16 storage): a warp per row, then rows
        // of zeros up to a multiple of 64 so that whole 64-row tiles can be fetched
        if (xp != nullptr && M < N) {
            __syncthreads();                      // this CTA's writes to ord[] are visible to it
            const int B = N - M, Bpad = (B + 63) & ~63;
            const int nvec = d >> 3;
            uint4 *seg = reinterpret_cast<uint4 *>(xp + (size_t)xp_row0(t_begin, img) * d);
            for (int j = warp; j < Bpad; j += (nth >> 5)) {
                uint4 *dst = seg + (size_t)j * nvec;
                if (j < B) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(Xb + (size_t)(t_begin + ord[M + j]) * d);
                    for (int v0 = lane; v0 < nvec; v0 += 128) {
                        uint4 t[4];
#pragma unroll
                        for (int a = 0; a < 4; ++a)
                            t[a] = (v0 + 32 * a < nvec) ? __ldg(src + v0 + 32 * a) : make_uint4(0, 0, 0, 0);
#pragma unroll
                        for (int a = 0; a < 4; ++a)
                            if (v0 + 32 * a < nvec) dst[v0 + 32 * a] = t[a];
                    }
                } else {
                    for (int v = lane; v < nvec; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
                }
            }
        }
    } else if (tid == 0) {
        atomicOr(&hdr->status, RTPRUNE_DEV_BAD_OFFSETS);  // offsets broke the contract: the image yields no output
        counts[img] = 0;
        float *st = stats + (size_t)img * kStats;
        for (int q = 0; q < kStats; ++q) st[q] = 0.f;
    }

    // last CTA: out_offsets = exclusive prefix sum of counts
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const uint32_t prev = atomicAdd(&hdr->select_done, 1u);
        s_last = (prev == (uint32_t)batch - 1u);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) hdr->select_done = 0;  // ready for the next run
    const int ipt2 = (batch + nth - 1) / nth;
    const int b0 = min(tid * ipt2, batch), b1 = min(b0 + ipt2, batch);
    int sum = 0;
    for (int b = b0; b < b1; ++b) sum += __ldcg(counts + b);
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_redi[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < (nth >> 5)) ? s_redi[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        s_redi[lane] = wi - w;
    }
    __syncthreads();
    int run = s_redi[warp] + incl - sum;
    for (int b = b0; b < b1; ++b) {
        out_offsets[b] = run;
        run += __ldcg(counts + b);
    }
    if (tid == nth - 1) out_offsets[batch] = run;  // the last thread's running sum is the total
}

}  // namespace rtp
