// The transport problem of Eq. 2-6 solved exactly, one CTA per image.  With the dustbins of Eq. 5 the linear
// program is a maximum-weight partial matching between kept and pruned tokens whose pair (i, j) gains
// S_ij - z over leaving both in the dustbins; a vertex of the polytope pairs every token at most once.  The
// kernel finds it by shortest augmenting paths on the gains clipped at zero (a pair of clipped gain 0 is left
// unpaired afterwards), the smaller side being the one whose tokens are inserted one by one.  Every step of a
// path search is one pass of the CTA over the other side: relax the reduced costs against the token reached
// last, take the block-wide minimum (ties to the lower index), shift the potentials by it.
//
// Outputs: the pairs (merge_partner = kept position or -1, merge_weight = 1 or 0) and the plan of zeros and
// ones that Eq. 7 then uses as it uses Sinkhorn's: alpha at the paired cells of the bf16 plan buffer, or 1 in
// place in the fp32 workspace tile.  stats[5] = path-search steps taken, stats[6] = 0.
#pragma once
#include "common.cuh"
#include "sinkhorn.cuh"

namespace rtp {

constexpr int kExThreads = 512;
constexpr int kExWarps = kExThreads / 32;

// Words of shared memory the search arrays take for images of at most max_tokens tokens: two potentials, the
// reduced-cost minima, the assignment, the path links and the visited marks, each of at most max_tokens + 1.
__host__ __device__ inline size_t exact_array_words(int max_tokens) { return 6 * (size_t)(max_tokens + 8); }

// Dynamic shared memory of a launch: the arrays, then as many clipped gains as the limit leaves (an image
// whose n x m gains fit keeps them there, the others read the workspace tile at every step).
__host__ inline size_t exact_smem_bytes(int max_tokens, size_t limit)
{
    const size_t arrays = 4 * exact_array_words(max_tokens);
    const size_t half = (size_t)(max_tokens + 1) / 2;
    const size_t gains = 4 * half * ((size_t)max_tokens - half + 1);
    return arrays + gains <= limit ? arrays + gains : limit;
}

__global__ void __launch_bounds__(kExThreads)
exact_pairing_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                     const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                     float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams prm,
                     int smem_words, __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch,
                     int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                     float *__restrict__ merge_weight, float *__restrict__ stats, WsHeader *__restrict__ hdr)
{
    extern __shared__ __align__(16) float sm[];
    __shared__ float s_val[2][kExWarps];
    __shared__ int s_idx[2][kExWarps];
    const int img = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0) return;
    const bool transposed = B > M;            // rows of the assignment = the smaller side
    const int n = transposed ? M : B, m = transposed ? B : M;
    const int cap = max_tokens + 8;
    float *u = sm;                            // [n]   potentials of the rows
    float *v = u + cap;                       // [m+1] potentials of the columns (column m: the root of a search)
    float *minv = v + cap;                    // [m+1] smallest reduced cost seen for each column in this search
    int *asg = reinterpret_cast<int *>(minv + cap);   // [m+1] row assigned to each column, -1: free
    int *way = asg + cap;                     // [m+1] column the search reached this column from
    int *used = way + cap;                    // [m+1] column is in the search tree
    float *gains = reinterpret_cast<float *>(used + cap);
    const bool staged = (long long)n * m <= (long long)smem_words - (long long)exact_array_words(max_tokens);

    float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ldS = score_pitch(B);
    const float z = prm.z;
    // clipped gain of row r, column c
    auto gain_of = [&](int r, int c) -> float {
        const float s = transposed ? __ldcg(Sg + (size_t)r * ldS + c) : __ldcg(Sg + (size_t)c * ldS + r);
        return fmaxf(s - z, 0.f);
    };
    if (staged)
        for (int idx = tid; idx < n * m; idx += kExThreads) {
            const int r = idx / m, c = idx - r * m;
            gains[idx] = gain_of(r, c);
        }
    for (int r = tid; r < n; r += kExThreads) u[r] = 0.f;
    for (int c = tid; c <= m; c += kExThreads) {
        v[c] = 0.f;
        asg[c] = -1;
    }
    __syncthreads();

    int steps = 0;
    bool broken = false;                      // a non-finite score: no minimum exists (uniform over the CTA)
    for (int row = 0; row < n && !broken; ++row) {
        for (int c = tid; c < m; c += kExThreads) {
            minv[c] = INFINITY;
            used[c] = 0;
        }
        if (tid == 0) {
            used[m] = 1;
            asg[m] = row;
        }
        __syncthreads();
        int j0 = m;
        // each step puts one more column into the tree and there are m of them: the search ends within m steps
        for (int guard = 0; guard <= m; ++guard) {
            const int i0 = asg[j0];
            const float ui0 = u[i0];
            const float *grow = gains + (size_t)i0 * m;
            float best = INFINITY;
            int bj = 0x7fffffff;
            for (int c = tid; c < m; c += kExThreads) {
                if (used[c]) continue;
                const float g = staged ? grow[c] : gain_of(i0, c);
                const float cur = -g - ui0 - v[c];
                float mv = minv[c];
                if (cur < mv) {
                    mv = cur;
                    minv[c] = cur;
                    way[c] = j0;
                }
                if (mv < best) {              // c ascends within a thread: strict < keeps the lower column
                    best = mv;
                    bj = c;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
                if (ob < best || (ob == best && oj < bj)) {
                    best = ob;
                    bj = oj;
                }
            }
            const int par = steps & 1;
            if (lane == 0) {
                s_val[par][warp] = best;
                s_idx[par][warp] = bj;
            }
            __syncthreads();
            float delta = s_val[par][0];
            int j1 = s_idx[par][0];
#pragma unroll
            for (int w = 1; w < kExWarps; ++w) {
                const float ob = s_val[par][w];
                const int oj = s_idx[par][w];
                if (ob < delta || (ob == delta && oj < j1)) {
                    delta = ob;
                    j1 = oj;
                }
            }
            ++steps;
            if (j1 == 0x7fffffff) {
                broken = true;
                break;
            }
            for (int c = tid; c <= m; c += kExThreads) {
                if (used[c]) {
                    u[asg[c]] += delta;       // the rows of the tree's columns are distinct
                    v[c] -= delta;
                } else {
                    minv[c] -= delta;
                }
                if (c == j1) used[c] = 1;
            }
            __syncthreads();
            j0 = j1;
            if (asg[j0] < 0) break;           // a free column: the path is complete
        }
        if (broken) break;
        if (tid == 0) {
            // flip the path back to the root
            int c = j0;
            for (int guard = 0; guard <= m && c != m; ++guard) {
                const int prev = way[c];
                asg[c] = asg[prev];
                c = prev;
            }
        }
        __syncthreads();
    }

    // pairs by pruned token, in `way` (free now): kept position, or -1
    int *match = way;
    __syncthreads();
    for (int j = tid; j < B; j += kExThreads) match[j] = -1;
    __syncthreads();
    if (!broken) {
        for (int c = tid; c < m; c += kExThreads) {
            const int r = asg[c];
            if (r < 0) continue;
            const int i = transposed ? r : c, j = transposed ? c : r;
            if (__ldcg(Sg + (size_t)i * ldS + j) - z > 0.f) match[j] = i;   // clipped gain 0: both stay unpaired
        }
    } else if (tid == 0) {
        atomicOr(&hdr->status, RTPRUNE_DEV_NONFINITE);
    }
    __syncthreads();

    const int seg = t_begin - out_offsets[img];
    const int32_t *ord = order + t_begin;
    for (int j = tid; j < B; j += kExThreads) {
        merged_idx[seg + j] = ord[M + j];
        merge_partner[seg + j] = match[j];
        merge_weight[seg + j] = match[j] >= 0 ? 1.f : 0.f;
    }
    if (tid == 0) {
        stats[(size_t)img * kStats + 5] = (float)steps;
        stats[(size_t)img * kStats + 6] = 0.f;
    }

    if (pbuf) {
        // alpha P in bf16: rows by the kept token's position in X, columns up to the next multiple of 64
        const int kpad = (B + 63) & ~63;
        const int vec_per_row = kpad >> 3;
        __nv_bfloat16 *Pimg = pbuf + (size_t)t_begin * pbuf_pitch;
        for (int idx = tid; idx < M * vec_per_row; idx += kExThreads) {
            const int i = idx / vec_per_row, q = idx - i * vec_per_row;
            *reinterpret_cast<uint4 *>(Pimg + (size_t)ord[i] * pbuf_pitch + 8 * q) = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        const __nv_bfloat16 a = __float2bfloat16_rn(prm.alpha);
        for (int j = tid; j < B; j += kExThreads)
            if (match[j] >= 0) Pimg[(size_t)ord[match[j]] * pbuf_pitch + j] = a;
    } else {
        // fp32: the plan in place of the scores in the workspace tile (every read of S is behind the barrier above)
        for (int idx = tid; idx < M * B; idx += kExThreads) {
            const int i = idx / B, j = idx - i * B;
            Sg[(size_t)i * ldS + j] = match[j] == i ? 1.f : 0.f;
        }
    }
}

}  // namespace rtp
