// The transport problem of Eq. 2-6 solved exactly, one CTA per image.  With the dustbins of Eq. 5 the linear
// program is a maximum-weight partial matching between kept and pruned tokens whose pair (i, j) gains
// S_ij - z over leaving both in the dustbins; a vertex of the polytope pairs every token at most once.  The
// kernel finds it by shortest augmenting paths on the gains clipped at zero (a pair of clipped gain 0 is left
// unpaired afterwards).  The smaller side are the rows.  Start: every row's price is its best gain and rows
// whose best column nobody smaller wants take it (those edges are tight).  Then, for every row still free, a
// shortest-path search over the columns in the reduced costs: every thread owns fixed columns and keeps their
// distances, predecessors and marks to itself, so a step is one relaxation of the own columns against the
// column reached last plus one block-wide minimum (ties to the lower index): ONE block barrier per step.  The
// prices move once per search, after the free column is found (columns in the tree by their distance to it,
// rows from the tightness of their own edge), never during it.
//
// Outputs: the pairs (merge_partner = kept position or -1, merge_weight = 1 or 0) and the plan of zeros and
// ones that Eq. 7 then uses as it uses Sinkhorn's: alpha at the paired cells of the bf16 plan buffer, or 1 in
// place in the fp32 workspace tile.  stats[5] = search steps taken, stats[6] = rows the start assigned.
#pragma once
#include "common.cuh"
#include "sinkhorn.cuh"

namespace rtp {

constexpr int kExThreads = 512;
constexpr int kExWarps = kExThreads / 32;

// Words of shared memory the search arrays take for images of at most max_tokens tokens: two prices, the
// distances, the assignment by column and by row and the path links (a word per token each) and the marks (a
// byte per token): 205 KB at the plan's limit of 8192 tokens.
__host__ __device__ inline size_t exact_array_words(int max_tokens)
{
    const size_t cap = (size_t)(max_tokens + 8);
    return 6 * cap + (cap + 3) / 4;       // six arrays of words and the marks, a byte each
}

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
    __shared__ int s_started;
    const int img = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0) return;
    const bool transposed = B > M;            // rows of the assignment = the smaller side
    const int n = transposed ? M : B, m = transposed ? B : M;
    const int cap = max_tokens + 8;
    float *u = sm;                            // [n]   prices of the rows
    float *v = u + cap;                       // [m]   prices of the columns
    float *dist = v + cap;                    // [m]   shortest reduced-cost distance found for each column in this search
    int *asg = reinterpret_cast<int *>(dist + cap);   // [m] row assigned to each column, -1: free
    int *way = asg + cap;                     // [m]   column the search reached this column from (m: the free row itself)
    int *rowcol = way + cap;                  // [n]   column assigned to each row, -1: free
    unsigned char *used = reinterpret_cast<unsigned char *>(rowcol + cap);   // [m] column is in the search tree
    float *gains = reinterpret_cast<float *>(sm + exact_array_words(max_tokens));
    const bool staged = (long long)n * m <= (long long)smem_words - (long long)exact_array_words(max_tokens);

    float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ldS = score_pitch(B);
    const float z = prm.z;
    // clipped gain of row r, column c (the cost of the assignment problem is its negative)
    auto gain_global = [&](int r, int c) -> float {
        const float s = transposed ? __ldcg(Sg + (size_t)r * ldS + c) : __ldcg(Sg + (size_t)c * ldS + r);
        return fmaxf(s - z, 0.f);
    };
    if (staged)
        for (int idx = tid; idx < n * m; idx += kExThreads) {
            const int r = idx / m, c = idx - r * m;
            gains[idx] = gain_global(r, c);
        }
    for (int c = tid; c < m; c += kExThreads) {
        v[c] = 0.f;
        asg[c] = 0x7fffffff;
    }
    if (tid == 0) s_started = 0;
    __syncthreads();
    auto gain_of = [&](int r, int c) -> float { return staged ? gains[(size_t)r * m + c] : gain_global(r, c); };

    // ---- start: u_r = -(best gain of row r); the row takes its best column (lowest index on ties) if no
    // lower row wants the same one.  Reduced costs -g - u_r - 0 are >= 0, and 0 on the edges taken.
    for (int r = warp; r < n; r += kExWarps) {
        float best = -1.f;
        int bc = 0x7fffffff;
        for (int c = lane; c < m; c += 32) {
            const float g = gain_of(r, c);
            if (g > best) {
                best = g;
                bc = c;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oc = __shfl_xor_sync(0xffffffffu, bc, o);
            if (ob > best || (ob == best && oc < bc)) {
                best = ob;
                bc = oc;
            }
        }
        if (lane == 0) {
            u[r] = -best;
            way[r] = bc;                      // (scratch until the searches begin)
            if (bc < m) atomicMin(&asg[bc], r);
        }
    }
    __syncthreads();
    int started = 0;
    for (int r = tid; r < n; r += kExThreads) {
        const int bc = way[r];
        const bool won = bc < m && asg[bc] == r;
        rowcol[r] = won ? bc : -1;
        started += won ? 1 : 0;
    }
    if (started) atomicAdd(&s_started, started);
    __syncthreads();
    for (int c = tid; c < m; c += kExThreads)
        if (asg[c] == 0x7fffffff) asg[c] = -1;
    __syncthreads();

    int steps = 0;
    bool broken = false;                      // a non-finite score: no minimum exists (uniform over the CTA)
    for (int row = 0; row < n && !broken; ++row) {
        if (rowcol[row] >= 0) continue;       // (uniform: every thread reads the same word)
        // distances from the free row; every thread touches only its own columns until the path is flipped
        const float urow = u[row];
        float lbest = INFINITY;
        int lj = 0x7fffffff;
        for (int c = tid; c < m; c += kExThreads) {
            const float dc = -gain_of(row, c) - urow - v[c];
            dist[c] = dc;
            way[c] = m;
            used[c] = 0;
            if (dc < lbest) {                 // c ascends within a thread: strict < keeps the lower column
                lbest = dc;
                lj = c;
            }
        }
        int sink = -1;
        float mu = 0.f;
        // each step puts one more column into the tree and at most `row` of them are taken: the search ends
        for (int guard = 0; guard <= m; ++guard) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, lbest, o);
                const int oj = __shfl_xor_sync(0xffffffffu, lj, o);
                if (ob < lbest || (ob == lbest && oj < lj)) {
                    lbest = ob;
                    lj = oj;
                }
            }
            const int par = steps & 1;
            if (lane == 0) {
                s_val[par][warp] = lbest;
                s_idx[par][warp] = lj;
            }
            __syncthreads();
            float dmin = s_val[par][0];
            int jstar = s_idx[par][0];
#pragma unroll
            for (int w = 1; w < kExWarps; ++w) {
                const float ob = s_val[par][w];
                const int oj = s_idx[par][w];
                if (ob < dmin || (ob == dmin && oj < jstar)) {
                    dmin = ob;
                    jstar = oj;
                }
            }
            ++steps;
            if (jstar == 0x7fffffff) {
                broken = true;
                break;
            }
            mu = dmin;
            const int i2 = asg[jstar];
            if (i2 < 0) {                     // a free column: the shortest path ends here
                sink = jstar;
                break;
            }
            // relax the own columns against the row of the column just reached, and find the next minimum
            const float base = dmin - u[i2];
            lbest = INFINITY;
            lj = 0x7fffffff;
            for (int c = tid; c < m; c += kExThreads) {
                if (c == jstar) used[c] = 1;
                if (used[c]) continue;
                const float nd = base - gain_of(i2, c) - v[c];
                float dc = dist[c];
                if (nd < dc) {
                    dc = nd;
                    dist[c] = nd;
                    way[c] = jstar;
                }
                if (dc < lbest) {
                    lbest = dc;
                    lj = c;
                }
            }
        }
        if (broken || sink < 0) {
            broken = true;
            break;
        }
        // prices of the tree's columns (own columns), while one thread flips the path back to the free row
        for (int c = tid; c < m; c += kExThreads)
            if (used[c]) v[c] += dist[c] - mu;
        if (tid == 0) {
            int c = sink;
            for (int guard = 0; guard <= m; ++guard) {
                const int prev = way[c];
                if (prev >= m) {
                    asg[c] = row;
                    rowcol[row] = c;
                    break;
                }
                const int r = asg[prev];
                asg[c] = r;
                rowcol[r] = c;
                c = prev;
            }
        }
        __syncthreads();
        // prices of the tree's rows from the tightness of the edges they now hold
        for (int c = tid; c < m; c += kExThreads)
            if (used[c] || c == sink) {
                const int r = asg[c];
                u[r] = -gain_of(r, c) - v[c];
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
        stats[(size_t)img * kStats + 6] = (float)s_started;
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
