// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C), one CTA per
// image.  The (M+1) x (B+1) matrix stays in shared memory across all iterations when it fits, else
// it is iterated in place in the image's L2-resident workspace tile.
#pragma once
#include "common.cuh"

namespace rtp {

struct OtParams {
    float z, alpha, eps;
    int iters;
    int stop_fp;
    float tol;
};

constexpr int kSinkThreads = 512;

constexpr int kSfThreads = 512;
constexpr int kSfWarps = kSfThreads / 32;
constexpr int kSfMaxNc = 20;           // the cluster kernel takes tiles of at most 32 * 20 columns

// Row pitch (floats) of K in the cluster kernel (sinkhorn_cluster.cuh): the widths its lane layouts cover.
__host__ __device__ inline int sinkhorn_ldk(int B)
{
    if (B <= 128) return B <= 32 ? 32 : (B <= 64 ? 64 : 128);
    if (B <= 256) return B <= 192 ? 192 : 256;
    return B <= 384 ? 384 : (B <= 512 ? 512 : 640);
}
// Shared-memory floats one CTA of the cluster kernel needs for an M x B tile split over C CTAs, K
// aside: per-warp and per-CTA partials of the column sums (the same space serves the pairing), duals,
// token positions, scratch.
__host__ __device__ inline long long sinkhorn_cluster_aux_floats(int M, int B, int C)
{
    const long long ldk = sinkhorn_ldk(B);
    const long long rows_per = (M + C - 1) / C;
    return 2 * kSfWarps * ldk + 2 * C * ldk + 2 * (rows_per + 8) + (ldk + 4) + kSfWarps + 16 + 16;
}
// The same with the CTA's rows of K (padded to the pitch) in shared memory too.
__host__ __device__ inline long long sinkhorn_cluster_floats(int M, int B, int C)
{
    const long long rows_per = (M + C - 1) / C;
    return rows_per * sinkhorn_ldk(B) + sinkhorn_cluster_aux_floats(M, B, C);
}
// K fits the cluster's shared memory.
__host__ __device__ inline bool sinkhorn_cluster_fits(int M, int B, int C, int smem_floats)
{
    return B >= 1 && B <= 32 * kSfMaxNc && sinkhorn_cluster_floats(M, B, C) <= (long long)smem_floats;
}
// The cluster kernel solves the tile: with K in shared memory if it fits, else in the workspace tile.
__host__ __device__ inline bool sinkhorn_cluster_handles(int M, int B, int C, int smem_floats)
{
    return B >= 1 && B <= 32 * kSfMaxNc && sinkhorn_cluster_aux_floats(M, B, C) <= (long long)smem_floats;
}

// True if two positive floats differ by more than one unit in the last place.
__device__ inline bool ulp_far(float a, float b)
{
    const int d = (int)__float_as_uint(a) - (int)__float_as_uint(b);
    return d > 1 || d < -1;
}

__device__ inline void lse_merge(float &m, float &s, float m2, float s2)
{
    const float mm = fmaxf(m, m2);
    if (mm == -INFINITY) {
        s = 0.f;
        m = mm;
        return;
    }
    s = s * expf(m - mm) + s2 * expf(m2 - mm);
    m = mm;
}

// LOG = true : Z_ij = S-bar_ij / eps, duals u, v in the log domain,
//              u_i = log mu_i - LSE_j(Z_ij + v_j), v_j = log nu_j - LSE_i(Z_ij + u_i).
// LOG = false: K_ij = exp((S-bar_ij - c)/eps), c = max(1, z); duals carried as U = e^u and
//              V = e^{v + c/eps} (V starts at e^{c/eps}, i.e. v = 0), so that U K V = exp(Z + u + v)
//              after any number of iterations, zero included:
//              U_i = mu_i / sum_j K_ij V_j, V_j = nu_j / sum_i K_ij U_i.
// mu = [1_M, B], nu = [1_B, M].  Plan: P_ij = U_i K_ij V_j  (= exp(Z_ij + u_i + v_j)).
template <bool LOG>
__global__ void __launch_bounds__(kSinkThreads)
sinkhorn_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                int smem_floats, __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch,
                int32_t *__restrict__ merged_idx,
                int32_t *__restrict__ merge_partner, float *__restrict__ merge_weight,
                float *__restrict__ stats, int fast_cluster, int fast_smem_floats, int tall_max_b)
{
    extern __shared__ __align__(16) float sm[];
    __shared__ float s_red[32];
    const int img = blockIdx.x, tid = threadIdx.x;
    constexpr int nth = kSinkThreads;
    const int lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = nth / 32;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0) return;
    // images the cluster kernel launched before this one takes were solved there
    if (fast_cluster > 0 && sinkhorn_cluster_handles(M, B, fast_cluster, fast_smem_floats)) return;
    if (B <= tall_max_b) return;     // solved by the kernel for wide tiles (sinkhorn_tall.cuh)
    const int R = M + 1, Cc = B + 1;

    float *u = sm;
    float *v = u + R;
    float *part = v + Cc;                       // [2][nth]: partial column results and a second lane
    constexpr int part_floats = 2 * nth;        // (running maxima for LOG, indices for the pairing)
    float *Ks = part + part_floats;
    const int lds = Cc | 1;                     // odd row stride: conflict-free column walks
    const bool in_smem = (long long)R * lds + (R + Cc + part_floats) <= (long long)smem_floats;
    float *Kg = kmat + kmat_offset(kmat_stride, t_begin, img);
    float *Kp = in_smem ? Ks : Kg;
    const int ldg = score_pitch(B);             // pitch of the workspace tile
    const int ld = in_smem ? lds : ldg;

    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);

    // build Z or K from the raw cosines (dustbin row and column = z, Eq. 5)
    for (int idx = tid; idx < R * Cc; idx += nth) {
        const int i = idx / Cc, j = idx - i * Cc;
        const float s = (i < M && j < B) ? Kg[(size_t)i * ldg + j] : p.z;
        Kp[(size_t)i * ld + j] = LOG ? s * inv_eps : expf((s - shift) * inv_eps);
    }
    const float v_init = LOG ? 0.f : expf(shift * inv_eps);
    for (int i = tid; i < R; i += nth) u[i] = LOG ? 0.f : 1.f;
    for (int j = tid; j < Cc; j += nth) v[j] = v_init;
    __syncthreads();

    const float mu_last = LOG ? logf((float)B) : (float)B;
    const float nu_last = LOG ? logf((float)M) : (float)M;
    const float mu_one = LOG ? 0.f : 1.f;

    const int cols_per_pass = min(Cc, nth);
    const int G = nth / cols_per_pass;
    const int passes = (Cc + cols_per_pass - 1) / cols_per_pass;
    const int cj = tid % cols_per_pass, cg = tid / cols_per_pass;
    const bool row_per_thread = in_smem && R >= 128;

    int done = 0;
    float last_move = 0.f;
    for (int it = 0; it < p.iters; ++it) {
        // ---- u from v -------------------------------------------------------------------------
        if (row_per_thread) {
            for (int i = tid; i < R; i += nth) {
                const float *row = Kp + (size_t)i * ld;
                if (LOG) {
                    float m = -INFINITY;
                    for (int j = 0; j < Cc; ++j) m = fmaxf(m, row[j] + v[j]);
                    float s = 0.f;
                    for (int j = 0; j < Cc; ++j) s += expf(row[j] + v[j] - m);
                    u[i] = (i < M ? mu_one : mu_last) - (m + logf(s));
                } else {
                    float s = 0.f;
                    for (int j = 0; j < Cc; ++j) s = fmaf(row[j], v[j], s);
                    u[i] = (i < M ? mu_one : mu_last) / s;
                }
            }
        } else {
            for (int i = warp; i < R; i += nwarps) {
                const float *row = Kp + (size_t)i * ld;
                if (LOG) {
                    float m = -INFINITY;
                    for (int j = lane; j < Cc; j += 32) m = fmaxf(m, row[j] + v[j]);
                    m = warp_max(m);
                    float s = 0.f;
                    for (int j = lane; j < Cc; j += 32) s += expf(row[j] + v[j] - m);
                    s = warp_sum(s);
                    if (lane == 0) u[i] = (i < M ? mu_one : mu_last) - (m + logf(s));
                } else {
                    float s = 0.f;
                    for (int j = lane; j < Cc; j += 32) s = fmaf(row[j], v[j], s);
                    s = warp_sum(s);
                    if (lane == 0) u[i] = (i < M ? mu_one : mu_last) / s;
                }
            }
        }
        __syncthreads();

        // ---- v from u -------------------------------------------------------------------------
        int cont = 0;
        last_move = 0.f;
        for (int ps = 0; ps < passes; ++ps) {
            const int j = ps * cols_per_pass + cj;
            const bool active = (cg < G) && (j < Cc);
            float m = -INFINITY, s = 0.f;
            if (active) {
                if (LOG) {
                    for (int i = cg; i < R; i += G) m = fmaxf(m, Kp[(size_t)i * ld + j] + u[i]);
                    for (int i = cg; i < R; i += G) s += expf(Kp[(size_t)i * ld + j] + u[i] - m);
                } else {
                    for (int i = cg; i < R; i += G) s = fmaf(Kp[(size_t)i * ld + j], u[i], s);
                }
            }
            if (G > 1) {
                if (active) {
                    part[cg * cols_per_pass + cj] = s;
                    if (LOG) part[nth + cg * cols_per_pass + cj] = m;
                }
                __syncthreads();
                if (active && cg == 0) {
                    for (int g = 1; g < G; ++g) {
                        if (LOG) lse_merge(m, s, part[nth + g * cols_per_pass + cj],
                                           part[g * cols_per_pass + cj]);
                        else s += part[g * cols_per_pass + cj];
                    }
                }
            }
            if (active && cg == 0) {
                const float nu = (j < B) ? mu_one : nu_last;
                const float nv = LOG ? nu - (m + logf(s)) : nu / s;
                const float ov = v[j];
                const float move = LOG ? fabsf(nv - ov) : fabsf(nv - ov) / fabsf(ov);
                last_move = fmaxf(last_move, move);
                if (p.tol > 0.f) cont |= (move > p.tol) ? 1 : 0;
                else cont |= p.stop_fp ? (LOG ? (__float_as_uint(nv) != __float_as_uint(ov)) : ulp_far(nv, ov)) : 1;
                v[j] = nv;
            }
            if (passes > 1 && G > 1) __syncthreads();
        }
        ++done;
        if (!__syncthreads_or(cont)) break;
    }
    __syncthreads();

    // largest dual move of the last executed iteration
    {
        float mv = warp_max(last_move);
        if (lane == 0) s_red[warp] = mv;
        __syncthreads();
        if (warp == 0) {
            mv = warp_max(lane < nwarps ? s_red[lane] : 0.f);
            if (lane == 0) {
                stats[(size_t)img * kStats + 5] = (float)done;
                stats[(size_t)img * kStats + 6] = mv;
            }
        }
    }

    // ---- pairing: partner_j = argmax_i P_ij = argmax_i (Z_ij + u_i), ties to the lower i -------
    // weight_j = (U_i K_ij) V_j, the same product the plan below stores, so weight == P there.
    const int seg = t_begin - out_offsets[img];
    const int32_t *ord = order + t_begin;
    int *parti = reinterpret_cast<int *>(part + nth);
    for (int ps = 0; ps < passes; ++ps) {
        const int j = ps * cols_per_pass + cj;
        const bool active = (cg < G) && (j < B);
        float best = -INFINITY;
        int bi = 0x7fffffff;
        if (active) {
            for (int i = cg; i < M; i += G) {
                const float k = Kp[(size_t)i * ld + j];
                const float key = LOG ? k + u[i] : k * u[i];
                if (key > best) {   // i ascends within a thread: strict > keeps the lower index
                    best = key;
                    bi = i;
                }
            }
        }
        if (G > 1) {
            __syncthreads();    // part[] may still be read by the previous pass / the sweeps
            if (active) {
                part[cg * cols_per_pass + cj] = best;
                parti[cg * cols_per_pass + cj] = bi;
            }
            __syncthreads();
            if (active && cg == 0) {
                for (int g = 1; g < G; ++g) {
                    const float ob = part[g * cols_per_pass + cj];
                    const int oi = parti[g * cols_per_pass + cj];
                    if (ob > best || (ob == best && oi < bi)) {
                        best = ob;
                        bi = oi;
                    }
                }
            }
        }
        if (active && cg == 0) {
            merged_idx[seg + j] = ord[M + j];
            merge_partner[seg + j] = bi;
            merge_weight[seg + j] = LOG ? expf(best + v[j]) : best * v[j];
        }
    }
    __syncthreads();

    // ---- plan P (non-dustbin block) ---------------------------------------------------------------
    if (pbuf) {
        // alpha P in bf16 for the tensor-core merge: row = the kept token's position in X, columns padded with zeros to
        // the next multiple of 64 (the contraction runs over whole 64-column blocks)
        const int kpad = (B + 63) & ~63;
        __nv_bfloat16 *Pimg = pbuf + (size_t)t_begin * pbuf_pitch;
        for (int idx = tid; idx < M * kpad; idx += nth) {
            const int i = idx / kpad, j = idx - i * kpad;
            float pv = 0.f;
            if (j < B) {
                const float k = Kp[(size_t)i * ld + j];
                pv = LOG ? expf(k + u[i] + v[j]) : (k * u[i]) * v[j];
            }
            Pimg[(size_t)ord[i] * pbuf_pitch + j] = __float2bfloat16_rn(p.alpha * pv);
        }
    } else {
        // fp32, in place in the workspace tile (row pitch score_pitch(B))
        for (int idx = tid; idx < M * B; idx += nth) {
            const int i = idx / B, j = idx - i * B;
            const float k = Kp[(size_t)i * ld + j];
            Kg[(size_t)i * ldg + j] = LOG ? expf(k + u[i] + v[j]) : (k * u[i]) * v[j];
        }
    }
}

}  // namespace rtp
