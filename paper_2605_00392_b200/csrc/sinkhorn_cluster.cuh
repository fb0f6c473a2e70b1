// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C) in scaling form, for
// score tiles that fit the shared memory of one thread-block cluster: the rows (kept tokens) of an
// image's tile are split over the C CTAs of a cluster, C = 1, 2, 4 or 8.
//
// The duals are carried as U = e^u, V = e^{v + c/eps} against K_ij = exp((S_ij - c)/eps), c = max(1, z),
// so that U_i K_ij V_j = exp(Z_ij + u_i + v_j) (Appendix C) after any number of iterations.  The
// dustbin row and column of S-bar are the constant z (Eq. 5), so they are not stored: with
// kappa = exp((z - c)/eps), mu = [1_M, B], nu = [1_B, M],
//     U_i = 1 / (sum_j K_ij V_j + kappa V_d)          U_d = B / (kappa (sum_j V_j + V_d))
//     V_j = 1 / (sum_i K_ij U_i + kappa U_d)          V_d = M / (kappa (sum_i U_i + U_d))
// One iteration is ONE pass over K in shared memory: a warp owns a few rows at a time, its lanes own
// the columns lane, lane + 32, ...; the row sums are reduced together across the warp, the new U_i
// multiply the same K values (still in registers) into per-lane column accumulators; the column sums
// are completed across the 16 warps through shared memory and across the CTAs through distributed
// shared memory: every CTA stores its partial column sums into every CTA of the cluster, one cluster
// barrier, and every warp of every CTA adds the C partials in the same order, so all of them hold
// bit-identical V and take the same decision to stop.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "sinkhorn.cuh"

namespace rtp {

// Sums of R per-lane values over the warp, all R at once: afterwards lanes q*(32/R) .. (q+1)*(32/R)-1
// hold the total of value q.  R - 1 + log2(32 / R) shuffles instead of 5 R.
template <int R>
__device__ inline float warp_sum_scatter(float (&p)[R], int lane)
{
    int off = 16;
#pragma unroll
    for (int n = R; n > 1; n >>= 1, off >>= 1) {
        const bool hi = (lane & off) != 0;
#pragma unroll
        for (int q = 0; q < n / 2; ++q) {
            const float keep = hi ? p[q + n / 2] : p[q];
            const float give = hi ? p[q] : p[q + n / 2];
            p[q] = keep + __shfl_xor_sync(0xffffffffu, give, off);
        }
    }
    float r = p[0];
#pragma unroll
    for (; off > 0; off >>= 1) r += __shfl_xor_sync(0xffffffffu, r, off);
    return r;
}

__device__ inline float rcp_fast(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// exp(x) by the hardware base-2 exponential (relative error about 2^-22).
__device__ inline float exp_fast(float x) { return exp2f(x * 1.4426950408889634f); }

struct ScState {
    int done;
    float last_move;
};

// Shared-memory regions of one CTA of the cluster kernel.
struct ScSmem {
    float *Ks;      // [rows_per][ldk]      this CTA's rows of K
    float *part;    // [2][16][ldk]         per-warp column partials; pairing values and indices
    float *xpart;   // [2][C][ldk]          per-CTA column partials, double-buffered by iteration parity
    float *us;      // [rows_per + 1]       U of this CTA's rows
    float *vs;      // [ldk + 4]            final V_j, V_d at [ldk]
    float *wsum;    // [16]                 per-warp sums of U
    float *xusum;   // [2][8]               per-CTA sums of U, double-buffered
    int *toks;      // [rows_per]           token position of each of this CTA's rows (for the plan write)
};

// The iterations, for tiles of at most 32 * NC columns; Ml = this CTA's rows.  A warp takes
// RPC = 32 / NC rows per step, so that the K values it holds in registers stay at 32 whatever the
// tile's width.  On return every warp of every CTA holds the final V (lane's columns lane + 32 c),
// V_d and U_d; U of this CTA's rows is in us[].
template <int NC>
__device__ inline ScState sinkhorn_cluster_iterate(const ScSmem &m, int Ml, int M, int B, int nc, int ldk,
                                                   uint32_t C, uint32_t rank, const OtParams &p, float kappa,
                                                   float v_init, float (&V)[NC], float &Vd, float &Ud)
{
    constexpr int RPC = 32 / NC;          // rows per step
    constexpr int LPR = 32 / RPC;         // lanes that end up holding one row's total
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float Bf = (float)B, Mf = (float)M;
#pragma unroll
    for (int c = 0; c < NC; ++c) V[c] = (c < nc && lane + 32 * c < B) ? v_init : 0.f;
    Vd = v_init;
    float sumV = Bf * v_init;
    Ud = 1.f;
    const int ngroups = (Ml + RPC - 1) / RPC;
    const uint32_t xpart_u32 = ptx::smem_u32(m.xpart), xusum_u32 = ptx::smem_u32(m.xusum);
    ScState st{0, 0.f};

    for (int it = 0; it < p.iters; ++it) {
        Ud = Bf * rcp_fast(kappa * (sumV + Vd));
        const float kVd = kappa * Vd;
        float colacc[NC];
#pragma unroll
        for (int c = 0; c < NC; ++c) colacc[c] = 0.f;
        float usum = 0.f;

        for (int g = warp; g < ngroups; g += kSfWarps) {
            const int i0 = g * RPC;
            float k[RPC][NC];
            float ps[RPC];
#pragma unroll
            for (int r = 0; r < RPC; ++r) {
                // rows past Ml repeat the last row: their values are computed and dropped
                const float *row = m.Ks + (size_t)min(i0 + r, Ml - 1) * ldk + lane;
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    k[r][c] = (c < nc) ? row[32 * c] : 0.f;
                    s = fmaf(k[r][c], V[c], s);
                }
                ps[r] = s;
            }
            const float tot = warp_sum_scatter<RPC>(ps, lane);
            const float Unew = rcp_fast(tot + kVd);         // lanes q LPR .. : row i0 + q
            if ((lane % LPR) == 0 && i0 + lane / LPR < Ml) m.us[i0 + lane / LPR] = Unew;
#pragma unroll
            for (int r = 0; r < RPC; ++r) {
                float Ur = __shfl_sync(0xffffffffu, Unew, LPR * r);
                Ur = (i0 + r < Ml) ? Ur : 0.f;
                usum += Ur;
#pragma unroll
                for (int c = 0; c < NC; ++c) colacc[c] = fmaf(k[r][c], Ur, colacc[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if (c < nc) m.part[warp * ldk + lane + 32 * c] = colacc[c];
        if (lane == 0) m.wsum[warp] = usum;
        __syncthreads();

        // this CTA's column sums and sum of U go to every CTA of the cluster (this one included)
        const uint32_t slot = (uint32_t)(it & 1) * C + rank;
        if (tid < ldk) {
            float cs = 0.f;
#pragma unroll
            for (int w = 0; w < kSfWarps; ++w) cs += m.part[w * ldk + tid];
            const uint32_t a = xpart_u32 + (slot * (uint32_t)ldk + (uint32_t)tid) * 4u;
            for (uint32_t r = 0; r < C; ++r) ptx::st_cluster_f32(ptx::map_to_rank(a, r), cs);
        }
        if (tid == kSfThreads - 1) {
            float su = 0.f;
#pragma unroll
            for (int w = 0; w < kSfWarps; ++w) su += m.wsum[w];
            const uint32_t a = xusum_u32 + slot * 4u;
            for (uint32_t r = 0; r < C; ++r) ptx::st_cluster_f32(ptx::map_to_rank(a, r), su);
        }
        ptx::cluster_sync_all();

        // ---- V from the completed column sums, in every warp of every CTA alike ----------------------
        const float *xb = m.xpart + (size_t)(it & 1) * C * ldk;
        const float *ub = m.xusum + (it & 1) * C;
        float cs[NC];
#pragma unroll
        for (int c = 0; c < NC; ++c) cs[c] = 0.f;
        float su = 0.f;
        for (uint32_t r = 0; r < C; ++r) {
#pragma unroll
            for (int c = 0; c < NC; ++c)
                if (c < nc) cs[c] += xb[r * ldk + lane + 32 * c];
            su += ub[r];
        }
        const float kUd = kappa * Ud;
        bool changed = false;
        float move = 0.f, sv = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const bool real = c < nc && lane + 32 * c < B;
            const float nv = real ? rcp_fast(cs[c] + kUd) : 0.f;
            changed |= __float_as_uint(nv) != __float_as_uint(V[c]);
            if (real) move = fmaxf(move, fabsf(nv - V[c]) * rcp_fast(V[c]));
            V[c] = nv;
            sv += nv;
        }
        const float nVd = Mf * rcp_fast(kappa * (su + Ud));
        changed |= __float_as_uint(nVd) != __float_as_uint(Vd);
        move = fmaxf(move, fabsf(nVd - Vd) * rcp_fast(Vd));
        Vd = nVd;
        sumV = warp_sum(sv);
        st.last_move = move;
        ++st.done;
        bool cont;
        if (p.tol > 0.f) cont = __any_sync(0xffffffffu, move > p.tol);
        else cont = p.stop_fp ? __any_sync(0xffffffffu, changed) : true;
        if (!cont) break;
    }
    st.last_move = warp_max(st.last_move);
    return st;
}

// grid = batch * C CTAs, clusters of C along x: CTA rank r of cluster i owns rows r*rows_per .. of
// image i's tile.  Every early return below depends on the image only, so a cluster leaves as a whole.
__global__ void __launch_bounds__(kSfThreads, 1)
sinkhorn_cluster_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                        const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                        float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                        int smem_floats, __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch,
                        int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                        float *__restrict__ merge_weight, float *__restrict__ stats)
{
    extern __shared__ __align__(16) float sm[];
    const uint32_t C = ptx::cluster_nctarank(), rank = ptx::cluster_ctarank();
    const int img = blockIdx.x / C, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();     // the scores come from the kernel ahead
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0 || !sinkhorn_cluster_fits(M, B, (int)C, smem_floats)) return;   // the general kernel takes it
    const int out0 = out_offsets[img];
    const int my_prop = (rank == 0 && tid < B) ? order[t_begin + M + tid] : 0;   // needed at the end

    const int nc = (B + 31) >> 5;
    const int ldk = nc << 5;
    const int rows_per = (M + (int)C - 1) / (int)C;
    const int row_lo = min(M, (int)rank * rows_per);
    const int Ml = min(M, row_lo + rows_per) - row_lo;       // this CTA's rows (may be 0)
    ScSmem m;
    m.Ks = sm;
    m.part = m.Ks + (size_t)rows_per * ldk;
    m.xpart = m.part + 2 * kSfWarps * ldk;
    m.us = m.xpart + 2 * C * ldk;
    m.vs = m.us + ((rows_per + 8) & ~3);
    m.wsum = m.vs + (ldk + 4);
    m.xusum = m.wsum + kSfWarps;
    m.toks = reinterpret_cast<int *>(m.xusum + 16);

    float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ldS = score_pitch(B);
    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);

    // ---- K = exp((S - c)/eps) of this CTA's rows, zero beyond column B ------------------------------
    {
        const int qpr = ldk >> 2;                     // float4 per row of Ks
        const int total_q = Ml * qpr;
        for (int q0 = tid; q0 < total_q; q0 += kSfThreads * 4) {
            float4 s[4];
            int ii[4], jj[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kSfThreads;
                ii[a] = q / qpr;
                jj[a] = (q - ii[a] * qpr) << 2;
                s[a] = (q < total_q && jj[a] < ldS)
                           ? __ldcg(reinterpret_cast<const float4 *>(Sg + (size_t)(row_lo + ii[a]) * ldS + jj[a]))
                           : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kSfThreads;
                if (q < total_q) {
                    float4 k;
                    k.x = (jj[a] + 0 < B) ? exp_fast((s[a].x - shift) * inv_eps) : 0.f;
                    k.y = (jj[a] + 1 < B) ? exp_fast((s[a].y - shift) * inv_eps) : 0.f;
                    k.z = (jj[a] + 2 < B) ? exp_fast((s[a].z - shift) * inv_eps) : 0.f;
                    k.w = (jj[a] + 3 < B) ? exp_fast((s[a].w - shift) * inv_eps) : 0.f;
                    *reinterpret_cast<float4 *>(m.Ks + (size_t)ii[a] * ldk + jj[a]) = k;
                }
            }
        }
    }
    const float v_init = expf(shift * inv_eps);       // v = 0
    for (int i = tid; i < Ml; i += kSfThreads) {
        m.us[i] = 1.f;                                            // u = 0
        m.toks[i] = __ldg(order + t_begin + row_lo + i);
    }
    // every CTA of the cluster is running and has its shared memory laid out before anyone writes into it
    ptx::cluster_sync_all();

    // ---- the iterations --------------------------------------------------------------------------------
    ScState st;
    float Vd, Ud;
    if (nc <= 2) {
        float V[2];
        st = sinkhorn_cluster_iterate<2>(m, Ml, M, B, nc, ldk, C, rank, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < 2; ++c) if (c < nc) m.vs[lane + 32 * c] = V[c];
        }
    } else if (nc <= 4) {
        float V[4];
        st = sinkhorn_cluster_iterate<4>(m, Ml, M, B, nc, ldk, C, rank, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) if (c < nc) m.vs[lane + 32 * c] = V[c];
        }
    } else {
        float V[8];
        st = sinkhorn_cluster_iterate<8>(m, Ml, M, B, nc, ldk, C, rank, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) if (c < nc) m.vs[lane + 32 * c] = V[c];
        }
    }
    if (tid == 0) {
        m.vs[ldk] = Vd;
        if (rank == 0) {
            stats[(size_t)img * kStats + 5] = (float)st.done;
            stats[(size_t)img * kStats + 6] = st.last_move;
        }
    }
    (void)Ud;
    // nobody reads xpart any more (it is reused below), and vs is visible to the CTA
    ptx::cluster_sync_all();

    // ---- pairing: partner_j = argmax_i P_ij = argmax_i K_ij U_i, ties to the lower i ----------------
    {
        float *pv = m.part;
        int *pi = reinterpret_cast<int *>(m.part + kSfWarps * ldk);
        for (int cb = 0; cb < nc; cb += 2) {          // two column blocks of 32 per sweep over the rows
            float best0 = -INFINITY, best1 = -INFINITY;
            int bi0 = 0x7fffffff, bi1 = 0x7fffffff;
            const bool two = cb + 1 < nc;
            for (int i = warp; i < Ml; i += kSfWarps) {
                const float ui = m.us[i];
                const float *row = m.Ks + (size_t)i * ldk + lane + 32 * cb;
                const float k0 = row[0] * ui;
                const float k1 = two ? row[32] * ui : -INFINITY;
                if (k0 > best0) { best0 = k0; bi0 = row_lo + i; }    // i ascends: strict > keeps the lower index
                if (k1 > best1) { best1 = k1; bi1 = row_lo + i; }
            }
            pv[warp * ldk + lane + 32 * cb] = best0;
            pi[warp * ldk + lane + 32 * cb] = bi0;
            if (two) {
                pv[warp * ldk + lane + 32 * cb + 32] = best1;
                pi[warp * ldk + lane + 32 * cb + 32] = bi1;
            }
        }
        __syncthreads();
        // this CTA's best per column goes to rank 0: values in xpart[0][rank][.], indices in xpart[1][rank][.]
        if (tid < B) {
            float b = pv[tid];
            int ib = pi[tid];
#pragma unroll
            for (int w = 1; w < kSfWarps; ++w) {
                const float ob = pv[w * ldk + tid];
                const int oi = pi[w * ldk + tid];
                if (ob > b || (ob == b && oi < ib)) {
                    b = ob;
                    ib = oi;
                }
            }
            const uint32_t base = ptx::map_to_rank(ptx::smem_u32(m.xpart), 0);
            ptx::st_cluster_f32(base + ((rank * (uint32_t)ldk) + (uint32_t)tid) * 4u, b);
            ptx::st_cluster_u32(base + (((C + rank) * (uint32_t)ldk) + (uint32_t)tid) * 4u, (uint32_t)ib);
        }
        ptx::cluster_sync_all();      // after this barrier nothing is written into another CTA any more
        if (rank == 0 && tid < B) {
            const int *xi = reinterpret_cast<const int *>(m.xpart + (size_t)C * ldk);
            float b = m.xpart[tid];
            int ib = xi[tid];
            for (uint32_t r = 1; r < C; ++r) {     // ranks hold ascending row ranges: strict > keeps the lower index
                const float ob = m.xpart[r * ldk + tid];
                if (ob > b) {
                    b = ob;
                    ib = xi[r * ldk + tid];
                }
            }
            const int seg = t_begin - out0;
            merged_idx[seg + tid] = my_prop;
            merge_partner[seg + tid] = ib;
            merge_weight[seg + tid] = b * m.vs[tid];    // (K U) V, the product the plan stores
        }
    }

    // ---- plan P = U K V (non-dustbin block), this CTA's rows --------------------------------------------
    if (pbuf) {
        // alpha P in bf16 for the tensor-core merge: row = the kept token's position in X; columns up to
        // the next multiple of 64 are written (zeros past B), 8 columns = 16 bytes per store
        const int kpad = (B + 63) & ~63;
        const int vpr = kpad >> 3;
        __nv_bfloat16 *Pimg = pbuf + (size_t)t_begin * pbuf_pitch;
        for (int idx = tid; idx < Ml * vpr; idx += kSfThreads) {
            const int i = idx / vpr, j0 = (idx - i * vpr) << 3;
            const int tok = m.toks[i];
            const float ui = m.us[i];
            __align__(16) float kk[8];
            __align__(16) float vv[8];
            if (j0 < ldk) {
                *reinterpret_cast<float4 *>(kk) = *reinterpret_cast<const float4 *>(m.Ks + (size_t)i * ldk + j0);
                *reinterpret_cast<float4 *>(kk + 4) = *reinterpret_cast<const float4 *>(m.Ks + (size_t)i * ldk + j0 + 4);
                *reinterpret_cast<float4 *>(vv) = *reinterpret_cast<const float4 *>(m.vs + j0);
                *reinterpret_cast<float4 *>(vv + 4) = *reinterpret_cast<const float4 *>(m.vs + j0 + 4);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) kk[e] = vv[e] = 0.f;
            }
            __nv_bfloat162 o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                // K is zero past column B, so those products are zero
                const float a = (kk[2 * e] * ui) * vv[2 * e];
                const float b = (kk[2 * e + 1] * ui) * vv[2 * e + 1];
                o[e] = __floats2bfloat162_rn(p.alpha * a, p.alpha * b);
            }
            *reinterpret_cast<uint4 *>(Pimg + (size_t)tok * pbuf_pitch + j0) = *reinterpret_cast<uint4 *>(o);
        }
    } else {
        // fp32, in place in the workspace tile (row pitch score_pitch(B))
        for (int idx = tid; idx < Ml * B; idx += kSfThreads) {
            const int i = idx / B, j = idx - i * B;
            Sg[(size_t)(row_lo + i) * ldS + j] = (m.Ks[(size_t)i * ldk + j] * m.us[i]) * m.vs[j];
        }
    }
}

}  // namespace rtp
