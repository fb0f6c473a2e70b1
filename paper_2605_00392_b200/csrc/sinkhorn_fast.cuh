// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C) in scaling form,
// one CTA per image, for score tiles that fit one CTA's shared memory.
//
// The duals are carried as U = e^u, V = e^{v + c/eps} against K_ij = exp((S_ij - c)/eps), c = max(1, z),
// so that U_i K_ij V_j = exp(Z_ij + u_i + v_j) (Appendix C) after any number of iterations.  The
// dustbin row and column of S-bar are the constant z (Eq. 5), so they are not stored: with
// kappa = exp((z - c)/eps), mu = [1_M, B], nu = [1_B, M],
//     U_i = 1 / (sum_j K_ij V_j + kappa V_d)          U_d = B / (kappa (sum_j V_j + V_d))
//     V_j = 1 / (sum_i K_ij U_i + kappa U_d)          V_d = M / (kappa (sum_i U_i + U_d))
// One iteration is ONE pass over K in shared memory: a warp owns four rows at a time, its lanes own
// the columns lane, lane + 32, ...; the four row sums are reduced together across the warp, the new
// U_i multiply the same K values (still in registers) into per-lane column accumulators, and the
// column sums are completed across the 16 warps through shared memory.
#pragma once
#include "common.cuh"
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

struct SfState {
    int done;
    float last_move;
};

// The iterations, for tiles of at most 32 * NC columns.  A warp takes RPC = 32 / NC rows per step, so
// that the K values it holds in registers stay at 32 whatever the tile's width.  Every warp completes
// the column sums for itself from the 16 warps' partials (same order in every warp, hence the same
// bits), so an iteration needs one CTA barrier; the partials are double-buffered.  On return every
// warp holds the final V (lane's columns lane + 32 c), V_d and U_d; U_i is in us[].
template <int NC>
__device__ inline SfState sinkhorn_fast_iterate(const float *__restrict__ Ks, int M, int B, int nc, int ldk,
                                                float *part, float *wsum, float *us, const OtParams &p,
                                                float kappa, float v_init, float (&V)[NC], float &Vd,
                                                float &Ud)
{
    constexpr int RPC = 32 / NC;          // rows per step
    constexpr int LPR = 32 / RPC;         // lanes that end up holding one row's total
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float Bf = (float)B, Mf = (float)M;
#pragma unroll
    for (int c = 0; c < NC; ++c) V[c] = (c < nc && lane + 32 * c < B) ? v_init : 0.f;
    Vd = v_init;
    float sumV = Bf * v_init;
    Ud = 1.f;
    const int ngroups = (M + RPC - 1) / RPC;
    SfState st{0, 0.f};

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
                // rows past M repeat the last row: their values are computed and dropped
                const float *row = Ks + (size_t)min(i0 + r, M - 1) * ldk + lane;
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
            if ((lane % LPR) == 0 && i0 + lane / LPR < M) us[i0 + lane / LPR] = Unew;
#pragma unroll
            for (int r = 0; r < RPC; ++r) {
                float Ur = __shfl_sync(0xffffffffu, Unew, LPR * r);
                Ur = (i0 + r < M) ? Ur : 0.f;
                usum += Ur;
#pragma unroll
                for (int c = 0; c < NC; ++c) colacc[c] = fmaf(k[r][c], Ur, colacc[c]);
            }
        }
        float *pb = part + (it & 1) * kSfWarps * ldk;
        float *wb = wsum + (it & 1) * kSfWarps;
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if (c < nc) pb[warp * ldk + lane + 32 * c] = colacc[c];
        if (lane == 0) wb[warp] = usum;
        __syncthreads();

        // ---- V from the completed column sums, in every warp alike ---------------------------------
        float cs[NC];
#pragma unroll
        for (int c = 0; c < NC; ++c) cs[c] = 0.f;
        float su = 0.f;
#pragma unroll
        for (int w = 0; w < kSfWarps; ++w) {
#pragma unroll
            for (int c = 0; c < NC; ++c)
                if (c < nc) cs[c] += pb[w * ldk + lane + 32 * c];
            su += wb[w];
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

__global__ void __launch_bounds__(kSfThreads, 1)
sinkhorn_fast_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                     const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                     float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                     int smem_floats, __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch,
                     int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                     float *__restrict__ merge_weight, float *__restrict__ stats)
{
    extern __shared__ __align__(16) float sm[];
    const int img = blockIdx.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0 || !sinkhorn_fast_fits(M, B, kSfMaxNc, smem_floats)) return;   // the general kernel takes it
    const int out0 = out_offsets[img];
    const int my_prop = (tid < B) ? order[t_begin + M + tid] : 0;   // needed at the end: fetch it now

    const int nc = (B + 31) >> 5;
    const int ldk = nc << 5;
    // shared memory carve-up
    float *Ks = sm;                                   // [M][ldk]
    float *part = Ks + (size_t)M * ldk;               // [2][16][ldk] column partials / pairing values, indices
    float *us = part + 2 * kSfWarps * ldk;            // [M + 1] U_i, U_d
    float *vs = us + ((M + 8) & ~3);                  // [ldk + 4]: V_j, then V_d at [ldk]; 16-byte aligned
    float *wsum = vs + (ldk + 4);                     // [2][16] per-warp sums of U

    float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ldS = score_pitch(B);
    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);

    // ---- K = exp((S - c)/eps), zero beyond column B --------------------------------------------------
    {
        const int qpr = ldk >> 2;                     // float4 per row of Ks
        const int total_q = M * qpr;
        for (int q0 = tid; q0 < total_q; q0 += kSfThreads * 4) {
            float4 s[4];
            int ii[4], jj[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kSfThreads;
                ii[a] = q / qpr;
                jj[a] = (q - ii[a] * qpr) << 2;
                s[a] = (q < total_q && jj[a] < ldS)
                           ? __ldcg(reinterpret_cast<const float4 *>(Sg + (size_t)ii[a] * ldS + jj[a]))
                           : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kSfThreads;
                if (q < total_q) {
                    float4 k;
                    k.x = (jj[a] + 0 < B) ? expf((s[a].x - shift) * inv_eps) : 0.f;
                    k.y = (jj[a] + 1 < B) ? expf((s[a].y - shift) * inv_eps) : 0.f;
                    k.z = (jj[a] + 2 < B) ? expf((s[a].z - shift) * inv_eps) : 0.f;
                    k.w = (jj[a] + 3 < B) ? expf((s[a].w - shift) * inv_eps) : 0.f;
                    *reinterpret_cast<float4 *>(Ks + (size_t)ii[a] * ldk + jj[a]) = k;
                }
            }
        }
    }
    const float v_init = expf(shift * inv_eps);       // v = 0
    for (int i = tid; i < M; i += kSfThreads) us[i] = 1.f;     // u = 0
    __syncthreads();

    // ---- the iterations --------------------------------------------------------------------------------
    SfState st;
    float Vd, Ud;
    if (nc <= 2) {
        float V[2];
        st = sinkhorn_fast_iterate<2>(Ks, M, B, nc, ldk, part, wsum, us, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) { vs[lane] = V[0]; if (nc > 1) vs[lane + 32] = V[1]; }
    } else if (nc <= 4) {
        float V[4];
        st = sinkhorn_fast_iterate<4>(Ks, M, B, nc, ldk, part, wsum, us, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) if (c < nc) vs[lane + 32 * c] = V[c];
        }
    } else {
        float V[8];
        st = sinkhorn_fast_iterate<8>(Ks, M, B, nc, ldk, part, wsum, us, p, kappa, v_init, V, Vd, Ud);
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) if (c < nc) vs[lane + 32 * c] = V[c];
        }
    }
    if (tid == 0) {
        vs[ldk] = Vd;
        us[M] = Ud;
        stats[(size_t)img * kStats + 5] = (float)st.done;
        stats[(size_t)img * kStats + 6] = st.last_move;
    }
    __syncthreads();

    // ---- pairing: partner_j = argmax_i P_ij = argmax_i K_ij U_i, ties to the lower i ----------------
    {
        float *pv = part;
        int *pi = reinterpret_cast<int *>(part + kSfWarps * ldk);
        for (int cb = 0; cb < nc; cb += 2) {          // two column blocks of 32 per sweep over the rows
            float best0 = -INFINITY, best1 = -INFINITY;
            int bi0 = 0x7fffffff, bi1 = 0x7fffffff;
            const bool two = cb + 1 < nc;
            for (int i = warp; i < M; i += kSfWarps) {
                const float ui = us[i];
                const float *row = Ks + (size_t)i * ldk + lane + 32 * cb;
                const float k0 = row[0] * ui;
                const float k1 = two ? row[32] * ui : -INFINITY;
                if (k0 > best0) { best0 = k0; bi0 = i; }    // i ascends: strict > keeps the lower index
                if (k1 > best1) { best1 = k1; bi1 = i; }
            }
            pv[warp * ldk + lane + 32 * cb] = best0;
            pi[warp * ldk + lane + 32 * cb] = bi0;
            if (two) {
                pv[warp * ldk + lane + 32 * cb + 32] = best1;
                pi[warp * ldk + lane + 32 * cb + 32] = bi1;
            }
        }
        __syncthreads();
        const int seg = t_begin - out0;
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
            merged_idx[seg + tid] = my_prop;
            merge_partner[seg + tid] = ib;
            merge_weight[seg + tid] = b * vs[tid];    // (K U) V, the product the plan stores
        }
    }

    // ---- plan P = U K V (non-dustbin block) ---------------------------------------------------------
    if (pbuf) {
        // alpha P in bf16 for the tensor-core merge: row = the kept token's position in X; columns up to
        // the next multiple of 64 are written (zeros past B), 8 columns = 16 bytes per store
        const int kpad = (B + 63) & ~63;
        const int vpr = kpad >> 3;
        __nv_bfloat16 *Pimg = pbuf + (size_t)t_begin * pbuf_pitch;
        for (int idx = tid; idx < M * vpr; idx += kSfThreads) {
            const int i = idx / vpr, j0 = (idx - i * vpr) << 3;
            const int tok = __ldg(order + t_begin + i);
            const float ui = us[i];
            __align__(16) float kk[8];
            __align__(16) float vv[8];
            if (j0 < ldk) {
                *reinterpret_cast<float4 *>(kk) = *reinterpret_cast<const float4 *>(Ks + (size_t)i * ldk + j0);
                *reinterpret_cast<float4 *>(kk + 4) = *reinterpret_cast<const float4 *>(Ks + (size_t)i * ldk + j0 + 4);
                *reinterpret_cast<float4 *>(vv) = *reinterpret_cast<const float4 *>(vs + j0);
                *reinterpret_cast<float4 *>(vv + 4) = *reinterpret_cast<const float4 *>(vs + j0 + 4);
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
        for (int idx = tid; idx < M * B; idx += kSfThreads) {
            const int i = idx / B, j = idx - i * B;
            Sg[(size_t)i * ldS + j] = (Ks[(size_t)i * ldk + j] * us[i]) * vs[j];
        }
    }
}

}  // namespace rtp
