// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C) in scaling form, one
// thread-block cluster per image: the rows (kept tokens) of an image's score tile are split over the
// C CTAs of a cluster, C = 1, 2, 4 or 8.  Tiles of up to 640 pruned tokens are taken; K stays in the
// cluster's shared memory when it fits there, else it is built in place in the image's workspace
// tile and read through L2 in every iteration.
//
// The duals are carried as U = e^u, V = e^{v + c/eps} against K_ij = exp((S_ij - c)/eps), c = max(1, z),
// so that U_i K_ij V_j = exp(Z_ij + u_i + v_j) (Appendix C) after any number of iterations.  The
// dustbin row and column of S-bar are the constant z (Eq. 5), so they are not stored: with
// kappa = exp((z - c)/eps), mu = [1_M, B], nu = [1_B, M],
//     U_i = 1 / (sum_j K_ij V_j + kappa V_d)          U_d = B / (kappa (sum_j V_j + V_d))
//     V_j = 1 / (sum_i K_ij U_i + kappa U_d)          V_d = M / (kappa (sum_i U_i + U_d))
// One iteration is ONE pass over K: 8, 16 or 32 lanes share a row, the row sum is an
// all-reduce over them, the new U_i multiplies the same K values (still in registers) into per-lane
// column accumulators; the column sums are completed across the 16 warps through shared memory and
// across the CTAs through distributed shared memory: every CTA stores its partial column sums into
// every CTA of the cluster, one cluster barrier, and every CTA adds the C partials in the same order,
// so all of them hold bit-identical V and take the same decision to stop.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "sinkhorn.cuh"

namespace rtp {

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
    int ldr;        // pitch of K's rows: ldk in shared memory, the tile's pitch in the workspace
    float *Ks;      // [rows_per][ldr]      this CTA's rows of K (shared memory, or the workspace tile)
    float *part;    // [2][16][ldk]         per-warp column partials; pairing values and indices
    float *xpart;   // [2][C][ldk]          per-CTA column partials, double-buffered by iteration parity
    float *us;      // [rows_per + 1]       U of this CTA's rows
    float *vs;      // [ldk + 4]            final V_j, V_d at [ldk]
    float *wsum;    // [16]                 per-warp sums of U
    float *xusum;   // [2][8]               per-CTA sums of U, double-buffered
    int *toks;      // [rows_per]           token position of each of this CTA's rows (for the plan write)
};

// The iterations for a tile whose rows are ldk = LR * CPL floats wide; Ml = this CTA's rows.
// Lane layout of the row pass: LR consecutive lanes share a row, a warp takes 32 / LR rows per step;
// lane `sub` of a row owns the 16-byte column chunks sub, sub + LR, ... (CPL columns in all), so a
// row's lanes read consecutive chunks.  The row sum is an all-reduce over the LR lanes (every lane of
// the row then has U_i, no broadcast), the products K_ij U_i go to per-lane column accumulators, which
// are reduced over the warp's rows at the end of the pass, over the 16 warps through shared memory,
// and over the CTAs through distributed shared memory (one cluster barrier).  The threads then
// compute one V_j each (two for B > 512), the same in every CTA.  On return vs[] holds the final V (V_d at [ldk]) and
// us[] the U of this CTA's rows.
template <int LR, int CPL, bool KGLOBAL>
__device__ inline ScState sinkhorn_cluster_iterate(const ScSmem &m, int Ml, int M, int B, uint32_t C,
                                                   uint32_t rank, const OtParams &p, float kappa, float v_init)
{
    constexpr int ldk = LR * CPL;
    // K's rows: in shared memory (pitch ldk, zero from column B on) or, KGLOBAL, for tiles too large
    // for it, in the image's workspace tile (pitch m.ldr, which is also how many columns exist there;
    // zero from column B on)
    const float *Kbase = m.Ks;
    const int ldr = KGLOBAL ? m.ldr : ldk;
    constexpr int RPS = 32 / LR;          // rows per step of a warp
    constexpr int NQ = CPL / 4;           // 16-byte chunks per lane
    constexpr bool kOneColumn = ldk <= kSfThreads;                 // a thread per column is enough
    constexpr int kVWarps = kOneColumn ? ldk / 32 : kSfWarps;      // warps that hold sums of V
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;
    const float Bf = (float)B, Mf = (float)M;
    __shared__ float s_vsum[kSfWarps];    // per-warp sums of V (warps 0 .. ldk/32-1)

    for (int j = tid; j <= ldk; j += kSfThreads) m.vs[j] = (j < B || j == ldk) ? v_init : 0.f;
    if (tid < kSfWarps) s_vsum[tid] = (tid == 0) ? Bf * v_init : 0.f;
    __syncthreads();
    const int nsteps = (Ml + RPS - 1) / RPS;
    const uint32_t xpart_u32 = ptx::smem_u32(m.xpart), xusum_u32 = ptx::smem_u32(m.xusum);
    ScState st{0, 0.f};

    for (int it = 0; it < p.iters; ++it) {
        // this lane's V, the dustbin terms
        float4 V[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(m.vs + 4 * (q * LR + sub));
        float sumV = 0.f;
#pragma unroll
        for (int w = 0; w < kVWarps; ++w) sumV += s_vsum[w];
        const float Vd = m.vs[ldk];
        const float Ud = Bf * rcp_fast(kappa * (sumV + Vd));
        const float kVd = kappa * Vd;
        float4 colacc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) colacc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float usum = 0.f;

#pragma unroll 2
        for (int g = warp; g < nsteps; g += kSfWarps) {
            const int i = g * RPS + slot;
            const bool valid = i < Ml;
            // rows past Ml repeat the last row: their values are computed and dropped
            const float *row = Kbase + (size_t)min(i, Ml - 1) * ldr + 4 * sub;
            float4 k[NQ];
            float s = 0.f;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if constexpr (KGLOBAL)
                    k[q] = (4 * (q * LR + sub) < ldr) ? __ldcg(reinterpret_cast<const float4 *>(row + 4 * q * LR))
                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                else
                    k[q] = *reinterpret_cast<const float4 *>(row + 4 * q * LR);
                s = fmaf(k[q].x, V[q].x, s);
                s = fmaf(k[q].y, V[q].y, s);
                s = fmaf(k[q].z, V[q].z, s);
                s = fmaf(k[q].w, V[q].w, s);
            }
#pragma unroll
            for (int o = 1; o < LR; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const float U = valid ? rcp_fast(s + kVd) : 0.f;
            if (sub == 0 && valid) {
                m.us[i] = U;
                usum += U;
            }
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                colacc[q].x = fmaf(k[q].x, U, colacc[q].x);
                colacc[q].y = fmaf(k[q].y, U, colacc[q].y);
                colacc[q].z = fmaf(k[q].z, U, colacc[q].z);
                colacc[q].w = fmaf(k[q].w, U, colacc[q].w);
            }
        }
        // column partials over the warp's row slots, then to shared memory (lanes of slot 0)
#pragma unroll
        for (int o = LR; o < 32; o <<= 1) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                colacc[q].x += __shfl_xor_sync(0xffffffffu, colacc[q].x, o);
                colacc[q].y += __shfl_xor_sync(0xffffffffu, colacc[q].y, o);
                colacc[q].z += __shfl_xor_sync(0xffffffffu, colacc[q].z, o);
                colacc[q].w += __shfl_xor_sync(0xffffffffu, colacc[q].w, o);
            }
        }
        if (slot == 0) {
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                *reinterpret_cast<float4 *>(m.part + warp * ldk + 4 * (q * LR + sub)) = colacc[q];
        }
        usum = warp_sum(usum);
        if (lane == 0) m.wsum[warp] = usum;
        __syncthreads();

        // this CTA's column sums and sum of U go to every CTA of the cluster (this one included)
        const uint32_t slot_x = (uint32_t)(it & 1) * C + rank;
        for (int j = tid; j < ldk; j += kSfThreads) {       // one trip when ldk <= the thread count
            float cs = 0.f;
#pragma unroll
            for (int w = 0; w < kSfWarps; ++w) cs += m.part[w * ldk + j];
            const uint32_t a = xpart_u32 + (slot_x * (uint32_t)ldk + (uint32_t)j) * 4u;
            for (uint32_t r = 0; r < C; ++r) ptx::st_cluster_f32(ptx::map_to_rank(a, r), cs);
        }
        if (tid == kSfThreads - 1) {
            float su = 0.f;
#pragma unroll
            for (int w = 0; w < kSfWarps; ++w) su += m.wsum[w];
            const uint32_t a = xusum_u32 + slot_x * 4u;
            for (uint32_t r = 0; r < C; ++r) ptx::st_cluster_f32(ptx::map_to_rank(a, r), su);
        }
        ptx::cluster_sync_all();

        // ---- V from the completed column sums: one thread per column, the same in every CTA ----------
        const float *xb = m.xpart + (size_t)(it & 1) * C * ldk;
        const float *ub = m.xusum + (it & 1) * C;
        int cont = 0;
        float move = 0.f;
        if constexpr (kOneColumn) {
            if (tid < ldk) {
                float nv = 0.f;
                if (tid < B) {
                    float cs = 0.f;
                    for (uint32_t r = 0; r < C; ++r) cs += xb[r * ldk + tid];
                    nv = rcp_fast(cs + kappa * Ud);
                    const float ov = m.vs[tid];
                    move = fabsf(nv - ov) * rcp_fast(ov);
                    cont = p.tol > 0.f ? (move > p.tol) : (p.stop_fp ? ulp_far(nv, ov) : 1);
                    m.vs[tid] = nv;
                }
                const float wv = warp_sum(nv);        // warps 0 .. ldk/32-1 lie entirely inside tid < ldk
                if (lane == 0) s_vsum[warp] = wv;
            }
        } else {
            float sv = 0.f;
            for (int j = tid; j < B; j += kSfThreads) {
                float cs = 0.f;
                for (uint32_t r = 0; r < C; ++r) cs += xb[r * ldk + j];
                const float nv = rcp_fast(cs + kappa * Ud);
                const float ov = m.vs[j];
                const float mj = fabsf(nv - ov) * rcp_fast(ov);
                move = fmaxf(move, mj);
                cont |= p.tol > 0.f ? (mj > p.tol) : (p.stop_fp ? ulp_far(nv, ov) : 1);
                m.vs[j] = nv;
                sv += nv;
            }
            sv = warp_sum(sv);
            if (lane == 0) s_vsum[warp] = sv;
        }
        if (tid == kSfThreads - 1) {                  // the dustbin column
            float su = 0.f;
            for (uint32_t r = 0; r < C; ++r) su += ub[r];
            const float nVd = Mf * rcp_fast(kappa * (su + Ud));
            const float mj = fabsf(nVd - Vd) * rcp_fast(Vd);
            move = fmaxf(move, mj);
            cont |= p.tol > 0.f ? (mj > p.tol) : (p.stop_fp ? ulp_far(nVd, Vd) : 1);
            m.vs[ldk] = nVd;
        }
        st.last_move = move;
        ++st.done;
        if (!__syncthreads_or(cont)) break;
    }
    // largest relative dual move of the last executed iteration, over the CTA
    float mv = warp_max(st.last_move);
    __syncthreads();
    if (lane == 0) s_vsum[warp] = mv;
    __syncthreads();
    mv = 0.f;
#pragma unroll
    for (int w = 0; w < kSfWarps; ++w) mv = fmaxf(mv, s_vsum[w]);
    st.last_move = mv;
    return st;
}

// This CTA has written everything it contributes to image `img`; the last CTA of the cluster to say so
// appends the image to the list that the merge kernel consumes in order of completion (it may already
// be running: it was launched as a programmatic dependent).  Called by every thread of the CTA.
__device__ inline void sinkhorn_publish(int img, uint32_t C, uint32_t *__restrict__ sink_done,
                                        int32_t *__restrict__ ready_list, WsHeader *__restrict__ hdr)
{
    if (!ready_list) return;
    ptx::fence_proxy_async_all();     // the plan rows are read by TMA over there
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t prev = atomicAdd(&sink_done[img], 1u);
        if (prev == C - 1u) {
            __threadfence();
            const uint32_t slot = atomicAdd(&hdr->n_ready, 1u);
            ptx::st_release_gpu(ready_list + slot, img + 1);
        }
    }
}

// grid = batch * C CTAs, clusters of C along x: CTA rank r of cluster i owns rows r*rows_per .. of
// image i's tile.  Every early return below depends on the image only, so a cluster leaves as a whole.
// Two instances: WIDE = false takes the tiles of up to 256 columns that fit shared memory (the common
// case, kept free of everything the others need) and is launched alone when no other tile is possible
// in the run; WIDE = true is launched instead when wider or taller tiles are possible, and then takes
// every tile of the family (takes_all), so that the images of a ragged batch are solved side by side
// by one grid rather than by two grids one after the other.
template <bool WIDE>
__global__ void __launch_bounds__(kSfThreads, 1)
sinkhorn_cluster_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                        const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                        float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                        int smem_floats, __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch,
                        int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                        float *__restrict__ merge_weight, float *__restrict__ stats,
                        uint32_t *__restrict__ sink_done, int32_t *__restrict__ ready_list,
                        WsHeader *__restrict__ hdr, const uint32_t *scores_done, int takes_all)
{
    extern __shared__ __align__(16) float sm[];
    const uint32_t C = ptx::cluster_nctarank(), rank = ptx::cluster_ctarank();
    const int img = blockIdx.x / C, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    ptx::grid_dep_launch();
    // The scores come from the kernel ahead: wait for that grid to end, or, with per-image counts of
    // finished score tiles, only for this image's tiles (and for the grid before leaving, so that this
    // grid's end still implies that one's).
    if (!scores_done) ptx::grid_dep_wait();
    int t_begin, N;
    // (a ready list is only passed when this instance is the only Sinkhorn kernel of the run, so an
    // image that leaves here needs no plan)
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) {
        sinkhorn_publish(img, C, sink_done, ready_list, hdr);
        if (scores_done) ptx::grid_dep_wait();
        return;
    }
    if (scores_done) {
        if (tid == 0) {
            const uint32_t want = (uint32_t)((N + 127) / 128);     // the scores kernel's 128-token tiles
            // first the run's number: before it is there the counts are what the run before left
            const bool tagged = ptx::wait_equal_gpu(&hdr->run_tag, ptx::ld_acquire_gpu(&hdr->launch_seq));
            bool ok = false;
            for (uint32_t i = 0; tagged && i < ptx::kSpinLimit && !ok; ++i) {
                ok = (uint32_t)ptx::ld_acquire_gpu(reinterpret_cast<const int *>(scores_done + img)) >= want;
                if (!ok) __nanosleep(200);
            }
            if (!ok) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
        }
        __syncthreads();
    }
    const int M = __ldcg(counts + img), B = N - M;
    if (B == 0 || !sinkhorn_cluster_handles(M, B, (int)C, smem_floats)) {   // the general kernel takes it
        sinkhorn_publish(img, C, sink_done, ready_list, hdr);
        if (scores_done) ptx::grid_dep_wait();
        return;
    }
    const bool in_smem = sinkhorn_cluster_fits(M, B, (int)C, smem_floats);
    const int ldk = sinkhorn_ldk(B);
    if (!(WIDE && takes_all) && (in_smem && ldk <= 256) == WIDE) {   // the other instance's tile
        if (scores_done) ptx::grid_dep_wait();
        return;
    }
    const int out0 = __ldcg(out_offsets + img);
    const int nc = ldk >> 5;
    const int rows_per = (M + (int)C - 1) / (int)C;
    const int row_lo = min(M, (int)rank * rows_per);
    const int Ml = min(M, row_lo + rows_per) - row_lo;       // this CTA's rows (may be 0)
    float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ldS = score_pitch(B);
    // K of this CTA's rows: in shared memory when the tile fits the cluster, else in place in the
    // workspace tile (read through L2 every iteration)
    ScSmem m;
    m.Ks = (!WIDE || in_smem) ? sm : Sg + (size_t)row_lo * ldS;
    m.ldr = (!WIDE || in_smem) ? ldk : ldS;
    m.part = (!WIDE || in_smem) ? sm + (size_t)rows_per * ldk : sm;
    m.xpart = m.part + 2 * kSfWarps * ldk;
    m.us = m.xpart + 2 * C * ldk;
    m.vs = m.us + ((rows_per + 8) & ~3);
    m.wsum = m.vs + (ldk + 4);
    m.xusum = m.wsum + kSfWarps;
    m.toks = reinterpret_cast<int *>(m.xusum + 16);

    const int ldr = m.ldr;
    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);

    for (int i = tid; i < Ml; i += kSfThreads) m.toks[i] = __ldcg(order + t_begin + row_lo + i);

    // ---- K = exp((S - c)/eps) of this CTA's rows, zero beyond column B ------------------------------
    {
        const int qpr = ldr >> 2;                     // float4 per row of K
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
                    *reinterpret_cast<float4 *>(m.Ks + (size_t)ii[a] * ldr + jj[a]) = k;
                }
            }
        }
    }
    const float v_init = expf(shift * inv_eps);       // v = 0
    for (int i = tid; i < Ml; i += kSfThreads) m.us[i] = 1.f;     // u = 0
    // every CTA of the cluster is running and has its shared memory laid out before anyone writes into it
    ptx::cluster_sync_all();

    // ---- the iterations --------------------------------------------------------------------------------
    ScState st;
#define RTP_SC_SMEM(LR, CPL) st = sinkhorn_cluster_iterate<LR, CPL, false>(m, Ml, M, B, C, rank, p, kappa, v_init)
#define RTP_SC_GLOBAL(LR, CPL) st = sinkhorn_cluster_iterate<LR, CPL, true>(m, Ml, M, B, C, rank, p, kappa, v_init)
#define RTP_SC_EITHER(LR, CPL)                                                                            \
    if (in_smem) RTP_SC_SMEM(LR, CPL);                                                                    \
    else RTP_SC_GLOBAL(LR, CPL)
    if constexpr (!WIDE) {
        if (ldk == 32) RTP_SC_SMEM(8, 4);
        else if (ldk == 64) RTP_SC_SMEM(8, 8);
        else if (ldk == 128) RTP_SC_SMEM(8, 16);
        else if (ldk == 192) RTP_SC_SMEM(16, 12);
        else RTP_SC_SMEM(16, 16);
    } else {
        switch (ldk) {
        case 32: RTP_SC_EITHER(8, 4); break;
        case 64: RTP_SC_EITHER(8, 8); break;
        case 128: RTP_SC_EITHER(8, 16); break;
        case 192: RTP_SC_EITHER(16, 12); break;
        case 256: RTP_SC_EITHER(16, 16); break;
        case 384: RTP_SC_EITHER(32, 12); break;
        case 512: RTP_SC_EITHER(32, 16); break;
        default: RTP_SC_EITHER(32, 20); break;
        }
    }
#undef RTP_SC_SMEM
#undef RTP_SC_GLOBAL
#undef RTP_SC_EITHER
    if (tid == 0 && rank == 0) {
        stats[(size_t)img * kStats + 5] = (float)st.done;
        stats[(size_t)img * kStats + 6] = st.last_move;
    }
    // ---- plan P = U K V (non-dustbin block), this CTA's rows --------------------------------------------
    // (needs this CTA's K and U and the V every CTA holds: no cluster barrier before it)
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
#pragma unroll
            for (int h = 0; h < 8; h += 4) {
                const bool have = j0 + h < ldk && j0 + h < ldr;      // beyond: columns past B, zero
                *reinterpret_cast<float4 *>(kk + h) =
                    have ? *reinterpret_cast<const float4 *>(m.Ks + (size_t)i * ldr + j0 + h) : make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4 *>(vv + h) =
                    have ? *reinterpret_cast<const float4 *>(m.vs + j0 + h) : make_float4(0.f, 0.f, 0.f, 0.f);
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
    }
    // the merge kernel may take the image from here: the pairs below are outputs of their own
    sinkhorn_publish(img, C, sink_done, ready_list, hdr);

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
                // columns past the row's end (workspace tile narrower than ldk) are past B: never read back
                const int c0 = lane + 32 * cb;
                const float *row = m.Ks + (size_t)i * ldr + c0;
                const float k0 = (c0 < ldr) ? row[0] * ui : 0.f;
                const float k1 = two ? ((c0 + 32 < ldr) ? row[32] * ui : 0.f) : -INFINITY;
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
        for (int j = tid; j < B; j += kSfThreads) {
            float b = pv[j];
            int ib = pi[j];
#pragma unroll
            for (int w = 1; w < kSfWarps; ++w) {
                const float ob = pv[w * ldk + j];
                const int oi = pi[w * ldk + j];
                if (ob > b || (ob == b && oi < ib)) {
                    b = ob;
                    ib = oi;
                }
            }
            const uint32_t base = ptx::map_to_rank(ptx::smem_u32(m.xpart), 0);
            ptx::st_cluster_f32(base + ((rank * (uint32_t)ldk) + (uint32_t)j) * 4u, b);
            ptx::st_cluster_u32(base + (((C + rank) * (uint32_t)ldk) + (uint32_t)j) * 4u, (uint32_t)ib);
        }
        ptx::cluster_sync_all();      // after this barrier nothing is written into another CTA any more
        if (rank == 0) {
            const int *xi = reinterpret_cast<const int *>(m.xpart + (size_t)C * ldk);
            const int seg = t_begin - out0;
            for (int j = tid; j < B; j += kSfThreads) {
                float b = m.xpart[j];
                int ib = xi[j];
                for (uint32_t r = 1; r < C; ++r) {     // ranks hold ascending row ranges: strict > keeps the lower index
                    const float ob = m.xpart[r * ldk + j];
                    if (ob > b) {
                        b = ob;
                        ib = xi[r * ldk + j];
                    }
                }
                merged_idx[seg + j] = __ldcg(order + t_begin + M + j);
                merge_partner[seg + j] = ib;
                merge_weight[seg + j] = b * m.vs[j];    // (K U) V, the product the plan stores
            }
        }
    }

    // fp32 storage: the plan in place in the workspace tile (row pitch score_pitch(B)), after the pairing
    // because the tile may be where K lives
    if (!pbuf) {
        for (int idx = tid; idx < Ml * B; idx += kSfThreads) {
            const int i = idx / B, j = idx - i * B;
            Sg[(size_t)(row_lo + i) * ldS + j] = (m.Ks[(size_t)i * ldr + j] * m.us[i]) * m.vs[j];
        }
    }
    if (scores_done) ptx::grid_dep_wait();
}

}  // namespace rtp
