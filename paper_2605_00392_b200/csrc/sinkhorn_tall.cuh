// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C) in scaling form for
// score tiles too wide for the kernels of sinkhorn_cluster.cuh: images with many tokens (thousands
// per image, as the OCR models with large visual token sets produce), up to 4092 pruned tokens.  One
// cluster of 8 CTAs per image (16 when the batch is small enough to leave SMs idle otherwise); the tile's rows (kept tokens) are split over the CTAs; K =
// exp((S - c)/eps) is built in place in the image's workspace tile and read once per iteration
// through L2: a CTA's rows are contiguous there, so one thread streams them block by block into a ring
// of shared-memory stages with 1-D bulk copies, a few blocks ahead of the threads (the tile does not
// change between iterations, so the stream runs on across the end of an iteration).
//
// Same recursion and notation as sinkhorn_cluster.cuh (U = e^u, V = e^{v + c/eps}, the dustbin row and
// column carried as scalars).  What differs is the layout: a thread owns fixed columns (16-byte chunks
// ct, ct + W, ...) of every row of its row group, so the column sums K^T U live in registers across
// the whole pass; the row sums K V are completed across the W threads of a row by shuffles and one
// __syncthreads per block of R rows.  The column sums are reduce-scattered over the cluster: CTA r
// owns a slice of the columns, receives the other CTAs' partial sums for it through distributed shared
// memory, adds them in rank order, computes V for the slice and broadcasts it, so every CTA holds
// bit-identical V and takes the same decision to stop.  Two cluster barriers per iteration.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "sinkhorn.cuh"
#include "sinkhorn_cluster.cuh"

namespace rtp {

constexpr int kTallC = 8;             // CTAs per image
constexpr int kTallCMax = 16;         // with few images and a device that schedules such clusters: 16
constexpr int kTallThreads = 512;
constexpr int kTallMaxB = 4092;       // row pitch (B + 4) & ~3 <= 4096 floats = 512 threads x 2 chunks
// The fixed-point test of this kernel: a dual here is the reciprocal of a sum of a thousand or more
// products, whose rounding noise is a few units in the last place, so "the iteration reproduces its
// input" is tested within four units (4 x 2^-23 relative).  With the one-unit test of the smaller tiles,
// images of 4512 tokens spent up to 81 iterations on noise of one or two units after reaching this level
// in 6; against all 100 iterations the plan then differs by 5.5e-7 relative at most.
constexpr float kTallFixedPointTol = 4.76837158e-7f;

// Dynamic shared memory (floats) of sinkhorn_tall_kernel for tiles of at most maxB columns and maxM rows.
__host__ __device__ inline size_t sinkhorn_tall_smem_floats(int maxB, int maxM, int C = kTallC)
{
    const size_t qpr = (size_t)score_pitch(maxB) / 4;
    const size_t sl = (qpr + C - 1) / C;
    const size_t rows_cap = ((size_t)maxM + C - 1) / C;
    return (4 * qpr + 4) + 2 * C * 4 * sl + 2048 + 256 + 64 + 64 + 2 * (rows_cap + 4) + 4;
}
constexpr int kTallMaxStages = 4;
constexpr int kTallStageFloatsMax = 16384;      // a block of rows is at most 64 KB (see the three layouts)

// Sums of R values over the 32 lanes of a warp in 9 (R = 8) or 6 (R = 4) shuffles: every step halves the
// values a lane carries (it keeps one half and hands the other to its partner), so the lanes end up
// holding the total of row `row_of_lane<R>(lane)`.  The order of the additions is the same in every warp.
template <int R> __device__ inline int row_of_lane(int lane)
{
    if constexpr (R == 8) return ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
    else return ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
}
template <int R> __device__ inline float warp_rows_sum(const float (&s)[R], int lane)
{
    static_assert(R == 8 || R == 4, "rows per block");
    float t2[2];
    if constexpr (R == 8) {
        float t4[4];
        const bool hi = lane & 16;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            t4[i] = (hi ? s[i + 4] : s[i]) + __shfl_xor_sync(0xffffffffu, hi ? s[i] : s[i + 4], 16);
        const bool hi8 = lane & 8;
#pragma unroll
        for (int i = 0; i < 2; ++i)
            t2[i] = (hi8 ? t4[i + 2] : t4[i]) + __shfl_xor_sync(0xffffffffu, hi8 ? t4[i] : t4[i + 2], 8);
        const bool hi4 = lane & 4;
        float t = (hi4 ? t2[1] : t2[0]) + __shfl_xor_sync(0xffffffffu, hi4 ? t2[0] : t2[1], 4);
        t += __shfl_xor_sync(0xffffffffu, t, 2);
        t += __shfl_xor_sync(0xffffffffu, t, 1);
        return t;
    } else {
        const bool hi = lane & 16;
#pragma unroll
        for (int i = 0; i < 2; ++i)
            t2[i] = (hi ? s[i + 2] : s[i]) + __shfl_xor_sync(0xffffffffu, hi ? s[i] : s[i + 2], 16);
        const bool hi8 = lane & 8;
        float t = (hi8 ? t2[1] : t2[0]) + __shfl_xor_sync(0xffffffffu, hi8 ? t2[0] : t2[1], 8);
        t += __shfl_xor_sync(0xffffffffu, t, 4);
        t += __shfl_xor_sync(0xffffffffu, t, 2);
        t += __shfl_xor_sync(0xffffffffu, t, 1);
        return t;
    }
}

// One image's tile on one CTA of the cluster.  W threads share a row (G = 512 / W row groups), a thread
// owns NQ 16-byte column chunks, rows are taken R per group at a time.
template <int W, int NQ, int R>
__device__ inline void sinkhorn_tall_solve(float *Kg, int ldS, int M, int B, int Ml, int row_lo, uint32_t rank,
                                           const OtParams &p, float *sm, int smem_floats, uint64_t *full,
                                           WsHeader *__restrict__ hdr, int rows_cap,
                                           const int32_t *__restrict__ ord, __nv_bfloat16 *__restrict__ Pimg,
                                           int pbuf_pitch, int32_t *__restrict__ merged_seg,
                                           int32_t *__restrict__ partner_seg, float *__restrict__ weight_seg,
                                           float *__restrict__ stats_img)
{
    const int C = (int)ptx::cluster_nctarank();      // 8 or 16
    constexpr int G = kTallThreads / W;
    constexpr int WPG = W / 32;
    constexpr int kWarps = kTallThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ct = tid % W, g = tid / W;
    const int qpr = ldS >> 2;                 // 16-byte chunks per row of the tile
    const int ldc = qpr * 4;
    const int sl = (qpr + C - 1) / C;         // chunks per owner slice
    const int slc = 4 * sl;                   // columns per owner slice (<= 512)

    float *vs = sm;                           // [ldc + 4]      V of every column
    float *xrecv = vs + ldc + 4;              // [2][C][slc]    partial column sums received (pairing: values, indices)
    float *cpart = xrecv + 2 * C * slc;       // [2][1024]      row group 1's column partials (pairing: values, indices)
    float *red = cpart + 2048;                // [2][16][8]     per-warp row-sum partials, double-buffered by block
    float *wred = red + 256;                  // [2][16] + [2]  per-warp sums of V and moves; the groups' sums of U
    float *xs = wred + 64;                    // [4][C]         per-CTA sums of U, sums of V, continue flags, moves
    float *us = xs + 64;                      // [rows_cap + 4] U of this CTA's rows
    int *toks = reinterpret_cast<int *>(us + rows_cap + 4);   // [rows_cap] token position of this CTA's rows
    const int fixed_floats = (int)((us + rows_cap + 4 + rows_cap) - sm + 3) & ~3;
    float *ring = sm + fixed_floats;          // [NS][G R ldS]  blocks of rows of K on their way to the threads
    const int stage_floats = G * R * ldS;
    const int NS = max(1, min(kTallMaxStages, (smem_floats - fixed_floats) / stage_floats));

    int cq[NQ];
    bool cv[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        cq[q] = q * W + ct;
        cv[q] = cq[q] < qpr;
    }
    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);
    const float v_init = expf(shift * inv_eps);       // v = 0
    const float Bf = (float)B, Mf = (float)M;

    for (int i = tid; i < Ml; i += kTallThreads) {
        toks[i] = __ldcg(ord + row_lo + i);
        us[i] = 1.f;                                  // u = 0
    }
    // ---- K = exp((S - c)/eps) of this CTA's rows, in place, zero from column B on ---------------------
    {
        const int total_q = Ml * qpr;
        for (int q0 = tid; q0 < total_q; q0 += kTallThreads * 4) {
            float4 s[4];
            int ii[4], jj[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kTallThreads;
                ii[a] = q / qpr;
                jj[a] = (q - ii[a] * qpr) << 2;
                s[a] = (q < total_q) ? __ldcg(reinterpret_cast<const float4 *>(Kg + (size_t)ii[a] * ldS + jj[a]))
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int q = q0 + a * kTallThreads;
                if (q < total_q) {
                    float4 k;
                    k.x = (jj[a] + 0 < B) ? exp_fast((s[a].x - shift) * inv_eps) : 0.f;
                    k.y = (jj[a] + 1 < B) ? exp_fast((s[a].y - shift) * inv_eps) : 0.f;
                    k.z = (jj[a] + 2 < B) ? exp_fast((s[a].z - shift) * inv_eps) : 0.f;
                    k.w = (jj[a] + 3 < B) ? exp_fast((s[a].w - shift) * inv_eps) : 0.f;
                    *reinterpret_cast<float4 *>(Kg + (size_t)ii[a] * ldS + jj[a]) = k;
                }
            }
        }
    }
    for (int j = tid; j < ldc; j += kTallThreads) vs[j] = (j < B) ? v_init : 0.f;
    if (tid == 0) {
        for (int s = 0; s < kTallMaxStages; ++s) ptx::mbar_init(&full[s], 1);
        ptx::fence_mbar_init();
    }
    ptx::fence_proxy_async_all();     // K was stored through the generic proxy; the bulk copies read it
    __syncthreads();              // K (re-read from L2 below by other threads of this CTA), vs, us, toks
    // every CTA of the cluster is running and has its shared memory laid out before anyone writes into it
    ptx::cluster_sync_all();

    // rows of block `blk` for this thread's group: blk * G * R + g * R + r
    auto load_block = [&](int blk, float4 (&k)[R][NQ]) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int i = (blk * G + g) * R + r;
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                k[r][q] = (i < Ml && cv[q]) ? __ldcg(reinterpret_cast<const float4 *>(Kg + (size_t)i * ldS) + cq[q])
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    const int nblk = (Ml + G * R - 1) / (G * R);
    // The stream of blocks: load n brings block n % nblk into stage n % NS; it is issued once every thread
    // has taken block n - NS out of that stage (the __syncthreads of that block).  At most iters * nblk
    // loads are ever needed; those still in flight when the loop ends early are waited for below.
    const uint32_t n_max = (uint32_t)min((long long)p.iters * nblk, 0x7fffffffLL);
    const uint32_t ring_u32 = ptx::smem_u32(ring);
    auto issue = [&](uint32_t n) {
        const int blk = (int)(n % (uint32_t)nblk), s = (int)(n % (uint32_t)NS);
        const int rows = min(G * R, Ml - blk * G * R);
        const uint32_t bytes = (uint32_t)rows * (uint32_t)ldS * 4u;
        ptx::mbar_arrive_expect_tx(&full[s], bytes);
        ptx::bulk_load(ring_u32 + (uint32_t)s * (uint32_t)stage_floats * 4u, Kg + (size_t)blk * G * R * ldS, bytes,
                       &full[s]);
    };
    if (tid == 0)
        for (uint32_t n = 0; n < min((uint32_t)NS, n_max); ++n) issue(n);
    uint32_t n = 0;               // blocks taken so far, over all iterations
    bool gave_up = false;
    // byte offsets inside a stage: this thread's row slot, a row, its chunks (a chunk past the row's end is
    // replaced by the thread's first one: it is read, weighted by V = 0, and its column sums are dropped)
    const uint32_t stage_bytes = (uint32_t)stage_floats * 4u, row_bytes = (uint32_t)ldS * 4u;
    const uint32_t lane_off = (uint32_t)g * (uint32_t)R * row_bytes;
    uint32_t chunk_off[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) chunk_off[q] = 16u * (uint32_t)(cv[q] ? cq[q] : (cv[0] ? cq[0] : 0));
    const uint32_t xrecv_u32 = ptx::smem_u32(xrecv), xs_u32 = ptx::smem_u32(xs), vs_u32 = ptx::smem_u32(vs);

    // ---- the iterations --------------------------------------------------------------------------------
    float sumV = Bf * v_init, Vd = v_init;    // the same in every thread of every CTA
    int done = 0;
    float last_move = 0.f;
    for (int it = 0; it < p.iters; ++it) {
        float4 V[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q)
            V[q] = cv[q] ? *reinterpret_cast<const float4 *>(vs + 4 * cq[q]) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float Ud = Bf * rcp_fast(kappa * (sumV + Vd));
        const float kVd = kappa * Vd;
        float4 colacc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) colacc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float usum = 0.f;

        // A block's work has two halves: (a) its rows out of the ring, their partial sums against V, this
        // warp's part of the R row sums to shared memory; (b) after a __syncthreads, the row sums, U, and the
        // column accumulation.  Half (a) of block b + 1 is issued ahead of half (b) of block b, so the two
        // dependent chains (shuffle trees, the reciprocal) overlap; one __syncthreads per block.
        auto first_half = [&](int blk, uint32_t nn, float4 (&kk)[R][NQ]) {
            const uint32_t stg = nn % (uint32_t)NS;
            if (!gave_up && !ptx::mbar_wait(&full[stg], (nn / (uint32_t)NS) & 1u)) gave_up = true;
            const uint32_t base = ring_u32 + stg * stage_bytes + lane_off;
            float s[R];
            if ((blk * G + g + 1) * R <= Ml && !gave_up) {       // all R rows exist: nothing to mask but the columns
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float a = 0.f;
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        // (threads past the row's end read a chunk of their own row slot: finite values
                        // from the tile, multiplied by V = 0 here and never sent on)
                        kk[r][q] = ptx::ld_shared_v4(base + (uint32_t)r * row_bytes + chunk_off[q]);
                        a = fmaf(kk[r][q].x, V[q].x, a);
                        a = fmaf(kk[r][q].y, V[q].y, a);
                        a = fmaf(kk[r][q].z, V[q].z, a);
                        a = fmaf(kk[r][q].w, V[q].w, a);
                    }
                    s[r] = a;
                }
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int i = (blk * G + g) * R + r;
                    float a = 0.f;
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        kk[r][q] = (i < Ml && cv[q] && !gave_up)
                                       ? ptx::ld_shared_v4(base + (uint32_t)r * row_bytes + chunk_off[q])
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                        a = fmaf(kk[r][q].x, V[q].x, a);
                        a = fmaf(kk[r][q].y, V[q].y, a);
                        a = fmaf(kk[r][q].z, V[q].z, a);
                        a = fmaf(kk[r][q].w, V[q].w, a);
                    }
                    s[r] = a;
                }
            }
            // this warp's part of the R row sums: one lane per row writes it
            const float wsum = warp_rows_sum<R>(s, lane);
            if ((lane & (32 / R - 1)) == 0) red[(blk & 1) * 128 + warp * 8 + row_of_lane<R>(lane)] = wsum;
        };
        float4 kn[R][NQ];
        if (nblk > 0) first_half(0, n, kn);
        for (int blk = 0; blk < nblk; ++blk, ++n) {
            __syncthreads();      // the parts of block blk's row sums are in; every thread holds its K values
            if (tid == 0 && n + (uint32_t)NS < n_max) issue(n + (uint32_t)NS);    // so its stage is free again
            float4 k[R][NQ];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int q = 0; q < NQ; ++q) k[r][q] = kn[r][q];
            if (blk + 1 < nblk) first_half(blk + 1, n + 1, kn);
            // every warp adds the WPG parts of each row in the same order: lane l takes row l % R
            const float *rb = red + (blk & 1) * 128;
            const int rr = lane % R, wq = lane / R;
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < WPG * R / 32; ++w) t += rb[(g * WPG + wq + w * (32 / R)) * 8 + rr];
#pragma unroll
            for (int o = R; o < 32; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            const int i0 = (blk * G + g) * R;
            const bool valid_own = i0 + rr < Ml;
            const float Uown = valid_own ? rcp_fast(t + kVd) : 0.f;
            if (ct < R && valid_own) us[i0 + rr] = Uown;      // ct < R: lane ct of the group's first warp, rr = ct
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float U = __shfl_sync(0xffffffffu, Uown, r);
                usum += U;                                    // (only the group's first thread's sum is used)
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    colacc[q].x = fmaf(k[r][q].x, U, colacc[q].x);
                    colacc[q].y = fmaf(k[r][q].y, U, colacc[q].y);
                    colacc[q].z = fmaf(k[r][q].z, U, colacc[q].z);
                    colacc[q].w = fmaf(k[r][q].w, U, colacc[q].w);
                }
            }
        }
        // the row groups' column partials and sums of U meet in group 0
        if (ct == 0) wred[32 + g] = usum;
        if constexpr (G == 2) {
            if (g == 1) {
#pragma unroll
                for (int q = 0; q < NQ; ++q)
                    if (cv[q]) *reinterpret_cast<float4 *>(cpart + 4 * cq[q]) = colacc[q];
            }
        }
        __syncthreads();
        if (g == 0) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (!cv[q]) continue;
                float4 cs = colacc[q];
                if constexpr (G == 2) {
                    const float4 o = *reinterpret_cast<const float4 *>(cpart + 4 * cq[q]);
                    cs.x += o.x;
                    cs.y += o.y;
                    cs.z += o.z;
                    cs.w += o.w;
                }
                // to the CTA that owns these columns
                const int owner = cq[q] / sl, off = cq[q] - owner * sl;
                const uint32_t a = ptx::map_to_rank(xrecv_u32 + (uint32_t)((rank * slc) + 4 * off) * 4u, (uint32_t)owner);
                ptx::st_cluster_f32(a, cs.x);
                ptx::st_cluster_f32(a + 4u, cs.y);
                ptx::st_cluster_f32(a + 8u, cs.z);
                ptx::st_cluster_f32(a + 12u, cs.w);
            }
        }
        if (tid == 0) {
            float su = wred[32];
            if constexpr (G == 2) su += wred[33];
            for (uint32_t r = 0; r < (uint32_t)C; ++r)
                ptx::st_cluster_f32(ptx::map_to_rank(xs_u32 + rank * 4u, r), su);
        }
        ptx::cluster_sync_all();

        // ---- this CTA's slice of V from the completed column sums, broadcast to the cluster -----------
        float su_all = 0.f;
        for (int r = 0; r < C; ++r) su_all += xs[r];          // read here: the next pass may overwrite it early
        int cont = 0;
        float move = 0.f, nv = 0.f;
        const int j = (int)rank * slc + tid;
        if (tid < slc && j < B) {
            float cs = 0.f;
            for (int r = 0; r < C; ++r) cs += xrecv[r * slc + tid];
            nv = rcp_fast(cs + kappa * Ud);
            const float ov = vs[j];
            move = fabsf(nv - ov) * rcp_fast(ov);
            cont = p.tol > 0.f ? (move > p.tol) : (p.stop_fp ? (move > kTallFixedPointTol) : 1);
            const uint32_t a = vs_u32 + (uint32_t)j * 4u;
            for (uint32_t r = 0; r < (uint32_t)C; ++r) ptx::st_cluster_f32(ptx::map_to_rank(a, r), nv);
        }
        const float wv = warp_sum(nv), wm = warp_max(move);
        if (lane == 0) {
            wred[warp] = wv;
            wred[16 + warp] = wm;
        }
        cont = __syncthreads_or(cont);
        if (tid == 0) {
            float sv = 0.f, mv = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                sv += wred[w];
                mv = fmaxf(mv, wred[16 + w]);
            }
            for (uint32_t r = 0; r < (uint32_t)C; ++r) {
                ptx::st_cluster_f32(ptx::map_to_rank(xs_u32 + (uint32_t)(C + rank) * 4u, r), sv);
                ptx::st_cluster_f32(ptx::map_to_rank(xs_u32 + (uint32_t)(2 * C + rank) * 4u, r), cont ? 1.f : 0.f);
                ptx::st_cluster_f32(ptx::map_to_rank(xs_u32 + (uint32_t)(3 * C + rank) * 4u, r), mv);
            }
        }
        ptx::cluster_sync_all();

        // every thread of every CTA: the sums, the dustbin column, the decision to go on
        const float nVd = Mf * rcp_fast(kappa * (su_all + Ud));
        const float md = fabsf(nVd - Vd) * rcp_fast(Vd);
        bool go = p.tol > 0.f ? (md > p.tol) : (p.stop_fp ? (md > kTallFixedPointTol) : true);
        float sv_all = 0.f, mv_all = md;
        for (int r = 0; r < C; ++r) {
            sv_all += xs[C + r];
            go = go || (xs[2 * C + r] != 0.f);
            mv_all = fmaxf(mv_all, xs[3 * C + r]);
        }
        sumV = sv_all;
        Vd = nVd;
        last_move = mv_all;
        ++done;
        if (!go) break;
    }
    if (rank == 0 && tid == 0) {
        stats_img[5] = (float)done;
        stats_img[6] = last_move;
    }
    // loads issued for iterations that did not run: wait for them before this CTA's shared memory goes away
    if (tid == 0) {
        const uint32_t n_issued = min(n + (uint32_t)NS, n_max);
        for (uint32_t m = n; m < n_issued; ++m)
            if (!ptx::mbar_wait(&full[m % (uint32_t)NS], (m / (uint32_t)NS) & 1u)) gave_up = true;
    }
    if (gave_up) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);

    // ---- plan P = U K V of this CTA's rows, and per column the best K_ij U_i over them ------------------
    const int kpad = (B + 63) & ~63;          // the tensor-core merge reads whole 64-column blocks
    {
        float4 V[NQ];
        float best[NQ][4];
        int bi[NQ][4];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            V[q] = cv[q] ? *reinterpret_cast<const float4 *>(vs + 4 * cq[q]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                best[q][e] = -INFINITY;
                bi[q][e] = 0x7fffffff;
            }
        }
        for (int blk = 0; blk < nblk; ++blk) {
            float4 k[R][NQ];
            load_block(blk, k);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int i = (blk * G + g) * R + r;
                if (i >= Ml) continue;
                const float U = us[i];
                const int tok = toks[i];
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (!cv[q]) continue;
                    const float ku[4] = {k[r][q].x * U, k[r][q].y * U, k[r][q].z * U, k[r][q].w * U};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (ku[e] > best[q][e]) {        // rows ascend within a thread: strict > keeps the lower index
                            best[q][e] = ku[e];
                            bi[q][e] = row_lo + i;
                        }
                    }
                    const float4 P = make_float4(ku[0] * V[q].x, ku[1] * V[q].y, ku[2] * V[q].z, ku[3] * V[q].w);
                    if (Pimg) {
                        if (4 * cq[q] < kpad) {          // alpha P in bf16, row = the kept token's position in X
                            __nv_bfloat162 o[2];
                            o[0] = __floats2bfloat162_rn(p.alpha * P.x, p.alpha * P.y);
                            o[1] = __floats2bfloat162_rn(p.alpha * P.z, p.alpha * P.w);
                            *reinterpret_cast<uint2 *>(Pimg + (size_t)tok * pbuf_pitch + 4 * cq[q]) =
                                *reinterpret_cast<uint2 *>(o);
                        }
                    } else {
                        *reinterpret_cast<float4 *>(Kg + (size_t)i * ldS + 4 * cq[q]) = P;   // fp32: in place
                    }
                }
            }
        }
        if (Pimg && kpad > ldc) {             // zero columns between the tile's pitch and the 64-column block's end
            const int zq = (kpad - ldc) >> 2;
            for (int idx = tid; idx < Ml * zq; idx += kTallThreads) {
                const int i = idx / zq, c = idx - i * zq;
                *reinterpret_cast<uint2 *>(Pimg + (size_t)toks[i] * pbuf_pitch + ldc + 4 * c) = make_uint2(0u, 0u);
            }
        }
        // pairing: the row groups meet in group 0, the CTAs in the owner of the column
        int *cparti = reinterpret_cast<int *>(cpart + 1024);
        if constexpr (G == 2) {
            if (g == 1) {
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (!cv[q]) continue;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        cpart[4 * cq[q] + e] = best[q][e];
                        cparti[4 * cq[q] + e] = bi[q][e];
                    }
                }
            }
            __syncthreads();
        }
        if (g == 0) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (!cv[q]) continue;
                const int owner = cq[q] / sl, off = cq[q] - owner * sl;
                const uint32_t a = ptx::map_to_rank(xrecv_u32 + (uint32_t)((rank * slc) + 4 * off) * 4u, (uint32_t)owner);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float b = best[q][e];
                    int ib = bi[q][e];
                    if constexpr (G == 2) {
                        const float ob = cpart[4 * cq[q] + e];
                        const int oi = cparti[4 * cq[q] + e];
                        if (ob > b || (ob == b && oi < ib)) {
                            b = ob;
                            ib = oi;
                        }
                    }
                    ptx::st_cluster_f32(a + 4u * e, b);
                    ptx::st_cluster_u32(a + (uint32_t)(C * slc) * 4u + 4u * e, (uint32_t)ib);
                }
            }
        }
        ptx::cluster_sync_all();      // after this barrier nothing is written into another CTA any more
        const int j = (int)rank * slc + tid;
        if (tid < slc && j < B) {
            const int *xi = reinterpret_cast<const int *>(xrecv + C * slc);
            float b = xrecv[tid];
            int ib = xi[tid];
            for (int r = 1; r < C; ++r) {      // ranks hold ascending row ranges: strict > keeps the lower index
                const float ob = xrecv[r * slc + tid];
                if (ob > b) {
                    b = ob;
                    ib = xi[r * slc + tid];
                }
            }
            merged_seg[j] = __ldcg(ord + M + j);
            partner_seg[j] = ib;
            weight_seg[j] = b * vs[j];          // (K U) V, the product the plan stores
        }
    }
}

// grid = batch * 8 CTAs, clusters of 8 along x.  Takes the images that the cluster kernels ahead of it
// left (fast_c, fast_floats: their cluster size and shared-memory floats) and whose B <= kTallMaxB; every
// early return depends on the image only, so a cluster leaves as a whole.
__global__ void __launch_bounds__(kTallThreads, 1)
sinkhorn_tall_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                     const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                     float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                     __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch, int32_t *__restrict__ merged_idx,
                     int32_t *__restrict__ merge_partner, float *__restrict__ merge_weight,
                     float *__restrict__ stats, int fast_c, int fast_floats, int smem_floats,
                     WsHeader *__restrict__ hdr)
{
    extern __shared__ __align__(16) float sm[];
    __shared__ uint64_t s_full[kTallMaxStages];
    const uint32_t rank = ptx::cluster_ctarank();
    const int nC = (int)ptx::cluster_nctarank();
    const int img = blockIdx.x / nC;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();         // scores, counts and order come from the kernels ahead
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = __ldcg(counts + img), B = N - M;
    if (B == 0 || B > kTallMaxB) return;
    if (fast_c > 0 && sinkhorn_cluster_handles(M, B, fast_c, fast_floats)) return;   // solved ahead of this kernel
    const int rows_per = (M + nC - 1) / nC;
    const int row_lo = min(M, (int)rank * rows_per);
    const int Ml = min(M, row_lo + rows_per) - row_lo;       // this CTA's rows (may be 0)
    const int ldS = score_pitch(B);
    float *Kg = kmat + kmat_offset(kmat_stride, t_begin, img) + (size_t)row_lo * ldS;
    const int seg = t_begin - __ldcg(out_offsets + img);
    __nv_bfloat16 *Pimg = pbuf ? pbuf + (size_t)t_begin * pbuf_pitch : nullptr;
    const int qpr = ldS >> 2;
#define RTP_TALL(W, NQ, R)                                                                                     \
    sinkhorn_tall_solve<W, NQ, R>(Kg, ldS, M, B, Ml, row_lo, rank, p, sm, smem_floats, s_full, hdr, rows_per,  \
                                  order + t_begin, Pimg,                                                      \
                                  pbuf_pitch, merged_idx + seg, merge_partner + seg, merge_weight + seg,      \
                                  stats + (size_t)img * kStats)
    if (qpr <= 256) RTP_TALL(256, 1, 8);
    else if (qpr <= 512) RTP_TALL(512, 1, 8);
    else RTP_TALL(512, 2, 4);
#undef RTP_TALL
}

}  // namespace rtp
