// Stage 2 of Algorithm 1 in ONE kernel, one cluster of two CTAs per image: cosine scores (Section
// 3.3.2) on the tcgen05 tensor cores, dustbin augmentation and Sinkhorn iterations (Eq. 5, Appendix C)
// with the kernel matrix K held in REGISTERS, and the merge T_k + alpha P T_p (Eq. 7) on the tensor
// cores again, written packed.  Nothing goes through global memory between the steps: S lives in
// tensor memory, K in registers, the plan P in shared memory.
//
// Taken by runs whose images all have at most kFuMaxTok tokens and at most kFuMaxB pruned tokens, bf16
// storage, width a multiple of 64, scaling form (fused_eligible() on the host); everything else keeps
// the separate kernels.
//
// Work split inside a cluster (rank r = 0, 1): rank r owns the kept positions [r * half, ...) of the
// image, half = ceil(M / 2): its rows of S, K, P and of the output Y.  Both CTAs need all B pruned rows.
//
// Operand fetch: kept and pruned rows are scattered over the image, so the operand tiles are gathered
// by eleven producer warps with 16-byte cp.async copies straight into the 128-byte-swizzled layout
// the UMMA descriptors expect, k-block by k-block, several k-blocks in flight.  Measured on a B200, per
// SM, on rows that sit in L2: 16-byte loads through the load/store path 70 B/clk, tiled TMA boxes of
// 128-byte rows 31 B/clk, tile::gather4 7 B/clk; so the gather is faster than a tiled copy of a compact
// copy would be, and moves only the rows that are needed.
//
// Sinkhorn iteration: as in sinkhorn_cluster.cuh (one pass per iteration, LR lanes share a row, column
// sums completed over the warps in shared memory and over the two CTAs through distributed shared
// memory), but a thread's K values never leave its registers.
// Merge: for each tile of 64 output columns, D = [I | alpha P] . [T_k rows of the tile ; T_p] (the
// identity block carries the kept token's own row through the tensor cores, exact in the fp32
// accumulator); four accumulator stages in tensor memory; the epilogue converts to bf16, stages a
// warp's 32 rows in shared memory and writes them with coalesced 16-byte stores (the rows of a CTA are
// consecutive rows of Y).
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "sinkhorn.cuh"
#include "sinkhorn_cluster.cuh"

namespace rtp {

constexpr int kFuThreads = 512;
constexpr int kFuWarps = kFuThreads / 32;
// Warp roles.  Scores: warp 0 lane 0 issues the UMMAs, warps 1-15 gather the operands.  Merge: warps 0-7 are
// the epilogue (TMEM lane quarter warp % 4 of row tile warp / 4), warp 8 lane 0 issues the UMMAs, warps
// 9-15 gather the operands.
constexpr int kFuScProducers = (kFuWarps - 1) * 32;
constexpr int kFuEpiWarps = 8;
constexpr int kFuMmaWarp = 8;
constexpr int kFuMgProducers = (kFuWarps - kFuMmaWarp - 1) * 32;
constexpr int kFuStageRowsMax = 448;      // rows of a stage (kept rows of the CTA + pruned rows, each rounded up to 16)
constexpr int kFuScChunks = (8 * kFuStageRowsMax + kFuScProducers - 1) / kFuScProducers;   // copies per producer thread and stage
constexpr int kFuMgChunks = (8 * kFuStageRowsMax + kFuMgProducers - 1) / kFuMgProducers;
constexpr int kFuMaxTok = 512;            // tokens per image
constexpr int kFuMaxB = 256;              // pruned tokens per image: one UMMA N, half of tensor memory
constexpr int kFuMaxRows = 256;           // kept rows per CTA: two tiles of 128
constexpr int kFuKRegs = 64;              // K values a thread may hold
constexpr int kFuTileM = 128;
constexpr int kFuBK = 64;                 // bf16 per k-block = one 128-byte swizzle row
constexpr int kFuNT = 64;                 // output columns per merge tile
constexpr int kFuABytes = kFuTileM * 128; // 16 KB: 128 rows x 64 bf16, K-major
constexpr int kFuBoxBytes = 64 * 128;     // 8 KB: 64 rows x 64 bf16
constexpr int kFuScStages = 6;            // at most
constexpr int kFuMgStages = 6;            // at most
constexpr int kFuAccStages = 4;           // accumulator stages of the merge (128 TMEM columns each)
constexpr int kFuSharedBytes = 15360;     // FuShared, rounded up
constexpr int kFuArenaBytes = 210 * 1024;
constexpr int kFuPartBytes = 32 * 1024;   // column partials of the iterations, then of the pairing
constexpr int kFuPartOffset = kFuArenaBytes - kFuPartBytes;
constexpr int kFuSmemBytes = 1024 + kFuSharedBytes + kFuArenaBytes;
static_assert(kFuSmemBytes <= 227 * 1024, "more shared memory than a CTA can have");

struct FuShared {
    uint64_t sc_full[kFuScStages], sc_empty[kFuScStages], sc_accum;
    uint64_t mg_full[kFuMgStages], mg_empty[kFuMgStages];
    uint64_t acc_full[kFuAccStages], acc_empty[kFuAccStages];
    uint64_t xbar[2];                           // the other CTA's column sums of an iteration have arrived (by parity)
    uint32_t tmem_base;
    volatile int abort_flag;
    int out0;
    float vsum[kFuWarps];
    float wsum[kFuWarps];
    __align__(16) float xusum[2][4];            // the other CTA's sum of U, by iteration parity
    __align__(16) float inv_nj[kFuMaxB];        // 1 / |x_j| of the pruned tokens
    __align__(16) float inv_ni[kFuMaxRows];     // 1 / |x_i| of this CTA's kept rows
    __align__(16) float vs[kFuMaxB + 8];        // V_j, V_d at [ldk]: read as 16-byte vectors
    int rowtok[kFuMaxRows + kFuMaxB + 32];      // image-local token of each row of a stage (-1: a row of zeros)
    __align__(16) float xpart[2][kFuMaxB];      // the other CTA's column partials, by iteration parity
    float pairv[2][kFuMaxB];                    // rank 0: per-CTA column maxima of K U ...
    int pairi[2][kFuMaxB];                      // ... and their rows
};
static_assert(sizeof(FuShared) <= kFuSharedBytes, "FuShared outgrew its region");

// K values per thread for a tile of `rows` rows (one CTA's share) and B columns; 0 if no layout fits.
__host__ __device__ inline int fused_k_regs(int rows, int B)
{
    const int ldk = sinkhorn_ldk(B);
    if (ldk > 256) return 0;
    const int lr = ldk <= 128 ? 8 : 16;
    const int rows_per_step = kFuWarps * (32 / lr);
    const int ns = (rows + rows_per_step - 1) / rows_per_step;
    return (ns < 1 ? 1 : ns) * (ldk / lr);
}

// Operand arrays in shared memory are rows of 128 bytes (64 bf16), eight-row groups of 1024 bytes, the
// 16-byte pieces of a row XOR-swizzled by the row's place in its group: what a UMMA descriptor with the
// 128-byte swizzle addresses, as a K-major operand (rows = M or N index) or as an MN-major one (rows = k
// index).  A stage of either ring holds this CTA's kept rows (rounded up to 16 rows, zeros past the last)
// followed by the pruned rows (likewise); the plan is one such array of the CTA's rows per 64 columns.
// A 128-row UMMA operand that starts at row 128 t of an array with fewer than 128 (t + 1) rows reads on
// into whatever follows (rows nobody uses): sizes below keep those reads inside the arena.
__host__ __device__ inline int fused_stage_bytes(int rows, int B)
{
    return (((rows + 15) & ~15) + ((B + 15) & ~15)) * 128;
}
__host__ __device__ inline int fused_plan_bytes(int rows, int B)
{
    return ((B + 63) / 64) * ((rows + 15) & ~15) * 128;
}

// Every image of a run with at most max_tokens tokens and max_b pruned tokens fits the fused kernel:
// K in 64 registers per thread, at least two stages in either ring.
__host__ inline bool fused_eligible(int d, int max_tokens, int max_b)
{
    if (d % 64 != 0 || max_tokens > kFuMaxTok || max_b > kFuMaxB) return false;
    for (int b = 0; b <= max_b; ++b) {
        const int m = max_tokens - b > 1 ? max_tokens - b : 1;
        const int rows = (m + 1) / 2;
        if (rows > kFuMaxRows) return false;
        if (b > 0) {
            const int regs = fused_k_regs(rows, b);
            if (regs == 0 || regs > kFuKRegs) return false;
        }
        if (fused_stage_bytes(rows, b) > kFuStageRowsMax * 128) return false;
        if (2 * fused_stage_bytes(rows, b) + kFuABytes > kFuArenaBytes) return false;
        if (fused_plan_bytes(rows, b) + 2 * fused_stage_bytes(rows, b) + kFuABytes > kFuArenaBytes) return false;
    }
    return true;
}

__device__ inline void mbar_inval(uint64_t *bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}

struct FuImage {
    int t_begin, N, M, B;
    int half, row_lo, Ml, ntile;  // this CTA's kept rows
    int ldk, nkb;
    int Ra, Rb;                   // rows a stage holds: kept rows and pruned rows, each rounded up to 16
};

struct FuIterState {
    int done;
    float last_move;
};

// One 32-bit word into the other CTA's shared memory, counted (4 bytes) on a barrier there when it has landed.
__device__ inline void st_async_peer(uint32_t remote_addr, uint32_t value, uint32_t remote_bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];" ::"r"(remote_addr), "r"(value),
                 "r"(remote_bar)
                 : "memory");
}

// The iterations, K in registers.  Row i of this CTA (kept position row_lo + i) lives in the LR lanes
// (step s, warp w, slot) with i = (s * 16 + w) * (32 / LR) + slot; lane `sub` of a row holds the 16-byte
// column chunks sub, sub + LR, ...  Column sums: over a warp's row slots by shuffles, over the warps in
// shared memory, over the two CTAs by sending this CTA's sums into the other's shared memory with
// asynchronous stores that are counted on a barrier there: no cluster-wide barrier in the loop.  Both
// CTAs add the two partial sums of a column (a + b = b + a), so they hold bit-identical V and leave the
// loop together.  `round` counts the exchanges of the kernel (the barriers' phases run on across images).
// On return vs[] holds the final V (V_d at [ldk]) and U[] the final U of the thread's rows.
template <int LR, int CPL, int NS>
__device__ inline FuIterState fused_iterate(const float4 (&k)[NS][CPL / 4], float (&U)[NS], FuShared *sh, float *part,
                                            int Ml, int M, int B, uint32_t rank, const OtParams &p, float kappa,
                                            float v_init, uint32_t &round, WsHeader *hdr)
{
    constexpr int ldk = LR * CPL;
    constexpr int RPS = 32 / LR;
    constexpr int NQ = CPL / 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;
    const float Bf = (float)B, Mf = (float)M;

    for (int j = tid; j <= ldk; j += kFuThreads) sh->vs[j] = (j < B || j == ldk) ? v_init : 0.f;
#pragma unroll
    for (int s = 0; s < NS; ++s) U[s] = 0.f;
    __syncthreads();
    const uint32_t peer = rank ^ 1u;
    const uint32_t xpart_peer = ptx::map_to_rank(ptx::smem_u32(&sh->xpart[0][0]), peer);
    const uint32_t xusum_peer = ptx::map_to_rank(ptx::smem_u32(&sh->xusum[0][0]), peer);
    const uint32_t xbar_peer = ptx::map_to_rank(ptx::smem_u32(&sh->xbar[0]), peer);
    FuIterState st{0, 0.f};

    for (int it = 0; it < p.iters; ++it, ++round) {
        const uint32_t par = round & 1u, phase = (round >> 1) & 1u;
        float4 V[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(sh->vs + 4 * (q * LR + sub));
        // sum of V over the real columns (V is 0 past column B): the LR lanes of a row hold all columns between
        // them, so the sum comes out of the same shuffles as a row sum, in every thread and in the same order
        float sumV = 0.f;
#pragma unroll
        for (int q = 0; q < NQ; ++q) sumV += (V[q].x + V[q].y) + (V[q].z + V[q].w);
#pragma unroll
        for (int o = 1; o < LR; o <<= 1) sumV += __shfl_xor_sync(0xffffffffu, sumV, o);
        const float Vd = sh->vs[ldk];
        const float Ud = Bf * rcp_fast(kappa * (sumV + Vd));
        const float kVd = kappa * Vd;
        float4 colacc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) colacc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float usum = 0.f;
        // this exchange's arrival on the local barrier: the other CTA's ldk column sums and its sum of U
        if (tid == 0) ptx::mbar_arrive_expect_tx(&sh->xbar[par], (uint32_t)(ldk + 1) * 4u);

#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const int i = (s * kFuWarps + warp) * RPS + slot;
            const bool valid = i < Ml;
            // four partial sums: a chain of NQ dependent multiply-adds instead of 4 NQ
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                s0 = fmaf(k[s][q].x, V[q].x, s0);
                s1 = fmaf(k[s][q].y, V[q].y, s1);
                s2 = fmaf(k[s][q].z, V[q].z, s2);
                s3 = fmaf(k[s][q].w, V[q].w, s3);
            }
            float sd = (s0 + s1) + (s2 + s3);
#pragma unroll
            for (int o = 1; o < LR; o <<= 1) sd += __shfl_xor_sync(0xffffffffu, sd, o);
            const float u = valid ? rcp_fast(sd + kVd) : 0.f;
            U[s] = u;
            if (sub == 0) usum += u;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                colacc[q].x = fmaf(k[s][q].x, u, colacc[q].x);
                colacc[q].y = fmaf(k[s][q].y, u, colacc[q].y);
                colacc[q].z = fmaf(k[s][q].z, u, colacc[q].z);
                colacc[q].w = fmaf(k[s][q].w, u, colacc[q].w);
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
                *reinterpret_cast<float4 *>(part + warp * ldk + 4 * (q * LR + sub)) = colacc[q];
        }
        usum = warp_sum(usum);
        if (lane == 0) sh->wsum[warp] = usum;
        __syncthreads();

        // V: thread j completes column j over the warps, sends the sum to the other CTA, waits for that CTA's
        int cont = 0;
        float move = 0.f;
        if (tid < ldk) {
            float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
#pragma unroll
            for (int w = 0; w < kFuWarps; w += 4) {
                c0 += part[(w + 0) * ldk + tid];
                c1 += part[(w + 1) * ldk + tid];
                c2 += part[(w + 2) * ldk + tid];
                c3 += part[(w + 3) * ldk + tid];
            }
            const float cs = (c0 + c1) + (c2 + c3);
            st_async_peer(xpart_peer + (par * (uint32_t)kFuMaxB + (uint32_t)tid) * 4u, __float_as_uint(cs), xbar_peer + par * 8u);
            if (!ptx::mbar_wait(&sh->xbar[par], phase)) {
                sh->abort_flag = 1;
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
            }
            float nv = 0.f;
            if (tid < B) {
                nv = rcp_fast((cs + sh->xpart[par][tid]) + kappa * Ud);
                const float ov = sh->vs[tid];
                move = fabsf(nv - ov) * rcp_fast(ov);
                cont = p.tol > 0.f ? (move > p.tol) : (p.stop_fp ? ulp_far(nv, ov) : 1);
                sh->vs[tid] = nv;
            }
        }
        if (tid == kFuThreads - 1) {              // the dustbin column
            float su = 0.f;
#pragma unroll
            for (int w = 0; w < kFuWarps; ++w) su += sh->wsum[w];
            st_async_peer(xusum_peer + par * 16u, __float_as_uint(su), xbar_peer + par * 8u);
            if (!ptx::mbar_wait(&sh->xbar[par], phase)) {
                sh->abort_flag = 1;
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
            }
            const float nVd = Mf * rcp_fast(kappa * ((su + sh->xusum[par][0]) + Ud));
            const float mj = fabsf(nVd - Vd) * rcp_fast(Vd);
            move = fmaxf(move, mj);
            cont |= p.tol > 0.f ? (mj > p.tol) : (p.stop_fp ? ulp_far(nVd, Vd) : 1);
            sh->vs[ldk] = nVd;
        }
        st.last_move = move;
        ++st.done;
        if (!__syncthreads_or(cont)) {
            ++round;
            break;
        }
    }
    // largest relative dual move of the last executed iteration, over the CTA
    float mv = warp_max(st.last_move);
    __syncthreads();
    if (lane == 0) sh->wsum[warp] = mv;
    __syncthreads();
    mv = 0.f;
#pragma unroll
    for (int w = 0; w < kFuWarps; ++w) mv = fmaxf(mv, sh->wsum[w]);
    st.last_move = mv;
    return st;
}

// Pairing, one CTA's part: per column the largest K_ij U_i over this CTA's rows and its row (ties to the
// lower row): over the thread's steps, over the warp's row slots, over the warps in shared memory; the
// result goes to rank 0's pairv / pairi (the cluster barrier that must follow makes it visible there).
template <int LR, int CPL, int NS>
__device__ inline void fused_pair_partials(const float4 (&k)[NS][CPL / 4], const float (&U)[NS], FuShared *sh, float *part,
                                           int Ml, int row_lo, int B, uint32_t rank)
{
    constexpr int ldk = LR * CPL;
    constexpr int RPS = 32 / LR;
    constexpr int NQ = CPL / 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;
    // ---- pairing, this CTA's part: per column the largest K_ij U_i over this CTA's rows and its row
    // (ties to the lower row).  Chunk by chunk: over the thread's steps, over the warp's row slots, to
    // shared memory per warp.
    float *pv = part;
    int *pi = reinterpret_cast<int *>(part + kFuWarps * ldk);
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        float bv[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        int bi[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};
#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const int i = (s * kFuWarps + warp) * RPS + slot;
            if (i < Ml) {
                const float e[4] = {k[s][q].x * U[s], k[s][q].y * U[s], k[s][q].z * U[s], k[s][q].w * U[s]};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (e[c] > bv[c]) {          // rows ascend with s: strict > keeps the lower row
                        bv[c] = e[c];
                        bi[c] = row_lo + i;
                    }
            }
        }
#pragma unroll
        for (int o = LR; o < 32; o <<= 1) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv[c], o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi[c], o);
                if (ov > bv[c] || (ov == bv[c] && oi < bi[c])) {
                    bv[c] = ov;
                    bi[c] = oi;
                }
            }
        }
        if (slot == 0) {
            const int col = 4 * (q * LR + sub);
            *reinterpret_cast<float4 *>(pv + warp * ldk + col) = make_float4(bv[0], bv[1], bv[2], bv[3]);
            *reinterpret_cast<int4 *>(pi + warp * ldk + col) = make_int4(bi[0], bi[1], bi[2], bi[3]);
        }
    }
    __syncthreads();
    if (tid < B) {
        float b = pv[tid];
        int ib = pi[tid];
#pragma unroll
        for (int w = 1; w < kFuWarps; ++w) {
            const float ob = pv[w * ldk + tid];
            const int oi = pi[w * ldk + tid];
            if (ob > b || (ob == b && oi < ib)) {
                b = ob;
                ib = oi;
            }
        }
        ptx::st_cluster_f32(ptx::map_to_rank(ptx::smem_u32(&sh->pairv[rank][tid]), 0), b);
        ptx::st_cluster_u32(ptx::map_to_rank(ptx::smem_u32(&sh->pairi[rank][tid]), 0), (uint32_t)ib);
    }
}

// Everything between the scores and the merge for one tile layout: K into registers, the iterations,
// alpha P of this CTA's rows into its plan arrays, the per-CTA column maxima of K U for the pairing
// (sent to rank 0).  kbuf: this CTA's K rows, pitch ldk + 4 floats, in shared memory (the arena's start,
// which the plan arrays then overwrite: every thread has its K in registers by then).
template <int LR, int CPL, int NS>
__device__ inline FuIterState fused_sinkhorn(FuShared *sh, const float *kbuf, uint8_t *arena, const FuImage &im,
                                             uint32_t rank, const OtParams &p, float kappa, float v_init,
                                             uint32_t &round, WsHeader *hdr)
{
    constexpr int ldk = LR * CPL;
    constexpr int RPS = 32 / LR;
    constexpr int NQ = CPL / 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;
    float *part = reinterpret_cast<float *>(arena + kFuPartOffset);

    float4 k[NS][NQ];
    float U[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const int i = (s * kFuWarps + warp) * RPS + slot;
#pragma unroll
        for (int q = 0; q < NQ; ++q)
            k[s][q] = (i < im.Ml) ? *reinterpret_cast<const float4 *>(kbuf + (size_t)i * (ldk + 4) + 4 * (q * LR + sub))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
    }

    const FuIterState st = fused_iterate<LR, CPL, NS>(k, U, sh, part, im.Ml, im.M, im.B, rank, p, kappa, v_init, round, hdr);
    if (p.iters == 0) {
#pragma unroll
        for (int s = 0; s < NS; ++s) U[s] = ((s * kFuWarps + warp) * RPS + slot < im.Ml) ? 1.f : 0.f;   // u = 0
        __syncthreads();          // every thread has its K before the plan arrays overwrite the buffer
    }

    // ---- alpha P = alpha U K V in bf16 into this CTA's plan arrays (A operand, K-major): one array of the
    // CTA's Ra rows per 64 columns, at arena + kb * Ra * 128.  Columns from B up to the next multiple of 16
    // are zeros (K is zero there): the contraction runs over whole 16-column steps.
    float4 V[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(sh->vs + 4 * (q * LR + sub));
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const int i = (s * kFuWarps + warp) * RPS + slot;
        if (i < im.Ml) {
            const uint32_t row_off = (uint32_t)(i >> 3) * 1024u + (uint32_t)(i & 7) * 128u;
            const float au = p.alpha * U[s];
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int col = 4 * (q * LR + sub);
                if (col < im.Rb) {
                    const int kb = col >> 6, c16 = (col & 63) >> 3;
                    const __nv_bfloat162 lo = __floats2bfloat162_rn((k[s][q].x * au) * V[q].x, (k[s][q].y * au) * V[q].y);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn((k[s][q].z * au) * V[q].z, (k[s][q].w * au) * V[q].w);
                    const uint32_t off = (uint32_t)kb * (uint32_t)(im.Ra * 128) + row_off +
                                         (uint32_t)((c16 ^ (i & 7)) << 4) + (uint32_t)(col & 4) * 2u;
                    *reinterpret_cast<uint2 *>(arena + off) =
                        make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
                }
            }
        }
    }

    fused_pair_partials<LR, CPL, NS>(k, U, sh, part, im.Ml, im.row_lo, im.B, rank);
    return st;
}

// The 16-byte copies of one stage, shared out over NPROD producer threads (this one is number pt): piece
// c = pt + NPROD q is the 16 bytes c & 7 of stage row c >> 3 and lands at its swizzled place; a row without
// a token (rowtok < 0) is written as zeros.  The table holds, per piece, where it comes from in the image
// (64-column block 0) and where it goes in a stage.
template <int NCH>
struct FuChunks {
    uint32_t src_off[NCH];
    uint32_t dst_off[NCH];
    uint32_t real;      // bit q: the piece exists in the image
    int n;              // pieces of this thread
};

template <int NCH, int NPROD>
__device__ inline void fused_chunk_table(FuChunks<NCH> &ck, const FuShared *sh, const FuImage &im, int pt, uint32_t row_bytes)
{
    ck.real = 0;
    ck.n = 0;
    const int total = 8 * (im.Ra + im.Rb);
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
        const int c = pt + NPROD * q;
        ck.src_off[q] = 0;
        ck.dst_off[q] = 0;
        if (c < total) {
            ck.n = q + 1;
            const int row = c >> 3, ch = c & 7;      // Ra is a multiple of 16: row & 7 is the row's place in its group
            const int tok = sh->rowtok[row];
            ck.dst_off[q] = (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((ch ^ (row & 7)) << 4));
            ck.src_off[q] = (uint32_t)max(tok, 0) * row_bytes + (uint32_t)ch * 16u;
            if (tok >= 0) ck.real |= 1u << q;
        }
    }
}

template <int NCH>
__device__ inline void fused_issue_stage(const FuChunks<NCH> &ck, const uint8_t *img_base, uint32_t col_bytes, uint32_t stage_u32)
{
#pragma unroll
    for (int q = 0; q < NCH; ++q)
        if (q < ck.n)
            ptx::cp_async_16(stage_u32 + ck.dst_off[q], img_base + ck.src_off[q] + col_bytes, ((ck.real >> q) & 1u) ? 16u : 0u);
    ptx::cp_async_commit();
}

// Waits until all but the `lag` most recent copy groups of this thread have landed.
__device__ inline void fused_wait_groups(int lag)
{
    if (lag >= 4) ptx::cp_async_wait<4>();
    else if (lag == 3) ptx::cp_async_wait<3>();
    else if (lag == 2) ptx::cp_async_wait<2>();
    else if (lag == 1) ptx::cp_async_wait<1>();
    else ptx::cp_async_wait<0>();
}

__device__ inline void fused_init_barriers(FuShared *sh, bool again)
{
    for (int s = 0; s < kFuScStages; ++s) {
        if (again) {
            mbar_inval(&sh->sc_full[s]);
            mbar_inval(&sh->sc_empty[s]);
        }
        ptx::mbar_init(&sh->sc_full[s], kFuScProducers / 32);
        ptx::mbar_init(&sh->sc_empty[s], 1);
    }
    if (again) mbar_inval(&sh->sc_accum);
    ptx::mbar_init(&sh->sc_accum, 1);
    for (int s = 0; s < kFuMgStages; ++s) {
        if (again) {
            mbar_inval(&sh->mg_full[s]);
            mbar_inval(&sh->mg_empty[s]);
        }
        ptx::mbar_init(&sh->mg_full[s], kFuMgProducers / 32);
        ptx::mbar_init(&sh->mg_empty[s], kFuEpiWarps);
    }
    for (int s = 0; s < kFuAccStages; ++s) {
        if (again) {
            mbar_inval(&sh->acc_full[s]);
            mbar_inval(&sh->acc_empty[s]);
        }
        ptx::mbar_init(&sh->acc_full[s], 1);
        ptx::mbar_init(&sh->acc_empty[s], kFuEpiWarps);
    }
    ptx::fence_mbar_init();
}

__global__ void __launch_bounds__(kFuThreads, 1)
stage2_fused_kernel(const __nv_bfloat16 *__restrict__ X, const int32_t *__restrict__ offsets, int d, int batch,
                    const int32_t *__restrict__ counts, const int32_t *__restrict__ order,
                    const float *__restrict__ norms, int max_tokens, int total, OtParams p,
                    __nv_bfloat16 *__restrict__ Y, int32_t *__restrict__ out_offsets, int32_t *__restrict__ kept_idx,
                    int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                    float *__restrict__ merge_weight, float *__restrict__ stats, WsHeader *__restrict__ hdr)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FuShared *sh = reinterpret_cast<FuShared *>(smem);
    uint8_t *arena = smem + kFuSharedBytes;
    const uint32_t arena_u32 = ptx::smem_u32(arena);
    const uint32_t rank = ptx::cluster_ctarank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
    const uint32_t row_bytes = (uint32_t)d * 2u;

    // ---- set-up that needs nothing from the kernels ahead ------------------------------------------------
    if (tid == 0) {
        fused_init_barriers(sh, false);
        ptx::mbar_init(&sh->xbar[0], 1);
        ptx::mbar_init(&sh->xbar[1], 1);
        sh->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == kFuMmaWarp) {
        ptx::tmem_alloc(&sh->tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();          // the selection comes from the kernel ahead
    // both CTAs are running and have their barriers in place before anyone writes into the other's shared memory
    ptx::cluster_sync_all();

    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);
    const float v_init = expf(shift * inv_eps);
    const int nct = d / kFuNT;
    const int nkblk = d / kFuBK;
    uint32_t round = 0;            // exchanges of column sums so far (the same in both CTAs)
    bool first = true;

    for (int img = cluster_id; img < batch; img += nclusters) {
        FuImage im;
        if (!image_range(offsets, img, max_tokens, total, im.t_begin, im.N)) {
            // no output rows; the image's slot of out_offsets still has to be right
            if (rank == 0 && warp == 0) {
                int s = 0;
                for (int b = lane; b < img; b += 32) s += __ldcg(counts + b);
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) {
                    out_offsets[img] = s;
                    if (img == batch - 1) out_offsets[batch] = s;
                }
            }
            continue;
        }
        const uint8_t *img_base = reinterpret_cast<const uint8_t *>(X + (size_t)im.t_begin * d);
        // the ring barriers start every image in phase 0 (the rings differ from image to image)
        if (!first && tid == 0) fused_init_barriers(sh, true);
        if (!first) __syncthreads();
        first = false;

        {
            im.M = __ldcg(counts + img);
            im.B = im.N - im.M;
            im.half = (im.M + 1) >> 1;
            im.row_lo = min(im.M, (int)rank * im.half);
            im.Ml = min(im.M, im.row_lo + im.half) - im.row_lo;
            im.ntile = (im.Ml + kFuTileM - 1) / kFuTileM;
            im.ldk = im.B > 0 ? sinkhorn_ldk(im.B) : 32;
            im.nkb = (im.B + 63) >> 6;
            im.Ra = (im.Ml + 15) & ~15;
            im.Rb = (im.B + 15) & ~15;
            // which token each row of a stage is (one trip to L2)
            const int32_t *ord = order + im.t_begin;
            for (int r = tid; r < im.Ra + im.Rb; r += kFuThreads) {
                int tok = -1;
                if (r < im.Ml) tok = __ldcg(ord + im.row_lo + r);
                else if (r >= im.Ra && r - im.Ra < im.B) tok = __ldcg(ord + im.M + (r - im.Ra));
                sh->rowtok[r] = tok;
            }
        }
        // out0 = number of kept rows of the images before this one
        if (warp == kFuWarps - 1) {
            int s = 0;
            for (int b = lane; b < img; b += 32) s += __ldcg(counts + b);
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) {
                sh->out0 = s;
                if (rank == 0) {
                    out_offsets[img] = s;
                    if (img == batch - 1) out_offsets[batch] = s + im.M;
                }
            }
        }
        __syncthreads();

        FuIterState ist{0, 0.f};
        if (im.B > 0) {
            // ---- scores: D[tile] = T_k[tile rows] . T_p^T over the full width ------------------------------
            const int stage_bytes = fused_stage_bytes(im.Ml, im.B);
            const int nstages = im.ntile > 0 ? min(kFuScStages, (kFuArenaBytes - kFuABytes) / stage_bytes) : 1;
            const int lag = max(0, nstages - 2);          // copy groups a producer keeps in flight behind the newest
            if (warp >= 1 && im.ntile > 0) {
                const int pt = tid - 32;
                FuChunks<kFuScChunks> ck;
                fused_chunk_table<kFuScChunks, kFuScProducers>(ck, sh, im, pt, row_bytes);
                bool ok = true;
                for (int kb = 0; kb < nkblk; ++kb) {
                    const int s = kb % nstages;
                    if (ok && kb >= nstages && !ptx::mbar_wait(&sh->sc_empty[s], ((kb / nstages) - 1) & 1)) ok = false;
                    if (ok) fused_issue_stage(ck, img_base, (uint32_t)kb * 128u, arena_u32 + s * stage_bytes);
                    else ptx::cp_async_commit();
                    if (kb >= lag) {
                        fused_wait_groups(lag);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&sh->sc_full[(kb - lag) % nstages]);
                    }
                }
                for (int kb = max(nkblk - lag, 0); kb < nkblk; ++kb) {
                    ptx::cp_async_wait<0>();
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&sh->sc_full[kb % nstages]);
                }
                if (!ok) {
                    sh->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                }
                // the norms of the rows, while the last k-blocks are multiplied
                {
                    for (int i = pt; i < im.Ml; i += kFuScProducers)
                        sh->inv_ni[i] = 1.f / fmaxf(__ldcg(norms + im.t_begin + sh->rowtok[i]), kNormFloor);
                    for (int j = pt; j < im.B; j += kFuScProducers)
                        sh->inv_nj[j] = 1.f / fmaxf(__ldcg(norms + im.t_begin + sh->rowtok[im.Ra + j]), kNormFloor);
                }
            } else if (warp == 0) {
                if (lane == 0 && im.ntile > 0) {
                    const uint32_t idesc = ptx::idesc_bf16(kFuTileM, im.Rb, false, false);
                    for (int kb = 0; kb < nkblk && !sh->abort_flag; ++kb) {
                        const int s = kb % nstages;
                        if (!ptx::mbar_wait(&sh->sc_full[s], (kb / nstages) & 1)) {
                            sh->abort_flag = 1;
                            atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                            break;
                        }
                        ptx::tc_fence_after();
                        const uint32_t a_base = arena_u32 + s * stage_bytes;
                        const uint32_t b_base = a_base + im.Ra * 128;
                        for (int t = 0; t < im.ntile; ++t) {
#pragma unroll
                            for (int k = 0; k < kFuBK / 16; ++k) {
                                const uint64_t da = ptx::smem_desc_sw128(a_base + t * kFuABytes + k * 32, 16, 1024);
                                const uint64_t db = ptx::smem_desc_sw128(b_base + k * 32, 16, 1024);
                                ptx::umma_bf16(tmem_base + (uint32_t)(t * 256), da, db, idesc, (kb | k) != 0);
                            }
                        }
                        ptx::umma_commit(&sh->sc_empty[s]);
                    }
                    ptx::umma_commit(&sh->sc_accum);
                }
            }
            __syncwarp();
            // everybody: the accumulators are complete (and with them every read of the ring)
            if (im.ntile > 0 && !ptx::mbar_wait(&sh->sc_accum, 0)) {
                sh->abort_flag = 1;
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
            }
            ptx::tc_fence_after();
            __syncthreads();               // inv_ni, inv_nj; and nobody still waits on the ring's barriers

            // ---- epilogue: K = exp((S - c) / eps) of this CTA's rows into shared memory (the ring is free) ----
            // warp (quarter q = warp % 4, g = warp / 4): tile g & 1, column chunks of 32 from (g >> 1), step 2.
            // Row pitch ldk + 4 floats: a warp's 32 rows of 16 bytes fall into distinct banks.
            float *kbuf = reinterpret_cast<float *>(arena);
            if (!sh->abort_flag) {
                const int q = warp & 3, g = warp >> 2;
                const int tile = g & 1;
                const int nchunk = im.ldk >> 5;
                if (tile < im.ntile) {
                    const int i = tile * kFuTileM + q * 32 + lane;
                    const bool have = i < im.Ml;
                    const float inv_ni = have ? sh->inv_ni[i] : 0.f;
                    float *krow = kbuf + (size_t)min(i, kFuMaxRows - 1) * (im.ldk + 4);
                    for (int c = (g >> 1); c < nchunk; c += 2) {
                        uint32_t r[32];
                        ptx::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tile * 256 + c * 32), r);
                        ptx::tmem_ld_wait();
                        if (have) {
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                float4 kv;
                                const int j = c * 32 + 4 * v;
                                kv.x = (j + 0 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 0]) * inv_ni * sh->inv_nj[j + 0] - shift) * inv_eps) : 0.f;
                                kv.y = (j + 1 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 1]) * inv_ni * sh->inv_nj[min(j + 1, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                kv.z = (j + 2 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 2]) * inv_ni * sh->inv_nj[min(j + 2, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                kv.w = (j + 3 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 3]) * inv_ni * sh->inv_nj[min(j + 3, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                *reinterpret_cast<float4 *>(krow + j) = kv;
                            }
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            __syncthreads();
            ptx::tc_fence_after();

            // ---- Sinkhorn on this CTA's rows ---------------------------------------------------------------
            const int rps = im.ldk <= 128 ? 4 : 2;
            const int ns = max(1, (im.half + kFuWarps * rps - 1) / (kFuWarps * rps));
#define RTP_FU(LR, CPL, NS) ist = fused_sinkhorn<LR, CPL, NS>(sh, kbuf, arena, im, rank, p, kappa, v_init, round, hdr)
#define RTP_FU_NS(LR, CPL, NSMAX)                                 \
    switch (ns) {                                                 \
    case 1: RTP_FU(LR, CPL, 1); break;                            \
    case 2: RTP_FU(LR, CPL, 2); break;                            \
    case 3: if (NSMAX >= 3) { RTP_FU(LR, CPL, (NSMAX >= 3 ? 3 : 1)); } break; \
    case 4: if (NSMAX >= 4) { RTP_FU(LR, CPL, (NSMAX >= 4 ? 4 : 1)); } break; \
    default: if (NSMAX >= 5) { RTP_FU(LR, CPL, (NSMAX >= 5 ? 5 : 1)); } break; \
    }
            switch (im.ldk) {
            case 32: RTP_FU_NS(8, 4, 4); break;
            case 64: RTP_FU_NS(8, 8, 4); break;
            case 128: RTP_FU_NS(8, 16, 4); break;
            case 192: RTP_FU_NS(16, 12, 5); break;
            default: RTP_FU_NS(16, 16, 4); break;
            }
#undef RTP_FU_NS
#undef RTP_FU
            if (tid == 0 && rank == 0) {
                stats[(size_t)img * kStats + 5] = (float)ist.done;
                stats[(size_t)img * kStats + 6] = ist.last_move;
            }
            ptx::fence_proxy_async_smem();     // the plan arrays (ordinary stores) feed UMMAs
        }
        // the pairing partials are with rank 0; the plan arrays and out0 are in place
        ptx::cluster_sync_all();

        const int out0 = sh->out0;
        // ---- merge: for every tile of 64 output columns, acc = alpha P . T_p on the tensor cores; the epilogue
        // adds the kept token's own row (it sits in the stage, fetched with the pruned rows), rounds to bf16
        // in place there, and writes the rows out with coalesced 16-byte stores (they are consecutive rows of Y).
        // arena: plan arrays | ring (it takes the place of the column partials, consumed before the barrier above)
        const int plan_bytes = fused_plan_bytes(im.Ml, im.B);
        const int mstage_bytes = fused_stage_bytes(im.Ml, im.B);
        const int mstages = im.ntile > 0 ? min(kFuMgStages, (kFuArenaBytes - plan_bytes) / mstage_bytes) : 1;
        const uint32_t ring_off = (uint32_t)plan_bytes;
        const int ksteps_p = im.Rb >> 4;                        // 16-row steps over the pruned rows
        if (warp > kFuMmaWarp && im.ntile > 0) {
            const int pt = tid - (kFuMmaWarp + 1) * 32;
            if (im.B > 0 && rank == 0) {
                // the pairs: rank 1 holds the higher rows, so strict > keeps the lower row on ties
                const int seg = im.t_begin - out0;
                for (int j = pt; j < im.B; j += kFuMgProducers) {
                    float b = sh->pairv[0][j];
                    int ib = sh->pairi[0][j];
                    const float ob = sh->pairv[1][j];
                    if (ob > b) {
                        b = ob;
                        ib = sh->pairi[1][j];
                    }
                    merged_idx[seg + j] = sh->rowtok[im.Ra + j];
                    merge_partner[seg + j] = ib;
                    merge_weight[seg + j] = b * sh->vs[j];
                }
            }
            for (int i = pt; i < im.Ml; i += kFuMgProducers) kept_idx[out0 + im.row_lo + i] = sh->rowtok[i];
            // the rows sit in L2 (this SM fetched them for the scores): a group lands while the next one is issued
            const int mlag = min(1, mstages - 1);
            FuChunks<kFuMgChunks> ck;
            fused_chunk_table<kFuMgChunks, kFuMgProducers>(ck, sh, im, pt, row_bytes);
            bool ok = true;
            for (int ct = 0; ct < nct; ++ct) {
                const int s = ct % mstages;
                if (ok && ct >= mstages && !ptx::mbar_wait(&sh->mg_empty[s], ((ct / mstages) - 1) & 1)) ok = false;
                if (ok) fused_issue_stage(ck, img_base, (uint32_t)ct * (kFuNT * 2), arena_u32 + ring_off + s * mstage_bytes);
                else ptx::cp_async_commit();
                if (ct >= mlag) {
                    fused_wait_groups(mlag);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&sh->mg_full[(ct - mlag) % mstages]);
                }
            }
            for (int ct = max(nct - mlag, 0); ct < nct; ++ct) {
                ptx::cp_async_wait<0>();
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sh->mg_full[ct % mstages]);
            }
            if (!ok) {
                sh->abort_flag = 1;
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
            }
        } else if (warp == kFuMmaWarp) {
            if (lane == 0 && im.ntile > 0) {
                ptx::fence_proxy_async_smem();
                const uint32_t idesc = ptx::idesc_bf16(kFuTileM, kFuNT, false, true);
                bool failed = false;
                for (int ct = 0; ct < nct && !sh->abort_flag && !failed; ++ct) {
                    const int s = ct % mstages, as = ct % kFuAccStages;
                    if (ct >= kFuAccStages) {
                        if (!ptx::mbar_wait(&sh->acc_empty[as], ((ct / kFuAccStages) - 1) & 1)) {
                            failed = true;
                            break;
                        }
                        ptx::tc_fence_after();
                    }
                    if (!ptx::mbar_wait(&sh->mg_full[s], (ct / mstages) & 1)) {
                        failed = true;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t stage = arena_u32 + ring_off + s * mstage_bytes;
                    for (int t = 0; t < im.ntile; ++t) {
                        const uint32_t d_tmem = tmem_base + (uint32_t)(as * 128 + t * 64);
                        for (int ks = 0; ks < ksteps_p; ++ks) {
                            const int kb = ks >> 2, k = ks & 3;
                            const uint64_t da = ptx::smem_desc_sw128(arena_u32 + (uint32_t)(kb * im.Ra * 128 + t * kFuABytes) + k * 32, 16, 1024);
                            const uint64_t db = ptx::smem_desc_sw128(stage + (im.Ra + ks * 16) * 128, kFuBoxBytes, 1024);
                            ptx::umma_bf16(d_tmem, da, db, idesc, ks != 0);
                        }
                    }
                    ptx::umma_commit(&sh->acc_full[as]);      // (at once when nothing is pruned: no UMMA was issued)
                }
                if (failed) {
                    sh->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                }
            }
        } else if (warp < kFuEpiWarps && im.ntile > 0) {
            // ---- epilogue: warp (tile t = warp / 4, quarter q = warp % 4) owns rows 128 t + 32 q .. + 31 -------------
            const int q = warp & 3, t = warp >> 2;
            const int i0 = t * kFuTileM + q * 32;
            const int i = i0 + lane;
            const bool has_rows = t < im.ntile && i0 < im.Ml;
            const uint32_t my_row = (uint32_t)((i >> 3) * 1024 + (i & 7) * 128);
            bool dead = false;
            for (int ct = 0; ct < nct; ++ct) {
                const int s = ct % mstages, as = ct % kFuAccStages;
                uint8_t *stage = arena + ring_off + s * mstage_bytes;
                uint8_t *xrow = stage + my_row;              // this thread's row: T_k now, the output row below
                // the stage first (it has been there for a while: the copies run ahead), and the row's eight
                // 16-byte cells while the accumulator is waited for
                bool ok = !dead && !sh->abort_flag && ptx::mbar_wait(&sh->mg_full[s], (ct / mstages) & 1);
                uint4 xv[8];
                if (ok && has_rows) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) xv[g] = *reinterpret_cast<const uint4 *>(xrow + ((g ^ (i & 7)) << 4));
                }
                ok = ok && ptx::mbar_wait(&sh->acc_full[as], (ct / kFuAccStages) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    if (!dead) {
                        sh->abort_flag = 1;
                        if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                    }
                    dead = true;
                    continue;
                }
                ptx::tc_fence_after();
                if (has_rows) {
                    // both halves of the accumulator row into registers, then the accumulator stage is free
                    uint32_t r0[32], r1[32];
                    if (im.B > 0) {
                        ptx::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * 128 + t * 64), r0);
                        ptx::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * 128 + t * 64 + 32), r1);
                        ptx::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) r0[e] = r1[e] = 0u;
                    }
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&sh->acc_empty[as]);
                    __nv_bfloat16 *yrow0 = Y + (size_t)(out0 + im.row_lo + i0) * d + ct * kFuNT;
                    // 32 columns at a time: add, round, back into the row's cells; then 4 lanes write a row's 64
                    // bytes, 8 rows per instruction
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const __nv_bfloat162 *xh = reinterpret_cast<const __nv_bfloat162 *>(&xv[4 * h + g]);
                            __nv_bfloat162 o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 xf = __bfloat1622float2(xh[e]);
                                const uint32_t a0 = h ? r1[8 * g + 2 * e] : r0[8 * g + 2 * e];
                                const uint32_t a1 = h ? r1[8 * g + 2 * e + 1] : r0[8 * g + 2 * e + 1];
                                o[e] = __floats2bfloat162_rn(xf.x + __uint_as_float(a0), xf.y + __uint_as_float(a1));
                            }
                            *reinterpret_cast<uint4 *>(xrow + (((4 * h + g) ^ (i & 7)) << 4)) = *reinterpret_cast<uint4 *>(o);
                        }
                        __syncwarp();
                        uint4 yv[4];
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr) {
                            const int ir = i0 + 8 * rr + (lane >> 2);
                            yv[rr] = *reinterpret_cast<const uint4 *>(stage + (ir >> 3) * 1024 + (ir & 7) * 128 +
                                                                      (((4 * h + (lane & 3)) ^ (ir & 7)) << 4));
                        }
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr) {
                            const int row = 8 * rr + (lane >> 2);
                            if (i0 + row < im.Ml)
                                *reinterpret_cast<uint4 *>(yrow0 + (size_t)row * d + (4 * h + (lane & 3)) * 8) = yv[rr];
                        }
                    }
                } else if (lane == 0) {
                    ptx::mbar_arrive(&sh->acc_empty[as]);
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&sh->mg_empty[s]);          // the stage's rows have been read (and written out)
            }
        }
        // every role is done with the image before the next one reuses the arena and the barriers
        ptx::tc_fence_before();
        __syncthreads();
        ptx::tc_fence_after();
    }

    ptx::tc_fence_before();
    __syncthreads();
    // no CTA leaves while the other may still write into its shared memory
    ptx::cluster_sync_all();
    if (warp == kFuMmaWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace rtp
