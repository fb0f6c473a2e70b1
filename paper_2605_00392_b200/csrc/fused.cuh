// Stage 2 of Algorithm 1 in ONE kernel, one cluster of two CTAs per image: cosine scores (Section
// 3.3.2) on the tcgen05 tensor cores, dustbin augmentation and Sinkhorn iterations (Eq. 5, Appendix C)
// with the kernel matrix K held in REGISTERS, and the merge T_k + alpha P T_p (Eq. 7) on the tensor
// cores again, written packed.  Nothing but the compact copy of the pruned rows goes through global
// memory between the steps: S lives in tensor memory, K in registers, the plan P in shared memory.
//
// Taken by runs whose images all have at most kFuMaxTok tokens and at most kFuMaxB pruned tokens, bf16
// storage, width a multiple of 64, scaling form (fused_eligible() on the host); everything else keeps
// the separate kernels.
//
// Work split inside a cluster (rank r = 0, 1):
//   * tokens: rank r owns the image's tokens [r * tpc, min(N, (r + 1) * tpc)), tpc = ceil(N / 2): at most
//     two tiles of 128 CONSECUTIVE tokens, fetched by tiled TMA (kept and pruned alike; rows of pruned
//     tokens are computed and dropped, as contiguous rows are what TMA moves at full speed: a
//     tile::gather4 load moves 512 bytes in about 70 cycles, a tiled load 16 KB in about 400).
//   * pruned rows: the cluster first copies the image's B pruned rows to a compact scratch in global
//     memory (they are L2 hits: stage 1 has just read them), so that both contractions can fetch them
//     as tiles too.
//   * kept rows of the Sinkhorn problem: rank r owns kept positions [r * half, ...), half = ceil(M / 2),
//     whatever tokens they are; the scores epilogue sends K = exp((S - c) / eps) of a row to its owner
//     through distributed shared memory, and the owner sends the row of alpha P back to the owner of the
//     token when the iterations are done.
// Sinkhorn iteration: as in sinkhorn_cluster.cuh (one pass per iteration, LR lanes share a row, column
// sums completed over the warps in shared memory and over the two CTAs through distributed shared
// memory, one cluster barrier), but a thread's K values never leave its registers.
// Merge: for each tile of 64 output columns, D = [I | alpha P] . [T_v rows of the token tile ; T_p]
// (the identity block carries the kept token's own row through the tensor cores, exact in the fp32
// accumulator); four accumulator stages in tensor memory; the epilogue converts to bf16, stages a
// warp's 32 rows in shared memory and writes the kept ones with coalesced 16-byte stores.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "sinkhorn.cuh"
#include "sinkhorn_cluster.cuh"

namespace rtp {

constexpr int kFuThreads = 512;
constexpr int kFuWarps = kFuThreads / 32;
constexpr int kFuMaxTok = 512;            // tokens per image: two tiles of 128 per CTA
constexpr int kFuMaxB = 256;              // pruned tokens per image: one UMMA N, half of tensor memory
constexpr int kFuKRegs = 64;              // K values a thread may hold
constexpr int kFuTileM = 128;
constexpr int kFuBK = 64;                 // bf16 per k-block = one 128-byte swizzle row
constexpr int kFuNT = 64;                 // output columns per merge tile
constexpr int kFuABytes = kFuTileM * 128; // 16 KB: 128 rows x 64 bf16, K-major
constexpr int kFuBoxBytes = 64 * 128;     // 8 KB: 64 rows x 64 bf16
constexpr int kFuIdentBytes = 3 * (kFuABytes / 2);
constexpr int kFuScStages = 4;            // at most
constexpr int kFuMgStages = 4;            // B-operand ring of the merge
constexpr int kFuAccStages = 4;           // accumulator stages of the merge (128 TMEM columns each)
constexpr int kFuSharedBytes = 12288;     // FuShared, rounded up
constexpr int kFuArenaBytes = 180 * 1024;
constexpr int kFuPartOffset = 128 * 1024; // arena offsets: P tiles at 0, column partials / merge ring here
constexpr int kFuStagePitch = kFuNT * 2 + 16;                 // bytes per staged output row
constexpr int kFuStagingOffset = kFuPartOffset + 32 * 1024;   // 4 warps x 32 rows x kFuStagePitch
constexpr int kFuSmemBytes = 1024 + kFuIdentBytes + kFuSharedBytes + kFuArenaBytes;

struct FuShared {
    uint64_t sc_full[kFuScStages], sc_empty[kFuScStages], sc_accum;
    uint64_t mg_full[kFuMgStages], mg_empty[kFuMgStages];
    uint64_t acc_full[kFuAccStages], acc_empty[kFuAccStages];
    uint32_t tmem_base;
    volatile int abort_flag;
    int out0;
    float vsum[kFuWarps];
    float wsum[kFuWarps];
    float xusum[2][2];
    __align__(16) float inv_nj[kFuMaxB];   // 1 / |x_j| of the pruned tokens
    __align__(16) float vs[kFuMaxB + 8];   // V_j, V_d at [ldk]: read as 16-byte vectors
    int toks[kFuMaxTok / 2 + 8];      // image-local token of each of this CTA's kept rows
    __align__(16) float xpart[2][2][kFuMaxB];   // per-CTA column partials by iteration parity
    float pairv[2][kFuMaxB];          // rank 0: per-CTA column maxima of K U ...
    int pairi[2][kFuMaxB];            // ... and their rows
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

// Every image of a run with at most max_tokens tokens and max_b pruned tokens fits the fused kernel.
__host__ inline bool fused_eligible(int d, int max_tokens, int max_b)
{
    if (d % 64 != 0 || max_tokens > kFuMaxTok || max_b > kFuMaxB) return false;
    for (int b = 1; b <= max_b; ++b) {
        const int m = max_tokens - b > 1 ? max_tokens - b : 1;
        const int regs = fused_k_regs((m + 1) / 2, b);
        if (regs == 0 || regs > kFuKRegs) return false;
    }
    return true;
}

__device__ inline void st_cluster_v4(uint32_t addr, float4 v)
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ inline void st_cluster_v2_u32(uint32_t addr, uint32_t a, uint32_t b)
{
    asm volatile("st.shared::cluster.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
__device__ inline void mbar_inval(uint64_t *bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}

struct FuImage {
    int t_begin, N, M, B;
    int tok_lo, ntok, ntile;      // this CTA's tokens
    int half, row_lo, Ml;         // this CTA's kept rows of the Sinkhorn problem
    int ldk, nkb, nbox, BN;
    int tpc;
};

struct FuIterState {
    int done;
    float last_move;
};

// The iterations, K in registers.  Row i of this CTA (kept position row_lo + i) lives in the LR lanes
// (step s, warp w, slot) with i = (s * 16 + w) * (32 / LR) + slot; lane `sub` of a row holds the 16-byte
// column chunks sub, sub + LR, ...  On return vs[] holds the final V (V_d at [ldk]) and U[] the final
// U of the thread's rows (0 for rows past Ml).
template <int LR, int CPL, int NS>
__device__ inline FuIterState fused_iterate(const float4 (&k)[NS][CPL / 4], float (&U)[NS], FuShared *sh, float *part,
                                            int Ml, int M, int B, uint32_t rank, const OtParams &p, float kappa,
                                            float v_init)
{
    constexpr int ldk = LR * CPL;
    constexpr int RPS = 32 / LR;
    constexpr int NQ = CPL / 4;
    constexpr int kVWarps = ldk / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;
    const float Bf = (float)B, Mf = (float)M;
    constexpr uint32_t C = 2;

    for (int j = tid; j <= ldk; j += kFuThreads) sh->vs[j] = (j < B || j == ldk) ? v_init : 0.f;
    if (tid < kFuWarps) sh->vsum[tid] = (tid == 0) ? Bf * v_init : 0.f;
#pragma unroll
    for (int s = 0; s < NS; ++s) U[s] = 0.f;
    __syncthreads();
    const uint32_t xpart_u32 = ptx::smem_u32(&sh->xpart[0][0][0]), xusum_u32 = ptx::smem_u32(&sh->xusum[0][0]);
    FuIterState st{0, 0.f};

    for (int it = 0; it < p.iters; ++it) {
        float4 V[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(sh->vs + 4 * (q * LR + sub));
        float sumV = 0.f;
#pragma unroll
        for (int w = 0; w < kVWarps; ++w) sumV += sh->vsum[w];
        const float Vd = sh->vs[ldk];
        const float Ud = Bf * rcp_fast(kappa * (sumV + Vd));
        const float kVd = kappa * Vd;
        float4 colacc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) colacc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float usum = 0.f;

#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const int i = (s * kFuWarps + warp) * RPS + slot;
            const bool valid = i < Ml;
            float sd = 0.f;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                sd = fmaf(k[s][q].x, V[q].x, sd);
                sd = fmaf(k[s][q].y, V[q].y, sd);
                sd = fmaf(k[s][q].z, V[q].z, sd);
                sd = fmaf(k[s][q].w, V[q].w, sd);
            }
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

        // this CTA's column sums and sum of U go to both CTAs of the cluster
        const uint32_t slot_x = (uint32_t)(it & 1) * C + rank;
        if (tid < ldk) {
            float cs = 0.f;
#pragma unroll
            for (int w = 0; w < kFuWarps; ++w) cs += part[w * ldk + tid];
            const uint32_t a = xpart_u32 + (slot_x * (uint32_t)kFuMaxB + (uint32_t)tid) * 4u;
            ptx::st_cluster_f32(ptx::map_to_rank(a, 0), cs);
            ptx::st_cluster_f32(ptx::map_to_rank(a, 1), cs);
        }
        if (tid == kFuThreads - 1) {
            float su = 0.f;
#pragma unroll
            for (int w = 0; w < kFuWarps; ++w) su += sh->wsum[w];
            const uint32_t a = xusum_u32 + slot_x * 4u;
            ptx::st_cluster_f32(ptx::map_to_rank(a, 0), su);
            ptx::st_cluster_f32(ptx::map_to_rank(a, 1), su);
        }
        ptx::cluster_sync_all();

        // V from the completed column sums: one thread per column, the same in both CTAs
        const float *xb = &sh->xpart[it & 1][0][0];
        const float *ub = &sh->xusum[it & 1][0];
        int cont = 0;
        float move = 0.f;
        if (tid < ldk) {
            float nv = 0.f;
            if (tid < B) {
                const float cs = xb[tid] + xb[kFuMaxB + tid];
                nv = rcp_fast(cs + kappa * Ud);
                const float ov = sh->vs[tid];
                move = fabsf(nv - ov) * rcp_fast(ov);
                cont = p.tol > 0.f ? (move > p.tol) : (p.stop_fp ? ulp_far(nv, ov) : 1);
                sh->vs[tid] = nv;
            }
            const float wv = warp_sum(nv);        // warps 0 .. ldk/32-1 lie entirely inside tid < ldk
            if (lane == 0) sh->vsum[warp] = wv;
        }
        if (tid == kFuThreads - 1) {              // the dustbin column
            const float su = ub[0] + ub[1];
            const float nVd = Mf * rcp_fast(kappa * (su + Ud));
            const float mj = fabsf(nVd - Vd) * rcp_fast(Vd);
            move = fmaxf(move, mj);
            cont |= p.tol > 0.f ? (mj > p.tol) : (p.stop_fp ? ulp_far(nVd, Vd) : 1);
            sh->vs[ldk] = nVd;
        }
        st.last_move = move;
        ++st.done;
        if (!__syncthreads_or(cont)) break;
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

// Everything between the K exchange and the merge for one tile layout: K into registers, the
// iterations, alpha P into the A-operand tiles of the token owners, the per-CTA column maxima of
// K U for the pairing (into rank 0's xpart).  kbuf: this CTA's K rows [Ml][ldk] in shared memory.
template <int LR, int CPL, int NS>
__device__ inline FuIterState fused_sinkhorn(FuShared *sh, const float *kbuf, uint8_t *arena, const FuImage &im,
                                             uint32_t rank, const OtParams &p, float kappa, float v_init)
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
            k[s][q] = (i < im.Ml) ? *reinterpret_cast<const float4 *>(kbuf + (size_t)i * ldk + 4 * (q * LR + sub))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // with no iteration there is no barrier between this load and the plan rows the other CTA will write
    // over the K buffer
    if (p.iters == 0) ptx::cluster_sync_all();

    const FuIterState st = fused_iterate<LR, CPL, NS>(k, U, sh, part, im.Ml, im.M, im.B, rank, p, kappa, v_init);
    if (p.iters == 0) {
#pragma unroll
        for (int s = 0; s < NS; ++s) U[s] = ((s * kFuWarps + warp) * RPS + slot < im.Ml) ? 1.f : 0.f;   // u = 0
    }

    // ---- alpha P = alpha U K V in bf16 into the A tiles (128 rows x 64 columns, K-major, 128-byte swizzle)
    // of the CTA that owns the token: tile (token tile, k-block) at arena + (tile * nkb + kb) * 16 KB
    float4 V[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(sh->vs + 4 * (q * LR + sub));
    const uint32_t arena_u32 = ptx::smem_u32(arena);
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const int i = (s * kFuWarps + warp) * RPS + slot;
        if (i < im.Ml) {
            const int tok = sh->toks[i];
            const uint32_t owner = tok >= im.tpc ? 1u : 0u;
            const int tr = tok - (int)owner * im.tpc;
            const int tile = tr >> 7, r = tr & 127;
            const uint32_t row_off = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u;
            const float au = p.alpha * U[s];
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int col = 4 * (q * LR + sub);
                if (col < 64 * im.nkb) {
                    const int kb = col >> 6, c16 = (col & 63) >> 3;
                    const __nv_bfloat162 lo = __floats2bfloat162_rn((k[s][q].x * au) * V[q].x, (k[s][q].y * au) * V[q].y);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn((k[s][q].z * au) * V[q].z, (k[s][q].w * au) * V[q].w);
                    const uint32_t off = (uint32_t)(tile * im.nkb + kb) * (uint32_t)kFuABytes + row_off +
                                         (uint32_t)((c16 ^ (r & 7)) << 4) + (uint32_t)(col & 4) * 2u;
                    st_cluster_v2_u32(ptx::map_to_rank(arena_u32 + off, owner),
                                      *reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
                }
            }
            if (ldk < 64) {       // columns 32 .. 63 of the only k-block: zeros (they meet the zero rows of T_p)
                const int col = 32 + 4 * sub;
                const int c16 = col >> 3;
                const uint32_t off = (uint32_t)(tile * im.nkb) * (uint32_t)kFuABytes + row_off +
                                     (uint32_t)((c16 ^ (r & 7)) << 4) + (uint32_t)(col & 4) * 2u;
                st_cluster_v2_u32(ptx::map_to_rank(arena_u32 + off, owner), 0u, 0u);
            }
        }
    }

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
            if (i < im.Ml) {
                const float e[4] = {k[s][q].x * U[s], k[s][q].y * U[s], k[s][q].z * U[s], k[s][q].w * U[s]};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (e[c] > bv[c]) {          // rows ascend with s: strict > keeps the lower row
                        bv[c] = e[c];
                        bi[c] = im.row_lo + i;
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
    if (tid < im.B) {
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
        // to rank 0 (these arrays are not the ones the last iteration's V update may still be reading there)
        ptx::st_cluster_f32(ptx::map_to_rank(ptx::smem_u32(&sh->pairv[rank][tid]), 0), b);
        ptx::st_cluster_u32(ptx::map_to_rank(ptx::smem_u32(&sh->pairi[rank][tid]), 0), (uint32_t)ib);
    }
    return st;
}

__global__ void __launch_bounds__(kFuThreads, 1)
stage2_fused_kernel(const __grid_constant__ CUtensorMap tmapXa,    // X, boxes of 64 columns x 128 rows
                    const __grid_constant__ CUtensorMap tmapXb,    // X, boxes of 64 columns x 64 rows
                    const __grid_constant__ CUtensorMap tmapXp,    // compact copy, boxes of 64 x 64
                    const __nv_bfloat16 *__restrict__ X, const int32_t *__restrict__ offsets, int d, int batch,
                    const int32_t *__restrict__ counts, const int32_t *__restrict__ order,
                    const int32_t *__restrict__ kpos, const float *__restrict__ norms, __nv_bfloat16 *__restrict__ xp,
                    int max_tokens, int total, OtParams p, __nv_bfloat16 *__restrict__ Y,
                    int32_t *__restrict__ out_offsets, int32_t *__restrict__ kept_idx,
                    int32_t *__restrict__ merged_idx, int32_t *__restrict__ merge_partner,
                    float *__restrict__ merge_weight, float *__restrict__ stats, WsHeader *__restrict__ hdr)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *ident = smem;
    FuShared *sh = reinterpret_cast<FuShared *>(smem + kFuIdentBytes);
    uint8_t *arena = smem + kFuIdentBytes + kFuSharedBytes;
    const uint32_t arena_u32 = ptx::smem_u32(arena);
    const uint32_t rank = ptx::cluster_ctarank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;

    // ---- set-up that needs nothing from the kernels ahead: identity block, tensor memory ---------------
    // rows 64 .. 127 of a 192-row region hold I_64 (ones at (64 + r, k = r)) in the swizzled K-major
    // layout, the other rows are zero: the view that starts at row 64 has its ones in rows 0-63, the view
    // that starts at row 0 in rows 64-127.
    for (int v = tid; v < kFuIdentBytes / 16; v += kFuThreads) reinterpret_cast<uint4 *>(ident)[v] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    if (tid < 64) {
        const int r = 64 + tid, k = tid;
        const uint32_t off = (r >> 3) * 1024 + (r & 7) * 128 + (((k >> 3) ^ (r & 7)) << 4) + (k & 7) * 2;
        *reinterpret_cast<uint16_t *>(ident + off) = 0x3F80;   // bf16 1.0
    }
    ptx::fence_proxy_async_smem();
    if (tid == 0) {
        for (int s = 0; s < kFuScStages; ++s) {
            ptx::mbar_init(&sh->sc_full[s], 1);
            ptx::mbar_init(&sh->sc_empty[s], 1);
        }
        ptx::mbar_init(&sh->sc_accum, 1);
        for (int s = 0; s < kFuMgStages; ++s) {
            ptx::mbar_init(&sh->mg_full[s], 1);
            ptx::mbar_init(&sh->mg_empty[s], 1);
        }
        for (int s = 0; s < kFuAccStages; ++s) {
            ptx::mbar_init(&sh->acc_full[s], 1);
            ptx::mbar_init(&sh->acc_empty[s], 128);
        }
        sh->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmapXa);
        ptx::prefetch_tensormap(&tmapXb);
        ptx::prefetch_tensormap(&tmapXp);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&sh->tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();          // the selection comes from the kernel ahead
    // both CTAs are running and have their shared memory laid out before anyone writes into the other's
    ptx::cluster_sync_all();

    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);
    const float v_init = expf(shift * inv_eps);
    const int nct = d / kFuNT;
    const int nkblk = d / kFuBK;
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
        im.M = __ldcg(counts + img);
        im.B = im.N - im.M;
        im.tpc = (im.N + 1) >> 1;
        im.tok_lo = min(im.N, (int)rank * im.tpc);
        im.ntok = min(im.N, im.tok_lo + im.tpc) - im.tok_lo;
        im.ntile = (im.ntok + kFuTileM - 1) / kFuTileM;
        im.half = (im.M + 1) >> 1;
        im.row_lo = min(im.M, (int)rank * im.half);
        im.Ml = min(im.M, im.row_lo + im.half) - im.row_lo;
        im.ldk = im.B > 0 ? sinkhorn_ldk(im.B) : 32;
        im.nkb = (im.B + 63) >> 6;
        im.nbox = im.nkb;
        im.BN = (im.B + 15) & ~15;
        const int xp0 = xp_row0(im.t_begin, img);
        const int32_t *ord = order + im.t_begin;

        if (!first) {
            // the barriers start every image in phase 0 (their rings differ from image to image)
            __syncthreads();
            if (tid == 0) {
                for (int s = 0; s < kFuScStages; ++s) {
                    mbar_inval(&sh->sc_full[s]);
                    mbar_inval(&sh->sc_empty[s]);
                    ptx::mbar_init(&sh->sc_full[s], 1);
                    ptx::mbar_init(&sh->sc_empty[s], 1);
                }
                mbar_inval(&sh->sc_accum);
                ptx::mbar_init(&sh->sc_accum, 1);
                for (int s = 0; s < kFuMgStages; ++s) {
                    mbar_inval(&sh->mg_full[s]);
                    mbar_inval(&sh->mg_empty[s]);
                    ptx::mbar_init(&sh->mg_full[s], 1);
                    ptx::mbar_init(&sh->mg_empty[s], 1);
                }
                for (int s = 0; s < kFuAccStages; ++s) {
                    mbar_inval(&sh->acc_full[s]);
                    mbar_inval(&sh->acc_empty[s]);
                    ptx::mbar_init(&sh->acc_full[s], 1);
                    ptx::mbar_init(&sh->acc_empty[s], 128);
                }
                ptx::fence_mbar_init();
            }
            __syncthreads();
        }
        first = false;

        // ---- out0 = number of kept rows of the images before this one (warp 15) ----------------------------
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

        FuIterState ist{0, 0.f};
        if (im.B > 0) {
            // ---- compact copy of the pruned rows: rows j = warp of the cluster, + 32, ...; zero rows up to
            // a multiple of 64 (whole 64-row boxes are fetched)
            {
                const int nvec = d >> 3;
                const int gw = (int)rank * kFuWarps + warp;
                uint4 *seg = reinterpret_cast<uint4 *>(xp + (size_t)xp0 * d);
                for (int j = gw; j < 64 * im.nkb; j += 2 * kFuWarps) {
                    const uint4 *src = (j < im.B)
                                           ? reinterpret_cast<const uint4 *>(X + (size_t)(im.t_begin + __ldcg(ord + im.M + j)) * d)
                                           : nullptr;
                    for (int v0 = lane; v0 < nvec; v0 += 32 * 5) {
                        uint4 t[5];
#pragma unroll
                        for (int b = 0; b < 5; ++b) {
                            const int v = v0 + 32 * b;
                            t[b] = (src && v < nvec) ? __ldg(src + v) : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int b = 0; b < 5; ++b) {
                            const int v = v0 + 32 * b;
                            if (v < nvec) seg[(size_t)j * nvec + v] = t[b];
                        }
                    }
                }
            }
            // 1 / |x_j| of the pruned tokens; tokens of this CTA's kept rows
            for (int j = tid; j < im.B; j += kFuThreads)
                sh->inv_nj[j] = 1.f / fmaxf(__ldcg(norms + im.t_begin + __ldcg(ord + im.M + j)), kNormFloor);
            for (int i = tid; i < im.Ml; i += kFuThreads) sh->toks[i] = __ldcg(ord + im.row_lo + i);
            __threadfence();
            ptx::fence_proxy_async_all();      // the copy is read by TMA
            ptx::cluster_sync_all();           // #0: the whole compact copy is in place

            // ---- scores: D[tile] = X[tile rows] . T_p^T over the full width --------------------------------
            const int stage_bytes = im.ntile * kFuABytes + im.nbox * kFuBoxBytes;
            const int nstages = min(kFuScStages, kFuArenaBytes / stage_bytes);
            if (warp == 0) {
                if (lane == 0) {
                    ptx::fence_proxy_async_all();
                    for (int kb = 0; kb < nkblk && !sh->abort_flag; ++kb) {
                        const int s = kb % nstages;
                        if (kb >= nstages && !ptx::mbar_wait(&sh->sc_empty[s], ((kb / nstages) - 1) & 1)) {
                            sh->abort_flag = 1;
                            atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                            break;
                        }
                        const uint32_t dst = arena_u32 + s * stage_bytes;
                        ptx::mbar_arrive_expect_tx(&sh->sc_full[s], (uint32_t)stage_bytes);
                        for (int t = 0; t < im.ntile; ++t)
                            ptx::tma_load_2d(dst + t * kFuABytes, &tmapXa, &sh->sc_full[s], kb * kFuBK,
                                             im.t_begin + im.tok_lo + t * kFuTileM);
                        for (int b = 0; b < im.nbox; ++b)
                            ptx::tma_load_2d(dst + im.ntile * kFuABytes + b * kFuBoxBytes, &tmapXp, &sh->sc_full[s],
                                             kb * kFuBK, xp0 + b * 64);
                    }
                }
            } else if (warp == 1) {
                if (lane == 0) {
                    const uint32_t idesc = ptx::idesc_bf16(kFuTileM, im.BN, false, false);
                    for (int kb = 0; kb < nkblk && !sh->abort_flag; ++kb) {
                        const int s = kb % nstages;
                        if (!ptx::mbar_wait(&sh->sc_full[s], (kb / nstages) & 1)) {
                            sh->abort_flag = 1;
                            atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                            break;
                        }
                        ptx::tc_fence_after();
                        const uint32_t a_base = arena_u32 + s * stage_bytes;
                        const uint32_t b_base = a_base + im.ntile * kFuABytes;
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
            {
                bool ok = im.ntile == 0 || ptx::mbar_wait(&sh->sc_accum, 0);
                if (!ok) {
                    sh->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                }
            }
            ptx::tc_fence_after();
            ptx::cluster_sync_all();           // #1: both rings are free: the K rows may land on them

            // ---- epilogue: K = exp((S - c) / eps) of a kept token's row to the owner of its kept position --
            // warp (quarter q = warp % 4, g = warp / 4): tile g & 1, column chunks of 32 from (g >> 1), step 2
            if (!sh->abort_flag) {
                const int q = warp & 3, g = warp >> 2;
                const int tile = g & 1;
                const int nchunk = im.ldk >> 5;
                if (tile < im.ntile) {
                    const int tr = tile * kFuTileM + q * 32 + lane;
                    const int tok = im.tok_lo + tr;
                    const int pk = (tr < im.ntok) ? __ldcg(kpos + im.t_begin + tok) : -1;
                    const float inv_ni = (pk >= 0) ? 1.f / fmaxf(__ldcg(norms + im.t_begin + tok), kNormFloor) : 0.f;
                    const uint32_t owner = (pk >= im.half) ? 1u : 0u;
                    const uint32_t krow = ptx::map_to_rank(arena_u32, owner) +
                                          (uint32_t)(max(pk, 0) - (int)owner * im.half) * (uint32_t)im.ldk * 4u;
                    for (int c = (g >> 1); c < nchunk; c += 2) {
                        uint32_t r[32];
                        ptx::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tile * 256 + c * 32), r);
                        ptx::tmem_ld_wait();
                        if (pk >= 0) {
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                float4 kv;
                                const int j = c * 32 + 4 * v;
                                kv.x = (j + 0 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 0]) * inv_ni * sh->inv_nj[j + 0] - shift) * inv_eps) : 0.f;
                                kv.y = (j + 1 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 1]) * inv_ni * sh->inv_nj[min(j + 1, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                kv.z = (j + 2 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 2]) * inv_ni * sh->inv_nj[min(j + 2, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                kv.w = (j + 3 < im.B) ? exp_fast((__uint_as_float(r[4 * v + 3]) * inv_ni * sh->inv_nj[min(j + 3, kFuMaxB - 1)] - shift) * inv_eps) : 0.f;
                                st_cluster_v4(krow + (uint32_t)j * 4u, kv);
                            }
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::cluster_sync_all();           // #2: every K row is with its owner
            ptx::tc_fence_after();

            // ---- Sinkhorn on this CTA's rows ---------------------------------------------------------------
            const float *kbuf = reinterpret_cast<const float *>(arena);
            const int rps = im.ldk <= 128 ? 4 : 2;
            const int ns = max(1, (im.half + kFuWarps * rps - 1) / (kFuWarps * rps));
#define RTP_FU(LR, CPL, NS) ist = fused_sinkhorn<LR, CPL, NS>(sh, kbuf, arena, im, rank, p, kappa, v_init)
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
            ptx::fence_proxy_async_all();      // the plan rows (ordinary stores, some into the other CTA) feed UMMAs
            ptx::cluster_sync_all();           // #3: plan tiles and pairing partials are in place
        }

        __syncthreads();                       // out0 (with nothing pruned no barrier has passed since it was written)
        // ---- rank 0, warps 8-15: the pairs ---------------------------------------------------------------
        if (im.B > 0 && rank == 0 && warp >= 8) {
            const int out0 = sh->out0;
            const int seg = im.t_begin - out0;
            for (int j = tid - 256; j < im.B; j += 256) {
                float b = sh->pairv[0][j];
                int ib = sh->pairi[0][j];
                const float ob = sh->pairv[1][j];      // rank 1 holds the higher rows: strict > keeps the lower
                if (ob > b) {
                    b = ob;
                    ib = sh->pairi[1][j];
                }
                merged_idx[seg + j] = __ldcg(ord + im.M + j);
                merge_partner[seg + j] = ib;
                merge_weight[seg + j] = b * sh->vs[j];
            }
        }

        // ---- merge: for every tile of 64 output columns, [I | alpha P] . [X rows of the token tiles ; T_p] ----
        const int nident0 = im.ntile > 0 ? (min(im.ntok, kFuTileM) > 64 ? 2 : 1) : 0;
        const int nident1 = im.ntile > 1 ? (im.ntok - kFuTileM > 64 ? 2 : 1) : 0;
        if (warp == 0) {
            if (lane == 0 && im.ntile > 0) {
                ptx::fence_proxy_async_all();
                uint32_t it = 0;
                for (int ct = 0; ct < nct && !sh->abort_flag; ++ct) {
                    const int nload = nident0 + nident1 + im.nkb;
                    for (int l = 0; l < nload; ++l, ++it) {
                        const int s = it % kFuMgStages;
                        if (it >= (uint32_t)kFuMgStages &&
                            !ptx::mbar_wait(&sh->mg_empty[s], ((it / kFuMgStages) - 1) & 1)) {
                            sh->abort_flag = 1;
                            atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                            break;
                        }
                        const uint32_t dst = arena_u32 + kFuPartOffset + s * kFuBoxBytes;
                        ptx::mbar_arrive_expect_tx(&sh->mg_full[s], kFuBoxBytes);
                        if (l < nident0 + nident1) {
                            const int t = l < nident0 ? 0 : 1, kb = l < nident0 ? l : l - nident0;
                            ptx::tma_load_2d(dst, &tmapXb, &sh->mg_full[s], ct * kFuNT,
                                             im.t_begin + im.tok_lo + t * kFuTileM + kb * 64);
                        } else {
                            ptx::tma_load_2d(dst, &tmapXp, &sh->mg_full[s], ct * kFuNT, xp0 + (l - nident0 - nident1) * 64);
                        }
                    }
                }
            }
        } else if (warp == 1) {
            if (lane == 0 && im.ntile > 0) {
                ptx::fence_proxy_async_smem();
                const uint32_t idesc = ptx::idesc_bf16(kFuTileM, kFuNT, false, true);
                const uint32_t ident_u32 = ptx::smem_u32(ident);
                uint32_t it = 0;
                bool failed = false;
                for (int ct = 0; ct < nct && !sh->abort_flag && !failed; ++ct) {
                    const int as = ct % kFuAccStages;
                    if (ct >= kFuAccStages) {
                        if (!ptx::mbar_wait(&sh->acc_empty[as], ((ct / kFuAccStages) - 1) & 1)) {
                            failed = true;
                            break;
                        }
                        ptx::tc_fence_after();
                    }
                    const uint32_t d_tmem = tmem_base + (uint32_t)(as * 128);
                    for (int t = 0; t < im.ntile && !failed; ++t) {
                        const int ni = t == 0 ? nident0 : nident1;
                        for (int kb = 0; kb < ni; ++kb, ++it) {
                            const int s = it % kFuMgStages;
                            if (!ptx::mbar_wait(&sh->mg_full[s], (it / kFuMgStages) & 1)) {
                                failed = true;
                                break;
                            }
                            ptx::tc_fence_after();
                            const uint32_t a_base = ident_u32 + (1 - kb) * (kFuABytes / 2);
                            const uint32_t b_base = arena_u32 + kFuPartOffset + s * kFuBoxBytes;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint64_t da = ptx::smem_desc_sw128(a_base + k * 32, 16, 1024);
                                const uint64_t db = ptx::smem_desc_sw128(b_base + k * 2048, kFuBoxBytes, 1024);
                                ptx::umma_bf16(d_tmem + (uint32_t)(t * 64), da, db, idesc, (kb | k) != 0);
                            }
                            ptx::umma_commit(&sh->mg_empty[s]);
                        }
                    }
                    for (int kb = 0; kb < im.nkb && !failed; ++kb, ++it) {
                        const int s = it % kFuMgStages;
                        if (!ptx::mbar_wait(&sh->mg_full[s], (it / kFuMgStages) & 1)) {
                            failed = true;
                            break;
                        }
                        ptx::tc_fence_after();
                        const uint32_t b_base = arena_u32 + kFuPartOffset + s * kFuBoxBytes;
                        for (int t = 0; t < im.ntile; ++t) {
                            const uint32_t a_base = arena_u32 + (uint32_t)(t * im.nkb + kb) * kFuABytes;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint64_t da = ptx::smem_desc_sw128(a_base + k * 32, 16, 1024);
                                const uint64_t db = ptx::smem_desc_sw128(b_base + k * 2048, kFuBoxBytes, 1024);
                                ptx::umma_bf16(d_tmem + (uint32_t)(t * 64), da, db, idesc, 1u);
                            }
                        }
                        ptx::umma_commit(&sh->mg_empty[s]);
                    }
                    if (!failed) ptx::umma_commit(&sh->acc_full[as]);
                }
                if (failed) {
                    sh->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                }
            }
        } else if (warp >= 4 && warp < 8 && im.ntile > 0) {
            // ---- epilogue: TMEM -> bf16 -> this warp's staging rows -> coalesced stores of the kept rows ------
            const int q = warp - 4;
            const int out0 = sh->out0;
            uint8_t *stg = arena + kFuStagingOffset + q * 32 * kFuStagePitch;
            int pk[2], tokv[2];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int tr = t * kFuTileM + q * 32 + lane;
                tokv[t] = im.tok_lo + tr;
                pk[t] = (t < im.ntile && tr < im.ntok) ? __ldcg(kpos + im.t_begin + tokv[t]) : -1;
                if (pk[t] >= 0) kept_idx[out0 + pk[t]] = tokv[t];
            }
            bool dead = false;
            for (int ct = 0; ct < nct; ++ct) {
                const int as = ct % kFuAccStages;
                bool ok = !dead && !sh->abort_flag && ptx::mbar_wait(&sh->acc_full[as], (ct / kFuAccStages) & 1);
                if (!__all_sync(0xffffffffu, ok)) {
                    if (!dead) {
                        sh->abort_flag = 1;
                        if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                    }
                    dead = true;
                    continue;
                }
                ptx::tc_fence_after();
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    // a warp whose 32 rows all lie past the CTA's tokens has nothing to convert or store
                    if (t >= im.ntile || t * kFuTileM + q * 32 >= im.ntok) continue;
#pragma unroll
                    for (int c0 = 0; c0 < kFuNT; c0 += 32) {
                        uint32_t r[32];
                        ptx::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * 128 + t * 64 + c0), r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            __nv_bfloat162 o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                o[e] = __floats2bfloat162_rn(__uint_as_float(r[8 * g + 2 * e]),
                                                             __uint_as_float(r[8 * g + 2 * e + 1]));
                            *reinterpret_cast<uint4 *>(stg + lane * kFuStagePitch + (c0 + 8 * g) * 2) =
                                *reinterpret_cast<uint4 *>(o);
                        }
                    }
                    __syncwarp();
                    // 8 lanes write one row's 128 bytes: 4 rows per instruction
#pragma unroll
                    for (int rr = 0; rr < 32; rr += 4) {
                        const int row = rr + (lane >> 3);
                        const int prow = __shfl_sync(0xffffffffu, pk[t], row);
                        if (prow >= 0) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(stg + row * kFuStagePitch + (lane & 7) * 16);
                            *reinterpret_cast<uint4 *>(Y + (size_t)(out0 + prow) * d + ct * kFuNT + (lane & 7) * 8) = v;
                        }
                    }
                    __syncwarp();
                }
                ptx::tc_fence_before();
                ptx::mbar_arrive(&sh->acc_empty[as]);
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
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace rtp
