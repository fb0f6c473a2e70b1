// Dustbin-augmented optimal transport by Sinkhorn iterations (Eq. 5, Appendix C) in scaling form, one
// cluster of two CTAs per image, the kernel matrix K of a thread's rows held in its REGISTERS across the
// iterations, and the two CTAs' column sums exchanged by asynchronous stores counted on a barrier (no
// cluster-wide barrier in the loop).  The iteration itself is fused_iterate (fused.cuh); this kernel is
// its stand-alone form for the schedule of separate kernels: it reads the scores from the workspace tile,
// writes alpha P (bf16, row = token position) for the tensor-core merge, hands the image to the merge
// kernel as soon as that is done, and then writes the pairs.  Taken instead of sinkhorn_cluster_kernel when
// every tile the run can hold fits: at most 256 pruned tokens, 64 K values per thread.
#pragma once
#include "fused.cuh"

namespace rtp {

// K into registers, the iterations, alpha P to the plan buffer, the pairing partials to rank 0.
template <int LR, int CPL, int NS>
__device__ inline FuIterState reg_sinkhorn(FuShared *sh, const float *kbuf, float *part, int Ml, int row_lo, int M, int B,
                                           uint32_t rank, const OtParams &p, float kappa, float v_init, uint32_t &round,
                                           WsHeader *hdr, __nv_bfloat16 *__restrict__ Pimg, int pbuf_pitch, int img,
                                           uint32_t *__restrict__ sink_done, int32_t *__restrict__ ready_list)
{
    constexpr int ldk = LR * CPL;
    constexpr int RPS = 32 / LR;
    constexpr int NQ = CPL / 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LR, slot = lane / LR;

    float4 k[NS][NQ];
    float U[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const int i = (s * kFuWarps + warp) * RPS + slot;
#pragma unroll
        for (int q = 0; q < NQ; ++q)
            k[s][q] = (i < Ml) ? *reinterpret_cast<const float4 *>(kbuf + (size_t)i * (ldk + 4) + 4 * (q * LR + sub))
                               : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const FuIterState st = fused_iterate<LR, CPL, NS>(k, U, sh, part, Ml, M, B, rank, p, kappa, v_init, round, hdr);
    if (p.iters == 0) {
#pragma unroll
        for (int s = 0; s < NS; ++s) U[s] = ((s * kFuWarps + warp) * RPS + slot < Ml) ? 1.f : 0.f;   // u = 0
    }

    // alpha P = alpha U K V in bf16: row = the kept token's position in X, columns up to the next multiple
    // of 64 (zeros past B: K is zero there), 4 columns = 8 bytes per store
    const int kpad = (B + 63) & ~63;
    float4 V[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) V[q] = *reinterpret_cast<const float4 *>(sh->vs + 4 * (q * LR + sub));
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        const int i = (s * kFuWarps + warp) * RPS + slot;
        if (i < Ml) {
            __nv_bfloat16 *prow = Pimg + (size_t)sh->rowtok[i] * pbuf_pitch;
            const float au = p.alpha * U[s];
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int col = 4 * (q * LR + sub);
                if (col < kpad) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn((k[s][q].x * au) * V[q].x, (k[s][q].y * au) * V[q].y);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn((k[s][q].z * au) * V[q].z, (k[s][q].w * au) * V[q].w);
                    *reinterpret_cast<uint2 *>(prow + col) =
                        make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
                }
            }
            if (ldk < 64) *reinterpret_cast<uint2 *>(prow + 32 + 4 * sub) = make_uint2(0u, 0u);   // columns 32 .. 63
        }
    }
    // the merge kernel may take the image from here: the pairs below are outputs of their own
    sinkhorn_publish(img, 2u, sink_done, ready_list, hdr);

    fused_pair_partials<LR, CPL, NS>(k, U, sh, part, Ml, row_lo, B, rank);
    return st;
}

// grid = 2 * batch CTAs of kFuThreads threads, clusters of 2 along x.  Dynamic shared memory: kFuSmemBytes.
__global__ void __launch_bounds__(kFuThreads, 1)
sinkhorn_reg_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                    const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                    const float *__restrict__ kmat, int kmat_stride, int max_tokens, int total, OtParams p,
                    __nv_bfloat16 *__restrict__ pbuf, int pbuf_pitch, int32_t *__restrict__ merged_idx,
                    int32_t *__restrict__ merge_partner, float *__restrict__ merge_weight, float *__restrict__ stats,
                    uint32_t *__restrict__ sink_done, int32_t *__restrict__ ready_list, WsHeader *__restrict__ hdr,
                    const uint32_t *scores_done)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FuShared *sh = reinterpret_cast<FuShared *>(smem);
    uint8_t *arena = smem + kFuSharedBytes;
    float *kbuf = reinterpret_cast<float *>(arena);
    float *part = reinterpret_cast<float *>(arena + kFuPartOffset);
    const uint32_t rank = ptx::cluster_ctarank();
    const int img = blockIdx.x >> 1, tid = threadIdx.x;
    if (tid == 0) {
        ptx::mbar_init(&sh->xbar[0], 1);
        ptx::mbar_init(&sh->xbar[1], 1);
        sh->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    ptx::grid_dep_launch();
    // The scores come from the kernel ahead: wait for that grid to end, or, with per-image counts of
    // finished score tiles, only for this image's tiles (and for the grid before leaving, so that this
    // grid's end still implies that one's).
    if (!scores_done) ptx::grid_dep_wait();
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) {
        sinkhorn_publish(img, 2u, sink_done, ready_list, hdr);
        if (scores_done) ptx::grid_dep_wait();
        return;
    }
    if (scores_done) {
        if (tid == 0) {
            const uint32_t want = (uint32_t)((N + 127) / 128);     // the scores kernel's 128-token tiles
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
    const int M = __ldcg(counts + img), out0 = __ldcg(out_offsets + img), B = N - M;     // (one trip to L2 for both)
    if (B == 0) {
        sinkhorn_publish(img, 2u, sink_done, ready_list, hdr);
        if (scores_done) ptx::grid_dep_wait();
        return;
    }
    const int half = (M + 1) >> 1;
    const int row_lo = min(M, (int)rank * half);
    const int Ml = min(M, row_lo + half) - row_lo;
    const int ldk = sinkhorn_ldk(B);
    const int ldS = score_pitch(B);
    const float *Sg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const float inv_eps = 1.f / p.eps;
    const float shift = fmaxf(1.f, p.z);
    const float kappa = expf((p.z - shift) * inv_eps);
    const float v_init = expf(shift * inv_eps);

    for (int i = tid; i < Ml; i += kFuThreads) sh->rowtok[i] = __ldcg(order + t_begin + row_lo + i);
    // ---- K = exp((S - c)/eps) of this CTA's rows into shared memory (pitch ldk + 4), zero beyond column B ----
    {
        const int qpr = ldk >> 2;                     // float4 per row of K
        const int total_q = Ml * qpr;
        constexpr int kInFlight = 8;                  // 16-byte loads a thread has in flight per trip to L2
        for (int q0 = tid; q0 < total_q; q0 += kFuThreads * kInFlight) {
            float4 s4[kInFlight];
            int ii[kInFlight], jj[kInFlight];
#pragma unroll
            for (int a = 0; a < kInFlight; ++a) {
                const int q = q0 + a * kFuThreads;
                ii[a] = q / qpr;
                jj[a] = (q - ii[a] * qpr) << 2;
                s4[a] = (q < total_q && jj[a] < ldS)
                            ? __ldcg(reinterpret_cast<const float4 *>(Sg + (size_t)(row_lo + ii[a]) * ldS + jj[a]))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int a = 0; a < kInFlight; ++a) {
                const int q = q0 + a * kFuThreads;
                if (q < total_q) {
                    float4 kv;
                    kv.x = (jj[a] + 0 < B) ? exp_fast((s4[a].x - shift) * inv_eps) : 0.f;
                    kv.y = (jj[a] + 1 < B) ? exp_fast((s4[a].y - shift) * inv_eps) : 0.f;
                    kv.z = (jj[a] + 2 < B) ? exp_fast((s4[a].z - shift) * inv_eps) : 0.f;
                    kv.w = (jj[a] + 3 < B) ? exp_fast((s4[a].w - shift) * inv_eps) : 0.f;
                    *reinterpret_cast<float4 *>(kbuf + (size_t)ii[a] * (ldk + 4) + jj[a]) = kv;
                }
            }
        }
    }
    __syncthreads();
    // both CTAs are running and have their barriers in place before anything is sent to the other
    ptx::cluster_sync_all();

    uint32_t round = 0;
    FuIterState ist{0, 0.f};
    __nv_bfloat16 *Pimg = pbuf + (size_t)t_begin * pbuf_pitch;
    const int rps = ldk <= 128 ? 4 : 2;
    const int ns = max(1, (half + kFuWarps * rps - 1) / (kFuWarps * rps));
#define RTP_RG(LR, CPL, NS) \
    ist = reg_sinkhorn<LR, CPL, NS>(sh, kbuf, part, Ml, row_lo, M, B, rank, p, kappa, v_init, round, hdr, Pimg, pbuf_pitch, img, sink_done, ready_list)
#define RTP_RG_NS(LR, CPL, NSMAX)                                 \
    switch (ns) {                                                 \
    case 1: RTP_RG(LR, CPL, 1); break;                            \
    case 2: RTP_RG(LR, CPL, 2); break;                            \
    case 3: if (NSMAX >= 3) { RTP_RG(LR, CPL, (NSMAX >= 3 ? 3 : 1)); } break; \
    case 4: if (NSMAX >= 4) { RTP_RG(LR, CPL, (NSMAX >= 4 ? 4 : 1)); } break; \
    default: if (NSMAX >= 5) { RTP_RG(LR, CPL, (NSMAX >= 5 ? 5 : 1)); } break; \
    }
    switch (ldk) {
    case 32: RTP_RG_NS(8, 4, 4); break;
    case 64: RTP_RG_NS(8, 8, 4); break;
    case 128: RTP_RG_NS(8, 16, 4); break;
    case 192: RTP_RG_NS(16, 12, 5); break;
    default: RTP_RG_NS(16, 16, 4); break;
    }
#undef RTP_RG_NS
#undef RTP_RG
    if (tid == 0 && rank == 0) {
        stats[(size_t)img * kStats + 5] = (float)ist.done;
        stats[(size_t)img * kStats + 6] = ist.last_move;
    }
    ptx::cluster_sync_all();          // the pairing partials are with rank 0; nothing is sent to another CTA after this
    if (rank == 0) {
        const int seg = t_begin - out0;
        for (int j = tid; j < B; j += kFuThreads) {
            float b = sh->pairv[0][j];
            int ib = sh->pairi[0][j];
            const float ob = sh->pairv[1][j];      // rank 1 holds the higher rows: strict > keeps the lower row
            if (ob > b) {
                b = ob;
                ib = sh->pairi[1][j];
            }
            merged_idx[seg + j] = __ldcg(order + t_begin + M + j);
            merge_partner[seg + j] = ib;
            merge_weight[seg + j] = b * sh->vs[j];
        }
    }
    if (scores_done) ptx::grid_dep_wait();
}

// Every tile a run with at most max_tokens tokens and max_b pruned tokens per image can produce fits.
__host__ inline bool sinkhorn_reg_eligible(int max_tokens, int max_b)
{
    if (max_b > kFuMaxB || max_b < 1) return false;
    for (int b = 1; b <= max_b; ++b) {
        const int m = max_tokens - b > 1 ? max_tokens - b : 1;
        const int rows = (m + 1) / 2;
        if (rows > kFuMaxRows) return false;
        const int regs = fused_k_regs(rows, b);
        if (regs == 0 || regs > kFuKRegs) return false;
    }
    return true;
}

}  // namespace rtp
