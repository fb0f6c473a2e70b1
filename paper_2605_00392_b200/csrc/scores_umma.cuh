// Cosine scores S = T_kept T_prop^T / (|.| |.|) (Section 3.3.2, Appendix C) on the tcgen05 tensor
// cores, bf16 inputs, fp32 accumulation in tensor memory.
//
// One CTA computes a 128-token x B tile of one image over the full width d.
//   * A operand: 128 CONSECUTIVE tokens of the image (kept and pruned alike), fetched by tiled TMA
//     (64-column boxes, 128-byte swizzle).  Rows of pruned tokens are computed and dropped: kept
//     tokens are ~84 % of an image, and contiguous rows are what TMA moves at full speed.
//   * B operand: the image's pruned tokens, read from the compact copy the selection kernel made,
//     so that they too are contiguous rows for tiled TMA (64-row boxes).  Rows past B inside the last
//     box are zeros or another image's tokens; they only reach accumulator columns nobody reads.
//   * D: 128 TMEM lanes x BN columns (BN = B rounded up to 16, at most 256 per pass).
// Warp roles (192 threads): warps 0-3 run the epilogue (TMEM -> registers -> divide by the two norms
// -> global); warp 4 issues the TMA loads (those of a k-block from several lanes at once); warp 5 owns TMEM and its
// lane 0 issues the UMMAs.  A
// ring of shared-memory stages (as many as fit in 96 KB: 4 for B <= 64, 2 for B = 256) is handed over
// with mbarriers.  The ring is sized so that two CTAs share an SM: a whole Large batch is one wave.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace rtp {

constexpr int kScTileM = 128;
constexpr int kScBK = 64;            // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kScMaxStages = 8;
constexpr int kScBNMax = 256;
constexpr int kScBBoxRows = 64;      // rows per TMA box of the B operand
constexpr int kScThreads = 192;
constexpr int kScABytes = kScTileM * 128;    // 16 KB
constexpr int kScBBoxBytes = kScBBoxRows * 128;  // 8 KB
constexpr int kScRingBytes = 96 * 1024;
constexpr int kScSmemBytes = kScRingBytes + 1024 /*alignment*/ + 2048 /*barriers, norms*/;

struct ScoresBarriers {
    uint64_t full[kScMaxStages];
    uint64_t empty[kScMaxStages];
    uint64_t accum_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    volatile int abort_flag;
    float inv_nj[kScBNMax];          // 1 / |x_j| of the current pass's pruned tokens
};

__global__ void __launch_bounds__(kScThreads, 2)
scores_umma_kernel(const __grid_constant__ CUtensorMap tmapX, const __grid_constant__ CUtensorMap tmapXp,
                   const int32_t *__restrict__ offsets, int d, const int32_t *__restrict__ counts,
                   const int32_t *__restrict__ order, const int32_t *__restrict__ kpos,
                   const float *__restrict__ norms, float *__restrict__ kmat, int kmat_stride,
                   int max_tokens, int total, WsHeader *__restrict__ hdr, uint32_t *__restrict__ scores_done)
{
    extern __shared__ uint8_t smem_raw[];
    const int img = blockIdx.y, mt = blockIdx.x;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();     // counts, order, norms and the compact copy come from the kernels ahead
    int t_begin, N;
    const int M = __ldcg(counts + img);       // (issued with the two offsets: one trip to L2)
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int B = N - M;
    if (mt * kScTileM >= N) return;
    // With scores_done, every tile of a valid image is counted when it is complete (at once if nothing is
    // pruned): the Sinkhorn kernel, launched as a programmatic dependent, starts on an image when its
    // tiles are in.
    if (B == 0) {
        if (scores_done && threadIdx.x == 0) atomicAdd(&scores_done[img], 1u);
        return;
    }

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    ScoresBarriers *bars = reinterpret_cast<ScoresBarriers *>(smem + kScRingBytes);
    // stage = A tile + the B boxes of the widest pass; as many stages as fit in the ring
    const int boxes_max = (min(kScBNMax, B) + kScBBoxRows - 1) / kScBBoxRows;
    const int stage_bytes = kScABytes + boxes_max * kScBBoxBytes;
    const int kScStages = min(kScMaxStages, kScRingBytes / stage_bytes);   // 2 .. 4
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = (d + kScBK - 1) / kScBK;
    const int nbt = (B + kScBNMax - 1) / kScBNMax;
    const int32_t *ord = order + t_begin;
    const int xp0 = xp_row0(t_begin, img);

    if (tid == 0) {
        for (int s = 0; s < kScMaxStages; ++s) {
            ptx::mbar_init(&bars->full[s], 1);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        ptx::mbar_init(&bars->accum_full, 1);
        ptx::mbar_init(&bars->tmem_empty, 128);
        bars->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 5) {
        ptx::tmem_alloc(&bars->tmem_base, kScBNMax);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t smem_base = ptx::smem_u32(smem);

    if (warp == 4) {
        // ---------------- producer: tiled TMA for both operands -----------------------------------
        // The whole warp walks the k-blocks in step; the loads of a k-block are issued by as many lanes at
        // once (lane 0: the A tile, lanes 1-4: the B boxes) instead of by one thread one after the other.
        {
            if (lane == 0) {
                ptx::prefetch_tensormap(&tmapX);
                ptx::prefetch_tensormap(&tmapXp);
            }
            uint32_t it = 0;
            bool alive = true;
            for (int bt = 0; bt < nbt && alive && !bars->abort_flag; ++bt) {
                const int nbox = (min(kScBNMax, B - bt * kScBNMax) + kScBBoxRows - 1) / kScBBoxRows;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kScStages;
                    const bool ok = it < (uint32_t)kScStages || ptx::mbar_wait(&bars->empty[s], ((it / kScStages) - 1) & 1);
                    if (!__all_sync(0xffffffffu, ok)) {
                        bars->abort_flag = 1;
                        if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        alive = false;
                        break;
                    }
                    const uint32_t a_dst = smem_base + s * stage_bytes;
                    if (lane == 0) ptx::mbar_arrive_expect_tx(&bars->full[s], kScABytes + nbox * kScBBoxBytes);
                    __syncwarp();
                    if (lane == 0)
                        ptx::tma_load_2d(a_dst, &tmapX, &bars->full[s], kb * kScBK, t_begin + mt * kScTileM);
                    else if (lane <= nbox)
                        ptx::tma_load_2d(a_dst + kScABytes + (lane - 1) * kScBBoxBytes, &tmapXp, &bars->full[s],
                                         kb * kScBK, xp0 + bt * kScBNMax + (lane - 1) * kScBBoxRows);
                }
            }
        }
    } else if (warp == 5) {
        // ---------------- UMMA issuer -----------------------------------------------------------
        if (lane == 0) {
            uint32_t it = 0;
            for (int bt = 0; bt < nbt && !bars->abort_flag; ++bt) {
                const int BN = min(kScBNMax, (B - bt * kScBNMax + 15) & ~15);
                const uint32_t idesc = ptx::idesc_bf16(kScTileM, BN, false, false);
                if (bt > 0) {
                    if (!ptx::mbar_wait(&bars->tmem_empty, (bt - 1) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::tc_fence_after();
                }
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kScStages;
                    if (!ptx::mbar_wait(&bars->full[s], (it / kScStages) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a_base = smem_base + s * stage_bytes;
                    const uint32_t b_base = a_base + kScABytes;
#pragma unroll
                    for (int k = 0; k < kScBK / 16; ++k) {
                        const uint64_t da = ptx::smem_desc_sw128(a_base + k * 32, 16, 1024);
                        const uint64_t db = ptx::smem_desc_sw128(b_base + k * 32, 16, 1024);
                        ptx::umma_bf16(tmem_base, da, db, idesc, (kb | k) != 0);
                    }
                    ptx::umma_commit(&bars->empty[s]);
                }
                ptx::umma_commit(&bars->accum_full);
            }
        }
    } else {
        // ---------------- warps 0-3: epilogue -----------------------------------------------------
        float *Simg = kmat + kmat_offset(kmat_stride, t_begin, img);
        const int ldS = score_pitch(B);
        const int row = tid;                       // TMEM lane = tile row
        const int k_tok = mt * kScTileM + row;
        const int p = (k_tok < N) ? kpos[t_begin + k_tok] : -1;
        const float inv_ni = (p >= 0) ? 1.f / fmaxf(norms[t_begin + k_tok], kNormFloor) : 1.f;
        bool dead = false;     // a wait gave up: keep taking the named barriers, skip the rest
        for (int bt = 0; bt < nbt; ++bt) {
            const int j0 = bt * kScBNMax;
            const int BN = min(kScBNMax, (B - j0 + 15) & ~15);
            // 1/|x_j| of this pass's columns, shared by the 128 epilogue threads (the first barrier
            // keeps a fast warp from overwriting values a slow one still reads)
            if (bt > 0) asm volatile("bar.sync 1, 128;" ::: "memory");
            for (int j = tid; j < min(B - j0, kScBNMax); j += 128)
                bars->inv_nj[j] = 1.f / fmaxf(norms[t_begin + ord[M + j0 + j]], kNormFloor);
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (dead) continue;
            // the TMEM loads below are warp-collective: take the go / no-go decision per warp
            bool ok = !bars->abort_flag && ptx::mbar_wait(&bars->accum_full, bt & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                bars->abort_flag = 1;
                if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                dead = true;
                continue;
            }
            ptx::tc_fence_after();
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
                ptx::tmem_ld_wait();
                if (p >= 0) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const int j = j0 + c0 + 4 * g;
                        if (j < B) {
                            float o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int je = min(j + e, B - 1) - j0;
                                o[e] = __uint_as_float(r[4 * g + e]) * inv_ni * bars->inv_nj[je];
                            }
                            *reinterpret_cast<float4 *>(Simg + (size_t)p * ldS + j) =
                                make_float4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&bars->tmem_empty);
        }
    }

    ptx::tc_fence_before();
    if (scores_done) __threadfence();          // the epilogue's stores, before the count below
    __syncthreads();
    if (scores_done && tid == 0) {
        __threadfence();
        atomicAdd(&scores_done[img], 1u);
    }
    if (warp == 5) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kScBNMax);
    }
}

}  // namespace rtp
