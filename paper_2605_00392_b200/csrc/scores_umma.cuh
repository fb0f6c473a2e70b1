// Cosine scores S = T_kept T_prop^T / (|.| |.|) (Section 3.3.2, Appendix C) on the tcgen05 tensor
// cores, bf16 inputs, fp32 accumulation in tensor memory.
//
// One CTA computes a 128-token x B tile of one image over the full width d.
//   * A operand: 128 CONSECUTIVE tokens of the image (kept and pruned alike), fetched by tiled TMA
//     (64-column boxes, 128-byte swizzle).  Rows of pruned tokens are computed and dropped: kept
//     tokens are ~84 % of an image, and contiguous rows are what TMA moves at full speed.
//   * B operand: the image's pruned tokens, gathered row by row with 16-byte cp.async copies into
//     the same swizzled K-major layout (a gather cannot be expressed as one tiled box).
//   * D: 128 TMEM lanes x BN columns (BN = B rounded up to 16, at most 256 per pass).
// Warp roles (192 threads): warps 0-3 gather B, then run the epilogue (TMEM -> registers -> divide by
// the two norms -> global); warp 4 lane 0 issues the TMA loads; warp 5 owns TMEM and lane 0 issues
// the UMMAs.  A ring of shared-memory stages (as many as fit: 8 for B <= 64, 4 for B = 256) is handed
// over with mbarriers; the gather keeps kScLag stages of copies in flight per thread.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace rtp {

constexpr int kScTileM = 128;
constexpr int kScBK = 64;            // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kScMaxStages = 8;
constexpr int kScLag = 3;            // stages of gather copies in flight per thread (< stages)
constexpr int kScBNMax = 256;
constexpr int kScThreads = 192;
constexpr int kScABytes = kScTileM * 128;    // 16 KB
constexpr int kScRingBytes = 4 * (kScABytes + kScBNMax * 128);   // 192 KB of stage buffers
constexpr int kScSmemBytes = kScRingBytes + 1024 /*alignment*/ + 2048 /*barriers, norms*/;

struct ScoresBarriers {
    uint64_t full[kScMaxStages];
    uint64_t empty[kScMaxStages];
    uint64_t accum_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    volatile int abort_flag;
    float inv_nj[kScBNMax];          // 1 / |x_j| of the first pass's pruned tokens
};

__global__ void __launch_bounds__(kScThreads, 1)
scores_umma_kernel(const __grid_constant__ CUtensorMap tmapX, const __nv_bfloat16 *__restrict__ X,
                   const int32_t *__restrict__ offsets, int d, const int32_t *__restrict__ counts,
                   const int32_t *__restrict__ order, const int32_t *__restrict__ kpos,
                   const float *__restrict__ norms, float *__restrict__ kmat, int kmat_stride,
                   int max_tokens, int total, WsHeader *__restrict__ hdr)
{
    extern __shared__ uint8_t smem_raw[];
    const int img = blockIdx.y, mt = blockIdx.x;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    if (B == 0 || mt * kScTileM >= N) return;

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    ScoresBarriers *bars = reinterpret_cast<ScoresBarriers *>(smem + kScRingBytes);
    // stage = A tile + this image's B tile; as many stages as fit in the ring
    const int stage_bytes = kScABytes + min(kScBNMax, (B + 15) & ~15) * 128;
    const int kScStages = min(kScMaxStages, kScRingBytes / stage_bytes);   // 4 .. 8
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = (d + kScBK - 1) / kScBK;
    const int nbt = (B + kScBNMax - 1) / kScBNMax;
    const int32_t *ord = order + t_begin;

    if (tid == 0) {
        for (int s = 0; s < kScMaxStages; ++s) {
            ptx::mbar_init(&bars->full[s], 1 + 128);
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
        // ---------------- A producer: tiled TMA ------------------------------------------------
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmapX);
            uint32_t it = 0;
            for (int bt = 0; bt < nbt && !bars->abort_flag; ++bt) {
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kScStages;
                    if (it >= (uint32_t)kScStages &&
                        !ptx::mbar_wait(&bars->empty[s], ((it / kScStages) - 1) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(&bars->full[s], kScABytes);
                    ptx::tma_load_2d(smem_base + s * stage_bytes, &tmapX, &bars->full[s], kb * kScBK,
                                     t_begin + mt * kScTileM);
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
        // ---------------- warps 0-3: gather B, then epilogue ------------------------------------
        const int c = tid & 7, rbase = tid >> 3;
        uint32_t it = 0;
        float *Simg = kmat + kmat_offset(kmat_stride, t_begin, img);
        const int ldS = score_pitch(B);
        const int row = tid;                       // TMEM lane = tile row
        const int k_tok = mt * kScTileM + row;
        const int p = (k_tok < N) ? kpos[t_begin + k_tok] : -1;
        const float inv_ni = (p >= 0) ? 1.f / fmaxf(norms[t_begin + k_tok], kNormFloor) : 1.f;
        // 1/|x_j| of the first pass's columns, shared by the 128 epilogue threads.  The barrier is
        // reached unconditionally: nothing can have failed yet.
        for (int j = tid; j < min(B, kScBNMax); j += 128)
            bars->inv_nj[j] = 1.f / fmaxf(norms[t_begin + ord[M + j]], kNormFloor);
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int bt = 0; bt < nbt; ++bt) {
            if (bt > 0 && __any_sync(0xffffffffu, bars->abort_flag != 0)) break;  // warp-uniform
            const int j0 = bt * kScBNMax;
            const int BN = min(kScBNMax, (B - j0 + 15) & ~15);
            int tok[kScBNMax / 16];
#pragma unroll
            for (int q = 0; q < kScBNMax / 16; ++q) {
                const int j = j0 + rbase + 16 * q;
                tok[q] = (16 * q < BN && j < B) ? t_begin + ord[M + j] : -1;
            }
            bool failed = false;
            const uint32_t it0 = it;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % kScStages;
                if (it >= (uint32_t)kScStages &&
                    !ptx::mbar_wait(&bars->empty[s], ((it / kScStages) - 1) & 1)) {
                    failed = true;
                    break;
                }
                const uint32_t b_base = smem_base + s * stage_bytes + kScABytes;
                const int kcol = kb * kScBK + c * 8;
#pragma unroll
                for (int q = 0; q < kScBNMax / 16; ++q) {
                    if (16 * q < BN) {
                        const int r = rbase + 16 * q;
                        const bool ok = tok[q] >= 0 && kcol < d;
                        const __nv_bfloat16 *src = ok ? X + (size_t)tok[q] * d + kcol : X;
                        const uint32_t dst = b_base + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
                        ptx::cp_async_16(dst, src, ok ? 16u : 0u);
                    }
                }
                ptx::cp_async_commit();
                if (kb >= kScLag) {     // the copies issued kScLag k-blocks ago have landed
                    ptx::cp_async_wait<kScLag>();
                    ptx::fence_proxy_async_smem();
                    ptx::mbar_arrive(&bars->full[(it - kScLag) % kScStages]);
                }
            }
            ptx::cp_async_wait<0>();
            if (!failed) {
                ptx::fence_proxy_async_smem();
                for (uint32_t q = (it - it0 > (uint32_t)kScLag ? it - kScLag : it0); q < it; ++q)
                    ptx::mbar_arrive(&bars->full[q % kScStages]);
            }
            // the TMEM loads below are warp-collective: take the go / no-go decision per warp
            bool ok = !__any_sync(0xffffffffu, failed);
            if (ok) ok = ptx::mbar_wait(&bars->accum_full, bt & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                bars->abort_flag = 1;
                if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                break;
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
                                const int je = min(j + e, B - 1);
                                const float inv_nj =
                                    (bt == 0) ? bars->inv_nj[je]
                                              : 1.f / fmaxf(__ldg(norms + t_begin + ord[M + je]), kNormFloor);
                                o[e] = __uint_as_float(r[4 * g + e]) * inv_ni * inv_nj;
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
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kScBNMax);
    }
}

}  // namespace rtp
