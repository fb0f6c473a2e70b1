// Merge + pack (Eq. 7 and the output of Algorithm 1): Y = T_k + alpha * P T_p, written packed, with
// the P T_p contraction on the tcgen05 tensor cores (bf16 inputs, fp32 accumulation in TMEM).
//
// One CTA owns 128 kept tokens of one image and walks the width d in tiles of 256 columns.
//   * A operand: the plan rows P[i][0..B) in bf16, K-major, fetched by tiled TMA from the packed plan
//     buffer (row = packed output row, so consecutive kept tokens are consecutive rows).
//   * B operand: the pruned tokens' rows, gathered with 16-byte cp.async copies into the MN-major
//     128-byte-swizzled layout (the contraction index j is the row, the output column c is
//     contiguous): slab (c / 64) holds rows j of 128 bytes, 8-row groups 1024 bytes apart.
//   * D: two 128-lane x 256-column fp32 accumulators in TMEM, so that the epilogue of one column
//     tile overlaps the UMMAs of the next.
// Warp roles (320 threads): warps 0-3 epilogue (TMEM -> registers, add the kept token's own row,
// round to bf16, store); warps 4-7 gather B; warp 8 lane 0 issues TMA; warp 9 owns TMEM and issues
// the UMMAs.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace rtp {

constexpr int kMgTileM = 128;
constexpr int kMgTileN = 256;        // output columns per accumulator
constexpr int kMgBK = 64;            // pruned tokens (contraction rows) per step
constexpr int kMgStages = 4;
constexpr int kMgThreads = 320;
constexpr int kMgABytes = kMgTileM * 128;            // P tile: 128 rows x 64 bf16
constexpr int kMgBBytes = kMgBK * kMgTileN * 2;      // X_p tile: 64 rows x 256 bf16 = 32 KB
constexpr int kMgStageBytes = kMgABytes + kMgBBytes; // 48 KB
constexpr int kMgSmemBytes = kMgStages * kMgStageBytes + 1024 + 256;

struct MergeBarriers {
    uint64_t full[kMgStages];
    uint64_t empty[kMgStages];
    uint64_t accum_full[2];
    uint64_t accum_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__global__ void __launch_bounds__(kMgThreads, 1)
merge_umma_kernel(const __grid_constant__ CUtensorMap tmapP, const __nv_bfloat16 *__restrict__ X,
                  const int32_t *__restrict__ offsets, int d, const int32_t *__restrict__ counts,
                  const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ order,
                  int max_tokens, int total, float alpha, __nv_bfloat16 *__restrict__ Y,
                  int32_t *__restrict__ kept_idx, WsHeader *__restrict__ hdr)
{
    extern __shared__ uint8_t smem_raw[];
    const int img = blockIdx.y, mt = blockIdx.x;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    const int i0 = mt * kMgTileM;
    if (i0 >= M) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int32_t *ord = order + t_begin;
    const int out0 = out_offsets[img];

    if (B == 0) {
        // retention 1: the output rows are the input rows
        const int rows = min(kMgTileM, M - i0);
        const int vec_per_row = d / 8;
        for (int v = tid; v < rows * vec_per_row; v += kMgThreads) {
            const int r = v / vec_per_row, cv = v - r * vec_per_row;
            const uint4 val = ldg_vec(X + (size_t)(t_begin + ord[i0 + r]) * d + cv * 8);
            *reinterpret_cast<uint4 *>(Y + (size_t)(out0 + i0 + r) * d + cv * 8) = val;
        }
        for (int r = tid; r < rows; r += kMgThreads) kept_idx[out0 + i0 + r] = ord[i0 + r];
        return;
    }

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    MergeBarriers *bars = reinterpret_cast<MergeBarriers *>(smem + kMgStages * kMgStageBytes);
    const int nct = (d + kMgTileN - 1) / kMgTileN;   // column tiles
    const int nkb = (B + kMgBK - 1) / kMgBK;          // contraction steps per column tile

    if (tid == 0) {
        for (int s = 0; s < kMgStages; ++s) {
            ptx::mbar_init(&bars->full[s], 1 + 128);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&bars->accum_full[b], 1);
            ptx::mbar_init(&bars->accum_empty[b], 128);
        }
        bars->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 9) {
        ptx::tmem_alloc(&bars->tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t smem_base = ptx::smem_u32(smem);

    if (warp == 8) {
        // ---------------- A producer: plan tile by TMA ------------------------------------------
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmapP);
            uint32_t it = 0;
            for (int ct = 0; ct < nct && !bars->abort_flag; ++ct) {
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kMgStages;
                    if (it >= (uint32_t)kMgStages &&
                        !ptx::mbar_wait(&bars->empty[s], ((it / kMgStages) - 1) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(&bars->full[s], kMgABytes);
                    ptx::tma_load_2d(smem_base + s * kMgStageBytes, &tmapP, &bars->full[s], kb * kMgBK,
                                     out0 + i0);
                }
            }
        }
    } else if (warp == 9) {
        // ---------------- UMMA issuer -----------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_bf16(kMgTileM, kMgTileN, false, true);
            uint32_t it = 0;
            for (int ct = 0; ct < nct && !bars->abort_flag; ++ct) {
                const int buf = ct & 1;
                if (ct >= 2) {
                    if (!ptx::mbar_wait(&bars->accum_empty[buf], ((ct >> 1) - 1) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::tc_fence_after();
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kMgTileN);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kMgStages;
                    if (!ptx::mbar_wait(&bars->full[s], (it / kMgStages) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a_base = smem_base + s * kMgStageBytes;
                    const uint32_t b_base = a_base + kMgABytes;
#pragma unroll
                    for (int k = 0; k < kMgBK / 16; ++k) {
                        // A: K-major, 32 bytes further along the 128-byte row per 16 k.
                        // B: MN-major, 16 k-rows = 2 groups of 8 rows = 2048 bytes further; 64-column
                        //    slabs are kMgBK * 128 bytes apart, 8-row groups 1024 bytes apart.
                        const uint64_t da = ptx::smem_desc_sw128(a_base + k * 32, 16, 1024);
                        const uint64_t db = ptx::smem_desc_sw128(b_base + k * 2048, kMgBK * 128, 1024);
                        ptx::umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0);
                    }
                    ptx::umma_commit(&bars->empty[s]);
                }
                ptx::umma_commit(&bars->accum_full[buf]);
            }
        }
    } else if (warp >= 4) {
        // ---------------- warps 4-7: gather the pruned tokens' rows -----------------------------
        const int lt = tid - 128;             // 0..127
        const int cch = lt & 31;              // 16-byte chunk within the 512-byte row segment
        const int rbase = lt >> 5;            // rows rbase + 4 q
        uint32_t it = 0;
        bool failed = false;
        for (int ct = 0; ct < nct && !failed; ++ct) {
            const int col = ct * kMgTileN + cch * 8;
            const int slab = cch >> 3, cc = cch & 7;
            const uint32_t it0 = it;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % kMgStages;
                if (it >= (uint32_t)kMgStages &&
                    !ptx::mbar_wait(&bars->empty[s], ((it / kMgStages) - 1) & 1)) {
                    failed = true;
                    break;
                }
                const uint32_t b_base = smem_base + s * kMgStageBytes + kMgABytes + slab * (kMgBK * 128);
#pragma unroll 4
                for (int q = 0; q < kMgBK / 4; ++q) {
                    const int r = rbase + 4 * q;
                    const int j = kb * kMgBK + r;
                    const bool ok = j < B && col < d;
                    const __nv_bfloat16 *src = ok ? X + (size_t)(t_begin + ord[M + j]) * d + col : X;
                    const uint32_t dst = b_base + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
                    ptx::cp_async_16(dst, src, ok ? 16u : 0u);
                }
                ptx::cp_async_commit();
                if (kb >= 1) {
                    ptx::cp_async_wait<1>();
                    ptx::fence_proxy_async_smem();
                    ptx::mbar_arrive(&bars->full[(it - 1) % kMgStages]);
                }
            }
            ptx::cp_async_wait<0>();
            if (!failed && it > it0) {
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(&bars->full[(it - 1) % kMgStages]);
            }
        }
        if (failed) {
            bars->abort_flag = 1;
            atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
        }
    } else {
        // ---------------- warps 0-3: epilogue ---------------------------------------------------
        const int row = tid;                                  // TMEM lane = tile row
        const bool valid = i0 + row < M;
        const int tok = valid ? ord[i0 + row] : 0;
        if (valid) kept_idx[out0 + i0 + row] = tok;
        const __nv_bfloat16 *xrow = X + (size_t)(t_begin + tok) * d;
        __nv_bfloat16 *yrow = Y + (size_t)(out0 + i0 + row) * d;
        for (int ct = 0; ct < nct; ++ct) {
            const int buf = ct & 1;
            bool ok = !bars->abort_flag && ptx::mbar_wait(&bars->accum_full[buf], (ct >> 1) & 1);
            if (!__all_sync(0xffffffffu, ok)) {      // warp-uniform: the TMEM loads are collective
                bars->abort_flag = 1;
                if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                break;
            }
            ptx::tc_fence_after();
            const int ncols = min(kMgTileN, d - ct * kMgTileN);
            for (int c0 = 0; c0 < ncols; c0 += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * kMgTileN + c0), r);
                ptx::tmem_ld_wait();
                if (valid) {
                    const int col = ct * kMgTileN + c0;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (col + 8 * g < d) {
                            float xf[8];
                            Elem<__nv_bfloat16>::unpack(ldg_vec(xrow + col + 8 * g), xf);
                            __nv_bfloat162 o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float y0 = fmaf(alpha, __uint_as_float(r[8 * g + 2 * e]), xf[2 * e]);
                                const float y1 = fmaf(alpha, __uint_as_float(r[8 * g + 2 * e + 1]), xf[2 * e + 1]);
                                o[e] = __floats2bfloat162_rn(y0, y1);
                            }
                            *reinterpret_cast<uint4 *>(yrow + col + 8 * g) = *reinterpret_cast<uint4 *>(o);
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&bars->accum_empty[buf]);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace rtp
