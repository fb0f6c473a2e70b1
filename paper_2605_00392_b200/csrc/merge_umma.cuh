// Merge + pack (Eq. 7 and the output of Algorithm 1): Y = T_k + alpha * P T_p, written packed, on the
// tcgen05 tensor cores (bf16 inputs, fp32 accumulation in TMEM), every operand fetched by tiled TMA.
//
// A work unit is (image, tile of 128 CONSECUTIVE tokens, tile of 256 output columns).  The kept
// token's own row enters through the tensor cores too: the contraction of a unit is
//     D = [ I_128 | alpha P_tok ] . [ T_v rows of the token tile ; T_p ]
// so the accumulator already holds T_k + alpha P T_p (1.0 x bf16 is exact in the fp32 accumulator) and
// the epilogue reads no global memory.  Rows of pruned tokens are computed and dropped.
//   * A operand: two constant identity tiles (built once in shared memory), then the plan rows
//     alpha P[token][0..B) in bf16, K-major, from the plan buffer whose rows are token positions.
//   * B operand, MN-major (row = contraction index, 64-column slabs of 128 bytes, 128-byte swizzle):
//     the token tile's rows of X (k-blocks 0, 1), then the image's pruned rows from the compact copy,
//     whose zero rows pad B to a multiple of 64.
//   * D: two 128-lane x 256-column fp32 accumulators in TMEM, so that the epilogue of one unit
//     overlaps the loads and UMMAs of the next.
// The kernel is persistent: CTA c takes units c, c + gridDim.x, ...  When the Sinkhorn kernel ahead
// publishes a list of finished images, the units follow that list (its s-th entry takes the place of
// image s), the CTAs draw them from a counter, and the scheduler waits, bounded, for the entry it
// needs: the kernel is launched as a programmatic dependent and merges the first images on whatever
// SMs are free while the last ones still iterate.  Warp roles (224 threads):
// warps 0-3 epilogue (TMEM -> registers -> bf16 -> own row of a padded staging tile -> one bulk store
// per kept row); warp 4 issues the TMA loads (the loads of a k-block from several lanes at once); warp 5 owns TMEM and
// its lane 0 issues the UMMAs;
// warp 6 lane 0 is the scheduler: it draws the units, looks up what the other roles need to know about
// them (a chain of dependent loads from L2) a few units ahead and hands them over through a small queue
// in shared memory.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace rtp {

constexpr int kMgTileM = 128;
constexpr int kMgTileN = 256;        // output columns per unit
constexpr int kMgBK = 64;            // contraction rows per k-block
constexpr int kMgBStages = 3;        // ring of B tiles (every k-block)
constexpr int kMgAStages = 2;        // ring of plan tiles (k-blocks after the identity ones)
constexpr int kMgThreads = 224;
constexpr int kMgLookahead = 1;       // units the scheduler may be ahead of the producer
constexpr int kMgABytes = kMgTileM * 128;            // A tile: 128 rows x 64 bf16
constexpr int kMgBBytes = kMgBK * kMgTileN * 2;      // B tile: 64 rows x 256 bf16 = 32 KB
constexpr int kMgBBoxBytes = kMgBK * 128;            // one 64-column slab of it
// I_128 as two 128 x 64 K-major views of [64 zero rows][I_64][64 zero rows]: the view that starts at
// the I_64 block has its ones in rows 0-63, the view that starts 64 rows earlier in rows 64-127.
constexpr int kMgIdentBytes = 3 * (kMgABytes / 2);
constexpr int kMgIdentKb = 2;                        // k-blocks that carry the token tile's own rows (one, if
                                                     // the image ends within the tile's first 64 rows)
constexpr int kMgStagePitch = kMgTileN * 2 + 16;     // bytes per staging row: padded, conflict-free
constexpr int kMgStagingBytes = kMgTileM * kMgStagePitch;
constexpr int kMgSmemBytes = kMgBStages * kMgBBytes + kMgAStages * kMgABytes + kMgIdentBytes +
                             kMgStagingBytes + 1024 /*alignment*/ + 1024 /*barriers, unit queue*/;

constexpr int kMgQueue = 16;         // ring of units between the producer and the other roles (about 6 in flight)

struct MergeBarriers {
    uint64_t full[kMgBStages];       // B tile (and, for plan k-blocks, the A tile) of a k-block has landed
    uint64_t empty[kMgBStages];      // the k-block's UMMAs have read them
    uint64_t accum_full[2];
    uint64_t accum_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

// What every role needs to know about a unit.  img = -1 ends the queue.
struct MergeUnit {
    int img, mt, ct;
    int t_begin, N, M, B, out0;
    int nident;       // identity k-blocks: 64-row blocks of the tile that hold tokens of the image
    bool valid;
    bool timed_out;   // the image's list entry never came
};

struct MergeQueue {
    volatile uint32_t head;          // units pushed by the scheduler
    volatile uint32_t prod;          // units the producer has taken
    volatile uint32_t tail;          // units every role is done with
    MergeUnit e[kMgQueue];
};

// Bounded wait for the n-th unit of the queue.  false = gave up, or the kernel is being abandoned.
__device__ inline bool merge_pop(MergeQueue *mq, const MergeBarriers *bars, uint32_t n, MergeUnit &q)
{
    for (uint32_t i = 0; i < ptx::kSpinLimit && !bars->abort_flag; ++i) {
        if (mq->head > n) {
            __threadfence_block();
            q = mq->e[n % kMgQueue];
            return true;
        }
        __nanosleep(40);
    }
    return false;
}

// Image in slot `slot` of the list of finished plans (bounded wait), -1 if it never shows up.
__device__ inline int merge_wait_image(const int32_t *ready_list, int slot)
{
    for (uint32_t i = 0; i < ptx::kSpinLimit; ++i) {
        const int v = ptx::ld_acquire_gpu(ready_list + slot);
        if (v != 0) return v - 1;
        __nanosleep(200);
    }
    return -1;
}

__device__ inline MergeUnit merge_unit(int u, int mtiles, int nct, const int32_t *__restrict__ offsets,
                                       const int32_t *__restrict__ counts,
                                       const int32_t *__restrict__ out_offsets, int max_tokens, int total,
                                       const int32_t *ready_list)
{
    MergeUnit q;
    q.ct = u % nct;
    const int v = u / nct;
    q.mt = v % mtiles;
    q.img = v / mtiles;
    q.timed_out = false;
    if (ready_list) {
        q.img = merge_wait_image(ready_list, q.img);
        if (q.img < 0) {
            q.valid = false;
            q.timed_out = true;
            return q;
        }
    }
    // L2 loads (with a ready list this kernel may have started before the selection wrote these), all issued
    // before the first use: one trip, not one per value (img is a valid image number either way)
    const int o_lo = __ldcg(offsets + q.img), o_hi = __ldcg(offsets + q.img + 1);
    const int m_img = __ldcg(counts + q.img), out0 = __ldcg(out_offsets + q.img);
    q.t_begin = o_lo;
    q.N = o_hi - o_lo;
    q.valid = q.N >= 1 && q.N <= max_tokens && o_lo >= 0 && o_hi <= total && q.mt * kMgTileM < q.N;
    q.M = q.valid ? m_img : 0;
    q.B = q.N - q.M;
    q.out0 = q.valid ? out0 : 0;
    q.nident = (q.N - q.mt * kMgTileM <= kMgBK) ? 1 : kMgIdentKb;
    return q;
}

__global__ void __launch_bounds__(kMgThreads, 1)
merge_umma_kernel(const __grid_constant__ CUtensorMap tmapX, const __grid_constant__ CUtensorMap tmapXp,
                  const __grid_constant__ CUtensorMap tmapP, const int32_t *__restrict__ offsets, int d,
                  int batch, int mtiles, const int32_t *__restrict__ counts,
                  const int32_t *__restrict__ out_offsets, const int32_t *__restrict__ kpos,
                  int max_tokens, int total, __nv_bfloat16 *__restrict__ Y, int32_t *__restrict__ kept_idx,
                  WsHeader *__restrict__ hdr, const int32_t *ready_list)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_ring = smem + kMgBStages * kMgBBytes;
    uint8_t *ident = a_ring + kMgAStages * kMgABytes;
    uint8_t *staging = ident + kMgIdentBytes;
    MergeBarriers *bars = reinterpret_cast<MergeBarriers *>(staging + kMgStagingBytes);
    MergeQueue *mq = reinterpret_cast<MergeQueue *>(staging + kMgStagingBytes + 256);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nct = (d + kMgTileN - 1) / kMgTileN;
    const int nunits = batch * mtiles * nct;

    // identity block: rows 64 .. 127 of the 192-row region hold I_64 (ones at (64 + r, k = r)), in the
    // swizzled K-major layout; the other rows are zero
    for (int v = tid; v < kMgIdentBytes / 16; v += kMgThreads)
        reinterpret_cast<uint4 *>(ident)[v] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    if (tid < 64) {
        const int r = 64 + tid, k = tid;
        const uint32_t off = (r >> 3) * 1024 + (r & 7) * 128 + (((k >> 3) ^ (r & 7)) << 4) + (k & 7) * 2;
        *reinterpret_cast<uint16_t *>(ident + off) = 0x3F80;   // bf16 1.0
    }
    ptx::fence_proxy_async_smem();
    if (tid == 0) {
        for (int s = 0; s < kMgBStages; ++s) {
            ptx::mbar_init(&bars->full[s], 1);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&bars->accum_full[b], 1);
            ptx::mbar_init(&bars->accum_empty[b], 128);
        }
        bars->abort_flag = 0;
        mq->head = 0;
        mq->prod = 0;
        mq->tail = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 5) {
        ptx::tmem_alloc(&bars->tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t smem_base = ptx::smem_u32(smem);
    // everything above is local set-up; the plan, the selection and the compact copy come from the
    // kernels ahead in the stream: wait for them to end, or, with a list of finished images, for each
    // image's entry (which is published after everything the image needs has been written)
    ptx::grid_dep_launch();
    if (!ready_list) ptx::grid_dep_wait();

    if (warp == 4) {
        // ---------------- producer: tiled TMA for every operand -------------------------------------
        // The whole warp walks the units and k-blocks in step (every lane takes the same waits); the loads of a
        // k-block are issued by as many lanes at once, one load each (lanes 0-3: the 64-column slabs of the B
        // tile, lane 4: the plan tile): one thread issuing them one after the other spent about 145 cycles in
        // each issue, 40 % of the kernel's time.
        {
            if (lane == 0) {
                ptx::prefetch_tensormap(&tmapX);
                ptx::prefetch_tensormap(&tmapXp);
                ptx::prefetch_tensormap(&tmapP);
            }
            // `it` counts k-blocks (B ring), `ia` plan k-blocks (A ring).  a_user[slot] is the k-block that
            // last read the A slot: its UMMAs must have finished before the slot is refilled.
            uint32_t it = 0, ia = 0;
            uint32_t a_user[kMgAStages];
            for (int s = 0; s < kMgAStages; ++s) a_user[s] = 0xffffffffu;
            bool alive = true;
            for (uint32_t n = 0; alive && !bars->abort_flag; ++n) {
                MergeUnit q;
                const bool got = merge_pop(mq, bars, n, q);
                if (!__all_sync(0xffffffffu, got)) {
                    bars->abort_flag = 1;
                    if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                    break;
                }
                if (q.img < 0) break;
                __syncwarp();                         // every lane has read the entry before it may be reused
                if (lane == 0) mq->prod = n + 1;
                if (ready_list) ptx::fence_proxy_async_all();   // the plan was written with ordinary stores
                const int nkb = q.nident + (q.B + kMgBK - 1) / kMgBK;
                const int row0 = q.t_begin + q.mt * kMgTileM;
                const int xp0 = xp_row0(q.t_begin, q.img);
                const int col0 = q.ct * kMgTileN;
                const int nslab = min(kMgTileN, d - col0 + 63) / 64;   // 64-column slabs with any column < d
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kMgBStages;
                    bool ok = it < (uint32_t)kMgBStages || ptx::mbar_wait(&bars->empty[s], ((it / kMgBStages) - 1) & 1);
                    const uint32_t b_dst = smem_base + s * kMgBBytes;
                    const bool own = kb < q.nident;         // the token tile's own rows: A is the identity
                    int sa = 0;
                    if (!own) {
                        sa = ia % kMgAStages;
                        const uint32_t prev = a_user[sa];
                        // k-blocks up to it - kMgBStages are known to be done (the wait above); a younger
                        // reader of this A slot is the latest user of its B slot: wait for that phase
                        if (ok && prev != 0xffffffffu && prev + kMgBStages > it)
                            ok = ptx::mbar_wait(&bars->empty[prev % kMgBStages], (prev / kMgBStages) & 1);
                        a_user[sa] = it;
                        ++ia;
                    }
                    if (!__all_sync(0xffffffffu, ok)) {
                        bars->abort_flag = 1;
                        if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        alive = false;
                        break;
                    }
                    if (lane == 0)
                        ptx::mbar_arrive_expect_tx(&bars->full[s], (own ? 0 : kMgABytes) + nslab * kMgBBoxBytes);
                    __syncwarp();
                    if (lane < nslab) {
                        const CUtensorMap *bm = own ? &tmapX : &tmapXp;
                        const int brow = own ? row0 + kb * kMgBK : xp0 + (kb - q.nident) * kMgBK;
                        ptx::tma_load_2d(b_dst + lane * kMgBBoxBytes, bm, &bars->full[s], col0 + lane * 64, brow);
                    } else if (lane == 4 && !own) {
                        ptx::tma_load_2d(ptx::smem_u32(a_ring) + sa * kMgABytes, &tmapP, &bars->full[s],
                                         (kb - q.nident) * kMgBK, row0);
                    }
                }
            }
        }
    } else if (warp == 6) {
        // ---------------- scheduler -------------------------------------------------------------------
        if (lane == 0) {
            uint32_t pushed = 0, drawn = 0;
            auto push = [&](const MergeUnit &q) {
                // stay a few units ahead of the producer, no more: a unit drawn is a unit no other CTA
                // can take.  (The queue itself cannot fill up: fewer units are in flight than it holds.)
                for (uint32_t i = 0; pushed - mq->prod >= (uint32_t)kMgLookahead ||
                                     pushed - mq->tail >= (uint32_t)kMgQueue; ++i) {
                    if (i >= ptx::kSpinLimit || bars->abort_flag) return false;
                    __nanosleep(100);
                }
                mq->e[pushed % kMgQueue] = q;
                __threadfence_block();
                mq->head = ++pushed;
                return true;
            };
            // with a list of finished images: not before the run's number is there (until then the list
            // and the unit counter are what the run before left)
            bool ok = !ready_list || ptx::wait_equal_gpu(&hdr->run_tag, ptx::ld_acquire_gpu(&hdr->launch_seq));
            while (ok && !bars->abort_flag) {
                // next unit: from the shared counter when the units follow the list of finished images
                const int u = ready_list ? (int)atomicAdd(&hdr->merge_next, 1u)
                                         : (int)(blockIdx.x + drawn++ * gridDim.x);
                if (u >= nunits) break;
                const MergeUnit q = merge_unit(u, mtiles, nct, offsets, counts, out_offsets, max_tokens, total,
                                               ready_list);
                if (q.timed_out) ok = false;
                else if (q.valid) ok = push(q);
            }
            MergeUnit end{};
            end.img = -1;
            if (ok) ok = push(end);
            if (!ok && !bars->abort_flag) {
                bars->abort_flag = 1;
                atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
            }
        }
    } else if (warp == 5) {
        // ---------------- UMMA issuer -----------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_bf16(kMgTileM, kMgTileN, false, true);
            uint32_t it = 0, ia = 0, acc = 0;
            for (uint32_t n = 0; !bars->abort_flag; ++n) {
                MergeUnit q;
                if (!merge_pop(mq, bars, n, q)) {
                    bars->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                    break;
                }
                if (q.img < 0) break;
                const int nkb = q.nident + (q.B + kMgBK - 1) / kMgBK;
                const int buf = acc & 1;
                if (acc >= 2) {
                    if (!ptx::mbar_wait(&bars->accum_empty[buf], ((acc >> 1) - 1) & 1)) {
                        bars->abort_flag = 1;
                        atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                        break;
                    }
                    ptx::tc_fence_after();
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kMgTileN);
                bool failed = false;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kMgBStages;
                    if (!ptx::mbar_wait(&bars->full[s], (it / kMgBStages) & 1)) {
                        failed = true;
                        break;
                    }
                    ptx::tc_fence_after();
                    // identity k-block 0: the view whose rows 0-63 are I_64; k-block 1: rows 64-127
                    uint32_t a_base;
                    if (kb < q.nident) {
                        a_base = ptx::smem_u32(ident) + (1 - kb) * (kMgABytes / 2);
                    } else {
                        a_base = ptx::smem_u32(a_ring) + (ia % kMgAStages) * kMgABytes;
                        ++ia;
                    }
                    const uint32_t b_base = smem_base + s * kMgBBytes;
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
                if (failed) {
                    bars->abort_flag = 1;
                    atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                    break;
                }
                ptx::umma_commit(&bars->accum_full[buf]);
                ++acc;
            }
        }
    } else {
        // ---------------- warps 0-3: epilogue ---------------------------------------------------------
        const int row = tid;                                  // TMEM lane = row of the token tile
        uint8_t *srow = staging + row * kMgStagePitch;        // this thread's staging row, nobody else's
        const uint32_t srow_u32 = ptx::smem_u32(srow);
        uint32_t acc = 0;
        for (uint32_t n = 0;; ++n) {
            MergeUnit q;
            const bool got = merge_pop(mq, bars, n, q);
            if (!__all_sync(0xffffffffu, got)) {
                bars->abort_flag = 1;
                if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                break;
            }
            if (q.img < 0) break;
            const int tok = q.mt * kMgTileM + row;            // image-local token of this row
            const int p = (tok < q.N) ? __ldcg(kpos + q.t_begin + tok) : -1;   // >= 0: position among kept
            const int buf = acc & 1;
            // the TMEM loads below are warp-collective: take the go / no-go decision per warp
            bool ok = !bars->abort_flag && ptx::mbar_wait(&bars->accum_full[buf], (acc >> 1) & 1);
            if (!__all_sync(0xffffffffu, ok)) {
                bars->abort_flag = 1;
                if (lane == 0) atomicOr(&hdr->status, RTPRUNE_DEV_TIMEOUT);
                break;
            }
            ptx::tc_fence_after();
            // unit n's accumulator is complete, so every epilogue thread is done with unit n - 2 (its
            // accumulator buffer was handed back) and the UMMA issuer is past it: those entries are free
            if (tid == 0 && n >= 1) mq->tail = n - 1;
            ptx::bulk_wait_read<0>();                         // the previous unit's store has read this row
            const int col0 = q.ct * kMgTileN;
            const int ncols = min(kMgTileN, d - col0);
            // a warp whose 32 rows all lie past the image's end has nothing to convert or store
            const bool warp_has_rows = q.mt * kMgTileM + warp * 32 < q.N;
            for (int c0 = 0; c0 < (warp_has_rows ? ncols : 0); c0 += 32) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * kMgTileN + c0), r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    __nv_bfloat162 o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        o[e] = __floats2bfloat162_rn(__uint_as_float(r[8 * g + 2 * e]),
                                                     __uint_as_float(r[8 * g + 2 * e + 1]));
                    *reinterpret_cast<uint4 *>(srow + (c0 + 8 * g) * 2) = *reinterpret_cast<uint4 *>(o);
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&bars->accum_empty[buf]);
            ++acc;
            if (p >= 0) {
                ptx::fence_proxy_async_smem();
                ptx::bulk_store(Y + (size_t)(q.out0 + p) * d + col0, srow_u32, (uint32_t)ncols * 2u);
                if (q.ct == 0) kept_idx[q.out0 + p] = tok;
            }
            ptx::bulk_commit();
        }
        ptx::bulk_wait<0>();                                  // stores complete before the CTA retires
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
    // keep the stream's order: this grid does not end before the ones ahead of it have
    if (ready_list) ptx::grid_dep_wait();
}

}  // namespace rtp
