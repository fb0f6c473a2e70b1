// Shared device helpers and the workspace layout of the RTPrune kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rtprune.h"

namespace rtp {

constexpr int kChunkTokens = 32;       // tokens per CTA of the norm/statistics pass
constexpr float kNormFloor = 1e-12f;   // divisor floor for a zero-norm token
constexpr int kStats = RTPRUNE_STATS_STRIDE;

// Workspace header (first 256 bytes of the workspace).
struct WsHeader {
    uint32_t status;       // RTPRUNE_DEV_* bits
    uint32_t select_done;  // images whose selection has been published
    uint32_t n_ready;      // images whose transport plan has been published (entries of ready_list)
    uint32_t merge_next;   // next unit of the merge kernel when its CTAs draw units from a counter
    int32_t run_tag;       // number of the run whose counters and lists below are in place
    int32_t launch_seq;    // number of the run in flight on this workspace: stage 1 counts it up on the device, so a
                           // run captured into a CUDA graph gets a new number at every replay
    uint32_t pad[58];
};

// Byte offsets of the workspace regions; computed on the host from the plan's maxima.
struct WsLayout {
    size_t header;     // WsHeader
    size_t img_done;   // uint32 [batch]           chunks of each image that have finished their pass
    size_t sink_done;  // uint32 [batch]           CTAs of each image's cluster that have written their plan rows
    size_t ready_list; // int32 [batch]            1 + image, in the order the plans were finished
    size_t scores_done; // uint32 [batch]          score tiles of each image that are complete
    size_t clear_bytes;  // the workspace's first clear_bytes bytes (header, counters) start at zero
    size_t norms;      // float [total]            l2 norms (the criterion C_k of Eq. 1)
    size_t crit;       // float [total]            C_k of a run that ranks by variance or entropy
    size_t spart;      // float [batch][chunks][d] partial sums of the unit tokens
    size_t order;      // int32 [total]            per image: kept indices then pruned indices
    size_t kpos;       // int32 [total]            per token: position among kept, or -1 - position
                       //                          among pruned
    size_t kmat;       // float [kmat_floats]      per-image score / kernel / plan matrix
    size_t xp;         // bf16 [total + 64 batch][d] compact copy of the pruned tokens (bf16 mode): image
                       //                          i's B rows start at row xp_row0(offsets[i], i), followed
                       //                          by zero rows up to a multiple of 64
    size_t pbuf;       // bf16 [total][pbuf_pitch] plan rows for the tensor-core merge (bf16 mode)
    int pbuf_pitch_max;  // elements; a run uses round_up(its largest possible B, 64) <= this
    size_t total;      // bytes
    int chunks;        // chunks per image = ceil(max_tokens_per_image / kChunkTokens)
    int kmat_stride;   // floats of kmat per token-unit, see kmat_offset()
};

// Row pitch (floats) of an image's score / plan matrix: B real columns + the dustbin column,
// rounded up to a multiple of 4 so that rows can be written as 16-byte vectors.
__host__ __device__ inline int score_pitch(int B) { return (B + 4) & ~3; }

// Image i's matrix starts at float offset kmat_stride * (offsets[i] + 8 i), a multiple of 4.  Its
// (M+1) rows of score_pitch(B) floats always fit: (M+1)(B+4) <= (N+5)^2 / 4 <= kmat_stride * (N+8),
// kmat_stride being 4 * ceil((maxN+8)/16).
__host__ __device__ inline size_t kmat_offset(int kmat_stride, int tok_offset, int img)
{
    return (size_t)kmat_stride * (size_t)(tok_offset + 8 * img);
}

// First row of image `img`'s segment in the compact copy of pruned tokens.  Each image owns
// N + 64 rows there, enough for its B <= N - 1 rows rounded up to a multiple of 64.
__host__ __device__ inline int xp_row0(int tok_offset, int img) { return tok_offset + 64 * img; }

// Reads image `img`'s token range and checks it against the contract (1 <= N <= max_tokens, rows
// inside [0, total)).  Kernels skip an image that fails; the selection kernel reports it.
__device__ inline bool image_range(const int32_t *offsets, int img, int max_tokens, int total,
                                   int &t_begin, int &N)
{
    t_begin = offsets[img];
    const int t_end = offsets[img + 1];
    N = t_end - t_begin;
    return N >= 1 && N <= max_tokens && t_begin >= 0 && t_end <= total;
}

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;  // elements per 16-byte vector
    __device__ static inline void unpack(const uint4 &v, float (&f)[8])
    {
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __bfloat1622float2(h[i]);
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
    __device__ static inline float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static inline __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static inline void unpack(const uint4 &v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    __device__ static inline float to_float(float x) { return x; }
    __device__ static inline float from_float(float x) { return x; }
};

__device__ inline uint4 ldg_vec(const void *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }

__device__ inline float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ inline float warp_max(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// Sum over a CTA; `red` is shared scratch of at least 32 floats; every thread gets the result.
__device__ inline float block_sum(float x, float *red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    x = warp_sum(x);
    __syncthreads();
    if (lane == 0) red[warp] = x;
    __syncthreads();
    float t = (lane < nwarps) ? red[lane] : 0.f;
    return warp_sum(t);
}

}  // namespace rtp
