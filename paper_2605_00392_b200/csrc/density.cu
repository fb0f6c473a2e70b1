// Textual density rho of page images (Eq. 9; Appendix B): BT.601 grayscale, 3 x 3 Sobel gradient
// magnitude, threshold tau, fraction of edge pixels per token patch, mean over the patches.
//
// The arithmetic is exact.  With 8-bit channels, 1000 * 255 * I = 299 R + 587 G + 114 B is an integer
// below 2^18, the Sobel sums are integers below 2^21 in magnitude, and
//     G >= tau   <=>   Gx_int^2 + Gy_int^2 >= (255000 tau)^2,
// a comparison of a 64-bit integer with a constant the host rounds up once.  Every pixel's decision is
// therefore the one exact arithmetic takes, and the counts do not depend on the order of anything.
// Pixels outside the image take the value of the nearest pixel inside.
//
// One CTA of 288 threads per 64 x 64 tile of pixels (one token patch of 64 x 64, or 4 / 16 patches of
// 32 x 32 / 16 x 16):
//   1. a tile row is up to 192 contiguous bytes, 16-byte aligned (the image width is a multiple of
//      16): a thread fetches 48 bytes = 16 pixels with three 16-byte loads, and the one-pixel ring left
//      and right of the tile pixel by pixel; every load of the CTA is issued before the first use (one
//      trip to memory); the pixels become integer gray values in a 66-row tile in shared memory.  The
//      gray value of a pixel is two dp2a instructions on the words as loaded (16-bit weights against
//      the bytes of a word, whichever of the four alignments the 3-byte pixel has), no byte is
//      extracted;
//   2. 256 threads each walk down 8 rows of two adjacent columns with the horizontal sums of three
//      rows in registers: 1.5 shared-memory loads and about a dozen integer operations per pixel; the
//      rows and columns of a thread lie in one patch, so the counts are reduced over the lanes that
//      share a patch and added to the patch's counter in shared memory.
// The kernel is bound by instruction issue, not by memory, which is why the instruction count per
// pixel is what the layout above is about.
// The CTA writes its patches' counts and adds their sum to the image's count (integer atomics: the
// result does not depend on the order); a second small kernel turns the image counts into rho.
#include <cstdint>
#include <algorithm>
#include <cmath>

#include <cuda_runtime.h>

#include "../../include/rtprune.h"

namespace rtp {

constexpr int kDnTile = 64;                        // tile side in pixels
constexpr int kDnThreads = 288;                    // 66 rows x 4 groups of 16 pixels = 264 fetch tasks
constexpr int kDnRows = 8;                         // rows a thread of the Sobel walk covers (8 warps x 8 rows)
constexpr int kDnPitch = 72;                       // gray tile row: ring at [3], pixels at [4 .. 67], ring at [68]

__device__ inline int gray_of(uint32_t r, uint32_t g, uint32_t b) { return (int)(299u * r + 587u * g + 114u * b); }

// 16-bit weight pairs (low half | high half << 16) for dp2a: low half times the lower byte of the
// selected byte pair of the data word, high half times the upper one.
constexpr uint32_t kW_RG = 299u | (587u << 16);
constexpr uint32_t kW_B0 = 114u;
constexpr uint32_t kW_0R = 299u << 16;
constexpr uint32_t kW_GB = 587u | (114u << 16);

// Gray values of the 4 pixels whose 12 bytes are the words a, b, c (R G B R | G B R G | B R G B).
__device__ inline int4 gray4(uint32_t a, uint32_t b, uint32_t c)
{
    int4 o;
    o.x = (int)__dp2a_lo(kW_RG, a, __dp2a_hi(kW_B0, a, 0u));     // R, G = a[0], a[1]; B = a[2]
    o.y = (int)__dp2a_hi(kW_0R, a, __dp2a_lo(kW_GB, b, 0u));     // R = a[3]; G, B = b[0], b[1]
    o.z = (int)__dp2a_hi(kW_RG, b, __dp2a_lo(kW_B0, c, 0u));     // R, G = b[2], b[3]; B = c[0]
    o.w = (int)__dp2a_lo(kW_0R, c, __dp2a_hi(kW_GB, c, 0u));     // R = c[1]; G, B = c[2], c[3]
    return o;
}

// What a thread fetches for one tile: 16 pixels of a tile row (12 words) and, for the first 132
// threads, the word that holds one pixel of the ring left or right of the tile.
struct DnFetch {
    uint32_t w[12];
    uint32_t ring;
};

// A tile: image, origin, extent (the last tile of a row or column may be narrower).
struct DnTile {
    int img, x0, y0, tw, th;
};

// Issues the loads of a tile.  Task = (tile row ty = tid / 4, group of 16 pixels gx = tid % 4); the ring
// pixel of a row is the upper three bytes of the word that ends where the tile starts, or the lower
// three of the word that starts where it ends (3 x0 and 3 (x0 + tw) are multiples of 4); at the
// image's left and right border the nearest pixel inside sits at the other end of its word.
__device__ inline void dn_fetch(const uint8_t *__restrict__ images, int H, int W, const DnTile &q, int tid, DnFetch &f)
{
    const uint8_t *im = images + (size_t)q.img * H * W * 3;
    const int ty = tid >> 2, gx = tid & 3;
    if (ty < q.th + 2 && 16 * gx < q.tw) {
        const int y = min(max(q.y0 + ty - 1, 0), H - 1);
        const uint4 *src = reinterpret_cast<const uint4 *>(im + ((size_t)y * W + q.x0 + 16 * gx) * 3);
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const uint4 v = __ldg(src + k);
            f.w[4 * k] = v.x;
            f.w[4 * k + 1] = v.y;
            f.w[4 * k + 2] = v.z;
            f.w[4 * k + 3] = v.w;
        }
    }
    if (tid < 2 * (q.th + 2)) {
        const int ry = tid >> 1, right = tid & 1;
        const int y = min(max(q.y0 + ry - 1, 0), H - 1);
        const uint8_t *row = im + (size_t)y * W * 3;
        int off;                                     // byte offset of the word within the row
        if (right) off = (q.x0 + q.tw < W) ? 3 * (q.x0 + q.tw) : 3 * W - 4;
        else off = (q.x0 > 0) ? 3 * q.x0 - 4 : 0;
        f.ring = __ldg(reinterpret_cast<const uint32_t *>(row + off));
    }
}

// Gray values of what dn_fetch loaded, into the tile in shared memory.
__device__ inline void dn_store(int *s_gray, int W, const DnTile &q, int tid, const DnFetch &f)
{
    const int ty = tid >> 2, gx = tid & 3;
    if (ty < q.th + 2 && 16 * gx < q.tw) {
        int4 *dst = reinterpret_cast<int4 *>(s_gray + ty * kDnPitch + 4 + 16 * gx);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) dst[k4] = gray4(f.w[3 * k4], f.w[3 * k4 + 1], f.w[3 * k4 + 2]);
    }
    if (tid < 2 * (q.th + 2)) {
        const int right = tid & 1;
        // pixel in bytes 0-2 of the word: right ring inside the image, or left ring clamped to pixel 0
        const bool low = right ? (q.x0 + q.tw < W) : (q.x0 == 0);
        const uint32_t v = f.ring;
        const int g = low ? (int)__dp2a_lo(kW_RG, v, __dp2a_hi(kW_B0, v, 0u))
                          : (int)__dp2a_lo(kW_0R, v, __dp2a_hi(kW_GB, v, 0u));
        s_gray[(tid >> 1) * kDnPitch + (right ? 4 + q.tw : 3)] = g;
    }
}

// One CTA per tile.  grid = (tiles across, tiles down, batch).
__global__ void __launch_bounds__(kDnThreads, 7)
density_tile_kernel(const uint8_t *__restrict__ images, int H, int W, int p, unsigned long long thr2,
                    int32_t *__restrict__ edge_counts, uint32_t *__restrict__ image_counts)
{
    __shared__ __align__(16) int s_gray[(kDnTile + 2) * kDnPitch];
    __shared__ int s_cnt[16];                        // up to 4 x 4 patches in a tile
    const int tid = threadIdx.x;
    DnTile q;
    q.img = blockIdx.z;
    q.x0 = blockIdx.x * kDnTile;
    q.y0 = blockIdx.y * kDnTile;
    q.tw = min(kDnTile, W - q.x0);                   // multiples of the patch (and of 16)
    q.th = min(kDnTile, H - q.y0);
    const int npt = kDnTile / p;                     // patches per tile side
    DnFetch f;
    dn_fetch(images, H, W, q, tid, f);
    if (tid < 16) s_cnt[tid] = 0;
    dn_store(s_gray, W, q, tid, f);
    __syncthreads();

    // ---- Sobel, threshold, count: thread = (columns 2 cp and 2 cp + 1, block of kDnRows rows) ----------
    const int cp = tid & 31, r0 = (tid >> 5) * kDnRows;
    const bool active = tid < 256 && 2 * cp < q.tw && r0 < q.th;
    int cnt = 0;
    if (active) {
        // horizontal sums of a tile row at the two columns: smooth s = l + 2 m + r, difference d = r - l
        auto hrow = [&](int trow, int &s0, int &d0, int &s1, int &d1) {
            const int *g = s_gray + trow * kDnPitch + 3 + 2 * cp;    // image columns x-1 .. x+2, x = 2 cp
            const int g0 = g[0];
            const int2 g12 = *reinterpret_cast<const int2 *>(g + 1);
            const int g3 = g[3];
            s0 = g0 + 2 * g12.x + g12.y;
            d0 = g12.y - g0;
            s1 = g12.x + 2 * g12.y + g3;
            d1 = g3 - g12.x;
        };
        auto edge = [&](int gx, int gy) {
            const unsigned long long g2 =
                (unsigned long long)((long long)gx * gx) + (unsigned long long)((long long)gy * gy);
            return g2 >= thr2 ? 1 : 0;
        };
        int su0, du0, su1, du1, sm0, dm0, sm1, dm1, sd0, dd0, sd1, dd1;
        hrow(r0, su0, du0, su1, du1);                // tile row r0 = image row y0 + r0 - 1
        hrow(r0 + 1, sm0, dm0, sm1, dm1);
#pragma unroll
        for (int r = 0; r < kDnRows; ++r) {          // th is a multiple of 16: the block is whole
            hrow(r0 + r + 2, sd0, dd0, sd1, dd1);
            cnt += edge(du0 + 2 * dm0 + dd0, su0 - sd0);
            cnt += edge(du1 + 2 * dm1 + dd1, su1 - sd1);
            su0 = sm0; du0 = dm0; su1 = sm1; du1 = dm1;
            sm0 = sd0; dm0 = dd0; sm1 = sd1; dm1 = dd1;
        }
    }
    // the lanes that share a patch: p / 2 of them (a warp holds the 64 columns of one block of rows)
    if (tid < 256) {
        const int width = p >> 1;
        for (int o = width >> 1; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if ((cp & (width - 1)) == 0 && active) atomicAdd(&s_cnt[(r0 / p) * npt + (2 * cp) / p], cnt);
    }
    __syncthreads();
    if (tid < npt * npt) {
        const int pi = tid / npt, pj = tid - pi * npt;
        if (pi * p < q.th && pj * p < q.tw && edge_counts) {
            const int gy = q.y0 / p + pi, gx = q.x0 / p + pj;
            edge_counts[((size_t)q.img * (H / p) + gy) * (W / p) + gx] = s_cnt[tid];
        }
    }
    if (tid == 32) {
        int total = 0;
        for (int k = 0; k < npt * npt; ++k) total += s_cnt[k];
        atomicAdd(image_counts + q.img, (uint32_t)total);
    }
}

// rho = average over the patches of (edge pixels / patch pixels); the patches are equal, so this is the
// image's edge pixels over its pixels.
__global__ void density_finish_kernel(const uint32_t *__restrict__ image_counts, int batch, float inv_pixels,
                                      float *__restrict__ rho)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < batch) rho[i] = (float)image_counts[i] * inv_pixels;
}

}  // namespace rtp

extern "C" rtprune_status_t rtprune_density(void *cuda_stream, const uint8_t *images, int32_t batch, int32_t height,
                                            int32_t width, int32_t patch, float tau, float *rho,
                                            uint32_t *image_counts, int32_t *edge_counts)
{
    using namespace rtp;
    if (batch < 0 || height <= 0 || width <= 0) return RTPRUNE_ERR_INVALID_ARG;
    if (patch != 16 && patch != 32 && patch != 64) return RTPRUNE_ERR_UNSUPPORTED;
    if (height % patch || width % patch) return RTPRUNE_ERR_UNSUPPORTED;
    if (!(tau >= 0.f) || !std::isfinite(tau)) return RTPRUNE_ERR_INVALID_ARG;
    if (batch == 0) return RTPRUNE_OK;
    if (!images || !rho || !image_counts || ((uintptr_t)images & 15u)) return RTPRUNE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // G >= tau  <=>  Gx_int^2 + Gy_int^2 >= (255000 tau)^2; the left side is an integer
    const double t = (double)tau * 255000.0;
    const double t2 = std::ceil(t * t);
    const unsigned long long thr2 = t2 >= 1.8e19 ? ~0ull : (unsigned long long)t2;
    if (cudaMemsetAsync(image_counts, 0, sizeof(uint32_t) * (size_t)batch, st) != cudaSuccess) return RTPRUNE_ERR_CUDA;
    if (batch > 65535 || (height + kDnTile - 1) / kDnTile > 65535) return RTPRUNE_ERR_UNSUPPORTED;
    dim3 grid((unsigned)((width + kDnTile - 1) / kDnTile), (unsigned)((height + kDnTile - 1) / kDnTile), (unsigned)batch);
    density_tile_kernel<<<grid, kDnThreads, 0, st>>>(images, height, width, patch, thr2, edge_counts, image_counts);
    density_finish_kernel<<<(batch + 255) / 256, 256, 0, st>>>(image_counts, batch,
                                                             1.f / ((float)height * (float)width), rho);
    return cudaGetLastError() == cudaSuccess ? RTPRUNE_OK : RTPRUNE_ERR_CUDA;
}
