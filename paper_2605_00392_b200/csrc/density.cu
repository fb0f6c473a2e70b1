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
// One CTA of 256 threads per token patch (p x p pixels, p = 16, 32 or 64):
//   1. the patch's rows are 3p contiguous bytes, 16-byte aligned (p and the image width are multiples
//      of 16): a thread fetches 48 bytes = 16 pixels with three 16-byte loads, turns them into 16
//      integer gray values and stores those into a (p+2) x (p+2) tile in shared memory; the one-pixel
//      ring around the patch is fetched pixel by pixel;
//   2. a thread walks down a column of the patch over p*p/256 rows with the horizontal sums of three
//      rows in registers: three shared-memory loads and about a dozen integer operations per pixel.
// The CTA writes its patch's count and adds it to the image's count (integer atomics: the result does
// not depend on the order); a second small kernel turns the image counts into rho.
#include <cstdint>
#include <cmath>

#include <cuda_runtime.h>

#include "../../include/rtprune.h"

namespace rtp {

constexpr int kDnThreads = 256;
constexpr int kDnMaxPatch = 64;
constexpr int kDnPitch = kDnMaxPatch + 2 + 1;      // odd pitch of the gray tile: conflict-free column walks

__device__ inline int gray_of(uint32_t r, uint32_t g, uint32_t b) { return (int)(299u * r + 587u * g + 114u * b); }

__global__ void __launch_bounds__(kDnThreads)
density_patch_kernel(const uint8_t *__restrict__ images, int H, int W, int p, unsigned long long thr2,
                     int32_t *__restrict__ edge_counts, uint32_t *__restrict__ image_counts)
{
    __shared__ int s_gray[(kDnMaxPatch + 2) * kDnPitch];
    __shared__ int s_cnt[kDnThreads / 32];
    const int tid = threadIdx.x;
    const int px = blockIdx.x, py = blockIdx.y, img = blockIdx.z;
    const uint8_t *im = images + (size_t)img * H * W * 3;
    const int x0 = px * p, y0 = py * p;

    // ---- gray tile: rows y0-1 .. y0+p, columns x0-1 .. x0+p (tile coordinates 0 .. p+1) -------------
    const int groups = p >> 4;                       // 16-pixel groups per patch row
    for (int t = tid; t < (p + 2) * groups; t += kDnThreads) {
        const int ty = t / groups, gx = t - ty * groups;
        const int y = min(max(y0 + ty - 1, 0), H - 1);
        const uint4 *src = reinterpret_cast<const uint4 *>(im + ((size_t)y * W + x0 + 16 * gx) * 3);
        uint32_t w[12];
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const uint4 v = __ldg(src + q);
            w[4 * q] = v.x;
            w[4 * q + 1] = v.y;
            w[4 * q + 2] = v.z;
            w[4 * q + 3] = v.w;
        }
        int *dst = s_gray + ty * kDnPitch + 1 + 16 * gx;
#pragma unroll
        for (int k = 0; k < 16; ++k) {               // pixel k = bytes 3k .. 3k+2 of the 48
            uint32_t c[3];
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                const int byte = 3 * k + e;
                c[e] = (w[byte >> 2] >> (8 * (byte & 3))) & 0xffu;
            }
            dst[k] = gray_of(c[0], c[1], c[2]);
        }
    }
    for (int t = tid; t < 2 * (p + 2); t += kDnThreads) {    // left and right ring columns
        const int ty = t >> 1, right = t & 1;
        const int y = min(max(y0 + ty - 1, 0), H - 1);
        const int x = right ? min(x0 + p, W - 1) : max(x0 - 1, 0);
        const uint8_t *q = im + ((size_t)y * W + x) * 3;
        s_gray[ty * kDnPitch + (right ? p + 1 : 0)] = gray_of(__ldg(q), __ldg(q + 1), __ldg(q + 2));
    }
    __syncthreads();

    // ---- Sobel, threshold, count: thread = (column c, block of rows) -----------------------------------
    const int ngroups = kDnThreads / p;              // 4, 8 or 16 row blocks
    const int rows_per = p / ngroups;                // 16, 4 or 1
    const int c = tid % p, r0 = (tid / p) * rows_per;
    // horizontal sums of a tile row at this column: smooth s = l + 2 m + r, difference d = r - l
    auto hrow = [&](int trow, int &s, int &d) {
        const int *g = s_gray + trow * kDnPitch + c;          // tile columns c, c+1, c+2 = image x-1, x, x+1
        const int l = g[0], m = g[1], r = g[2];
        s = l + 2 * m + r;
        d = r - l;
    };
    int s_up, d_up, s_mid, d_mid, s_dn, d_dn;
    hrow(r0, s_up, d_up);                            // tile row r0 = image row y0 + r0 - 1
    hrow(r0 + 1, s_mid, d_mid);
    int cnt = 0;
    for (int r = 0; r < rows_per; ++r) {
        hrow(r0 + r + 2, s_dn, d_dn);
        const int gx = d_up + 2 * d_mid + d_dn;
        const int gy = s_up - s_dn;
        const unsigned long long g2 = (unsigned long long)((long long)gx * gx) + (unsigned long long)((long long)gy * gy);
        cnt += (g2 >= thr2) ? 1 : 0;
        s_up = s_mid;
        d_up = d_mid;
        s_mid = s_dn;
        d_mid = d_dn;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if ((tid & 31) == 0) s_cnt[tid >> 5] = cnt;
    __syncthreads();
    if (tid == 0) {
        int total = 0;
#pragma unroll
        for (int w = 0; w < kDnThreads / 32; ++w) total += s_cnt[w];
        if (edge_counts) edge_counts[((size_t)img * gridDim.y + py) * gridDim.x + px] = total;
        atomicAdd(image_counts + img, (uint32_t)total);
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
    if (batch > 65535 || height / patch > 65535) return RTPRUNE_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // G >= tau  <=>  Gx_int^2 + Gy_int^2 >= (255000 tau)^2; the left side is an integer
    const double t = (double)tau * 255000.0;
    const double t2 = std::ceil(t * t);
    const unsigned long long thr2 = t2 >= 1.8e19 ? ~0ull : (unsigned long long)t2;
    if (cudaMemsetAsync(image_counts, 0, sizeof(uint32_t) * (size_t)batch, st) != cudaSuccess) return RTPRUNE_ERR_CUDA;
    dim3 grid((unsigned)(width / patch), (unsigned)(height / patch), (unsigned)batch);
    density_patch_kernel<<<grid, kDnThreads, 0, st>>>(images, height, width, patch, thr2, edge_counts, image_counts);
    density_finish_kernel<<<(batch + 255) / 256, 256, 0, st>>>(image_counts, batch,
                                                             1.f / ((float)height * (float)width), rho);
    return cudaGetLastError() == cudaSuccess ? RTPRUNE_OK : RTPRUNE_ERR_CUDA;
}
