// fp32 SIMT versions of the two contractions of stage 2: the cosine scores (Section 3.3.2) and the
// merge T_k + alpha P T_p (Eq. 7).  They serve the fp32 storage mode, where products must be kept
// to full fp32 precision, and any shape the tensor-core kernels do not take.
#pragma once
#include "common.cuh"

namespace rtp {

constexpr int kSimtTile = 64;  // output tile is 64 x 64, 256 threads, 4 x 4 per thread
constexpr int kSimtBK = 32;

// ---------------------------------------------------------------------------------------------
// S_ij = x_i . x_j / (|x_i| |x_j|), i in T_kept, j in T_prop.  grid = (mtiles * btiles, batch).
// Rows are gathered through the image's order[] list.  Output: kmat[i * score_pitch(B) + j].
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
scores_simt_kernel(const T *__restrict__ X, const int32_t *__restrict__ offsets, int d,
                   int btiles_max, const int32_t *__restrict__ counts,
                   const int32_t *__restrict__ order, const float *__restrict__ norms,
                   float *__restrict__ kmat, int kmat_stride, int max_tokens, int total)
{
    constexpr int EPV = Elem<T>::kPerVec;
    constexpr int VPR = kSimtBK / EPV;  // vectors per row per k-block
    __shared__ __align__(16) float As[kSimtBK][kSimtTile + 4];
    __shared__ __align__(16) float Bs[kSimtBK][kSimtTile + 4];
    __shared__ int s_rowA[kSimtTile], s_rowB[kSimtTile];

    const int img = blockIdx.y;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    const int mt = blockIdx.x / btiles_max, bt = blockIdx.x % btiles_max;
    const int i0 = mt * kSimtTile, j0 = bt * kSimtTile;
    if (B == 0 || i0 >= M || j0 >= B) return;

    const int tid = threadIdx.x;
    const int32_t *ord = order + t_begin;
    if (tid < kSimtTile) {
        s_rowA[tid] = (i0 + tid < M) ? t_begin + ord[i0 + tid] : -1;
        s_rowB[tid] = (j0 + tid < B) ? t_begin + ord[M + j0 + tid] : -1;
    }
    __syncthreads();

    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    for (int k0 = 0; k0 < d; k0 += kSimtBK) {
        for (int v = tid; v < kSimtTile * VPR; v += 256) {
            const int row = v / VPR, kv = v % VPR;
            const int k = k0 + kv * EPV;
            float fa[EPV], fb[EPV];
            const int ra = s_rowA[row], rb = s_rowB[row];
            if (ra >= 0 && k < d) {
                Elem<T>::unpack(ldg_vec(X + (size_t)ra * d + k), fa);
            } else {
#pragma unroll
                for (int e = 0; e < EPV; ++e) fa[e] = 0.f;
            }
            if (rb >= 0 && k < d) {
                Elem<T>::unpack(ldg_vec(X + (size_t)rb * d + k), fb);
            } else {
#pragma unroll
                for (int e = 0; e < EPV; ++e) fb[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                As[kv * EPV + e][row] = fa[e];
                Bs[kv * EPV + e][row] = fb[e];
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kSimtBK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }

    float *Kimg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ld = score_pitch(B);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const int i = i0 + ty * 4 + p;
        if (i >= M) continue;
        const float ni = fmaxf(norms[s_rowA[ty * 4 + p]], kNormFloor);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = j0 + tx * 4 + q;
            if (j >= B) continue;
            const float nj = fmaxf(norms[s_rowB[tx * 4 + q]], kNormFloor);
            Kimg[(size_t)i * ld + j] = acc[p][q] / (ni * nj);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// y_i = x_i + alpha * sum_j P_ij x_j (Eq. 7), written packed: Y row out_offsets[img] + i, together
// with kept_idx.  grid = (mtiles * dtiles, batch).  P is read from kmat (row pitch score_pitch(B)).
// With B = 0 the rows are copied unchanged.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
merge_simt_kernel(const T *__restrict__ X, const int32_t *__restrict__ offsets, int d, int dtiles,
                  const int32_t *__restrict__ counts, const int32_t *__restrict__ out_offsets,
                  const int32_t *__restrict__ order, const float *__restrict__ kmat,
                  int kmat_stride, int max_tokens, int total, float alpha, T *__restrict__ Y,
                  int32_t *__restrict__ kept_idx)
{
    constexpr int BK = 16;
    __shared__ __align__(16) float Ps[BK][kSimtTile + 4];   // [j][i]
    __shared__ __align__(16) float Xs[BK][kSimtTile + 4];   // [j][c]
    __shared__ int s_rowA[kSimtTile];

    const int img = blockIdx.y;
    int t_begin, N;
    if (!image_range(offsets, img, max_tokens, total, t_begin, N)) return;
    const int M = counts[img], B = N - M;
    const int mt = blockIdx.x / dtiles, dt = blockIdx.x % dtiles;
    const int i0 = mt * kSimtTile, c0 = dt * kSimtTile;
    if (i0 >= M) return;

    const int tid = threadIdx.x;
    const int32_t *ord = order + t_begin;
    const int out0 = out_offsets[img];
    if (tid < kSimtTile) {
        const int i = i0 + tid;
        s_rowA[tid] = (i < M) ? ord[i] : -1;
        if (dt == 0 && i < M) kept_idx[out0 + i] = ord[i];
    }
    __syncthreads();

    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    const float *Pimg = kmat + kmat_offset(kmat_stride, t_begin, img);
    const int ld = score_pitch(B);
    for (int j0 = 0; j0 < B; j0 += BK) {
        for (int v = tid; v < BK * kSimtTile; v += 256) {
            {   // P tile: consecutive threads walk j (contiguous in memory)
                const int i = v / BK, j = v % BK;
                Ps[j][i] = (i0 + i < M && j0 + j < B) ? Pimg[(size_t)(i0 + i) * ld + j0 + j] : 0.f;
            }
            {   // X_p tile: consecutive threads walk c
                const int j = v / kSimtTile, c = v % kSimtTile;
                float x = 0.f;
                if (j0 + j < B && c0 + c < d)
                    x = Elem<T>::to_float(X[(size_t)(t_begin + ord[M + j0 + j]) * d + c0 + c]);
                Xs[j][c] = x;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&Ps[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Xs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const int il = ty * 4 + p;
        if (i0 + il >= M) continue;
        const T *xrow = X + (size_t)(t_begin + s_rowA[il]) * d;
        T *yrow = Y + (size_t)(out0 + i0 + il) * d;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int c = c0 + tx * 4 + q;
            if (c >= d) continue;
            const float x = Elem<T>::to_float(xrow[c]);
            yrow[c] = Elem<T>::from_float(B > 0 ? fmaf(alpha, acc[p][q], x) : x);
        }
    }
}

}  // namespace rtp
