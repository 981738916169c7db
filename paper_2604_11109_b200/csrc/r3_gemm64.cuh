// FP64 product with a lower-triangular matrix, shared by the append step of the fit and by the batch
// proposal (both need  A * W^T  or  A * W  for the inverse Cholesky factor W).
#pragma once

#include <cuda_runtime.h>

namespace r3 {

// C[M x N] = A[M x R] * op(Wm) with the lower-triangular Wm (upper part stored as zeros):
//   NT = true :  C[i][c] = sum_{r <= c} A[i][r] * Wm[c][r]      (A * Wm^T)
//   NT = false:  C[i][c] = sum_{r >= c} A[i][r] * Wm[r][c]      (A * Wm)
// FP64, 32 x 64 tile per block of 256 threads (2 x 4 per thread), reduction in steps of 16 over the part of
// r that can be non-zero for the tile's columns.
template <bool NT>
__global__ void __launch_bounds__(256) tri_gemm_kernel(const double* __restrict__ A, int lda, size_t strideA,
                                                       const double* __restrict__ Wm, int ldw, size_t strideW,
                                                       double* __restrict__ C, int ldc, size_t strideC, int M, int N)
{
    __shared__ double As[32][17], Bs[16][65];
    const int g = blockIdx.z;
    A += (size_t)g * strideA;
    Wm += (size_t)g * strideW;
    C += (size_t)g * strideC;
    const int i0 = blockIdx.y * 32, c0 = blockIdx.x * 64;
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    double acc[2][4] = {};
    const int r_begin = NT ? 0 : (c0 / 16) * 16;
    const int r_end = NT ? min(c0 + 64, N) : N;
    for (int r0 = r_begin; r0 < r_end; r0 += 16) {
        for (int e = t; e < 32 * 16; e += 256) {
            const int i = e / 16, r = e % 16;
            As[i][r] = (i0 + i < M && r0 + r < N) ? A[(size_t)(i0 + i) * lda + r0 + r] : 0.0;
        }
        for (int e = t; e < 16 * 64; e += 256) {
            if (NT) {
                const int c = e / 16, r = e % 16;   // consecutive threads walk r: 128 contiguous bytes per row of Wm
                Bs[r][c] = (c0 + c < N && r0 + r < N) ? Wm[(size_t)(c0 + c) * ldw + r0 + r] : 0.0;
            } else {
                const int r = e / 64, c = e % 64;
                Bs[r][c] = (c0 + c < N && r0 + r < N) ? Wm[(size_t)(r0 + r) * ldw + c0 + c] : 0.0;
            }
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            const double a0 = As[ty * 2][r], a1 = As[ty * 2 + 1][r];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const double b = Bs[r][tx * 4 + v];
                acc[0][v] = fma(a0, b, acc[0][v]);
                acc[1][v] = fma(a1, b, acc[1][v]);
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * 2 + u, c = c0 + tx * 4 + v;
            if (i < M && c < N) C[(size_t)i * ldc + c] = acc[u][v];
        }
}

}  // namespace r3
