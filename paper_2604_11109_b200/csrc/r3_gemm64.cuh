// FP64 product with a lower-triangular matrix, shared by the append step of the fit and by the batch
// proposal (both need  A * W^T  or  A * W  for the inverse Cholesky factor W).
#pragma once

#include <cuda_runtime.h>

namespace r3 {

// C[M x N] = A[M x R] * op(Wm) with the lower-triangular Wm (upper part stored as zeros):
//   NT = true :  C[i][c] = sum_{r <= c} A[i][r] * Wm[c][r]      (A * Wm^T)
//   NT = false:  C[i][c] = sum_{r >= c} A[i][r] * Wm[r][c]      (A * Wm)
// FP64, TM x 64 tile per block of 256 threads (TM / 16 x 4 results per thread; TM = 32 for the few rows of an
// append, 64 for the many of a proposal's shortlist), reduction in steps of 16 over the part of r that can be
// non-zero for the tile's columns; the next step's operands are fetched into registers during the current one.
// With few rows (an append's k <= 128) the tiles are too few to fill the GPU and the long reductions of the
// right-hand columns dominate: `splits` > 1 cuts every tile's reduction into that many parts (blockIdx.z = GP *
// splits + part), part p writing its partial product to C + p * strideSplit; tri_gemm_sum_kernel adds the parts
// in a fixed order.
template <bool NT, int TM = 32>
__global__ void __launch_bounds__(256) tri_gemm_kernel(const double* __restrict__ A, int lda, size_t strideA,
                                                       const double* __restrict__ Wm, int ldw, size_t strideW,
                                                       double* __restrict__ C, int ldc, size_t strideC, int M, int N,
                                                       int splits = 1, size_t strideSplit = 0)
{
    constexpr int RU = TM / 16;   // rows per thread
    __shared__ double As[TM][17], Bs[16][65];
    const int g = blockIdx.z / splits, part = blockIdx.z % splits;
    A += (size_t)g * strideA;
    Wm += (size_t)g * strideW;
    C += (size_t)g * strideC + (size_t)part * strideSplit;
    const int i0 = blockIdx.y * TM, c0 = blockIdx.x * 64;
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    double acc[RU][4] = {};
    int r_begin = NT ? 0 : (c0 / 16) * 16;
    int r_end = NT ? min(c0 + 64, N) : N;
    if (splits > 1) {
        const int steps = (r_end - r_begin + 15) / 16, per = (steps + splits - 1) / splits;
        r_begin += part * per * 16;
        r_end = min(r_end, r_begin + per * 16);
    }
    double ra[RU], rb[4];
    auto fetch = [&](int r0) {
#pragma unroll
        for (int q = 0; q < RU; ++q) {
            const int e = t + 256 * q;
            const int i = e / 16, r = e % 16;
            ra[q] = (i0 + i < M && r0 + r < N) ? A[(size_t)(i0 + i) * lda + r0 + r] : 0.0;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int e = t + 256 * q;
            if (NT) {
                const int c = e / 16, r = e % 16;   // consecutive threads walk r: 128 contiguous bytes per row of Wm
                rb[q] = (c0 + c < N && r0 + r < N) ? Wm[(size_t)(c0 + c) * ldw + r0 + r] : 0.0;
            } else {
                const int r = e / 64, c = e % 64;
                rb[q] = (c0 + c < N && r0 + r < N) ? Wm[(size_t)(r0 + r) * ldw + c0 + c] : 0.0;
            }
        }
    };
    if (r_begin < r_end) fetch(r_begin);
    for (int r0 = r_begin; r0 < r_end; r0 += 16) {
        if (r0 > r_begin) __syncthreads();
#pragma unroll
        for (int q = 0; q < RU; ++q) {
            const int e = t + 256 * q;
            As[e / 16][e % 16] = ra[q];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int e = t + 256 * q;
            if (NT)
                Bs[e % 16][e / 16] = rb[q];
            else
                Bs[e / 64][e % 64] = rb[q];
        }
        __syncthreads();
        if (r0 + 16 < r_end) fetch(r0 + 16);
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            double a[RU];
#pragma unroll
            for (int u = 0; u < RU; ++u) a[u] = As[ty * RU + u][r];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const double b = Bs[r][tx * 4 + v];
#pragma unroll
                for (int u = 0; u < RU; ++u) acc[u][v] = fma(a[u], b, acc[u][v]);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < RU; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * RU + u, c = c0 + tx * 4 + v;
            if (i < M && c < N) C[(size_t)i * ldc + c] = acc[u][v];
        }
}

// C[g][e] = sum over the parts, in order (C's parts lie strideSplit apart; the sum goes to part 0)
static __global__ void tri_gemm_sum_kernel(double* __restrict__ C, size_t count, size_t strideC, int splits, size_t strideSplit)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count) return;
    double* c = C + (size_t)blockIdx.y * strideC + e;
    double s = c[0];
    for (int p = 1; p < splits; ++p) s += c[(size_t)p * strideSplit];
    c[0] = s;
}

}  // namespace r3
