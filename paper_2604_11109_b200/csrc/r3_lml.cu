// Log marginal likelihood of the history and its gradient with respect to the logarithms of the
// hyper-parameters, from what the fit already holds (L, W = L^-1, alpha, X, y):
//     lml = -1/2 y.alpha - sum_i log L_ii - n/2 log(2 pi)
//     M   = alpha alpha^T - K^-1,   K^-1 = W^T W                     (kinv_kernel: n^3/3 FP64 FMAs)
//     d lml / d log ell_j = 1/2 sum_ik M_ik sf2 e^-s (5/3)(1 + s) u_j^2     (u_j = (x_ij - x_kj)/ell_j)
//     d lml / d log sf2   = 1/2 sum_ik M_ik Kf_ik,    d lml / d log sn2 = 1/2 sn2 trace(M)
// Everything in FP64; the pair sums use the symmetry of M (lower triangle, off-diagonal pairs twice) and
// are reduced in a fixed order (per-block partial sums, then one block adds them), so results repeat
// bit for bit.
#include <math.h>

#include <vector>

#include "r3_internal.cuh"

namespace r3 {

namespace {

// M[i][j] = alpha_i alpha_j - sum_{r >= i} W[r][i] W[r][j] for j <= i (64 x 64 tile per block, 4 x 4 per thread).
__global__ void __launch_bounds__(256) kinv_kernel(const double* __restrict__ W, const double* __restrict__ alpha, int n,
                                                   int npad, double* __restrict__ M)
{
    const int g = blockIdx.z;
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (tj > ti) return;
    W += (size_t)g * npad * npad;
    M += (size_t)g * npad * npad;
    alpha += (size_t)g * npad;
    __shared__ double Ai[16][65], Aj[16][65];
    const int i0 = ti * 64, j0 = tj * 64;
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    double acc[4][4] = {};
    for (int r0 = i0 / 16 * 16; r0 < n; r0 += 16) {
        for (int e = t; e < 16 * 64; e += 256) {
            const int r = e / 64, c = e % 64;
            const bool ok = r0 + r < n;
            Ai[r][c] = (ok && i0 + c < n) ? W[(size_t)(r0 + r) * npad + i0 + c] : 0.0;
            Aj[r][c] = (ok && j0 + c < n) ? W[(size_t)(r0 + r) * npad + j0 + c] : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a[u] = Ai[r][ty * 4 + u];
                b[u] = Aj[r][tx * 4 + u];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * 4 + u, j = j0 + tx * 4 + v;
            if (i < n && j <= i) M[(size_t)i * npad + j] = alpha[i] * alpha[j] - acc[u][v];
        }
}

// One 32 x 32 tile of pairs (i, k), k-tile <= i-tile, per block of 256 threads (thread: one i, four k).
// partial[block][0 .. d-1] = sum over the tile of w M_ik G_ik u_j^2, partial[block][d] = sum w M_ik Kf_ik,
// with w = 1 on the diagonal, 2 below it, 0 above.
__global__ void __launch_bounds__(256) lml_pairs_kernel(const float* __restrict__ X, const float* __restrict__ ell,
                                                        const float* __restrict__ sf2v, int n, int d, int npad,
                                                        const double* __restrict__ M, int tiles,
                                                        double* __restrict__ partial)
{
    // blockIdx.y: the GP
    const int g = blockIdx.y;
    X += (size_t)g * n * d;
    ell += (size_t)g * d;
    M += (size_t)g * npad * npad;
    partial += (size_t)g * tiles * (d + 1);
    const double sf2 = (double)sf2v[g];
    // tile index -> (ti, tk) of the lower triangle
    const int b = blockIdx.x;
    int ti = (int)((sqrt(8.0 * b + 1.0) - 1.0) * 0.5);
    while ((ti + 1) * (ti + 2) / 2 <= b) ++ti;
    while (ti * (ti + 1) / 2 > b) --ti;
    const int tk = b - ti * (ti + 1) / 2;
    __shared__ float xi[32][33], xk[32][33];
    __shared__ double sl[32];        // 1 / lengthscale (FP64 reciprocal, as in the fit's Gram kernel)
    __shared__ double red[8];
    __shared__ double redc[8][32];   // the warps' sums of 32 features' terms
    const int t = threadIdx.x, li = t % 32, lk0 = (t / 32) * 4;
    const int i = ti * 32 + li;
    double r2[4] = {0, 0, 0, 0};
    for (int c0 = 0; c0 < d; c0 += 32) {
        __syncthreads();
        for (int e = t; e < 32 * 32; e += 256) {
            const int r = e / 32, c = e % 32;
            const int gi = ti * 32 + r, gk = tk * 32 + r;
            xi[r][c] = (gi < n && c0 + c < d) ? X[(size_t)gi * d + c0 + c] : 0.f;
            xk[r][c] = (gk < n && c0 + c < d) ? X[(size_t)gk * d + c0 + c] : 0.f;
        }
        if (t < 32) sl[t] = (c0 + t < d) ? 1.0 / (double)ell[c0 + t] : 1.0;
        __syncthreads();
        const int cmax = min(32, d - c0);
        for (int c = 0; c < cmax; ++c) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const double u = ((double)xi[li][c] - (double)xk[lk0 + q][c]) * sl[c];
                r2[q] = fma(u, u, r2[q]);
            }
        }
    }
    double gk[4], kf_sum = 0.0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int k = tk * 32 + lk0 + q;
        double w = 0.0;
        if (i < n && k < n && k <= i) w = (k == i) ? 1.0 : 2.0;
        const double m = w != 0.0 ? M[(size_t)i * npad + k] : 0.0;
        const double s = sqrt(5.0) * sqrt(r2[q]);
        const double e = exp(-s);
        gk[q] = w * m * sf2 * e * (5.0 / 3.0) * (1.0 + s);
        kf_sum += w * m * sf2 * (1.0 + s + s * s / 3.0) * e;
    }
    double* out = partial + (size_t)b * (d + 1);
    // block sums: warp shuffle, then the eight warps in a fixed order
    auto block_sum = [&](double v, int slot) {
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();
        if ((t & 31) == 0) red[t / 32] = v;
        __syncthreads();
        if (t == 0) {
            double s = 0.0;
            for (int w = 0; w < 8; ++w) s += red[w];
            out[slot] = s;
        }
    };
    block_sum(kf_sum, d);
    for (int c0 = 0; c0 < d; c0 += 32) {
        __syncthreads();
        for (int e = t; e < 32 * 32; e += 256) {
            const int r = e / 32, c = e % 32;
            const int gi = ti * 32 + r, gk_ = tk * 32 + r;
            xi[r][c] = (gi < n && c0 + c < d) ? X[(size_t)gi * d + c0 + c] : 0.f;
            xk[r][c] = (gk_ < n && c0 + c < d) ? X[(size_t)gk_ * d + c0 + c] : 0.f;
        }
        if (t < 32) sl[t] = (c0 + t < d) ? 1.0 / (double)ell[c0 + t] : 1.0;
        __syncthreads();
        const int cmax = min(32, d - c0);
        for (int c = 0; c < cmax; ++c) {
            double v = 0.0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const double u = ((double)xi[li][c] - (double)xk[lk0 + q][c]) * sl[c];
                v = fma(gk[q], u * u, v);
            }
            // warp sum now, the eight warps in a fixed order once per 32 features
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if ((t & 31) == 0) redc[t / 32][c] = v;
        }
        __syncthreads();
        if (t < cmax) {
            double s = 0.0;
            for (int w = 0; w < 8; ++w) s += redc[w][t];
            out[c0 + t] = s;
        }
    }
}

// One block per GP: adds the tiles' partial sums in order, the trace term and the value.
__global__ void __launch_bounds__(256) lml_finish_kernel(const double* __restrict__ partial, int tiles, int d,
                                                         const double* __restrict__ M, const double* __restrict__ L,
                                                         const double* __restrict__ alpha, const float* __restrict__ y,
                                                         int n, int npad, const float* __restrict__ sn2v,
                                                         double* __restrict__ out)
{
    __shared__ double red[256];
    const int g = blockIdx.x;
    partial += (size_t)g * tiles * (d + 1);
    M += (size_t)g * npad * npad;
    L += (size_t)g * npad * npad;
    alpha += (size_t)g * npad;
    y += (size_t)g * n;
    out += (size_t)g * (d + 3);
    const double sn2 = (double)sn2v[g];
    const int t = threadIdx.x;
    auto block_sum = [&](double v) {
        red[t] = v;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (t < o) red[t] += red[t + o];
            __syncthreads();
        }
        const double s = red[0];
        __syncthreads();
        return s;
    };
    for (int j = 0; j <= d; ++j) {
        double v = 0.0;
        for (int b = t; b < tiles; b += 256) v += partial[(size_t)b * (d + 1) + j];
        const double s = block_sum(v);
        if (t == 0) out[1 + j] = 0.5 * s;
    }
    double tr = 0.0, quad = 0.0, logdet = 0.0;
    for (int i = t; i < n; i += 256) {
        tr += M[(size_t)i * npad + i];
        quad += (double)y[i] * alpha[i];
        logdet += log(L[(size_t)i * npad + i]);
    }
    tr = block_sum(tr);
    quad = block_sum(quad);
    logdet = block_sum(logdet);
    if (t == 0) {
        out[d + 2] = 0.5 * sn2 * tr;
        out[0] = -0.5 * quad - logdet - 0.5 * n * 1.8378770664093454836;   // log(2 pi)
    }
}

}  // namespace

// out_h: host [batch][d + 3] = {lml, d/dlog ell_1..d, d/dlog sf2, d/dlog sn2}.  Synchronises.
r3_status_t lml_device(r3_gp* gp, double* out_h, cudaStream_t stream)
{
    const int B = gp->batch, n = gp->n, d = gp->d, npad = gp->npad;
    const int t32 = (n + 31) / 32, tiles = t32 * (t32 + 1) / 2;
    double *M = nullptr, *partial = nullptr, *out = nullptr;
    auto done = [&](r3_status_t st) {
        dev_free(M);
        dev_free(partial);
        dev_free(out);
        return st;
    };
#define TRY_DONE(expr)                                                                             \
    do {                                                                                           \
        cudaError_t e__ = (expr);                                                                  \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("%s failed: %s", #expr, cudaGetErrorString(e__));                            \
            return done(e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA);            \
        }                                                                                          \
    } while (0)
    TRY_DONE(dev_malloc(&M, sizeof(double) * (size_t)B * npad * npad));
    TRY_DONE(dev_malloc(&partial, sizeof(double) * (size_t)B * tiles * (d + 1)));
    TRY_DONE(dev_malloc(&out, sizeof(double) * (size_t)B * (d + 3)));
    const int t64 = (n + 63) / 64;
    kinv_kernel<<<dim3(t64, t64, B), 256, 0, stream>>>(gp->W64, gp->alpha64, n, npad, M);
    ++g_launches;
    TRY_DONE(cudaGetLastError());
    lml_pairs_kernel<<<dim3(tiles, B), 256, 0, stream>>>(gp->X, gp->ell_d, gp->sf2_d, n, d, npad, M, tiles, partial);
    ++g_launches;
    TRY_DONE(cudaGetLastError());
    lml_finish_kernel<<<B, 256, 0, stream>>>(partial, tiles, d, M, gp->L64, gp->alpha64, gp->y, n, npad, gp->sn2_d, out);
    ++g_launches;
    TRY_DONE(cudaGetLastError());
    TRY_DONE(cudaMemcpyAsync(out_h, out, sizeof(double) * (size_t)B * (d + 3), cudaMemcpyDeviceToHost, stream));
    TRY_DONE(cudaStreamSynchronize(stream));
#undef TRY_DONE
    return done(R3_OK);
}

}  // namespace r3
