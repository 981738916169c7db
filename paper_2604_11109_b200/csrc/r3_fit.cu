// r3_gp_fit on the device: FP64 Gram matrix, blocked batched Cholesky, inverse factor, weights.
//
// Everything here runs once per BO round, in FP64, and is rounded to FP32 once at the end:
//   K = k(X,X) + noise*I           gram_kernel            (direct differences, like the definition)
//   K = L L^T                      potrf_diag / panel / syrk kernels, right-looking, block 32
//   W = L^-1                       diagonal-block inverses, then recursive doubling with two
//                                  batched GEMMs per level:  W21 = -W22 (L21 W11)
//   alpha = W^T (W y)              two triangular matrix-vector products
// All kernels take the GP index from blockIdx.z (or .y), so `batch` GPs are factored together.
// n is padded to a multiple of 32 with an identity block, which leaves L, W and alpha unchanged.
#include "r3_gemm64.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr int NB = kFitBlock;

// ------------------------------------------------------------------------------------ checks
__global__ void check_finite_kernel(const float* __restrict__ a, size_t count, int* status)
{
    bool bad = false;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count;
         i += (size_t)gridDim.x * blockDim.x)
        bad |= !isfinite(a[i]);
    if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, DEV_NONFINITE);
}

__global__ void min_y_kernel(const float* __restrict__ y, int n, float* best, float* yabs)
{
    __shared__ float s[256], a[256];
    const float* yg = y + (size_t)blockIdx.x * n;
    float v = INFINITY, m = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        v = fminf(v, yg[i]);
        m = fmaxf(m, fabsf(yg[i]));
    }
    s[threadIdx.x] = v;
    a[threadIdx.x] = m;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            s[threadIdx.x] = fminf(s[threadIdx.x], s[threadIdx.x + o]);
            a[threadIdx.x] = fmaxf(a[threadIdx.x], a[threadIdx.x + o]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        best[blockIdx.x] = s[0];
        yabs[blockIdx.x] = a[0];
    }
}

// ------------------------------------------------------------------------------------ Gram
// One 16x16 tile of the lower triangle per block; r^2 by direct differences in FP64, scaled by the FP64
// reciprocal of the lengthscale (one rounding more than a division, a relative 1e-16 in K, for a third of
// the kernel's time), the Matern-5/2 profile, noise on the diagonal.
__global__ void gram_kernel(const float* __restrict__ X, const float* __restrict__ ell,
                            const float* __restrict__ sf2, const float* __restrict__ sn2, int n, int d,
                            int npad, double* __restrict__ K)
{
    const int g = blockIdx.z;
    const int ti = blockIdx.y, tj = blockIdx.x;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int i = ti * 16 + ty, j = tj * 16 + tx;
    double* Kg = K + (size_t)g * npad * npad;
    if (tj > ti) {
        Kg[(size_t)i * npad + j] = 0.0;
        return;
    }
    __shared__ float sxi[16][33], sxj[16][33];
    __shared__ double sl[32];   // 1 / lengthscale
    const float* Xg = X + (size_t)g * n * d;
    double r2 = 0.0;
    for (int c0 = 0; c0 < d; c0 += 32) {
        const int t = ty * 16 + tx;  // 0..255
        for (int e = t; e < 16 * 32; e += 256) {
            int r = e / 32, c = e % 32;
            int gi = ti * 16 + r, gj = tj * 16 + r;
            sxi[r][c] = (gi < n && c0 + c < d) ? Xg[(size_t)gi * d + c0 + c] : 0.f;
            sxj[r][c] = (gj < n && c0 + c < d) ? Xg[(size_t)gj * d + c0 + c] : 0.f;
        }
        if (t < 32) sl[t] = (c0 + t < d) ? 1.0 / (double)ell[(size_t)g * d + c0 + t] : 1.0;
        __syncthreads();
        const int cmax = min(32, d - c0);
        for (int c = 0; c < cmax; ++c) {
            double diff = ((double)sxi[ty][c] - (double)sxj[tx][c]) * sl[c];
            r2 += diff * diff;
        }
        __syncthreads();
    }
    double v;
    if (i < n && j < n) {
        double s = sqrt(5.0) * sqrt(r2);
        v = (double)sf2[g] * (1.0 + s + s * s / 3.0) * exp(-s);
        if (i == j) v += (double)sn2[g];
        if (j > i) v = 0.0;
    } else {
        v = (i == j) ? 1.0 : 0.0;
    }
    Kg[(size_t)i * npad + j] = v;
}

// ------------------------------------------------------------------------------------ Cholesky
// One step of the factorisation for the 32 columns at j0, in ONE launch: every block factors the 32x32
// diagonal block itself (redundantly -- it is the latency of 32 dependent columns either way, and a second
// launch waiting for a first costs as much again) and then solves its share of the panel below it, one row
// per thread.  Block 0 also stores the factored diagonal block (to Ldiag, copied into place after the
// factorisation: the other blocks of this launch may still be reading the unfactored block) and its inverse
// (to Dinv[g][j0/32], for the inverse factor).
//
// Diagonal block: one barrier per column.  At step k every thread forms r = 1/sqrt(a_kk) itself and scales
// what it reads of column k by it, so that nothing has to be written (and waited for) between the pivot and
// the update; the column stays unscaled in shared memory until the end.  The inverse comes from the same
// sweep: with L = L_1 ... L_32 (L_k the identity with column k of L), L^-1 = L_32^-1 ... L_1^-1, and
// applying L_k^-1 to the running product M is the same rank-one update on the columns <= k that the
// factorisation does on the columns > k -- the threads of the finished columns do it.  Row k of M, like
// column k of A, is scaled by r only at the end.
//
// Panel: L_panel L_jj^T = A_panel by forward substitution.  (Multiplying by the explicit inverse of L_jj
// instead loses the small entries of an ill-conditioned factor: its error is relative to
// |A_panel| |L_jj^-1|, not to the result, and the pivots that follow inherit it -- on noise-free smooth data
// the log-determinant came out wrong in the third digit.)
constexpr int kPanelThreads = 256;   // 32 x 8: four rows of the diagonal block per thread, one panel row per thread
constexpr size_t kPanelSmem = sizeof(double) * (kPanelThreads / NB) * NB * (NB + 1);   // the warps' row tiles
__global__ void __launch_bounds__(kPanelThreads) potrf_panel_kernel(double* __restrict__ A, int npad, int j0,
                                                                    double* __restrict__ Dinv,
                                                                    double* __restrict__ Ldiag, int* status)
{
    const int g = blockIdx.y;
    const int tx = threadIdx.x, tq = threadIdx.y;   // rows tq, tq + 8, tq + 16, tq + 24 of the diagonal block
    double* Agp = A + (size_t)g * npad * npad;
    const double* Ag = Agp + (size_t)j0 * npad + j0;
    __shared__ double a[NB][NB + 1];
    __shared__ double m[NB][NB + 1];
    __shared__ double rk[NB], lkk[NB];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int ty = tq + 8 * i;
        a[ty][tx] = Ag[(size_t)ty * npad + tx];
        m[ty][tx] = (tx == ty) ? 1.0 : 0.0;
    }
    __syncthreads();
    for (int k = 0; k < NB; ++k) {
        double p = a[k][k];
        if (!(p > 0.0) || !isfinite(p)) {
            if (tx == 0 && tq == 0 && blockIdx.x == 0) {
                atomicOr(&status[0], DEV_NOT_PD);
                atomicMin(&status[1], j0 + k);
            }
            p = 1.0;  // keep going without NaNs; the call reports the failure
        }
        const double r = rsqrt(p);
        if (tx == 0 && tq == 0) {
            rk[k] = r;
            // sqrt(p) from r with one correction step (a second long-latency operation here would be on every
            // column's critical path): s = p r, s += r (p - s^2) / 2
            const double sq = p * r;
            lkk[k] = fma(0.5 * r, fma(-sq, sq, p), sq);
        }
        const double ck = tx > k ? a[tx][k] * r : m[k][tx] * r;   // what this thread's column contributes
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int ty = tq + 8 * i;
            if (ty > k) {
                const double lik = a[ty][k] * r;
                if (tx > k) {
                    if (ty >= tx) a[ty][tx] -= lik * ck;
                } else {
                    m[ty][tx] -= lik * ck;
                }
            }
        }
        __syncthreads();
    }
    // the factor in place of the block (upper part zero), for the substitution below and for block 0's stores
    double lij[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int ty = tq + 8 * i;
        lij[i] = (tx < ty) ? a[ty][tx] * rk[tx] : (tx == ty ? lkk[ty] : 0.0);
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int ty = tq + 8 * i;
        a[ty][tx] = lij[i];
        if (blockIdx.x == 0) {
            const size_t blk = ((size_t)g * (npad / NB) + j0 / NB) * NB * NB + ty * NB + tx;
            Ldiag[blk] = lij[i];
            Dinv[blk] = m[ty][tx] * rk[ty];
        }
    }
    __syncthreads();
    // Panel rows: warp tq owns rows r0 .. r0 + 31.  The rows go through shared memory so that global memory is
    // read and written a row at a time by the whole warp (256 contiguous bytes) while each thread works on its
    // own row.
    extern __shared__ double tile_all[];                  // [8 warps][32][33]
    double* tile = tile_all + (size_t)tq * NB * (NB + 1);
    const int r0 = j0 + NB + blockIdx.x * kPanelThreads + tq * NB;
    if (r0 >= npad) return;                               // whole warps only: the tile needs no block barrier
    const int nrows = min(NB, npad - r0);
    for (int i = 0; i < nrows; ++i) tile[i * (NB + 1) + tx] = Agp[(size_t)(r0 + i) * npad + j0 + tx];
    __syncwarp();
    if (tx < nrows) {
        double x[NB];
#pragma unroll
        for (int c = 0; c < NB; ++c) x[c] = tile[tx * (NB + 1) + c];
#pragma unroll
        for (int c = 0; c < NB; ++c) {
            double s0 = 0.0, s1 = 0.0;
#pragma unroll
            for (int k = 0; k + 1 < c; k += 2) {
                s0 = fma(x[k], a[c][k], s0);
                s1 = fma(x[k + 1], a[c][k + 1], s1);
            }
            if (c & 1) s0 = fma(x[c - 1], a[c][c - 1], s0);
            x[c] = (x[c] - (s0 + s1)) * rk[c];
        }
#pragma unroll
        for (int c = 0; c < NB; ++c) tile[tx * (NB + 1) + c] = x[c];
    }
    __syncwarp();
    for (int i = 0; i < nrows; ++i) Agp[(size_t)(r0 + i) * npad + j0 + tx] = tile[i * (NB + 1) + tx];
}

// After the factorisation: the factored diagonal blocks into their places.
__global__ void scatter_ldiag_kernel(const double* __restrict__ Ldiag, int npad, double* __restrict__ L)
{
    const int g = blockIdx.y, b = blockIdx.x;
    const double* Dg = Ldiag + ((size_t)g * (npad / NB) + b) * NB * NB;
    double* Lg = L + (size_t)g * npad * npad + (size_t)(b * NB) * npad + b * NB;
    Lg[(size_t)threadIdx.y * npad + threadIdx.x] = Dg[threadIdx.y * NB + threadIdx.x];
}

// Trailing update: A[i][j] -= sum_k A[i][k] A[j][k] over the kw finished columns from k0 (kw a multiple of
// 32), for rows i >= j >= base and columns j < col_end; 64x64 tiles of the lower triangle counted from
// `base`.  The factorisation calls it twice per 32 columns' worth of work: narrowly (kw = 32) for the
// columns that remain inside the current 128-column panel, and once per panel (kw = 128) for everything to
// the right of it, so that the large trailing matrix is read and written once per 128 columns.
__global__ void __launch_bounds__(256) syrk_kernel(double* __restrict__ A, int npad, int k0, int kw, int base,
                                                   int col_end)
{
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (tj > ti) return;
    const int g = blockIdx.z;
    double* Ag = A + (size_t)g * npad * npad;
    __shared__ double pi[64][NB + 1], pj[64][NB + 1];
    const int t = threadIdx.x;
    const int ty = t / 16, tx = t % 16;
    double acc[4][4] = {};
    // the next 32 columns of the two operands travel to registers while the current ones are multiplied
    double ri[8], rj[8];
    auto fetch = [&](int kc) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = t + 256 * i;
            const int r = e / NB, c = e % NB;
            const int gi = base + ti * 64 + r, gj = base + tj * 64 + r;
            ri[i] = (gi < npad) ? Ag[(size_t)gi * npad + k0 + kc + c] : 0.0;
            rj[i] = (gj < npad) ? Ag[(size_t)gj * npad + k0 + kc + c] : 0.0;
        }
    };
    fetch(0);
    for (int kc = 0; kc < kw; kc += NB) {
        if (kc > 0) __syncthreads();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int e = t + 256 * i;
            pi[e / NB][e % NB] = ri[i];
            pj[e / NB][e % NB] = rj[i];
        }
        __syncthreads();
        if (kc + NB < kw) fetch(kc + NB);
#pragma unroll 8
        for (int k = 0; k < NB; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a[u] = pi[ty + 16 * u][k];
                b[u] = pj[tx + 16 * u][k];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] += a[u] * b[v];
        }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            int gi = base + ti * 64 + ty + 16 * u, gj = base + tj * 64 + tx + 16 * v;
            if (gi < npad && gj <= gi && gj < col_end) Ag[(size_t)gi * npad + gj] -= acc[u][v];
        }
}

// ------------------------------------------------------------------------------------ inverse
__global__ void scatter_dinv_kernel(const double* __restrict__ Dinv, int npad, double* __restrict__ W)
{
    // W = block-diag(Dinv): one 32x32 block per blockIdx.x, GP per blockIdx.y; rest zero already
    const int g = blockIdx.y, b = blockIdx.x;
    const double* Dg = Dinv + ((size_t)g * (npad / NB) + b) * NB * NB;
    double* Wg = W + (size_t)g * npad * npad + (size_t)(b * NB) * npad + b * NB;
    Wg[(size_t)threadIdx.y * npad + threadIdx.x] = Dg[threadIdx.y * NB + threadIdx.x];
}

// Batched FP64 GEMM used by the recursive-doubling inverse.  For pair p (blockIdx.z % npairs) of
// GP g (blockIdx.z / npairs), with block size s:  rows2 = [(2p+1)s, min((2p+2)s, npad)),
// cols1 = [2p s, (2p+1)s).
//   mode 0:  T[rows2][cols1]  =  L[rows2][cols1] * W[cols1][cols1]     (W11 lower: k >= j)
//   mode 1:  W[rows2][cols1]  = -W[rows2][rows2] * T[rows2][cols1]     (W22 lower: k <= i)
__global__ void __launch_bounds__(256) trtri_gemm_kernel(const double* __restrict__ Amat,
                                                         const double* __restrict__ Bmat,
                                                         double* __restrict__ Cmat, int npad, int s,
                                                         int npairs, int mode)
{
    const int p = blockIdx.z % npairs, g = blockIdx.z / npairs;
    const int row2 = (2 * p + 1) * s, col1 = 2 * p * s;
    const int M = min(s, npad - row2);
    const int N = s;
    const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    if (i0 >= M || j0 >= N) return;
    const size_t gs = (size_t)g * npad * npad;
    const double* A;
    const double* B;
    double* C = Cmat + gs + (size_t)row2 * npad + col1;
    int K, kbeg, kend;
    if (mode == 0) {
        A = Amat + gs + (size_t)row2 * npad + col1;
        B = Bmat + gs + (size_t)col1 * npad + col1;
        K = s;
        kbeg = j0;  // W11[k][j] == 0 for k < j
        kend = K;
    } else {
        A = Amat + gs + (size_t)row2 * npad + row2;
        B = Bmat + gs + (size_t)row2 * npad + col1;
        K = M;
        kbeg = 0;
        kend = min(K, i0 + 64);  // W22[i][k] == 0 for k > i
    }
    __shared__ double sa[64][17], sb[16][65];
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    double acc[4][4] = {};
    // the next 16 columns of A and rows of B travel from global memory to registers while the current ones are
    // multiplied out of shared memory
    double ra[4], rb[4];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = t + 256 * i;
            const int r = e / 16, c = e % 16;
            ra[i] = (i0 + r < M && k0 + c < K) ? A[(size_t)(i0 + r) * npad + k0 + c] : 0.0;
            const int rr = e / 64, cc = e % 64;
            rb[i] = (k0 + rr < K && j0 + cc < N) ? B[(size_t)(k0 + rr) * npad + j0 + cc] : 0.0;
        }
    };
    if (kbeg < kend) fetch(kbeg);
    for (int k0 = kbeg; k0 < kend; k0 += 16) {
        if (k0 > kbeg) __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = t + 256 * i;
            sa[e / 16][e % 16] = ra[i];
            sb[e / 64][e % 64] = rb[i];
        }
        __syncthreads();
        if (k0 + 16 < kend) fetch(k0 + 16);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a[u] = sa[ty + 16 * u][k];
                b[u] = sb[k][tx + 16 * u];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] += a[u] * b[v];
        }
    }
    const double sign = mode == 0 ? 1.0 : -1.0;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            int i = i0 + ty + 16 * u, j = j0 + tx + 16 * v;
            if (i < M && j < N) C[(size_t)i * npad + j] = sign * acc[u][v];
        }
}

// ------------------------------------------------------------------------------------ weights
// u = W y (lower-triangular W, one warp per row); rows >= n give 0.
template <typename T>
__global__ void w_times_y_kernel(const double* __restrict__ W, const T* __restrict__ y, int ystride, int n,
                                 int npad, double* __restrict__ u)
{
    const int g = blockIdx.y;
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (row >= npad) return;
    const double* Wr = W + (size_t)g * npad * npad + (size_t)row * npad;
    double s = 0.0;
    if (row < n)
        for (int k = lane; k <= row; k += 32) s += Wr[k] * (double)y[(size_t)g * ystride + k];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) u[(size_t)g * npad + row] = s;
}

// alpha = W^T u in two steps so that n = 4096 still fills the GPU: the rows are cut into kRowSlabs
// slabs, each block sums one slab for 128 columns (coalesced across columns), then the slabs are added
// in a fixed order (deterministic).
constexpr int kRowSlabs = 32;
__global__ void wt_times_u_partial_kernel(const double* __restrict__ W, const double* __restrict__ u, int n,
                                          int npad, double* __restrict__ partial)
{
    const int g = blockIdx.z, slab = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= npad) return;
    const int rows = (npad + kRowSlabs - 1) / kRowSlabs;
    const int i0 = max(slab * rows, j), i1 = min(min((slab + 1) * rows, npad), n);
    const double* Wg = W + (size_t)g * npad * npad;
    double s = 0.0;
    if (j < n)
        for (int i = i0; i < i1; ++i) s += Wg[(size_t)i * npad + j] * u[(size_t)g * npad + i];
    partial[((size_t)g * kRowSlabs + slab) * npad + j] = s;
}

__global__ void wt_times_u_reduce_kernel(const double* __restrict__ partial, int npad,
                                         double* __restrict__ alpha64, float* __restrict__ alpha32)
{
    const int g = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= npad) return;
    double s = 0.0;
    for (int r = 0; r < kRowSlabs; ++r) s += partial[((size_t)g * kRowSlabs + r) * npad + j];
    alpha64[(size_t)g * npad + j] = s;
    alpha32[(size_t)g * npad + j] = (float)s;
}

// Power iteration on W^T W: v holds the current vector (unit norm after the call), lam its norm
// before normalisation, i.e. the current estimate of |W|_2^2.
__global__ void power_init_kernel(double* __restrict__ v, int n, int npad)
{
    const int g = blockIdx.x;
    for (int i = threadIdx.x; i < npad; i += blockDim.x)
        v[(size_t)g * npad + i] = (i < n) ? (1.0 + 0.37 * ((i * 2654435761u >> 16) & 0xff) / 255.0) : 0.0;
}

__global__ void power_normalize_kernel(double* __restrict__ v, int npad, double* __restrict__ lam)
{
    __shared__ double s[256];
    const int g = blockIdx.x;
    double* vg = v + (size_t)g * npad;
    double acc = 0.0;
    for (int i = threadIdx.x; i < npad; i += 256) acc += vg[i] * vg[i];
    s[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    const double nrm = sqrt(s[0]);
    if (threadIdx.x == 0) lam[g] = nrm;
    const double inv = nrm > 0.0 ? 1.0 / nrm : 0.0;
    for (int i = threadIdx.x; i < npad; i += 256) vg[i] *= inv;
}

__global__ void power_finish_kernel(const double* __restrict__ lam, double* __restrict__ wnorm, int batch)
{
    // lam ~ |W|_2^2 from below; 1.5 covers slow convergence
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g < batch) wnorm[g] = 1.5 * sqrt(lam[g]);
}

__global__ void to_float_kernel(const double* __restrict__ a, float* __restrict__ b, size_t count)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count;
         i += (size_t)gridDim.x * blockDim.x)
        b[i] = (float)a[i];
}

// From W and y: the estimate of |W|_2 (power iteration on W^T W; alpha64/alpha32 serve as scratch first),
// alpha = W^T (W y) in FP64 and FP32, and W rounded to FP32.  u: [B][npad] scratch; slabs: [B + B*kRowSlabs*npad].
r3_status_t finish_weights(int B, int n, int npad, const double* W64, const float* y, double* alpha64, float* alpha32,
                           float* W32, double* wnorm_d, double* u, double* slabs, cudaStream_t stream)
{
    double* pv = alpha64;
    double* lam = slabs;  // [B], followed by the row-slab partial sums
    double* part = slabs + B;
    R3_LAUNCH(power_init_kernel, B, 256, 0, stream, pv, n, npad);
    R3_LAUNCH(power_normalize_kernel, B, 256, 0, stream, pv, npad, lam);
    for (int it = 0; it < 12; ++it) {
        R3_LAUNCH(w_times_y_kernel<double>, dim3((npad + 7) / 8, B), 256, 0, stream, W64, pv, npad, n, npad, u);
        R3_LAUNCH(wt_times_u_partial_kernel, dim3((npad + 127) / 128, kRowSlabs, B), 128, 0, stream, W64, u, n, npad,
                  part);
        R3_LAUNCH(wt_times_u_reduce_kernel, dim3((npad + 127) / 128, B), 128, 0, stream, part, npad, pv, alpha32);
        R3_LAUNCH(power_normalize_kernel, B, 256, 0, stream, pv, npad, lam);
    }
    R3_LAUNCH(power_finish_kernel, (B + 255) / 256, 256, 0, stream, lam, wnorm_d, B);
    R3_LAUNCH(w_times_y_kernel<float>, dim3((npad + 7) / 8, B), 256, 0, stream, W64, y, n, n, npad, u);
    R3_LAUNCH(wt_times_u_partial_kernel, dim3((npad + 127) / 128, kRowSlabs, B), 128, 0, stream, W64, u, n, npad, part);
    R3_LAUNCH(wt_times_u_reduce_kernel, dim3((npad + 127) / 128, B), 128, 0, stream, part, npad, alpha64, alpha32);
    R3_LAUNCH(to_float_kernel, 1184, 256, 0, stream, W64, W32, (size_t)B * npad * npad);
    return R3_OK;
}

}  // namespace

// Runs the whole fit on `stream`.  gp->X, ell (device copies) and the scalar arrays are already in
// place; L64, W64, W32, alpha*, best_d are filled.  The caller synchronises and reads status_d.
r3_status_t fit_device(r3_gp* gp, const float* y, cudaStream_t stream)
{
    const int B = gp->batch, n = gp->n, d = gp->d, npad = gp->npad;
    const size_t mat = (size_t)npad * npad;
    double *Dinv = nullptr, *Ldiag = nullptr, *T = nullptr, *u = nullptr, *slabs = nullptr;
    // stream and events of the factorisation's look-ahead (see the panel loop)
    cudaStream_t aux = nullptr;
    cudaEvent_t panel_done = nullptr, wide_done = nullptr;
    R3_CUDA_TRY(dev_malloc(&Dinv, sizeof(double) * B * (size_t)(npad / NB) * NB * NB));
    auto fail = [&](r3_status_t st) {
        if (aux) {
            cudaStreamSynchronize(aux);
            cudaStreamDestroy(aux);
        }
        if (panel_done) cudaEventDestroy(panel_done);
        if (wide_done) cudaEventDestroy(wide_done);
        dev_free(Dinv);
        dev_free(Ldiag);
        dev_free(T);
        dev_free(u);
        dev_free(slabs);
        return st;
    };
#define TRY_OR_FAIL(expr)                                                                          \
    do {                                                                                           \
        cudaError_t e__ = (expr);                                                                  \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("%s failed: %s", #expr, cudaGetErrorString(e__));                            \
            return fail(e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA);            \
        }                                                                                          \
    } while (0)
#define LAUNCH_OR_FAIL(kernel, grid, block, ...)                                                   \
    do {                                                                                           \
        kernel<<<(grid), (block), 0, stream>>>(__VA_ARGS__);                                       \
        ++g_launches;                                                                              \
        cudaError_t e__ = cudaGetLastError();                                                      \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("launch of %s failed: %s", #kernel, cudaGetErrorString(e__));                \
            return fail(R3_ERR_CUDA);                                                              \
        }                                                                                          \
    } while (0)

    TRY_OR_FAIL(dev_malloc(&Ldiag, sizeof(double) * B * (size_t)(npad / NB) * NB * NB));
    TRY_OR_FAIL(dev_malloc(&T, sizeof(double) * B * mat));
    TRY_OR_FAIL(dev_malloc(&u, sizeof(double) * B * npad));
    TRY_OR_FAIL(dev_malloc(&slabs, sizeof(double) * ((size_t)B + (size_t)B * kRowSlabs * npad)));

    LAUNCH_OR_FAIL(check_finite_kernel, 296, 256, gp->X, (size_t)B * n * d, gp->status_d);
    LAUNCH_OR_FAIL(check_finite_kernel, 64, 256, y, (size_t)B * n, gp->status_d);
    LAUNCH_OR_FAIL(min_y_kernel, B, 256, y, n, gp->best_d, gp->yabs_d);

    LAUNCH_OR_FAIL(gram_kernel, dim3(npad / 16, npad / 16, B), dim3(16, 16), gp->X, gp->ell_d, gp->sf2_d,
                   gp->sn2_d, n, d, npad, gp->L64);

    TRY_OR_FAIL(cudaFuncSetAttribute(potrf_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPanelSmem));
    constexpr int kOuter = 4 * NB;   // columns per panel of the two-level right-looking factorisation
    // Look-ahead: a panel's update of everything to its right is split.  The columns of the NEXT panel are updated
    // first, and that panel's factorisation (a chain of eight short dependent launches) follows at once, both on a
    // stream of the highest priority so that their few blocks are placed ahead of the queued blocks of the wide
    // update; the update of the columns beyond -- most of the arithmetic -- runs on the caller's stream meanwhile.
    // The two touch disjoint columns; the next panel's own update waits for the wide one (same elements).
    const bool look_ahead = npad > 2 * kOuter;
    cudaStream_t cs = stream;   // the stream of the chain
    if (look_ahead) {
        int least = 0, greatest = 0;
        TRY_OR_FAIL(cudaDeviceGetStreamPriorityRange(&least, &greatest));
        TRY_OR_FAIL(cudaStreamCreateWithPriority(&aux, cudaStreamNonBlocking, greatest));
        TRY_OR_FAIL(cudaEventCreateWithFlags(&panel_done, cudaEventDisableTiming));
        TRY_OR_FAIL(cudaEventCreateWithFlags(&wide_done, cudaEventDisableTiming));
        cs = aux;
        TRY_OR_FAIL(cudaEventRecord(wide_done, stream));   // the Gram matrix is ready
        TRY_OR_FAIL(cudaStreamWaitEvent(cs, wide_done, 0));
    }
#define CHAIN_LAUNCH(kernel, grid, block, smem, ...)                                               \
    do {                                                                                           \
        kernel<<<(grid), (block), (smem), cs>>>(__VA_ARGS__);                                      \
        ++g_launches;                                                                              \
        cudaError_t e__ = cudaGetLastError();                                                      \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("launch of %s failed: %s", #kernel, cudaGetErrorString(e__));                \
            return fail(R3_ERR_CUDA);                                                              \
        }                                                                                          \
    } while (0)
    bool wide_pending = false;
    for (int J = 0; J < npad; J += kOuter) {
        const int panel_end = std::min(J + kOuter, npad);
        for (int j0 = J; j0 < panel_end; j0 += NB) {
            const int rows = npad - j0 - NB;
            CHAIN_LAUNCH(potrf_panel_kernel, dim3(rows > 0 ? (rows + kPanelThreads - 1) / kPanelThreads : 1, B),
                         dim3(NB, kPanelThreads / NB), kPanelSmem, gp->L64, npad, j0, Dinv, Ldiag, gp->status_d);
            if (rows <= 0) continue;
            const int tiles = (rows + 63) / 64;
            const int inner = panel_end - j0 - NB;   // columns of this panel still to be factored
            if (inner > 0)
                CHAIN_LAUNCH(syrk_kernel, dim3((inner + 63) / 64, tiles, B), 256, 0, gp->L64, npad, j0, NB, j0 + NB, panel_end);
        }
        const int rows = npad - panel_end;
        if (rows <= 0) continue;
        const int tiles = (rows + 63) / 64;
        if (!look_ahead) {
            LAUNCH_OR_FAIL(syrk_kernel, dim3(tiles, tiles, B), 256, gp->L64, npad, J, panel_end - J, panel_end, npad);
            continue;
        }
        TRY_OR_FAIL(cudaEventRecord(panel_done, cs));
        if (wide_pending) TRY_OR_FAIL(cudaStreamWaitEvent(cs, wide_done, 0));
        const int next_cols = std::min(kOuter, rows);
        CHAIN_LAUNCH(syrk_kernel, dim3((next_cols + 63) / 64, tiles, B), 256, 0, gp->L64, npad, J, panel_end - J, panel_end,
                     panel_end + next_cols);
        const int wide = rows - next_cols;
        if (wide > 0) {
            const int wtiles = (wide + 63) / 64;
            TRY_OR_FAIL(cudaStreamWaitEvent(stream, panel_done, 0));
            LAUNCH_OR_FAIL(syrk_kernel, dim3(wtiles, wtiles, B), 256, gp->L64, npad, J, panel_end - J, panel_end + next_cols,
                           npad);
            TRY_OR_FAIL(cudaEventRecord(wide_done, stream));
            wide_pending = true;
        }
    }
#undef CHAIN_LAUNCH
    if (look_ahead) {   // the caller's stream goes on when the chain has ended
        TRY_OR_FAIL(cudaEventRecord(panel_done, cs));
        TRY_OR_FAIL(cudaStreamWaitEvent(stream, panel_done, 0));
    }

    LAUNCH_OR_FAIL(scatter_ldiag_kernel, dim3(npad / NB, B), dim3(NB, NB), Ldiag, npad, gp->L64);
    TRY_OR_FAIL(cudaMemsetAsync(gp->W64, 0, sizeof(double) * B * mat, stream));
    LAUNCH_OR_FAIL(scatter_dinv_kernel, dim3(npad / NB, B), dim3(NB, NB), Dinv, npad, gp->W64);
    for (int s = NB; s < npad; s *= 2) {
        const int npairs = (npad + 2 * s - 1) / (2 * s);   // a last lone block has M <= 0 and exits
        const int tiles = (s + 63) / 64;
        dim3 grid(tiles, tiles, npairs * B);
        LAUNCH_OR_FAIL(trtri_gemm_kernel, grid, 256, gp->L64, gp->W64, T, npad, s, npairs, 0);
        LAUNCH_OR_FAIL(trtri_gemm_kernel, grid, 256, gp->W64, T, gp->W64, npad, s, npairs, 1);
    }

    {
        const r3_status_t st = finish_weights(B, n, npad, gp->W64, y, gp->alpha64, gp->alpha32, gp->W32, gp->wnorm_d, u,
                                              slabs, stream);
        if (st != R3_OK) return fail(st);
    }
    TRY_OR_FAIL(cudaMemcpyAsync(gp->status_h, gp->status_d, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    TRY_OR_FAIL(cudaStreamSynchronize(stream));
#undef TRY_OR_FAIL
#undef LAUNCH_OR_FAIL
    fail(R3_OK);  // frees the temporaries
    return R3_OK;
}

// =====================================================================================================
// r3_gp_append: k more observations per GP without refactoring what is already factored.
//
// With K' = [[K, B], [B^T, C]] (B = k(X, Xnew), C = k(Xnew, Xnew) + noise*I) and K = L L^T, W = L^-1:
//     L21 = (W B)^T,   S = C - L21 L21^T = L22 L22^T,   L' = [[L, 0], [L21, L22]],
//     W22 = L22^-1,    W21 = -W22 (L21 W),              W' = [[W, 0], [W21, W22]],
// then alpha' = W'^T (W' y') as in the fit.  Two k x n x n/2 products in FP64 dominate: O(k n^2) against
// the fit's O(n^3 / 3).  The results equal a fit of the concatenated history up to rounding.
namespace {

// k <= kAppendMax (r3_internal.cuh): S and W22 are handled by one block per GP

// Copy the leading n0 x n0 blocks of the old matrices into the (zeroed) new ones and put the identity
// on the padding rows.
__global__ void embed_kernel(const double* __restrict__ src, int np0, double* __restrict__ dst, int np1, int n0, int n1)
{
    const int g = blockIdx.y;
    const int i = blockIdx.x;
    const double* s = src + (size_t)g * np0 * np0 + (size_t)i * np0;
    double* t = dst + (size_t)g * np1 * np1 + (size_t)i * np1;
    if (i < n0) {
        for (int c = threadIdx.x; c <= i; c += blockDim.x) t[c] = s[c];
    } else if (i >= n1 && threadIdx.x == 0) {
        t[i] = 1.0;
    }
}

// Rows of the new observations of K' (lower triangle): row n0 + i, columns 0 .. n0 + i.
__global__ void cross_gram_kernel(const float* __restrict__ X, const float* __restrict__ ell,
                                  const float* __restrict__ sf2, const float* __restrict__ sn2, int n0, int n1, int d,
                                  int np1, double* __restrict__ K)
{
    const int g = blockIdx.z, i = n0 + blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c > i) return;
    const float* Xg = X + (size_t)g * n1 * d;
    const float* xi = Xg + (size_t)i * d;
    const float* xc = Xg + (size_t)c * d;
    const float* lg = ell + (size_t)g * d;
    double r2 = 0.0;
    for (int j = 0; j < d; ++j) {
        const double diff = ((double)xi[j] - (double)xc[j]) * (1.0 / (double)lg[j]);   // as gram_kernel does
        r2 += diff * diff;
    }
    const double s = sqrt(5.0) * sqrt(r2);
    double v = (double)sf2[g] * (1.0 + s + s * s / 3.0) * exp(-s);
    if (c == i) v += (double)sn2[g];
    K[(size_t)g * np1 * np1 + (size_t)i * np1 + c] = v;
}

// S[i][j] = C[i][j] - sum_c L21[i][c] L21[j][c] for j <= i, written over the C block of L' (one warp per entry).
__global__ void schur_kernel(const double* __restrict__ L21, int n0, int k, double* __restrict__ Lnew, int np1)
{
    const int g = blockIdx.z, i = blockIdx.y;
    const int j = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (j > i) return;
    const double* a = L21 + ((size_t)g * k + i) * n0;
    const double* b = L21 + ((size_t)g * k + j) * n0;
    double s = 0.0;
    for (int c = lane; c < n0; c += 32) s = fma(a[c], b[c], s);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) Lnew[(size_t)g * np1 * np1 + (size_t)(n0 + i) * np1 + n0 + j] -= s;
}

// Cholesky of the k x k block at (n0, n0) of L' (in place) and its inverse into W' (one block per GP, k <= 128).
// Both triangles live in shared memory, packed by rows (entry (i, c), c <= i, at i (i + 1) / 2 + c).
// Factor: one barrier per column -- every thread forms r = 1 / sqrt(s_jj) itself and scales what it reads of
// column j by it, the column itself stays unscaled until the end (as in the fit's diagonal blocks).  Inverse:
// forward substitution L22 v = e_c, one column per thread, out of shared memory.
__global__ void __launch_bounds__(256) small_chol_inv_kernel(double* __restrict__ Lnew, double* __restrict__ Wnew,
                                                              int np1, int n0, int k, int* __restrict__ status)
{
    const int g = blockIdx.x;
    double* S = Lnew + (size_t)g * np1 * np1 + (size_t)n0 * np1 + n0;   // S[i][j] at S[i * np1 + j]
    double* V = Wnew + (size_t)g * np1 * np1 + (size_t)n0 * np1 + n0;
    extern __shared__ double tri[];            // packed S, then packed V, then r_j
    const int nt = k * (k + 1) / 2;
    double* s = tri;
    double* v = tri + nt;
    double* rj = v + nt;
    auto at = [](int i, int c) { return i * (i + 1) / 2 + c; };
    for (int e = threadIdx.x; e < k * k; e += blockDim.x) {
        const int i = e / k, c = e % k;
        if (c <= i) s[at(i, c)] = S[(size_t)i * np1 + c];
    }
    __syncthreads();
    for (int j = 0; j < k; ++j) {
        double piv = s[at(j, j)];
        if (!(piv > 0.0)) {
            if (threadIdx.x == 0) {
                atomicOr(&status[0], DEV_NOT_PD);
                atomicMin(&status[1], n0 + j);
            }
            piv = 1.0;
        }
        const double r = rsqrt(piv);
        if (threadIdx.x == 0) rj[j] = r;
        // trailing update of the lower triangle: rows i > j, columns j < c <= i
        const int w = k - j - 1;
        for (int e = threadIdx.x; e < w * w; e += blockDim.x) {
            const int i = j + 1 + e / w, c = j + 1 + e % w;
            if (c <= i) s[at(i, c)] -= (s[at(i, j)] * r) * (s[at(c, j)] * r);
        }
        __syncthreads();
    }
    // scale the columns, diagonal = sqrt(pivot) from its reciprocal root with one correction step
    for (int e = threadIdx.x; e < k * k; e += blockDim.x) {
        const int i = e / k, c = e % k;
        if (c > i) continue;
        double val;
        if (c == i) {
            double p = s[at(i, i)];
            if (!(p > 0.0)) p = 1.0;
            const double sq = p * rj[i];
            val = fma(0.5 * rj[i], fma(-sq, sq, p), sq);
        } else {
            val = s[at(i, c)] * rj[c];
        }
        S[(size_t)i * np1 + c] = val;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < k * k; e += blockDim.x) {   // the factor itself into shared memory
        const int i = e / k, c = e % k;
        if (c <= i) s[at(i, c)] = S[(size_t)i * np1 + c];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < k; c += blockDim.x) {
        v[at(c, c)] = 1.0 / s[at(c, c)];
        for (int i = c + 1; i < k; ++i) {
            double acc = 0.0;
            for (int j = c; j < i; ++j) acc = fma(s[at(i, j)], v[at(j, c)], acc);
            v[at(i, c)] = -acc / s[at(i, i)];
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < k * k; e += blockDim.x) {
        const int i = e / k, c = e % k;
        if (c <= i) V[(size_t)i * np1 + c] = v[at(i, c)];
    }
}

// Rows of L' : copy L21 [k][n0] into rows n0.. of L'.  Rows of W' : W21 = -W22 T2.
__global__ void place_l21_kernel(const double* __restrict__ L21, int n0, int k, double* __restrict__ Lnew, int np1)
{
    const int g = blockIdx.z, i = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < n0) Lnew[(size_t)g * np1 * np1 + (size_t)(n0 + i) * np1 + c] = L21[((size_t)g * k + i) * n0 + c];
}

__global__ void w21_kernel(const double* __restrict__ T2, int n0, int k, double* __restrict__ Wnew, int np1)
{
    const int g = blockIdx.z, i = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n0) return;
    const double* W22 = Wnew + (size_t)g * np1 * np1 + (size_t)(n0 + i) * np1 + n0;   // row i of W22
    const double* T = T2 + (size_t)g * k * n0;
    double s = 0.0;
    for (int j = 0; j <= i; ++j) s = fma(W22[j], T[(size_t)j * n0 + c], s);
    Wnew[(size_t)g * np1 * np1 + (size_t)(n0 + i) * np1 + c] = -s;
}

// T = Bt - T for the k new rows (Bt: rows n0.. of the extended matrix, leading dimension np1; T: [k][n0])
__global__ void l21_residual_kernel(const double* __restrict__ Kext, int np1, int n0, int k, double* __restrict__ T)
{
    const int g = blockIdx.z, i = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n0) return;
    const size_t e = ((size_t)g * k + i) * n0 + c;
    T[e] = Kext[(size_t)g * np1 * np1 + (size_t)(n0 + i) * np1 + c] - T[e];
}

__global__ void add_rows_kernel(const double* __restrict__ D, size_t total, double* __restrict__ T)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < total) T[e] += D[e];
}

struct AppendBuffers {
    float *X = nullptr, *y = nullptr, *W32 = nullptr, *alpha32 = nullptr, *best = nullptr;   // best: [2][B]
    double *L64 = nullptr, *W64 = nullptr, *alpha64 = nullptr, *T1 = nullptr, *T2 = nullptr, *T3 = nullptr, *u = nullptr,
           *slabs = nullptr, *wnorm = nullptr;
    void release()
    {
        dev_free(X); dev_free(y); dev_free(W32); dev_free(alpha32); dev_free(L64); dev_free(W64); dev_free(alpha64);
        dev_free(T1); dev_free(T2); dev_free(T3); dev_free(u); dev_free(slabs); dev_free(best); dev_free(wnorm);
        *this = AppendBuffers();
    }
};

}  // namespace

r3_status_t append_device(r3_gp* gp, const float* Xnew, const float* ynew, int k, cudaStream_t stream)
{
    const size_t xnew_gp_stride = (size_t)k * gp->d, ynew_gp_stride = (size_t)k;
    const int B = gp->batch, d = gp->d, n0 = gp->n, n1 = n0 + k, np0 = gp->npad, np1 = round_up(n1, NB);
    const size_t mat1 = (size_t)np1 * np1;
    AppendBuffers nb;
    auto fail = [&](r3_status_t st) {
        nb.release();
        return st;
    };
#define TRY_OR_FAIL(expr)                                                                          \
    do {                                                                                           \
        cudaError_t e__ = (expr);                                                                  \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("%s failed: %s", #expr, cudaGetErrorString(e__));                            \
            return fail(e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA);            \
        }                                                                                          \
    } while (0)
#define LAUNCH_OR_FAIL(kernel, grid, block, ...)                                                   \
    do {                                                                                           \
        kernel<<<(grid), (block), 0, stream>>>(__VA_ARGS__);                                       \
        ++g_launches;                                                                              \
        cudaError_t e__ = cudaGetLastError();                                                      \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("launch of %s failed: %s", #kernel, cudaGetErrorString(e__));                \
            return fail(R3_ERR_CUDA);                                                              \
        }                                                                                          \
    } while (0)
    TRY_OR_FAIL(dev_malloc(&nb.X, sizeof(float) * B * (size_t)n1 * d));
    TRY_OR_FAIL(dev_malloc(&nb.y, sizeof(float) * B * (size_t)n1));
    TRY_OR_FAIL(dev_malloc(&nb.L64, sizeof(double) * B * mat1));
    TRY_OR_FAIL(dev_malloc(&nb.W64, sizeof(double) * B * mat1));
    TRY_OR_FAIL(dev_malloc(&nb.W32, sizeof(float) * B * mat1));
    TRY_OR_FAIL(dev_malloc(&nb.alpha64, sizeof(double) * B * np1));
    TRY_OR_FAIL(dev_malloc(&nb.alpha32, sizeof(float) * B * np1));
    // the triangular products of few rows are cut along their reductions so that they fill the GPU
    const dim3 ggrid0((n0 + 63) / 64, (k + 31) / 32, B);
    const size_t blocks0 = (size_t)ggrid0.x * ggrid0.y * ggrid0.z;
    const int splits = blocks0 >= 2 * 148 ? 1 : (int)std::min<size_t>(8, (6 * 148 + blocks0 - 1) / blocks0);
    const size_t part = (size_t)B * k * n0;   // doubles of one [B][k][n0] array: the parts of a product lie this far apart
    TRY_OR_FAIL(dev_malloc(&nb.T1, sizeof(double) * part * splits));
    TRY_OR_FAIL(dev_malloc(&nb.T2, sizeof(double) * part * splits));
    TRY_OR_FAIL(dev_malloc(&nb.u, sizeof(double) * B * np1));
    TRY_OR_FAIL(dev_malloc(&nb.slabs, sizeof(double) * ((size_t)B + (size_t)B * kRowSlabs * np1)));
    TRY_OR_FAIL(dev_malloc(&nb.best, sizeof(float) * 2 * B));
    TRY_OR_FAIL(dev_malloc(&nb.wnorm, sizeof(double) * B));
    LAUNCH_OR_FAIL(check_finite_kernel, 64, 256, Xnew, (size_t)B * k * d, gp->status_d);
    LAUNCH_OR_FAIL(check_finite_kernel, 64, 256, ynew, (size_t)B * k, gp->status_d);

    // histories: old rows then new rows, per GP
    TRY_OR_FAIL(cudaMemcpy2DAsync(nb.X, sizeof(float) * (size_t)n1 * d, gp->X, sizeof(float) * (size_t)n0 * d,
                                  sizeof(float) * (size_t)n0 * d, B, cudaMemcpyDeviceToDevice, stream));
    TRY_OR_FAIL(cudaMemcpy2DAsync(nb.X + (size_t)n0 * d, sizeof(float) * (size_t)n1 * d, Xnew,
                                  sizeof(float) * xnew_gp_stride, sizeof(float) * (size_t)k * d, B,
                                  cudaMemcpyDeviceToDevice, stream));
    TRY_OR_FAIL(cudaMemcpy2DAsync(nb.y, sizeof(float) * n1, gp->y, sizeof(float) * n0, sizeof(float) * n0, B,
                                  cudaMemcpyDeviceToDevice, stream));
    TRY_OR_FAIL(cudaMemcpy2DAsync(nb.y + n0, sizeof(float) * n1, ynew, sizeof(float) * ynew_gp_stride, sizeof(float) * k,
                                  B, cudaMemcpyDeviceToDevice, stream));
    TRY_OR_FAIL(cudaMemsetAsync(nb.L64, 0, sizeof(double) * B * mat1, stream));
    TRY_OR_FAIL(cudaMemsetAsync(nb.W64, 0, sizeof(double) * B * mat1, stream));
    LAUNCH_OR_FAIL(embed_kernel, dim3(np1, B), 128, gp->L64, np0, nb.L64, np1, n0, n1);
    LAUNCH_OR_FAIL(embed_kernel, dim3(np1, B), 128, gp->W64, np0, nb.W64, np1, n0, n1);
    LAUNCH_OR_FAIL(min_y_kernel, B, 256, nb.y, n1, nb.best, nb.best + B);

    // new rows of K', then L21 = B^T W^T
    LAUNCH_OR_FAIL(cross_gram_kernel, dim3((n1 + 127) / 128, k, B), 128, nb.X, gp->ell_d, gp->sf2_d, gp->sn2_d, n0, n1,
                   d, np1, nb.L64);
    const dim3 ggrid((n0 + 63) / 64, (k + 31) / 32, B * splits);
    const dim3 sgrid((unsigned)(((size_t)k * n0 + 255) / 256), B);
    LAUNCH_OR_FAIL(tri_gemm_kernel<true>, ggrid, 256, nb.L64 + (size_t)n0 * np1, np1, mat1, nb.W64, np1, mat1, nb.T1,
                   n0, (size_t)k * n0, k, n0, splits, part);
    if (splits > 1) LAUNCH_OR_FAIL(tri_gemm_sum_kernel, sgrid, 256, nb.T1, (size_t)k * n0, (size_t)k * n0, splits, part);
    // The product with the explicit inverse is as accurate as a triangular solve only while K is well
    // conditioned (its error is relative to |B| |W|, not to L21).  Beyond cond(K) of about 1e8 -- estimated by
    // |W|_2^2 (sigma_f^2 + sigma_n^2) -- one step of iterative refinement with the factor itself follows:
    // R = B^T - L21 L^T, L21 += R W^T.  Without it the Schur complement of a noise-free smooth history came out
    // indefinite where a fit of the whole history succeeds.
    bool refine = false;
    for (int g = 0; g < B; ++g)
        refine |= gp->wnorm[g] * gp->wnorm[g] * ((double)gp->sf2[g] + (double)gp->sn2[g]) > 1e8;
    if (refine) {
        TRY_OR_FAIL(dev_malloc(&nb.T3, sizeof(double) * part * splits));
        LAUNCH_OR_FAIL(tri_gemm_kernel<true>, ggrid, 256, nb.T1, n0, (size_t)k * n0, nb.L64, np1, mat1, nb.T2, n0,
                       (size_t)k * n0, k, n0, splits, part);
        if (splits > 1)
            LAUNCH_OR_FAIL(tri_gemm_sum_kernel, sgrid, 256, nb.T2, (size_t)k * n0, (size_t)k * n0, splits, part);
        LAUNCH_OR_FAIL(l21_residual_kernel, dim3((n0 + 127) / 128, k, B), 128, nb.L64, np1, n0, k, nb.T2);
        LAUNCH_OR_FAIL(tri_gemm_kernel<true>, ggrid, 256, nb.T2, n0, (size_t)k * n0, nb.W64, np1, mat1, nb.T3, n0,
                       (size_t)k * n0, k, n0, splits, part);
        if (splits > 1)
            LAUNCH_OR_FAIL(tri_gemm_sum_kernel, sgrid, 256, nb.T3, (size_t)k * n0, (size_t)k * n0, splits, part);
        const size_t total = (size_t)B * k * n0;
        LAUNCH_OR_FAIL(add_rows_kernel, (unsigned)((total + 255) / 256), 256, nb.T3, total, nb.T1);
    }
    LAUNCH_OR_FAIL(place_l21_kernel, dim3((n0 + 127) / 128, k, B), 128, nb.T1, n0, k, nb.L64, np1);
    LAUNCH_OR_FAIL(schur_kernel, dim3((k + 7) / 8, k, B), 256, nb.T1, n0, k, nb.L64, np1);
    {
        const size_t smem = sizeof(double) * ((size_t)k * (k + 1) + k);
        TRY_OR_FAIL(cudaFuncSetAttribute(small_chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        small_chol_inv_kernel<<<B, 256, smem, stream>>>(nb.L64, nb.W64, np1, n0, k, gp->status_d);
        ++g_launches;
        TRY_OR_FAIL(cudaGetLastError());
    }
    // W21 = -W22 (L21 W)
    LAUNCH_OR_FAIL(tri_gemm_kernel<false>, ggrid, 256, nb.T1, n0, (size_t)k * n0, nb.W64, np1, mat1, nb.T2, n0,
                   (size_t)k * n0, k, n0, splits, part);
    if (splits > 1) LAUNCH_OR_FAIL(tri_gemm_sum_kernel, sgrid, 256, nb.T2, (size_t)k * n0, (size_t)k * n0, splits, part);
    LAUNCH_OR_FAIL(w21_kernel, dim3((n0 + 127) / 128, k, B), 128, nb.T2, n0, k, nb.W64, np1);
    {
        const r3_status_t st = finish_weights(B, n1, np1, nb.W64, nb.y, nb.alpha64, nb.alpha32, nb.W32, nb.wnorm,
                                              nb.u, nb.slabs, stream);
        if (st != R3_OK) return fail(st);
    }
    TRY_OR_FAIL(cudaMemcpyAsync(gp->status_h, gp->status_d, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    TRY_OR_FAIL(cudaStreamSynchronize(stream));
#undef TRY_OR_FAIL
#undef LAUNCH_OR_FAIL
    if (gp->status_h[0] & (DEV_NOT_PD | DEV_NONFINITE)) return fail(R3_OK);   // the caller reports; nothing swapped
    // success: the new arrays replace the old ones
    if (cudaMemcpy(gp->best_d, nb.best, sizeof(float) * B, cudaMemcpyDeviceToDevice) != cudaSuccess ||
        cudaMemcpy(gp->yabs_d, nb.best + B, sizeof(float) * B, cudaMemcpyDeviceToDevice) != cudaSuccess ||
        cudaMemcpy(gp->wnorm_d, nb.wnorm, sizeof(double) * B, cudaMemcpyDeviceToDevice) != cudaSuccess) {
        set_error("r3_gp_append: copying the incumbent failed");
        return fail(R3_ERR_CUDA);
    }
    dev_free(gp->X); dev_free(gp->y); dev_free(gp->L64); dev_free(gp->W64); dev_free(gp->W32);
    dev_free(gp->alpha64); dev_free(gp->alpha32);
    gp->X = nb.X; gp->y = nb.y; gp->L64 = nb.L64; gp->W64 = nb.W64; gp->W32 = nb.W32;
    gp->alpha64 = nb.alpha64; gp->alpha32 = nb.alpha32;
    nb.X = nullptr; nb.y = nullptr; nb.L64 = nullptr; nb.W64 = nullptr; nb.W32 = nullptr;
    nb.alpha64 = nullptr; nb.alpha32 = nullptr;
    nb.release();
    gp->n = n1;
    gp->npad = np1;
    return R3_OK;
}

}  // namespace r3
