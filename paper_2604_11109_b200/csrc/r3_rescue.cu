// Accuracy guard and FP64 rescue pass.
//
// The scoring engines work at FP32 level.  That is enough for almost every candidate of a
// well-conditioned GP, but not where the posterior variance sf2 - |W k*|^2 is a small difference of
// two numbers close to sf2 (a candidate on top of an observation), nor where mu = k*.alpha cancels
// heavily (an ill-conditioned history with large weights).  Each engine therefore writes, next to
// its results, an estimate of its own rounding error in mu and in q.  Once the whole pool is scored:
//   max_ei_kernel  the largest EI of each GP (the EI tolerance is relative to it)
//   flag_kernel    lists the candidates whose estimated error exceeds half of the accuracy contract
//                  (1e-4 relative on mu and sigma with absolute floors, 1e-5 max(EI) on EI)
//   rescue_kernel  recomputes the listed candidates from the raw inputs entirely in FP64 --
//                  direct-difference distances with a true division by the lengthscale, FP64 weights
//                  and the FP64 inverse factor -- and overwrites their mu, sigma and EI.
#include "r3_epilogue.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr int RESCUE_GROUP = 4;   // candidates per block (they share every read of W)

__global__ void max_ei_kernel(const float* __restrict__ ei, long long m, unsigned* __restrict__ maxbits)
{
    const int g = blockIdx.y;
    const float* e = ei + (size_t)g * m;
    float v = 0.f;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x)
        v = fmaxf(v, e[i]);  // EI >= 0; NaN is ignored by fmaxf
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) atomicMax(&maxbits[g], __float_as_uint(v));  // order-preserving for v >= 0
}

__global__ void flag_kernel(const float* __restrict__ mu, const float* __restrict__ sigma,
                            const float* __restrict__ err_mu, const float* __restrict__ err_q,
                            const float* __restrict__ sf2v, const float* __restrict__ bestv,
                            const float* __restrict__ yabsv, const unsigned* __restrict__ maxbits, long long m,
                            int* __restrict__ count, int* __restrict__ list)
{
    const int g = blockIdx.y;
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= m) return;
    const size_t f = (size_t)g * m + i;
    const float sf2 = sf2v[g];
    const float mu_i = mu[f], sd = sigma[f], dmu = err_mu[f], dq = err_q[f];
    // d sigma = dq / (2 sigma); with sigma -> 0 every rounding error in q matters
    const float dsd = (sd > 0.f) ? dq / (2.f * sd) : ((dq > 0.f) ? INFINITY : 0.f);
    const float tol_mu = 1e-4f * fabsf(mu_i) + 1e-6f * yabsv[g];
    const float tol_sd = 1e-4f * sd + 1e-6f * sqrtf(sf2);
    bool flag = !(dmu <= 0.5f * tol_mu) || !(dsd <= 0.5f * tol_sd);
    // EI: dEI = Phi(z) dmu + phi(z) dsigma against 1e-5 of the pool's largest EI
    const float z = (sd > 0.f) ? (bestv[g] - mu_i) / sd : 0.f;
    const float Phi = 0.5f * erfcf(-z * 0.70710678f);
    const float phi = expf(-0.5f * z * z) * 0.39894228f;
    const float tol_ei = 1e-5f * __uint_as_float(maxbits[g]);
    if (isfinite(dsd)) flag |= !(Phi * dmu + phi * dsd <= 0.5f * tol_ei);
    flag |= !(sd * sd >= 1e-3f * sf2);   // deep cancellation: do not trust the estimates either
    if (flag) list[(size_t)g * m + atomicAdd(&count[g], 1)] = (int)i;
}

template <int R>
__global__ void __launch_bounds__(256) rescue_kernel(const float* __restrict__ X, const float* __restrict__ ell,
                                                     const float* __restrict__ sf2v, const float* __restrict__ bestv,
                                                     const double* __restrict__ alpha64, const double* __restrict__ W64,
                                                     int n, int d, int npad, const float* __restrict__ Xcand, long long m,
                                                     const int* __restrict__ count, const int* __restrict__ list,
                                                     float* __restrict__ mu, float* __restrict__ sigma,
                                                     float* __restrict__ ei)
{
    extern __shared__ double smem[];
    double* ks = smem;                        // [R][npad]
    double* zs = smem + (size_t)R * npad;     // [R][d] candidates
    double* ls = zs + (size_t)R * d;          // [d] lengthscales
    __shared__ double red[2][R][8];
    const int g = blockIdx.y;
    const int t = threadIdx.x, lane = t % 32, warp = t / 32;
    const int total = min(count[g], (int)min(m, (long long)INT_MAX));
    const float* Xg = X + (size_t)g * n * d;
    const double* Wg = W64 + (size_t)g * npad * npad;
    const double* ag = alpha64 + (size_t)g * npad;
    const double sf2 = (double)sf2v[g];
    for (int j = t; j < d; j += 256) ls[j] = (double)ell[(size_t)g * d + j];
    for (int e0 = blockIdx.x * R; e0 < total; e0 += gridDim.x * R) {
        const int nr = min(R, total - e0);
        __syncthreads();
        for (int e = t; e < R * d; e += 256) {
            const int r = e / d, j = e % d;
            const int c = list[(size_t)g * m + e0 + min(r, nr - 1)];
            zs[e] = (double)Xcand[((size_t)g * m + c) * d + j];
        }
        __syncthreads();
        double mu_part[R];
#pragma unroll
        for (int r = 0; r < R; ++r) mu_part[r] = 0.0;
        for (int i = t; i < n; i += 256) {
            double r2[R];
#pragma unroll
            for (int r = 0; r < R; ++r) r2[r] = 0.0;
            for (int j = 0; j < d; ++j) {
                const double x = (double)Xg[(size_t)i * d + j], l = ls[j];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const double df = (x - zs[r * d + j]) / l;
                    r2[r] += df * df;
                }
            }
            const double a = ag[i];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const double s = sqrt(5.0) * sqrt(r2[r]);
                const double kv = sf2 * (1.0 + s + s * s / 3.0) * exp(-s);
                ks[(size_t)r * npad + i] = kv;
                mu_part[r] += kv * a;
            }
        }
        __syncthreads();
        double q_part[R];
#pragma unroll
        for (int r = 0; r < R; ++r) q_part[r] = 0.0;
        for (int i = warp; i < n; i += 8) {
            const double* Wr = Wg + (size_t)i * npad;
            double v[R];
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = 0.0;
            for (int k = lane; k <= i; k += 32) {
                const double w = Wr[k];
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] += w * ks[(size_t)r * npad + k];
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                for (int o = 16; o > 0; o >>= 1) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
                q_part[r] += v[r] * v[r];  // identical in every lane; lane 0's copy is used
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            for (int o = 16; o > 0; o >>= 1) mu_part[r] += __shfl_xor_sync(0xffffffffu, mu_part[r], o);
            if (lane == 0) {
                red[0][r][warp] = mu_part[r];
                red[1][r][warp] = q_part[r];
            }
        }
        __syncthreads();
        if (t < nr) {
            double mu_s = 0.0, q = 0.0;
            for (int w = 0; w < 8; ++w) {
                mu_s += red[0][t][w];
                q += red[1][t][w];
            }
            const size_t f = (size_t)g * m + list[(size_t)g * m + e0 + t];
            const CandidateResult res = finalize_candidate(mu_s, q, sf2, (double)bestv[g]);
            mu[f] = res.mu;
            sigma[f] = res.sigma;
            ei[f] = res.ei;
        }
    }
}

}  // namespace

size_t guard_workspace_bytes(const r3_gp* gp, long long m)
{
    const size_t bm = (size_t)gp->batch * m;
    return 2 * bm * sizeof(float) + bm * sizeof(int) + 2 * (size_t)gp->batch * sizeof(int) + 256;
}

GuardBuffers guard_carve(const r3_gp* gp, long long m, void* ws)
{
    GuardBuffers b;
    const size_t bm = (size_t)gp->batch * m;
    char* p = (char*)ws;
    b.err_mu = (float*)p;
    p += bm * sizeof(float);
    b.err_q = (float*)p;
    p += bm * sizeof(float);
    b.list = (int*)p;
    p += bm * sizeof(int);
    b.count = (int*)p;
    p += (size_t)gp->batch * sizeof(int);
    b.maxbits = (unsigned*)p;
    return b;
}

r3_status_t guard_and_rescue(r3_gp* gp, const float* Xcand, long long m, const GuardBuffers& b, float* mu,
                             float* sigma, float* ei, cudaStream_t stream)
{
    const int B = gp->batch;
    R3_CUDA_TRY(cudaMemsetAsync(b.count, 0, 2 * (size_t)B * sizeof(int), stream));  // count and maxbits
    const unsigned gx = (unsigned)((m + 255) / 256);
    R3_LAUNCH(max_ei_kernel, dim3(gx < 1184u ? gx : 1184u, B), 256, 0, stream, ei, m, b.maxbits);
    R3_LAUNCH(flag_kernel, dim3(gx, B), 256, 0, stream, mu, sigma, b.err_mu, b.err_q, gp->sf2_d, gp->best_d,
              gp->yabs_d, b.maxbits, m, b.count, b.list);
    R3_CUDA_TRY(cudaMemcpyAsync(gp->rescued_h, b.count, sizeof(int) * (B < 64 ? B : 64), cudaMemcpyDeviceToHost,
                                stream));
    const int R = gp->npad <= 4096 ? RESCUE_GROUP : 1;
    const size_t smem = sizeof(double) * ((size_t)R * gp->npad + (size_t)R * gp->d + gp->d);
    const unsigned grid_x = B >= 8 ? 74 : 592;
    if (R == RESCUE_GROUP) {
        if (smem > 48 * 1024)
            R3_CUDA_TRY(cudaFuncSetAttribute(rescue_kernel<RESCUE_GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem));
        R3_LAUNCH(rescue_kernel<RESCUE_GROUP>, dim3(grid_x, B), 256, smem, stream, gp->X, gp->ell_d, gp->sf2_d,
                  gp->best_d, gp->alpha64, gp->W64, gp->n, gp->d, gp->npad, Xcand, m, b.count, b.list, mu, sigma, ei);
    } else {
        if (smem > 48 * 1024)
            R3_CUDA_TRY(cudaFuncSetAttribute(rescue_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        R3_LAUNCH(rescue_kernel<1>, dim3(grid_x, B), 256, smem, stream, gp->X, gp->ell_d, gp->sf2_d, gp->best_d,
                  gp->alpha64, gp->W64, gp->n, gp->d, gp->npad, Xcand, m, b.count, b.list, mu, sigma, ei);
    }
    return R3_OK;
}

}  // namespace r3
