// FP64 rescue pass.
//
// Near an observation the posterior variance sf2 - |W k*|^2 is the small difference of two numbers
// close to sf2, and an FP32-level |W k*|^2 cannot give sigma to four digits.  The scoring engines
// therefore list every candidate whose variance falls below a fixed fraction of sf2; this kernel
// recomputes those few candidates from the raw inputs entirely in FP64 -- direct-difference
// distances with a true division by the lengthscale, FP64 weights and the FP64 inverse factor --
// and overwrites their mu, sigma and EI.  One block per listed candidate, grid-stride over the list.
#include "r3_epilogue.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

__global__ void __launch_bounds__(256) rescue_kernel(const float* __restrict__ X, const float* __restrict__ ell,
                                                     const float* __restrict__ sf2v, const float* __restrict__ bestv,
                                                     const double* __restrict__ alpha64, const double* __restrict__ W64,
                                                     int n, int d, int npad, const float* __restrict__ Xcand, long long m,
                                                     const int* __restrict__ count, const long long* __restrict__ list,
                                                     long long cap, float* __restrict__ mu, float* __restrict__ sigma,
                                                     float* __restrict__ ei)
{
    extern __shared__ double smem[];
    double* ks = smem;                 // [npad]
    double* zs = smem + npad;          // [d] candidate, [d] lengthscale
    double* ls = zs + d;
    __shared__ double red[2][8];
    const int t = threadIdx.x, lane = t % 32, warp = t / 32;
    long long total = count[0];
    if (total > cap) total = cap;
    for (long long e = blockIdx.x; e < total; e += gridDim.x) {
        const long long flat = list[e];
        const int g = (int)(flat / m);
        const float* z = Xcand + (size_t)flat * d;
        const float* Xg = X + (size_t)g * n * d;
        const double* Wg = W64 + (size_t)g * npad * npad;
        const double sf2 = (double)sf2v[g];
        __syncthreads();
        for (int j = t; j < d; j += 256) {
            zs[j] = (double)z[j];
            ls[j] = (double)ell[(size_t)g * d + j];
        }
        __syncthreads();
        double mu_part = 0.0;
        for (int i = t; i < n; i += 256) {
            double r2 = 0.0;
            for (int j = 0; j < d; ++j) {
                double df = ((double)Xg[(size_t)i * d + j] - zs[j]) / ls[j];
                r2 += df * df;
            }
            const double s = sqrt(5.0) * sqrt(r2);
            const double kv = sf2 * (1.0 + s + s * s / 3.0) * exp(-s);
            ks[i] = kv;
            mu_part += kv * alpha64[(size_t)g * npad + i];
        }
        __syncthreads();
        double q_part = 0.0;
        for (int i = warp; i < n; i += 8) {
            const double* Wr = Wg + (size_t)i * npad;
            double v = 0.0;
            for (int k = lane; k <= i; k += 32) v += Wr[k] * ks[k];
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            q_part += v * v;  // identical in every lane; lane 0's copy is used
        }
        for (int o = 16; o > 0; o >>= 1) mu_part += __shfl_xor_sync(0xffffffffu, mu_part, o);
        if (lane == 0) {
            red[0][warp] = mu_part;
            red[1][warp] = q_part;
        }
        __syncthreads();
        if (t == 0) {
            double mu_s = 0.0, q = 0.0;
            for (int w = 0; w < 8; ++w) {
                mu_s += red[0][w];
                q += red[1][w];
            }
            double var = sf2 - q;
            if (!(var > 0.0)) var = 0.0;
            const double sd = sqrt(var);
            mu[flat] = (float)mu_s;
            sigma[flat] = (float)sd;
            ei[flat] = (float)ei_closed_form(mu_s, sd, (double)bestv[g]);
        }
    }
}

}  // namespace

r3_status_t rescue(r3_gp* gp, const float* Xcand, long long m, const int* count, const long long* list,
                   long long cap, float* mu, float* sigma, float* ei, cudaStream_t stream)
{
    const size_t smem = sizeof(double) * ((size_t)gp->npad + 2 * (size_t)gp->d);
    if (smem > 48 * 1024)
        R3_CUDA_TRY(cudaFuncSetAttribute(rescue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    R3_LAUNCH(rescue_kernel, 592, 256, smem, stream, gp->X, gp->ell_d, gp->sf2_d, gp->best_d,
              gp->alpha64, gp->W64, gp->n, gp->d, gp->npad, Xcand, m, count, list, cap, mu, sigma, ei);
    return R3_OK;
}

}  // namespace r3
