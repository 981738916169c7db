// SIMT (CUDA-core, FP32) scoring engine.
//
// Serves every (n, d); it is the engine of choice for small feature counts, where the squared
// distance is cheap to form by direct differences and keeps full FP32 accuracy for near pairs, and
// the on-device cross-check for the tensor-core engine.  Per slab of candidates of one GP:
//   kstar_kernel       k*[c][i] = sf2 * M52(|(z_c - x_i)/ell|) -> slab buffer; mu_c = k* . alpha
//   trigemm_sq_kernel  V = W k* over the lower triangle only (register-tiled FP32 GEMM),
//                      q_c = sum_i V[i][c]^2, then the FP64 epilogue (sigma, EI) and the outputs
// The slab buffer is the only intermediate; it is sized to stay within a fixed budget.
#include "r3_epilogue.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr size_t kSlabBytes = 256ull << 20;
// relative error of one k* entry on this path: FP32 differences, FMA chain, sqrtf, expf.  The squared
// distance is an FP32 sum over d features, so its rounding grows like sqrt(d); the figure is for d <= 16.
constexpr double kEpsSimt = 1.2e-7;
inline double eps_simt(int d) { return kEpsSimt * (d > 16 ? sqrt((double)d / 16.0) : 1.0); }

struct SimtWorkspace {
    float* ks;         // [slab][npad]
    double* mu64;      // [slab][3]: mu, sum (k* alpha)^2, sum k*^2
    GuardBuffers guard;
    long long slab;
};

long long slab_candidates(int npad, long long m)
{
    long long s = (long long)(kSlabBytes / ((size_t)npad * sizeof(float)));
    s = s / 128 * 128;
    if (s < 128) s = 128;
    long long mr = round_up_ll(m, 128);
    return s < mr ? s : mr;
}

SimtWorkspace carve(const r3_gp* gp, long long m, void* ws)
{
    SimtWorkspace w;
    w.slab = slab_candidates(gp->npad, m);
    char* p = (char*)ws;
    w.ks = (float*)p;
    p += (size_t)w.slab * gp->npad * sizeof(float);
    w.mu64 = (double*)p;
    p += (size_t)w.slab * 3 * sizeof(double);
    w.guard = guard_carve(gp, m, p);
    return w;
}

// 64 candidates x 64 training points per step; thread (ty, tx): candidates ty + 16u, points 4tx + v.
__global__ void __launch_bounds__(256) kstar_kernel(const float* __restrict__ X,       // [n][d]
                                                    const float* __restrict__ inv_ell, // [d]
                                                    const float* __restrict__ alpha,   // [npad]
                                                    float sf2, int n, int d, int npad,
                                                    const float* __restrict__ Z,       // [mc][d] this slab
                                                    long long mc, float* __restrict__ ks,
                                                    double* __restrict__ mu64, int* status)
{
    __shared__ float sz[64][33], sx[64][33], sl[32];
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    const long long c0 = (long long)blockIdx.x * 64;
    double mu_acc[4] = {0.0, 0.0, 0.0, 0.0}, a1_acc[4] = {0.0, 0.0, 0.0, 0.0}, s2_acc[4] = {0.0, 0.0, 0.0, 0.0};
    bool bad = false;
    for (int k0 = 0; k0 < npad; k0 += 64) {
        float r2[4][4] = {};
        for (int j0 = 0; j0 < d; j0 += 32) {
            for (int e = t; e < 64 * 32; e += 256) {
                int r = e / 32, c = e % 32;
                float zv = (c0 + r < mc && j0 + c < d) ? Z[(size_t)(c0 + r) * d + j0 + c] : 0.f;
                bad |= !isfinite(zv);
                sz[r][c] = zv;
                sx[r][c] = (k0 + r < n && j0 + c < d) ? X[(size_t)(k0 + r) * d + j0 + c] : 0.f;
            }
            if (t < 32) sl[t] = (j0 + t < d) ? inv_ell[j0 + t] : 0.f;
            __syncthreads();
            const int jmax = min(32, d - j0);
            for (int j = 0; j < jmax; ++j) {
                const float w = sl[j];
                float zc[4], xk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    zc[u] = sz[ty + 16 * u][j];
                    xk[u] = sx[tx * 4 + u][j];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        float df = (zc[u] - xk[v]) * w;
                        r2[u][v] = fmaf(df, df, r2[u][v]);
                    }
            }
            __syncthreads();
        }
        float al[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) al[v] = (k0 + tx * 4 + v < npad) ? alpha[k0 + tx * 4 + v] : 0.f;  // zero beyond n
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float kv[4];
            float part = 0.f, apart = 0.f, spart = 0.f;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                float s = sqrtf(5.0f * r2[u][v]);
                float val = sf2 * (1.0f + s + s * s * (1.0f / 3.0f)) * expf(-s);
                if (k0 + tx * 4 + v >= n) val = 0.f;
                kv[v] = val;
                part = fmaf(val, al[v], part);
                apart = fmaf(val * al[v], val * al[v], apart);
                spart = fmaf(val, val, spart);
            }
            mu_acc[u] += (double)part;
            a1_acc[u] += (double)apart;
            s2_acc[u] += (double)spart;
            const long long c = c0 + ty + 16 * u;
            if (c < mc && k0 + tx * 4 < npad)
                *reinterpret_cast<float4*>(ks + (size_t)c * npad + k0 + tx * 4) =
                    make_float4(kv[0], kv[1], kv[2], kv[3]);
        }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        double v = mu_acc[u], a = a1_acc[u], s = s2_acc[u];
        for (int o = 8; o > 0; o >>= 1) {
            v += __shfl_xor_sync(0xffffffffu, v, o);
            a += __shfl_xor_sync(0xffffffffu, a, o);
            s += __shfl_xor_sync(0xffffffffu, s, o);
        }
        const long long c = c0 + ty + 16 * u;
        if (tx == 0 && c < mc) {
            mu64[3 * c + 0] = v;
            mu64[3 * c + 1] = a;
            mu64[3 * c + 2] = s;
        }
    }
    if (__syncthreads_or(bad) && t == 0) atomicOr(status, DEV_NONFINITE);
}

// V = W k* restricted to k <= i, 128 candidates per block, all row tiles in turn.
// Thread (ty, tx): rows i0 + 4ty + {0..3} and i0 + 64 + 4ty + {0..3}; candidates 4tx + {0..3} and
// 64 + 4tx + {0..3}.
__global__ void __launch_bounds__(256) trigemm_sq_kernel(const float* __restrict__ W,   // [npad][npad]
                                                         const float* __restrict__ ks,  // [slab][npad]
                                                         const double* __restrict__ mu64, int npad,
                                                         long long mc, double sf2, double best, double eps_k, double wnorm,
                                                         float* __restrict__ mu, float* __restrict__ sigma,
                                                         float* __restrict__ ei, float* __restrict__ err_mu,
                                                         float* __restrict__ err_q, unsigned* __restrict__ maxbits)
{
    __shared__ __align__(16) float sw[16][132];
    __shared__ __align__(16) float sk[16][132];
    __shared__ double sq[16][128];
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    const long long c0 = (long long)blockIdx.x * 128;
    double qacc[8] = {};
    for (int i0 = 0; i0 < npad; i0 += 128) {
        float acc[8][8] = {};
        const int kend = min(npad, i0 + 128);
        for (int k0 = 0; k0 < kend; k0 += 16) {
            // 128 x 16 tiles of W and k*, read as float4 along k and stored transposed
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int e = t + 256 * it;      // 0..511
                const int r = e / 4, kq = (e % 4) * 4;
                float4 wv = make_float4(0.f, 0.f, 0.f, 0.f), kv = wv;
                if (i0 + r < npad) wv = *reinterpret_cast<const float4*>(W + (size_t)(i0 + r) * npad + k0 + kq);
                if (c0 + r < mc) kv = *reinterpret_cast<const float4*>(ks + (size_t)(c0 + r) * npad + k0 + kq);
                sw[kq + 0][r] = wv.x; sw[kq + 1][r] = wv.y; sw[kq + 2][r] = wv.z; sw[kq + 3][r] = wv.w;
                sk[kq + 0][r] = kv.x; sk[kq + 1][r] = kv.y; sk[kq + 2][r] = kv.z; sk[kq + 3][r] = kv.w;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) {
                const float4 a0 = *reinterpret_cast<const float4*>(&sw[kk][4 * ty]);
                const float4 a1 = *reinterpret_cast<const float4*>(&sw[kk][64 + 4 * ty]);
                const float4 b0 = *reinterpret_cast<const float4*>(&sk[kk][4 * tx]);
                const float4 b1 = *reinterpret_cast<const float4*>(&sk[kk][64 + 4 * tx]);
                const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int u = 0; u < 8; ++u)
#pragma unroll
                    for (int v = 0; v < 8; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            float part = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) part = fmaf(acc[u][v], acc[u][v], part);
            qacc[v] += (double)part;
        }
    }
#pragma unroll
    for (int v = 0; v < 8; ++v) sq[ty][(v < 4 ? 4 * tx + v : 64 + 4 * tx + (v - 4))] = qacc[v];
    __syncthreads();
    if (t < 128) {
        const long long c = c0 + t;
        float ei_mine = 0.f;
        if (c < mc) {
            double q = 0.0;
#pragma unroll
            for (int r = 0; r < 16; ++r) q += sq[r][t];
            const CandidateResult res = finalize_candidate(mu64[3 * c], q, sf2, best);
            mu[c] = res.mu;
            sigma[c] = res.sigma;
            ei[c] = res.ei;
            err_mu[c] = mu_error_estimate(eps_k, mu64[3 * c + 1]);
            err_q[c] = q_error_estimate(eps_k, wnorm, q, mu64[3 * c + 2]);
            if (res.ei == res.ei) ei_mine = res.ei;
        }
        // the pool's largest EI, for the guard's EI tolerance: one atomic per warp
        const unsigned ei_top = __reduce_max_sync(0xffffffffu, __float_as_uint(ei_mine));
        if ((t & 31) == 0 && ei_top) atomicMax(maxbits, ei_top);
    }
}

}  // namespace

size_t score_simt_workspace_bytes(const r3_gp* gp, long long m)
{
    const long long slab = slab_candidates(gp->npad, m);
    return (size_t)slab * gp->npad * sizeof(float) + (size_t)slab * 3 * sizeof(double) +
           guard_workspace_bytes(gp, m);
}

r3_status_t score_simt(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei,
                       void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (ws_bytes < score_simt_workspace_bytes(gp, m)) {
        set_error("internal: SIMT workspace too small");
        return R3_ERR_INVALID_ARG;
    }
    SimtWorkspace w = carve(gp, m, ws);
    const int n = gp->n, d = gp->d, npad = gp->npad;
    {
        const r3_status_t st0 = guard_begin(gp, w.guard, stream);
        if (st0 != R3_OK) return st0;
    }
    for (int g = 0; g < gp->batch; ++g) {
        for (long long s0 = 0; s0 < m; s0 += w.slab) {
            const long long mc = (m - s0) < w.slab ? (m - s0) : w.slab;
            const float* Z = Xcand + ((size_t)g * m + s0) * d;
            const size_t off = (size_t)g * m + s0;
            R3_LAUNCH(kstar_kernel, (unsigned)((mc + 63) / 64), 256, 0, stream,
                      gp->X + (size_t)g * n * d, gp->inv_ell + (size_t)g * d,
                      gp->alpha32 + (size_t)g * npad, gp->sf2[g], n, d, npad, Z, mc, w.ks, w.mu64,
                      gp->status_d);
            prof_begin(gp, stream);
            R3_LAUNCH(trigemm_sq_kernel, (unsigned)((mc + 127) / 128), 256, 0, stream,
                      gp->W32 + (size_t)g * npad * npad, w.ks, w.mu64, npad, mc, (double)gp->sf2[g],
                      (double)gp->best[g], eps_simt(d), gp->wnorm[g], mu + off, sigma + off, ei + off,
                      w.guard.err_mu + off, w.guard.err_q + off, w.guard.maxbits + g);
            prof_end(gp, stream);
        }
    }
    return guard_and_rescue(gp, Xcand, m, w.guard, mu, sigma, ei, true, stream);
}

}  // namespace r3
