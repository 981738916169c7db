// Greedy batch proposal by fantasies ("parallel" search of Section IV: several points of one search are
// replayed at once).  Definition: q times -- pick the not-yet-picked candidate of largest EI (incumbent
// fixed at the best observed value), then condition the GP on that point with a fantasised value (its
// posterior mean, "believer", or the incumbent, "liar").
//
// Refitting and rescoring the pool q times would cost q full scoring passes.  Conditioning on one point
// is a rank-one change of the posterior:
//     c(x) = cov(x, x_t),  s = var(x_t) + noise,
//     mu(x) += c(x) (value - mu(x_t)) / s,     var(x) -= c(x)^2 / s,
//     cov(x, x_t) = k(x, x_t) - v(x).v(x_t) - sum_{earlier picks u} c_u(x) c_u(x_t) / s_u,   v(x) = W k*(x),
// and with the believer's value the means never move while the variances only shrink, so EI (fixed
// incumbent) only drops: a candidate outside the R best of the first scoring can be picked only if some
// pick's EI falls below the (R+1)-th initial EI.  So: one full scoring, top-(R+1), then the q picks on the
// shortlist alone, in FP64 (k*, v = W k* by one triangular product, the moments recomputed), two small
// launches per pick.  The (R+1)-th initial EI is returned as the certificate's bound.
#include "r3_epilogue.cuh"
#include "r3_gemm64.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

// All GPs of the handle are processed together: blockIdx.z (or .y) is the GP.  Per-GP scalars come from
// device arrays; the shortlist state of GP g starts at g times the per-GP stride of each array.
struct ProposeArrays {
    const float* X;        // [B][n][d]
    const float* ell;      // [B][d]
    const float* sf2;      // [B]
    const float* sn2;      // [B]
    const float* best;     // [B]
    const double* alpha;   // [B][npad]
    const float* Xcand;    // [B][m][d]
    const int* sidx;       // [B][Rk] shortlist (pool indices), Rk >= R
    long long m;
    int n, d, npad, R, Rk, q;
    double *Ks, *V;        // [B][R][npad]
    double *C;             // [B][q][R]
    double *mu, *var;      // [B][R]
    double *S, *delta;     // [B][q]
    int *picked, *sel;     // [B][R], [B][q]
};

// Ks[r][i] = k(x_i, candidate sidx[r]) in FP64 by direct differences; zero in the padding columns.
__global__ void shortlist_kstar_kernel(const ProposeArrays a)
{
    const int g = blockIdx.z, r = blockIdx.y;
    const int n = a.n, d = a.d, npad = a.npad;
    const float* X = a.X + (size_t)g * n * d;
    const float* ell = a.ell + (size_t)g * d;
    const float* Xcand = a.Xcand + (size_t)g * a.m * d;
    const int* sidx = a.sidx + (size_t)g * a.Rk;
    double* Ks = a.Ks + (size_t)g * a.R * npad;
    const double sf2 = (double)a.sf2[g];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    __shared__ double inv[kMaxD];   // FP64 reciprocals of the lengthscales, as the fit's Gram kernel uses them
    for (int j = threadIdx.x; j < d; j += blockDim.x) inv[j] = 1.0 / (double)ell[j];
    __syncthreads();
    if (i >= npad) return;
    double v = 0.0;
    if (i < n) {
        const float* z = Xcand + (size_t)sidx[r] * d;
        const float* x = X + (size_t)i * d;
        double r2 = 0.0;
        for (int j = 0; j < d; ++j) {
            const double diff = ((double)x[j] - (double)z[j]) * inv[j];
            r2 += diff * diff;
        }
        const double s = sqrt(5.0) * sqrt(r2);
        v = sf2 * (1.0 + s + s * s / 3.0) * exp(-s);
    }
    Ks[(size_t)r * npad + i] = v;
}

// mu[r] = Ks[r].alpha, var[r] = sf2 - |V[r]|^2 (one warp per shortlisted candidate).
__global__ void shortlist_moments_kernel(const ProposeArrays a)
{
    const int g = blockIdx.y;
    const int n = a.n, npad = a.npad, R = a.R;
    const double* Ks = a.Ks + (size_t)g * R * npad;
    const double* V = a.V + (size_t)g * R * npad;
    const double* alpha = a.alpha + (size_t)g * npad;
    double* mu = a.mu + (size_t)g * R;
    double* var = a.var + (size_t)g * R;
    int* picked = a.picked + (size_t)g * R;
    const double sf2 = (double)a.sf2[g];
    const int r = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (r >= R) return;
    double m = 0.0, q = 0.0;
    for (int i = lane; i < n; i += 32) {
        m = fma(Ks[(size_t)r * npad + i], alpha[i], m);
        const double v = V[(size_t)r * npad + i];
        q = fma(v, v, q);
    }
    for (int o = 16; o > 0; o >>= 1) {
        m += __shfl_xor_sync(0xffffffffu, m, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (lane == 0) {
        mu[r] = m;
        var[r] = sf2 - q;
        picked[r] = 0;
    }
}

// One block: EI of every unpicked shortlisted candidate, the largest (ties: lower pool index) is pick t.
__global__ void __launch_bounds__(1024) pick_kernel(const ProposeArrays a, int liar, int t, int* __restrict__ idx_all,
                                                    float* __restrict__ ei_all, int* __restrict__ status)
{
    __shared__ double se[1024];
    __shared__ int sr[1024];
    const int g = blockIdx.x;
    const int R = a.R;
    const double* mu = a.mu + (size_t)g * R;
    const double* var = a.var + (size_t)g * R;
    int* picked = a.picked + (size_t)g * R;
    const int* sidx = a.sidx + (size_t)g * a.Rk;
    int* sel = a.sel + (size_t)g * a.q;
    double* S = a.S + (size_t)g * a.q;
    double* delta = a.delta + (size_t)g * a.q;
    int* idx_out = idx_all + (size_t)g * a.q;
    float* ei_out = ei_all ? ei_all + (size_t)g * a.q : nullptr;
    const double best = (double)a.best[g], sn2 = (double)a.sn2[g];
    const int r = threadIdx.x;
    double e = -1.0;
    if (r < R && !picked[r]) e = ei_closed_form(mu[r], sqrt(fmax(var[r], 0.0)), best);
    se[r] = e;
    sr[r] = r;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (r < o) {
            const double ea = se[r], eb = se[r + o];
            const int ra = sr[r], rb = sr[r + o];
            // an entry that is not a candidate (e < 0) always loses; equal EI: the lower pool index wins
            const bool take_b = (eb > ea) || (eb == ea && eb >= 0.0 && sidx[rb] < sidx[ra]);
            if (take_b) {
                se[r] = eb;
                sr[r] = rb;
            }
        }
        __syncthreads();
    }
    if (r == 0) {
        const int j = sr[0];
        sel[t] = j;
        picked[j] = 1;
        idx_out[t] = sidx[j];
        if (ei_out) ei_out[t] = (float)se[0];
        const double s = fmax(var[j], 0.0) + sn2;
        if (!(s > 0.0)) {   // a candidate on top of an observation with zero noise: nothing to condition on
            atomicOr(status, DEV_NOT_PD);
            S[t] = INFINITY;
            delta[t] = 0.0;
        } else {
            S[t] = s;
            // the fantasised value enters the history as an observation, i.e. rounded to FP32
            const double value = liar ? best : (double)(float)mu[j];
            delta[t] = (value - mu[j]) / s;
        }
    }
}

// One warp per shortlisted candidate r: c = cov(x_r, x_pick) under the posterior before pick t, then the
// rank-one update of its mean and variance.  C[t][r] keeps c for the later picks.
__global__ void condition_kernel(const ProposeArrays a, int t)
{
    const int g = blockIdx.y;
    const int n = a.n, d = a.d, npad = a.npad, R = a.R;
    const float* Xcand = a.Xcand + (size_t)g * a.m * d;
    const int* sidx = a.sidx + (size_t)g * a.Rk;
    const float* ell = a.ell + (size_t)g * d;
    const double sf2 = (double)a.sf2[g];
    const double* V = a.V + (size_t)g * R * npad;
    double* C = a.C + (size_t)g * a.q * R;
    const double* S = a.S + (size_t)g * a.q;
    const double* delta = a.delta + (size_t)g * a.q;
    const int* sel = a.sel + (size_t)g * a.q;
    double* mu = a.mu + (size_t)g * R;
    double* var = a.var + (size_t)g * R;
    const int r = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (r >= R) return;
    const int j = sel[t];
    const float* xr = Xcand + (size_t)sidx[r] * d;
    const float* xj = Xcand + (size_t)sidx[j] * d;
    double r2 = 0.0, dot = 0.0, prev = 0.0;
    for (int f = lane; f < d; f += 32) {
        const double diff = ((double)xr[f] - (double)xj[f]) / (double)ell[f];
        r2 = fma(diff, diff, r2);
    }
    for (int i = lane; i < n; i += 32) dot = fma(V[(size_t)r * npad + i], V[(size_t)j * npad + i], dot);
    for (int u = lane; u < t; u += 32) prev += C[(size_t)u * R + r] * C[(size_t)u * R + j] / S[u];
    for (int o = 16; o > 0; o >>= 1) {
        r2 += __shfl_xor_sync(0xffffffffu, r2, o);
        dot += __shfl_xor_sync(0xffffffffu, dot, o);
        prev += __shfl_xor_sync(0xffffffffu, prev, o);
    }
    if (lane == 0) {
        const double s = sqrt(5.0) * sqrt(r2);
        const double c = sf2 * (1.0 + s + s * s / 3.0) * exp(-s) - dot - prev;
        C[(size_t)t * R + r] = c;
        mu[r] += c * delta[t];
        var[r] -= c * c / S[t];
    }
}

}  // namespace

size_t propose_workspace_bytes(int batch, int npad, int R, int q)
{
    return (size_t)batch * (sizeof(double) * (2 * (size_t)R * npad + (size_t)q * R + 2 * (size_t)R + 2 * (size_t)q) +
                            sizeof(int) * ((size_t)R + q)) + 1024;
}

// The q picks of every GP of the handle.  sidx: device [batch][Rk] pool indices of the shortlists (by initial
// EI, descending; the first R of each row are used); idx_out / ei_out: device [batch][q].
// ws: propose_workspace_bytes(batch, npad, R, q) bytes.
r3_status_t propose_shortlist(r3_gp* gp, const float* Xcand, long long m, const int* sidx, int Rk, int R, int q, int liar,
                              int* idx_out, float* ei_out, void* ws, cudaStream_t stream)
{
    const int B = gp->batch, n = gp->n, d = gp->d, npad = gp->npad;
    char* p = (char*)ws;
    auto carve = [&](size_t bytes) {
        char* r = p;
        p += (bytes + 15) / 16 * 16;
        return r;
    };
    ProposeArrays a;
    a.X = gp->X;
    a.ell = gp->ell_d;
    a.sf2 = gp->sf2_d;
    a.sn2 = gp->sn2_d;
    a.best = gp->best_d;
    a.alpha = gp->alpha64;
    a.Xcand = Xcand;
    a.sidx = sidx;
    a.m = m;
    a.n = n;
    a.d = d;
    a.npad = npad;
    a.R = R;
    a.Rk = Rk;
    a.q = q;
    a.Ks = (double*)carve(sizeof(double) * (size_t)B * R * npad);
    a.V = (double*)carve(sizeof(double) * (size_t)B * R * npad);
    a.C = (double*)carve(sizeof(double) * (size_t)B * q * R);
    a.mu = (double*)carve(sizeof(double) * (size_t)B * R);
    a.var = (double*)carve(sizeof(double) * (size_t)B * R);
    a.S = (double*)carve(sizeof(double) * (size_t)B * q);
    a.delta = (double*)carve(sizeof(double) * (size_t)B * q);
    a.picked = (int*)carve(sizeof(int) * (size_t)B * R);
    a.sel = (int*)carve(sizeof(int) * (size_t)B * q);

    R3_LAUNCH(shortlist_kstar_kernel, dim3((npad + 127) / 128, R, B), 128, 0, stream, a);
    // V = Ks W^T (v_r = W k*_r): the same triangular product as the append step of the fit
    R3_LAUNCH((tri_gemm_kernel<true, 64>), dim3((n + 63) / 64, (R + 63) / 64, B), 256, 0, stream, a.Ks, npad,
              (size_t)R * npad, gp->W64, npad, (size_t)npad * npad, a.V, npad, (size_t)R * npad, R, n);
    R3_LAUNCH(shortlist_moments_kernel, dim3((R + 7) / 8, B), 256, 0, stream, a);
    for (int t = 0; t < q; ++t) {
        R3_LAUNCH(pick_kernel, B, 1024, 0, stream, a, liar, t, idx_out, ei_out, gp->status_d);
        if (t + 1 < q) R3_LAUNCH(condition_kernel, dim3((R + 7) / 8, B), 256, 0, stream, a, t);
    }
    return R3_OK;
}

}  // namespace r3
