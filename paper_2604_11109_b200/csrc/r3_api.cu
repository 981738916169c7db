// C ABI of libr3gp: argument validation, handle life cycle, engine dispatch.  See include/r3.h.
#include <limits.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>

#include <new>

#include "r3_internal.cuh"

namespace r3 {

static thread_local char g_error[512] = "";
thread_local unsigned long long g_launches = 0;

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
}

r3_status_t ensure_workspace(r3_gp* gp, size_t bytes)
{
    if (bytes <= gp->ws_bytes) return R3_OK;
    // growing synchronises the device: wait for work that may still use the old buffer
    R3_CUDA_TRY(cudaDeviceSynchronize());
    if (gp->ws) dev_free(gp->ws);
    gp->ws = nullptr;
    gp->ws_bytes = 0;
    const size_t want = (bytes + (1u << 20)) & ~((size_t)(1u << 20) - 1);
    R3_CUDA_TRY(dev_malloc(&gp->ws, want));
    gp->ws_bytes = want;
    return R3_OK;
}

void prof_begin(r3_gp* gp, cudaStream_t stream)
{
    if (!gp->profile) return;
    if (gp->events_used + 2 > gp->events.size()) {
        if (gp->events.size() >= 16384) return;  // cap: further launches go untimed
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess) return;
        if (cudaEventCreate(&b) != cudaSuccess) {
            cudaEventDestroy(a);
            return;
        }
        gp->events.push_back(a);
        gp->events.push_back(b);
    }
    cudaEventRecord(gp->events[gp->events_used], stream);
}

void prof_end(r3_gp* gp, cudaStream_t stream)
{
    if (!gp->profile || gp->events_used + 2 > gp->events.size()) return;
    cudaEventRecord(gp->events[gp->events_used + 1], stream);
    gp->events_used += 2;
}

constexpr int kAutoSimtMaxD = 8, kAutoSimtMaxN = 128;

static r3_engine_t pick_engine(const r3_gp* gp)
{
    const bool tc_ok = gp->tc != nullptr;
    switch (gp->engine_req) {
        case R3_ENGINE_SIMT: return R3_ENGINE_SIMT;
        case R3_ENGINE_TENSOR: return tc_ok ? R3_ENGINE_TENSOR : R3_ENGINE_SIMT;
        default:
            // Few features and a short history: the squared distance by direct differences costs next to nothing
            // and keeps full FP32 accuracy for the near pairs such pools are full of, whereas the norm expansion
            // of the tensor path sends a third of a pool like that to the FP64 pass.
            if (gp->d <= kAutoSimtMaxD && gp->n <= kAutoSimtMaxN) return R3_ENGINE_SIMT;
            return tc_ok ? R3_ENGINE_TENSOR : R3_ENGINE_SIMT;
    }
}

static size_t score_workspace_bytes(const r3_gp* gp, long long m)
{
    return pick_engine(gp) == R3_ENGINE_TENSOR ? score_tc_workspace_bytes(gp, m)
                                               : score_simt_workspace_bytes(gp, m);
}

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

static r3_status_t check_score_args(const r3_gp* gp, const void* Xcand, long long m, const void* mu,
                                    const void* sigma, const void* ei)
{
    if (!gp || !Xcand || !mu || !sigma || !ei) {
        set_error("r3_gp_score: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (m < 1 || m >= (1ll << 31)) {
        set_error("r3_gp_score: m=%lld out of range [1, 2^31)", m);
        return R3_ERR_INVALID_ARG;
    }
    return R3_OK;
}

static r3_status_t run_score(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei,
                             void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (pick_engine(gp) == R3_ENGINE_TENSOR) return score_tc(gp, Xcand, m, mu, sigma, ei, ws, ws_bytes, stream);
    return score_simt(gp, Xcand, m, mu, sigma, ei, ws, ws_bytes, stream);
}

}  // namespace r3

using namespace r3;

extern "C" {

int r3_version(void) { return 100; }

const char* r3_last_error(void) { return g_error; }

const char* r3_status_string(r3_status_t s)
{
    switch (s) {
        case R3_OK: return "ok";
        case R3_ERR_INVALID_ARG: return "invalid argument";
        case R3_ERR_NONFINITE: return "non-finite input";
        case R3_ERR_NOT_PD: return "covariance matrix is not positive definite";
        case R3_ERR_ALLOC: return "allocation failed";
        case R3_ERR_CUDA: return "CUDA error";
        case R3_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case R3_ERR_UNSUPPORTED: return "unsupported";
    }
    return "unknown status";
}

unsigned long long r3_launch_count(void) { return g_launches; }
void r3_launch_count_reset(void) { g_launches = 0; }

void r3_gp_free(r3_gp_t* gp)
{
    if (!gp) return;
    tc_release(gp);
    dev_free(gp->X);
    dev_free(gp->y);
    dev_free(gp->ell_d);
    dev_free(gp->inv_ell);
    dev_free(gp->sn2_d);
    dev_free(gp->sf2_d);
    dev_free(gp->best_d);
    dev_free(gp->yabs_d);
    dev_free(gp->wnorm_d);
    dev_free(gp->L64);
    dev_free(gp->W64);
    dev_free(gp->W32);
    dev_free(gp->alpha64);
    dev_free(gp->alpha32);
    dev_free(gp->status_d);
    pinned_word_release(gp->status_h);   // rescued_h lives in the same block
    for (cudaEvent_t e : gp->events) cudaEventDestroy(e);
    for (cudaEvent_t e : gp->copy_events) cudaEventDestroy(e);
    if (gp->copy_stream) cudaStreamDestroy(gp->copy_stream);
    dev_free(gp->ws);
    delete gp;
}

r3_status_t r3_gp_fit(const float* X, const float* y, const float* lengthscales, const float* signal_var,
                      const float* noise_var, int batch, int n, int d, void* cuda_stream, r3_gp_t** out)
{
    if (out) *out = nullptr;
    if (!X || !y || !lengthscales || !signal_var || !noise_var || !out) {
        set_error("r3_gp_fit: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (batch < 1 || batch > 4096 || n < 1 || n > kMaxN || d < 1 || d > kMaxD) {
        set_error("r3_gp_fit: sizes out of range (batch=%d in [1,4096], n=%d in [1,%d], d=%d in [1,%d])", batch,
                  n, kMaxN, d, kMaxD);
        return R3_ERR_INVALID_ARG;
    }
    for (int g = 0; g < batch; ++g) {
        if (!(signal_var[g] > 0.f) || !isfinite(signal_var[g]) || !(noise_var[g] >= 0.f) ||
            !isfinite(noise_var[g])) {
            set_error("r3_gp_fit: GP %d needs signal_var > 0 and noise_var >= 0", g);
            return R3_ERR_INVALID_ARG;
        }
        for (int j = 0; j < d; ++j) {
            const float l = lengthscales[(size_t)g * d + j];
            if (!(l > 0.f) || !isfinite(l)) {
                set_error("r3_gp_fit: GP %d lengthscale %d must be positive and finite", g, j);
                return R3_ERR_INVALID_ARG;
            }
        }
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    r3_gp* gp = new (std::nothrow) r3_gp;
    if (!gp) {
        set_error("r3_gp_fit: out of host memory");
        return R3_ERR_ALLOC;
    }
    auto bail = [&](r3_status_t st) {
        r3_gp_free(gp);
        return st;
    };
#define TRY_BAIL(expr)                                                                             \
    do {                                                                                           \
        cudaError_t e__ = (expr);                                                                  \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("%s failed: %s", #expr, cudaGetErrorString(e__));                            \
            return bail(e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA);            \
        }                                                                                          \
    } while (0)
    TRY_BAIL(cudaGetDevice(&gp->device));
    gp->batch = batch;
    gp->n = n;
    gp->d = d;
    gp->npad = round_up(n, kFitBlock);
    gp->ell.assign(lengthscales, lengthscales + (size_t)batch * d);
    gp->sf2.assign(signal_var, signal_var + batch);
    gp->sn2.assign(noise_var, noise_var + batch);
    gp->best.assign(batch, 0.f);
    std::vector<float> inv((size_t)batch * d);
    for (size_t i = 0; i < inv.size(); ++i) inv[i] = (float)(1.0 / (double)gp->ell[i]);

    const size_t mat = (size_t)gp->npad * gp->npad;
    TRY_BAIL(dev_malloc(&gp->X, sizeof(float) * batch * (size_t)n * d));
    TRY_BAIL(dev_malloc(&gp->y, sizeof(float) * batch * (size_t)n));
    TRY_BAIL(dev_malloc(&gp->ell_d, sizeof(float) * batch * d));
    TRY_BAIL(dev_malloc(&gp->inv_ell, sizeof(float) * batch * d));
    TRY_BAIL(dev_malloc(&gp->sn2_d, sizeof(float) * batch));
    TRY_BAIL(dev_malloc(&gp->sf2_d, sizeof(float) * batch));
    TRY_BAIL(dev_malloc(&gp->best_d, sizeof(float) * batch));
    TRY_BAIL(dev_malloc(&gp->yabs_d, sizeof(float) * batch));
    TRY_BAIL(dev_malloc(&gp->wnorm_d, sizeof(double) * batch));
    TRY_BAIL(dev_malloc(&gp->L64, sizeof(double) * batch * mat));
    TRY_BAIL(dev_malloc(&gp->W64, sizeof(double) * batch * mat));
    TRY_BAIL(dev_malloc(&gp->W32, sizeof(float) * batch * mat));
    TRY_BAIL(dev_malloc(&gp->alpha64, sizeof(double) * batch * gp->npad));
    TRY_BAIL(dev_malloc(&gp->alpha32, sizeof(float) * batch * gp->npad));
    TRY_BAIL(dev_malloc(&gp->status_d, 4 * sizeof(int)));
    TRY_BAIL(cudaMemsetAsync(gp->status_d, 0, 4 * sizeof(int), stream));
    gp->status_h = pinned_word_acquire();   // [4] status words, then [64] rescue counters
    if (!gp->status_h) {
        set_error("r3_gp_fit: no pinned host memory");
        return bail(R3_ERR_ALLOC);
    }
    gp->rescued_h = gp->status_h + 4;
    for (int i = 0; i < 64; ++i) gp->rescued_h[i] = 0;
    gp->status_h[0] = 0;
    gp->status_h[1] = INT_MAX;
    TRY_BAIL(cudaMemcpyAsync(gp->status_d, gp->status_h, 2 * sizeof(int), cudaMemcpyHostToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->X, X, sizeof(float) * batch * (size_t)n * d, cudaMemcpyDeviceToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->y, y, sizeof(float) * batch * (size_t)n, cudaMemcpyDeviceToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->ell_d, gp->ell.data(), sizeof(float) * batch * d, cudaMemcpyHostToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->inv_ell, inv.data(), sizeof(float) * batch * d, cudaMemcpyHostToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->sn2_d, gp->sn2.data(), sizeof(float) * batch, cudaMemcpyHostToDevice, stream));
    TRY_BAIL(cudaMemcpyAsync(gp->sf2_d, gp->sf2.data(), sizeof(float) * batch, cudaMemcpyHostToDevice, stream));
    TRY_BAIL(cudaStreamSynchronize(stream));  // `inv` is a pageable temporary
#undef TRY_BAIL

    r3_status_t st = fit_device(gp, y, stream);  // synchronises, fills status_h
    if (st != R3_OK) return bail(st);
    if (gp->status_h[0] & DEV_NONFINITE) {
        set_error("r3_gp_fit: X or y contains a non-finite value");
        return bail(R3_ERR_NONFINITE);
    }
    if (gp->status_h[0] & DEV_NOT_PD) {
        set_error("r3_gp_fit: pivot %d of K + noise*I is not positive (duplicate rows with zero noise?)",
                  gp->status_h[1]);
        return bail(R3_ERR_NOT_PD);
    }
    gp->y_absmax.assign(batch, 0.f);
    gp->wnorm.assign(batch, 0.0);
    if (cudaMemcpy(gp->best.data(), gp->best_d, sizeof(float) * batch, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(gp->y_absmax.data(), gp->yabs_d, sizeof(float) * batch, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(gp->wnorm.data(), gp->wnorm_d, sizeof(double) * batch, cudaMemcpyDeviceToHost) != cudaSuccess) {
        set_error("r3_gp_fit: reading back the incumbent failed");
        return bail(R3_ERR_CUDA);
    }
    if (tc_supported(n, d)) {
        st = tc_prepare(gp, stream);
        if (st != R3_OK) return bail(st);
    }
    *out = gp;
    return R3_OK;
}

r3_status_t r3_gp_lml(r3_gp_t* gp, double* lml, double* grad, void* cuda_stream)
{
    if (!gp || !lml) {
        set_error("r3_gp_lml: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    const int B = gp->batch, d = gp->d;
    std::vector<double> out((size_t)B * (d + 3));
    const r3_status_t st = lml_device(gp, out.data(), (cudaStream_t)cuda_stream);
    if (st != R3_OK) return st;
    for (int g = 0; g < B; ++g) {
        lml[g] = out[(size_t)g * (d + 3)];
        if (grad)
            for (int j = 0; j < d + 2; ++j) grad[(size_t)g * (d + 2) + j] = out[(size_t)g * (d + 3) + 1 + j];
    }
    return R3_OK;
}

r3_status_t r3_gp_propose(r3_gp_t* gp, const float* Xcand, long long m, int q, int shortlist, int lie, int* idx,
                          float* ei_pick, int* certified, void* cuda_stream)
{
    if (!gp || !Xcand || !idx) {
        set_error("r3_gp_propose: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (m < 1 || m >= (1ll << 31) || q < 1 || q > 256 || q > m || (lie != 0 && lie != 1)) {
        set_error("r3_gp_propose: need 1 <= m < 2^31, 1 <= q <= min(m, 256), lie in {0, 1} (m=%lld q=%d lie=%d)", m, q,
                  lie);
        return R3_ERR_INVALID_ARG;
    }
    const int rmax = (int)(m < 1023 ? m : 1023);
    int R = shortlist;
    if (R == 0) {
        R = 8 * q > 256 ? 8 * q : 256;
        if (R > rmax) R = rmax;
    }
    if (R < q || R > rmax) {
        set_error("r3_gp_propose: shortlist=%d outside [q, min(m, 1023)]", shortlist);
        return R3_ERR_INVALID_ARG;
    }
    const int B = gp->batch;
    const int Rk = (long long)R < m ? R + 1 : R;   // one more than the shortlist: the certificate's bound
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    r3_status_t st = ensure_workspace(gp, score_workspace_bytes(gp, m));
    if (st != R3_OK) return st;
    float *scores = nullptr, *sval = nullptr;
    int* sidx = nullptr;
    void *tws = nullptr, *pws = nullptr;
    const size_t bm = (size_t)B * m, tbytes = topk_workspace_bytes(B, m, Rk);
    auto done = [&](r3_status_t s) {
        cudaStreamSynchronize(stream);
        dev_free(scores); dev_free(sval); dev_free(sidx); dev_free(tws); dev_free(pws);
        return s;
    };
#define TRY_DONE(expr)                                                                             \
    do {                                                                                           \
        cudaError_t e__ = (expr);                                                                  \
        if (e__ != cudaSuccess) {                                                                  \
            set_error("%s failed: %s", #expr, cudaGetErrorString(e__));                            \
            return done(e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA);            \
        }                                                                                          \
    } while (0)
    TRY_DONE(dev_malloc(&scores, sizeof(float) * 3 * bm));
    TRY_DONE(dev_malloc(&sval, sizeof(float) * (size_t)B * Rk));
    TRY_DONE(dev_malloc(&sidx, sizeof(int) * (size_t)B * Rk));
    TRY_DONE(dev_malloc(&tws, tbytes));
    TRY_DONE(dev_malloc(&pws, propose_workspace_bytes(B, gp->npad, R, q)));
    float *mu = scores, *sigma = scores + bm, *ei = scores + 2 * bm;
    st = run_score(gp, Xcand, m, mu, sigma, ei, gp->ws, gp->ws_bytes, stream);
    if (st != R3_OK) return done(st);
    st = topk_device(ei, B, m, Rk, sidx, sval, tws, tbytes, stream);
    if (st != R3_OK) return done(st);
    st = propose_shortlist(gp, Xcand, m, sidx, Rk, R, q, lie, idx, ei_pick, pws, stream);
    if (st != R3_OK) return done(st);
    // certificate and latched device status
    std::vector<float> hval((size_t)B * Rk), hpick;
    TRY_DONE(cudaMemcpyAsync(hval.data(), sval, sizeof(float) * hval.size(), cudaMemcpyDeviceToHost, stream));
    TRY_DONE(cudaMemcpyAsync(gp->status_h, gp->status_d, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    if (ei_pick) {
        hpick.resize((size_t)B * q);
        TRY_DONE(cudaMemcpyAsync(hpick.data(), ei_pick, sizeof(float) * hpick.size(), cudaMemcpyDeviceToHost, stream));
    }
    TRY_DONE(cudaStreamSynchronize(stream));
#undef TRY_DONE
    if (gp->status_h[0] & DEV_NOT_PD) {
        gp->status_h[0] &= ~DEV_NOT_PD;
        cudaMemcpy(gp->status_d, gp->status_h, sizeof(int), cudaMemcpyHostToDevice);
        set_error("r3_gp_propose: a picked candidate has zero variance and the noise is zero (it duplicates an "
                  "observation); nothing to condition on");
        return done(R3_ERR_NOT_PD);
    }
    if (certified) {
        for (int g = 0; g < B; ++g) {
            if (Rk == R) {
                certified[g] = 1;   // the shortlist is the whole pool
            } else if (lie != 0 || !ei_pick) {
                certified[g] = 0;
            } else {
                // the first excluded candidate's initial EI (FP32, within the scoring tolerance of 1e-5 max EI)
                const double bound = hval[(size_t)g * Rk + R], top = hval[(size_t)g * Rk];
                double lowest = hpick[(size_t)g * q];
                for (int t = 1; t < q; ++t) lowest = hpick[(size_t)g * q + t] < lowest ? hpick[(size_t)g * q + t] : lowest;
                certified[g] = lowest >= bound + 4e-5 * top ? 1 : 0;
            }
        }
    }
    return done(R3_OK);
}

r3_status_t r3_gp_append(r3_gp_t* gp, const float* Xnew, const float* ynew, int k, void* cuda_stream)
{
    if (!gp || !Xnew || !ynew) {
        set_error("r3_gp_append: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (k < 1 || k > kAppendMax || gp->n + k > kMaxN) {
        set_error("r3_gp_append: need 1 <= k <= %d and n + k <= %d (n=%d, k=%d)", kAppendMax, kMaxN, gp->n, k);
        return R3_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // Bits that an earlier scoring call latched (a non-finite candidate, a wait that ran out) are not this
    // call's: they are taken out of the status word while the append's own checks use it, and put back after.
    R3_CUDA_TRY(cudaMemcpyAsync(gp->status_h, gp->status_d, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));
    const int latched = gp->status_h[0] & (DEV_NONFINITE | DEV_TIMEOUT);
    if (latched) R3_CUDA_TRY(cudaMemsetAsync(gp->status_d, 0, sizeof(int), stream));
    r3_status_t st = append_device(gp, Xnew, ynew, k, stream);
    const int bits = gp->status_h ? gp->status_h[0] : 0;
    const int pivot = gp->status_h ? gp->status_h[1] : 0;
    if (latched) {
        gp->status_h[0] = latched;
        if (cudaMemcpyAsync(gp->status_d, gp->status_h, sizeof(int), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) {
            set_error("r3_gp_append: restoring the latched status failed");
            return R3_ERR_CUDA;
        }
    }
    if (st == R3_OK && (bits & (DEV_NONFINITE | DEV_NOT_PD))) {
        // the handle was not touched; clear this call's bits so that it stays usable
        gp->status_h[0] = latched;
        gp->status_h[1] = INT_MAX;
        R3_CUDA_TRY(cudaMemcpyAsync(gp->status_d, gp->status_h, 2 * sizeof(int), cudaMemcpyHostToDevice, stream));
        R3_CUDA_TRY(cudaStreamSynchronize(stream));
        if (bits & DEV_NONFINITE) {
            set_error("r3_gp_append: Xnew or ynew contains a non-finite value");
            return R3_ERR_NONFINITE;
        }
        set_error("r3_gp_append: pivot %d of the extended K + noise*I is not positive (duplicate rows with zero noise?)",
                  pivot);
        return R3_ERR_NOT_PD;
    }
    if (st != R3_OK) return st;
    R3_CUDA_TRY(cudaMemcpy(gp->best.data(), gp->best_d, sizeof(float) * gp->batch, cudaMemcpyDeviceToHost));
    R3_CUDA_TRY(cudaMemcpy(gp->y_absmax.data(), gp->yabs_d, sizeof(float) * gp->batch, cudaMemcpyDeviceToHost));
    R3_CUDA_TRY(cudaMemcpy(gp->wnorm.data(), gp->wnorm_d, sizeof(double) * gp->batch, cudaMemcpyDeviceToHost));
    tc_release(gp);
    if (tc_supported(gp->n, gp->d)) {
        st = tc_prepare(gp, stream);
        // The history is extended at this point.  If only the tensor engine's operands could not be allocated,
        // the append stands and the CUDA-core engine serves the handle (r3_gp_engine tells).
        if (st != R3_OK && st != R3_ERR_ALLOC) return st;
    }
    return R3_OK;
}

int r3_gp_size(const r3_gp_t* gp) { return gp ? gp->n : 0; }

r3_status_t r3_gp_score(r3_gp_t* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei,
                        void* cuda_stream)
{
    r3_status_t st = check_score_args(gp, Xcand, m, mu, sigma, ei);
    if (st != R3_OK) return st;
    st = ensure_workspace(gp, score_workspace_bytes(gp, m));
    if (st != R3_OK) return st;
    return run_score(gp, Xcand, m, mu, sigma, ei, gp->ws, gp->ws_bytes, (cudaStream_t)cuda_stream);
}

unsigned long long r3_topk_scratch_bytes(int batch, long long m, int k)
{
    if (batch < 1 || m < 1 || k < 1) return 0;
    return topk_workspace_bytes(batch, m, k);
}

static r3_status_t check_topk_args(const void* ei, int batch, long long m, int k, const void* idx)
{
    if (!ei || !idx) {
        set_error("r3_topk: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (batch < 1 || m < 1 || m >= (1ll << 31) || k < 1 || k > kMaxK || k > m) {
        set_error("r3_topk: need batch >= 1, 1 <= m < 2^31, 1 <= k <= min(m, %d) (batch=%d m=%lld k=%d)", kMaxK,
                  batch, m, k);
        return R3_ERR_INVALID_ARG;
    }
    return R3_OK;
}

r3_status_t r3_topk(const float* ei, int batch, long long m, int k, int* idx, float* val, void* scratch,
                    unsigned long long scratch_bytes, void* cuda_stream)
{
    r3_status_t st = check_topk_args(ei, batch, m, k, idx);
    if (st != R3_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (scratch) return topk_device(ei, batch, m, k, idx, val, scratch, (size_t)scratch_bytes, stream);
    void* ws = nullptr;
    const size_t bytes = topk_workspace_bytes(batch, m, k);
    R3_CUDA_TRY(dev_malloc(&ws, bytes));
    st = topk_device(ei, batch, m, k, idx, val, ws, bytes, stream);
    cudaError_t e = cudaStreamSynchronize(stream);
    dev_free(ws);
    if (st == R3_OK && e != cudaSuccess) {
        set_error("r3_topk: %s", cudaGetErrorString(e));
        st = R3_ERR_CUDA;
    }
    return st;
}

r3_status_t r3_topk_noalloc(const float* ei, int batch, long long m, int k, int* idx, float* val, void* cuda_stream)
{
    r3_status_t st = check_topk_args(ei, batch, m, k, idx);
    if (st != R3_OK) return st;
    const size_t capacity = topk_static_capacity_bytes();
    if (topk_workspace_bytes(batch, m, k) > capacity) {
        set_error("r3_topk_noalloc: batch * ceil(m / 4096) * k = %lld exceeds the fixed capacity of %zu keys; use r3_topk",
                  (long long)batch * ((m + 4095) / 4096) * k, topk_static_capacity_keys());
        return R3_ERR_UNSUPPORTED;
    }
    void* scratch = nullptr;
    st = topk_static_scratch(&scratch);   // first call on a device: looks the array's address up (no allocation)
    if (st != R3_OK) return st;
    return topk_device(ei, batch, m, k, idx, val, scratch, capacity, (cudaStream_t)cuda_stream);
}

r3_status_t r3_gp_score_topk(r3_gp_t* gp, const float* Xcand, long long m, int k, float* mu, float* sigma,
                             float* ei, int* idx, float* val, void* cuda_stream)
{
    r3_status_t st = check_score_args(gp, Xcand, m, mu, sigma, ei);
    if (st != R3_OK) return st;
    st = check_topk_args(ei, gp->batch, m, k, idx);
    if (st != R3_OK) return st;
    const size_t sb = align256(score_workspace_bytes(gp, m));
    const size_t tb = guard_topk_workspace_bytes(gp->batch, m, k);
    st = ensure_workspace(gp, sb + tb);
    if (st != R3_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the selection rides on the scoring call: its first level is taken by the guard's kernel
    gp->topk_req.k = k;
    gp->topk_req.idx = idx;
    gp->topk_req.val = val;
    gp->topk_req.ws = (char*)gp->ws + sb;
    gp->topk_req.ws_bytes = tb;
    st = run_score(gp, Xcand, m, mu, sigma, ei, gp->ws, sb, stream);
    gp->topk_req = TopkRequest();
    return st;
}

r3_status_t r3_gp_score_topk_host(r3_gp_t* gp, const float* Xcand_host, long long m, int k, float* mu_host,
                                  float* sigma_host, float* ei_host, int* idx_host, float* val_host,
                                  void* cuda_stream)
{
    if (!gp || !Xcand_host || !idx_host) {
        set_error("r3_gp_score_topk_host: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (m < 1 || m >= (1ll << 31) || k < 1 || k > kMaxK || k > m) {
        set_error("r3_gp_score_topk_host: m or k out of range");
        return R3_ERR_INVALID_ARG;
    }
    const size_t B = gp->batch;
    const size_t sb = align256(score_workspace_bytes(gp, m));
    const size_t tb = align256(guard_topk_workspace_bytes(gp->batch, m, k));
    const size_t xb = align256(sizeof(float) * B * m * gp->d);
    const size_t ob = align256(sizeof(float) * B * m);
    const size_t kb = align256(sizeof(float) * B * k);
    r3_status_t st = ensure_workspace(gp, sb + tb + xb + 3 * ob + 2 * kb);
    if (st != R3_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* p = (char*)gp->ws + sb + tb;
    float* xc = (float*)p;
    p += xb;
    float* mu = (float*)p;
    p += ob;
    float* sg = (float*)p;
    p += ob;
    float* e = (float*)p;
    p += ob;
    int* idx = (int*)p;
    p += kb;
    float* val = (float*)p;
    gp->topk_req.k = k;
    gp->topk_req.idx = idx;
    gp->topk_req.val = val;
    gp->topk_req.ws = (char*)gp->ws + sb;
    gp->topk_req.ws_bytes = tb;
    struct ClearRequest {
        r3_gp* gp;
        ~ClearRequest() { gp->topk_req = TopkRequest(); }
    } clear_request{gp};
    // On the tensor engine a pool of several pieces travels on a second stream while the earlier pieces are
    // scored (a piece is about seven full waves of tiles on 148 SMs, so that no launch ends on a nearly empty
    // wave); the accuracy guard runs once over the whole pool, as in the device-buffer call, and the results are
    // identical.  Everything else: one copy, then the scoring.
    const long long tiles = pick_engine(gp) == R3_ENGINE_TENSOR ? score_tc_tiles(gp, m) : 0;
    const long long tiles_per_gp = B ? tiles / (long long)B : 0;
    // pieces are ranges of tiles that are contiguous in memory: any range for one GP, whole GPs for several
    long long piece_tiles = 148 * 7;
    if (B > 1) piece_tiles = std::max<long long>(1, (piece_tiles + tiles_per_gp / 2) / std::max<long long>(tiles_per_gp, 1)) * tiles_per_gp;
    const bool split = pick_engine(gp) == R3_ENGINE_TENSOR && score_tc_can_split(gp) && tiles > piece_tiles;
    if (split) {
        const int pieces = (int)((tiles + piece_tiles - 1) / piece_tiles);
        if (!gp->copy_stream) R3_CUDA_TRY(cudaStreamCreateWithFlags(&gp->copy_stream, cudaStreamNonBlocking));
        while ((int)gp->copy_events.size() < pieces + 1) {
            cudaEvent_t ev;
            R3_CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
            gp->copy_events.push_back(ev);
        }
        // the copies start once the caller's stream has reached this call (the staging buffer may still be read)
        R3_CUDA_TRY(cudaEventRecord(gp->copy_events[pieces], stream));
        R3_CUDA_TRY(cudaStreamWaitEvent(gp->copy_stream, gp->copy_events[pieces], 0));
        const long long rows = (long long)B * m;   // candidate rows of the whole call, GP after GP
        auto first_row = [&](long long tile) {      // the row at which a tile starts
            if (B == 1) return std::min<long long>(m, tile * 128);
            return std::min<long long>(rows, tile / tiles_per_gp * m);
        };
        for (int c = 0; c < pieces; ++c) {
            const long long lo = first_row(c * piece_tiles), hi = first_row(std::min(tiles, (c + 1) * piece_tiles));
            R3_CUDA_TRY(cudaMemcpyAsync(xc + lo * gp->d, Xcand_host + lo * gp->d, sizeof(float) * (hi - lo) * gp->d,
                                        cudaMemcpyHostToDevice, gp->copy_stream));
            R3_CUDA_TRY(cudaEventRecord(gp->copy_events[c], gp->copy_stream));
        }
        for (int c = 0; c < pieces; ++c) {
            R3_CUDA_TRY(cudaStreamWaitEvent(stream, gp->copy_events[c], 0));
            st = score_tc_part(gp, xc, m, mu, sg, e, gp->ws, sb, c * piece_tiles, (c + 1) * piece_tiles, false, stream);
            if (st != R3_OK) return st;
        }
        st = score_tc_guard(gp, xc, m, mu, sg, e, gp->ws, stream);
        if (st != R3_OK) return st;
    } else {
        R3_CUDA_TRY(cudaMemcpyAsync(xc, Xcand_host, sizeof(float) * B * m * gp->d, cudaMemcpyHostToDevice, stream));
        st = run_score(gp, xc, m, mu, sg, e, gp->ws, sb, stream);
        if (st != R3_OK) return st;
    }
    if (mu_host) R3_CUDA_TRY(cudaMemcpyAsync(mu_host, mu, sizeof(float) * B * m, cudaMemcpyDeviceToHost, stream));
    if (sigma_host) R3_CUDA_TRY(cudaMemcpyAsync(sigma_host, sg, sizeof(float) * B * m, cudaMemcpyDeviceToHost, stream));
    if (ei_host) R3_CUDA_TRY(cudaMemcpyAsync(ei_host, e, sizeof(float) * B * m, cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaMemcpyAsync(idx_host, idx, sizeof(int) * B * k, cudaMemcpyDeviceToHost, stream));
    if (val_host) R3_CUDA_TRY(cudaMemcpyAsync(val_host, val, sizeof(float) * B * k, cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));
    return R3_OK;
}

r3_status_t r3_gp_check(r3_gp_t* gp, void* cuda_stream)
{
    if (!gp) {
        set_error("r3_gp_check: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    R3_CUDA_TRY(cudaMemcpyAsync(gp->status_h, gp->status_d, 3 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaMemsetAsync(gp->status_d, 0, sizeof(int), stream));
    R3_CUDA_TRY(cudaMemsetAsync(gp->status_d + 2, 0, sizeof(int), stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));
    const int bits = gp->status_h[0];
    if (bits & DEV_BOUNDS) {
        set_error("bounds-checking build: an index check failed (source line %d of its kernel's file); results are invalid",
                  gp->status_h[2]);
        return R3_ERR_CUDA;
    }
    if (bits & DEV_TIMEOUT) {
        set_error("a bounded device-side wait ran out; results are invalid");
        return R3_ERR_DEVICE_TIMEOUT;
    }
    if (bits & DEV_NONFINITE) {
        set_error("a candidate contains a non-finite value");
        return R3_ERR_NONFINITE;
    }
    return R3_OK;
}

r3_status_t r3_gp_set_wait_limit(r3_gp_t* gp, long long cycles)
{
    if (!gp || cycles < 100000) {
        set_error("r3_gp_set_wait_limit: need a handle and at least 100000 cycles");
        return R3_ERR_INVALID_ARG;
    }
    gp->wait_limit_cycles = cycles;
    return R3_OK;
}

r3_status_t r3_gp_test_withhold(r3_gp_t* gp, long long chunk)
{
    if (!gp || chunk < 0) {
        set_error("r3_gp_test_withhold: need a handle and chunk >= 0");
        return R3_ERR_INVALID_ARG;
    }
    if (!gp->tc) {
        set_error("r3_gp_test_withhold: the tensor-core engine does not serve this handle");
        return R3_ERR_UNSUPPORTED;
    }
    gp->withhold_w = chunk;
    return R3_OK;
}

r3_status_t r3_gp_get_best(const r3_gp_t* gp, float* best)
{
    if (!gp || !best) {
        set_error("r3_gp_get_best: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    for (int g = 0; g < gp->batch; ++g) best[g] = gp->best[g];
    return R3_OK;
}

r3_status_t r3_gp_set_best(r3_gp_t* gp, const float* best)
{
    if (!gp || !best) {
        set_error("r3_gp_set_best: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    for (int g = 0; g < gp->batch; ++g)
        if (!isfinite(best[g])) {
            set_error("r3_gp_set_best: non-finite incumbent for GP %d", g);
            return R3_ERR_INVALID_ARG;
        }
    R3_CUDA_TRY(cudaDeviceSynchronize());
    R3_CUDA_TRY(cudaMemcpy(gp->best_d, best, sizeof(float) * gp->batch, cudaMemcpyHostToDevice));
    gp->best.assign(best, best + gp->batch);
    return R3_OK;
}

r3_status_t r3_gp_set_engine(r3_gp_t* gp, r3_engine_t engine)
{
    if (!gp || (int)engine < 0 || (int)engine > 2) {
        set_error("r3_gp_set_engine: invalid argument");
        return R3_ERR_INVALID_ARG;
    }
    if (engine == R3_ENGINE_TENSOR && !gp->tc) {
        set_error("r3_gp_set_engine: the tensor-core engine does not serve n=%d d=%d", gp->n, gp->d);
        return R3_ERR_UNSUPPORTED;
    }
    gp->engine_req = engine;
    return R3_OK;
}

r3_status_t r3_gp_last_rescued(r3_gp_t* gp, void* cuda_stream, long long* total)
{
    if (!gp || !total) {
        set_error("r3_gp_last_rescued: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    R3_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    long long t = 0;
    for (int g = 0; g < gp->batch && g < 64; ++g) t += gp->rescued_h[g];
    *total = t;
    return R3_OK;
}

r3_status_t r3_gp_tensor_info(const r3_gp_t* gp, int* info)
{
    if (!gp || !info) {
        set_error("r3_gp_tensor_info: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    tc_info(gp, info);
    return R3_OK;
}

r3_status_t r3_gp_profile(r3_gp_t* gp, int enable)
{
    if (!gp) {
        set_error("r3_gp_profile: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    gp->profile = enable != 0;
    gp->events_used = 0;
    return R3_OK;
}

r3_status_t r3_gp_profile_read(r3_gp_t* gp, double* kernel_ms, long long* launches)
{
    if (!gp || !kernel_ms || !launches) {
        set_error("r3_gp_profile_read: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    double total = 0.0;
    for (size_t i = 0; i + 1 < gp->events_used; i += 2) {
        R3_CUDA_TRY(cudaEventSynchronize(gp->events[i + 1]));
        float ms = 0.f;
        R3_CUDA_TRY(cudaEventElapsedTime(&ms, gp->events[i], gp->events[i + 1]));
        total += ms;
    }
    *kernel_ms = total;
    *launches = (long long)(gp->events_used / 2);
    gp->events_used = 0;
    return R3_OK;
}

r3_engine_t r3_gp_engine(const r3_gp_t* gp) { return gp ? pick_engine(gp) : R3_ENGINE_SIMT; }

r3_status_t r3_gp_get_factor(const r3_gp_t* gp, double* alpha, double* L)
{
    if (!gp) {
        set_error("r3_gp_get_factor: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    R3_CUDA_TRY(cudaDeviceSynchronize());
    const int n = gp->n, npad = gp->npad;
    for (int g = 0; g < gp->batch; ++g) {
        if (alpha)
            R3_CUDA_TRY(cudaMemcpy(alpha + (size_t)g * n, gp->alpha64 + (size_t)g * npad, sizeof(double) * n,
                                   cudaMemcpyDeviceToHost));
        if (L)
            R3_CUDA_TRY(cudaMemcpy2D(L + (size_t)g * n * n, sizeof(double) * n, gp->L64 + (size_t)g * npad * npad,
                                     sizeof(double) * npad, sizeof(double) * n, n, cudaMemcpyDeviceToHost));
    }
    return R3_OK;
}

}  // extern "C"
