// r3_bo_run: the inner search of Section IV as one call -- fit, propose a parallel batch, have the
// caller replay it, discard incorrect configurations, update the surrogate, until one of the paper's
// three stopping rules fires.  Host logic around r3_gp_fit / r3_gp_propose / r3_gp_append /
// r3_gp_optimize; the only kernels of its own move rows of the pool.
#include <math.h>

#include <chrono>
#include <vector>

#include "r3_internal.cuh"

namespace r3 {

namespace {

// rows[i] = pool[idx[i]]
__global__ void gather_rows_kernel(const float* __restrict__ pool, const int* __restrict__ idx, int q, int d,
                                   float* __restrict__ rows)
{
    const int i = blockIdx.x;
    for (int j = threadIdx.x; j < d; j += blockDim.x) rows[(size_t)i * d + j] = pool[(size_t)idx[i] * d + j];
}

// Removes the q proposed rows: the rows from the tail of the pool that are not themselves proposed move
// into the holes the proposed rows leave in the part that stays.  One thread per (proposed row, feature);
// the matching of holes and tail rows is recomputed by every block from the q indices (q <= 128).
__global__ void remove_rows_kernel(float* __restrict__ pool, long long m, const int* __restrict__ idx, int q, int d)
{
    __shared__ int holes[128], movers[128];
    __shared__ int nh;
    if (threadIdx.x == 0) {
        const long long keep = m - q;   // the pool shrinks to rows [0, keep)
        int h = 0, mv = 0;
        for (int i = 0; i < q; ++i)
            if (idx[i] < keep) holes[h++] = idx[i];
        for (long long r = keep; r < m; ++r) {
            bool proposed = false;
            for (int i = 0; i < q; ++i) proposed |= idx[i] == r;
            if (!proposed) movers[mv++] = (int)r;
        }
        nh = h;   // == mv
    }
    __syncthreads();
    const int i = blockIdx.x;
    if (i >= nh) return;
    for (int j = threadIdx.x; j < d; j += blockDim.x) pool[(size_t)holes[i] * d + j] = pool[(size_t)movers[i] * d + j];
}

}  // namespace

}  // namespace r3

using namespace r3;

extern "C" {

r3_status_t r3_bo_run(const float* X0, const float* y0, int n0, int d, const float* lengthscales, float signal_var,
                      float noise_var, const float* pool, long long m, const r3_bo_options_t* options,
                      r3_evaluate_fn evaluate, void* user, float* best_x, float* best_y, int* rounds, int* evaluated,
                      int* discarded, int* stop_reason, r3_gp_t** gp_out, void* cuda_stream)
{
    if (gp_out) *gp_out = nullptr;
    if (!X0 || !y0 || !lengthscales || !pool || !options || !evaluate || !best_x || !best_y) {
        set_error("r3_bo_run: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (n0 < 1 || n0 > kMaxN || d < 1 || d > kMaxD) {
        set_error("r3_bo_run: need 1 <= n0 <= %d and 1 <= d <= %d (n0=%d, d=%d)", kMaxN, kMaxD, n0, d);
        return R3_ERR_INVALID_ARG;
    }
    const r3_bo_options_t opt = *options;
    if (opt.q < 1 || opt.q > kAppendMax || opt.max_rounds < 1 || m < 1 || m >= (1ll << 31) || (opt.lie != 0 && opt.lie != 1)) {
        set_error("r3_bo_run: need 1 <= q <= %d, max_rounds >= 1, 1 <= m < 2^31, lie in {0, 1}", kAppendMax);
        return R3_ERR_INVALID_ARG;
    }
    if (opt.surrogate != 0 && opt.surrogate != 1) {
        set_error("r3_bo_run: surrogate must be 0 (GP) or 1 (TPE)");
        return R3_ERR_INVALID_ARG;
    }
    const bool tpe = opt.surrogate == 1;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    r3_gp_t* gp = nullptr;
    r3_status_t st = R3_OK;
    if (!tpe) {
        st = r3_gp_fit(X0, y0, lengthscales, &signal_var, &noise_var, 1, n0, d, cuda_stream, &gp);
        if (st != R3_OK) return st;
    }

    float *work = nullptr, *rows_d = nullptr, *y_d = nullptr, *hist_x = nullptr, *hist_y = nullptr, *score = nullptr;
    int* idx_d = nullptr;
    void* topk_ws = nullptr;
    auto done = [&](r3_status_t s) {
        cudaStreamSynchronize(stream);
        dev_free(work);
        dev_free(rows_d);
        dev_free(y_d);
        dev_free(idx_d);
        dev_free(hist_x);
        dev_free(hist_y);
        dev_free(score);
        dev_free(topk_ws);
        if (s == R3_OK && gp_out && gp)
            *gp_out = gp;
        else
            r3_gp_free(gp);
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
    TRY_DONE(dev_malloc(&work, sizeof(float) * (size_t)m * d));
    TRY_DONE(dev_malloc(&rows_d, sizeof(float) * (size_t)opt.q * d));
    TRY_DONE(dev_malloc(&y_d, sizeof(float) * (size_t)opt.q));
    TRY_DONE(dev_malloc(&idx_d, sizeof(int) * (size_t)opt.q));
    TRY_DONE(cudaMemcpyAsync(work, pool, sizeof(float) * (size_t)m * d, cudaMemcpyDeviceToDevice, stream));
    // Parzen estimator: the history lives here (it is refitted every round), up to the estimator's 4096 rows
    const int hist_cap = 4096;
    int hist_n = n0;
    std::vector<int> all_ordinal(d, 0);
    const size_t topk_bytes = tpe ? topk_workspace_bytes(1, m, opt.q) : 0;
    if (tpe) {
        if (n0 > hist_cap) {
            set_error("r3_bo_run: the Parzen estimator takes at most %d observations", hist_cap);
            return done(R3_ERR_INVALID_ARG);
        }
        TRY_DONE(dev_malloc(&hist_x, sizeof(float) * (size_t)hist_cap * d));
        TRY_DONE(dev_malloc(&hist_y, sizeof(float) * (size_t)hist_cap));
        TRY_DONE(dev_malloc(&score, sizeof(float) * (size_t)m));
        TRY_DONE(dev_malloc(&topk_ws, topk_bytes));
        TRY_DONE(cudaMemcpyAsync(hist_x, X0, sizeof(float) * (size_t)n0 * d, cudaMemcpyDeviceToDevice, stream));
        TRY_DONE(cudaMemcpyAsync(hist_y, y0, sizeof(float) * (size_t)n0, cudaMemcpyDeviceToDevice, stream));
    }

    // incumbent: the best of the initial history
    std::vector<float> hx((size_t)n0 * d), hy(n0);
    TRY_DONE(cudaMemcpyAsync(hx.data(), X0, sizeof(float) * hx.size(), cudaMemcpyDeviceToHost, stream));
    TRY_DONE(cudaMemcpyAsync(hy.data(), y0, sizeof(float) * hy.size(), cudaMemcpyDeviceToHost, stream));
    TRY_DONE(cudaStreamSynchronize(stream));
    int ib = 0;
    for (int i = 1; i < n0; ++i)
        if (hy[i] < hy[ib]) ib = i;
    float by = hy[ib];
    std::vector<float> bx(hx.begin() + (size_t)ib * d, hx.begin() + (size_t)(ib + 1) * d);

    const auto t0 = std::chrono::steady_clock::now();
    std::vector<float> rows((size_t)opt.q * d), ys(opt.q), keep_rows, keep_y;
    std::vector<int> valid(opt.q);
    int round = 0, n_eval = 0, n_disc = 0, since_better = 0, reason = R3_BO_MAX_ROUNDS;
    long long left = m;
    while (true) {
        if (round >= opt.max_rounds) { reason = R3_BO_MAX_ROUNDS; break; }
        if (opt.max_seconds > 0.0 &&
            std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() >= opt.max_seconds) {
            reason = R3_BO_MAX_SECONDS;
            break;
        }
        if (opt.patience > 0 && since_better >= opt.patience) { reason = R3_BO_NO_IMPROVEMENT; break; }
        const int q = (int)(left < opt.q ? left : opt.q);
        if (q < 1) { reason = R3_BO_POOL_EXHAUSTED; break; }
        if ((tpe ? hist_n : r3_gp_size(gp)) + q > (tpe ? hist_cap : kMaxN)) { reason = R3_BO_HISTORY_FULL; break; }
        if (tpe) {
            r3_tpe_t* est = nullptr;
            st = r3_tpe_fit(hist_x, hist_y, opt.levels ? opt.levels : all_ordinal.data(), hist_n, d,
                            opt.gamma > 0.f ? opt.gamma : 0.25f, 1.0f, cuda_stream, &est);
            if (st != R3_OK) return done(st);
            st = r3_tpe_score(est, work, left, score, cuda_stream);
            if (st == R3_OK) st = topk_device(score, 1, left, q, idx_d, nullptr, topk_ws, topk_bytes, stream);
            if (st == R3_OK) st = r3_tpe_check(est, cuda_stream);
            r3_tpe_free(est);
            if (st != R3_OK) return done(st);
        } else {
            if (opt.optimize_every > 0 && round > 0 && round % opt.optimize_every == 0) {
                st = r3_gp_optimize(gp, 40, 1e-2, nullptr, nullptr, nullptr, nullptr, nullptr, cuda_stream);
                if (st != R3_OK && st != R3_ERR_NOT_PD) return done(st);   // a failed search keeps the old values
                if (gp->sn2[0] < 1e-6f * gp->sf2[0]) {
                    // keep the condition number of K within what the later rank-k updates can take
                    const std::vector<float> ell = gp->ell;
                    const float sf2 = gp->sf2[0], sn2 = 1e-6f * sf2;
                    st = r3_gp_refit(gp, ell.data(), &sf2, &sn2, cuda_stream);
                    if (st != R3_OK && st != R3_ERR_NOT_PD) return done(st);
                }
            }
            st = r3_gp_propose(gp, work, left, q, 0, opt.lie, idx_d, nullptr, nullptr, cuda_stream);
            if (st != R3_OK) return done(st);
        }
        gather_rows_kernel<<<q, 128, 0, stream>>>(work, idx_d, q, d, rows_d);
        ++g_launches;
        TRY_DONE(cudaGetLastError());
        TRY_DONE(cudaMemcpyAsync(rows.data(), rows_d, sizeof(float) * (size_t)q * d, cudaMemcpyDeviceToHost, stream));
        remove_rows_kernel<<<q, 128, 0, stream>>>(work, left, idx_d, q, d);
        ++g_launches;
        TRY_DONE(cudaGetLastError());
        TRY_DONE(cudaStreamSynchronize(stream));
        left -= q;
        for (int i = 0; i < q; ++i) valid[i] = 1;
        const int stop = evaluate(rows.data(), q, d, ys.data(), valid.data(), user);
        ++round;
        keep_rows.clear();
        keep_y.clear();
        bool better = false;
        for (int i = 0; i < q; ++i) {
            ++n_eval;
            if (!valid[i] || !isfinite(ys[i])) {   // an incorrect kernel (or no measurement): discarded
                ++n_disc;
                continue;
            }
            keep_rows.insert(keep_rows.end(), rows.begin() + (size_t)i * d, rows.begin() + (size_t)(i + 1) * d);
            keep_y.push_back(ys[i]);
            if (ys[i] < by) {
                by = ys[i];
                bx.assign(rows.begin() + (size_t)i * d, rows.begin() + (size_t)(i + 1) * d);
                better = true;
            }
        }
        since_better = better ? 0 : since_better + 1;
        if (!keep_y.empty()) {
            const int k = (int)keep_y.size();
            TRY_DONE(cudaMemcpyAsync(rows_d, keep_rows.data(), sizeof(float) * (size_t)k * d, cudaMemcpyHostToDevice,
                                     stream));
            TRY_DONE(cudaMemcpyAsync(y_d, keep_y.data(), sizeof(float) * (size_t)k, cudaMemcpyHostToDevice, stream));
            if (tpe) {
                TRY_DONE(cudaMemcpyAsync(hist_x + (size_t)hist_n * d, rows_d, sizeof(float) * (size_t)k * d,
                                         cudaMemcpyDeviceToDevice, stream));
                TRY_DONE(cudaMemcpyAsync(hist_y + hist_n, y_d, sizeof(float) * (size_t)k, cudaMemcpyDeviceToDevice,
                                         stream));
                TRY_DONE(cudaStreamSynchronize(stream));   // keep_rows / keep_y are reused next round
                hist_n += k;
            } else {
                // Hyper-parameters chosen by the optimiser can leave the extended covariance matrix numerically
                // singular (tiny noise, long lengthscales, a new point next to an old one): raise the noise
                // by factors of ten and refit until the update goes through.
                st = r3_gp_append(gp, rows_d, y_d, k, cuda_stream);
                for (int attempt = 0; st == R3_ERR_NOT_PD && attempt < 6; ++attempt) {
                    const std::vector<float> ell = gp->ell;
                    const float sf2 = gp->sf2[0];
                    const float sn2 = fmaxf(gp->sn2[0] * 10.f, 1e-8f * sf2);
                    st = r3_gp_refit(gp, ell.data(), &sf2, &sn2, cuda_stream);
                    if (st == R3_OK) st = r3_gp_append(gp, rows_d, y_d, k, cuda_stream);
                }
                if (st != R3_OK) return done(st);
            }
        }
        if (stop) { reason = R3_BO_STOPPED_BY_CALLER; break; }
    }
#undef TRY_DONE
    for (int j = 0; j < d; ++j) best_x[j] = bx[j];
    *best_y = by;
    if (rounds) *rounds = round;
    if (evaluated) *evaluated = n_eval;
    if (discarded) *discarded = n_disc;
    if (stop_reason) *stop_reason = reason;
    return done(R3_OK);
}

}  // extern "C"
