// r3_gp_refit and r3_gp_optimize: hyper-parameter fitting by maximising the log marginal likelihood.
//
// The device work is the fit (r3_fit.cu) and the evidence with its gradient (r3_lml.cu); this file is
// the host logic around them: one limited-memory BFGS optimiser per GP, written as ask/tell so that the
// GPs of a batch are evaluated together (one batched refit and one evidence call per round).
#include <limits.h>
#include <math.h>

#include <algorithm>
#include <deque>
#include <vector>

#include "r3_internal.cuh"

namespace r3 {

namespace {

// Uploads the handle's host hyper-parameters, refits, returns the latched status bits in *bits.
r3_status_t refit_device(r3_gp* gp, cudaStream_t stream, int* bits, int* pivot = nullptr)
{
    const int B = gp->batch, d = gp->d;
    std::vector<float> inv((size_t)B * d);
    for (size_t i = 0; i < inv.size(); ++i) inv[i] = (float)(1.0 / (double)gp->ell[i]);
    gp->status_h[0] = 0;
    gp->status_h[1] = INT_MAX;
    R3_CUDA_TRY(cudaMemcpyAsync(gp->status_d, gp->status_h, 2 * sizeof(int), cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaMemcpyAsync(gp->ell_d, gp->ell.data(), sizeof(float) * B * d, cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaMemcpyAsync(gp->inv_ell, inv.data(), sizeof(float) * B * d, cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaMemcpyAsync(gp->sf2_d, gp->sf2.data(), sizeof(float) * B, cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaMemcpyAsync(gp->sn2_d, gp->sn2.data(), sizeof(float) * B, cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));   // `inv` is a pageable temporary
    const r3_status_t st = fit_device(gp, gp->y, stream);   // synchronises, fills status_h
    if (st != R3_OK) return st;
    *bits = gp->status_h[0];
    if (pivot) *pivot = gp->status_h[1];
    if (*bits & (DEV_NOT_PD | DEV_NONFINITE)) {
        gp->status_h[0] = 0;
        gp->status_h[1] = INT_MAX;
        R3_CUDA_TRY(cudaMemcpy(gp->status_d, gp->status_h, 2 * sizeof(int), cudaMemcpyHostToDevice));
    }
    return R3_OK;
}

// After the last refit: host copies of the incumbent and the norm estimate, tensor-engine operands.
r3_status_t refresh_after_fit(r3_gp* gp, cudaStream_t stream)
{
    R3_CUDA_TRY(cudaMemcpy(gp->best.data(), gp->best_d, sizeof(float) * gp->batch, cudaMemcpyDeviceToHost));
    R3_CUDA_TRY(cudaMemcpy(gp->y_absmax.data(), gp->yabs_d, sizeof(float) * gp->batch, cudaMemcpyDeviceToHost));
    R3_CUDA_TRY(cudaMemcpy(gp->wnorm.data(), gp->wnorm_d, sizeof(double) * gp->batch, cudaMemcpyDeviceToHost));
    tc_release(gp);
    if (tc_supported(gp->n, gp->d)) return tc_prepare(gp, stream);
    return R3_OK;
}

// Minimises F = -lml over a box by L-BFGS with backtracking; the caller evaluates the points it asks for.
class Lbfgs {
public:
    Lbfgs(std::vector<double> x0, std::vector<double> lo, std::vector<double> hi, double gtol)
        : x_(std::move(x0)), lo_(std::move(lo)), hi_(std::move(hi)), gtol_(gtol)
    {
        trial_ = x_;
    }
    bool done() const { return done_; }
    const std::vector<double>& ask() const { return trial_; }
    const std::vector<double>& best() const { return x_; }
    double best_value() const { return f_; }

    // F and its gradient at ask(); ok = false when the point could not be evaluated
    void tell(bool ok, double F, const std::vector<double>& grad)
    {
        if (done_) return;
        if (!started_) {
            if (!ok) {   // the start itself must be valid; nothing to do otherwise
                done_ = true;
                return;
            }
            started_ = true;
            f_ = F;
            g_ = grad;
            new_direction();
            return;
        }
        const double armijo = f_ + 1e-4 * alpha_ * slope_;
        if (ok && isfinite(F) && F <= armijo) {
            std::vector<double> s(x_.size()), yv(x_.size());
            double sy = 0.0;
            for (size_t i = 0; i < x_.size(); ++i) {
                s[i] = trial_[i] - x_[i];
                yv[i] = grad[i] - g_[i];
                sy += s[i] * yv[i];
            }
            const double improvement = f_ - F;
            if (sy > 1e-12) {
                S_.push_back(s);
                Y_.push_back(yv);
                if (S_.size() > 8) {
                    S_.pop_front();
                    Y_.pop_front();
                }
            }
            x_ = trial_;
            f_ = F;
            g_ = grad;
            if (improvement <= 1e-10 * std::max(1.0, fabs(F))) {
                done_ = true;
                return;
            }
            new_direction();
        } else {
            alpha_ *= 0.5;
            if (alpha_ < 1e-8) {
                if (!S_.empty()) {   // one restart along the steepest descent before giving up
                    S_.clear();
                    Y_.clear();
                    new_direction();
                } else {
                    done_ = true;
                }
                return;
            }
            make_trial();
        }
    }

private:
    double projected_gradient_norm() const
    {
        double m = 0.0;
        for (size_t i = 0; i < x_.size(); ++i) {
            double gi = g_[i];
            if ((x_[i] <= lo_[i] && gi > 0.0) || (x_[i] >= hi_[i] && gi < 0.0)) gi = 0.0;   // pushing outwards
            m = std::max(m, fabs(gi));
        }
        return m;
    }
    void new_direction()
    {
        if (projected_gradient_norm() <= gtol_) {
            done_ = true;
            return;
        }
        // two-loop recursion on the gradient with the outward components at active bounds removed
        const size_t n = x_.size();
        std::vector<double> q(n);
        for (size_t i = 0; i < n; ++i) {
            q[i] = g_[i];
            if ((x_[i] <= lo_[i] && q[i] > 0.0) || (x_[i] >= hi_[i] && q[i] < 0.0)) q[i] = 0.0;
        }
        std::vector<double> a(S_.size());
        for (int k = (int)S_.size() - 1; k >= 0; --k) {
            double sy = 0.0, sq = 0.0;
            for (size_t i = 0; i < n; ++i) {
                sy += S_[k][i] * Y_[k][i];
                sq += S_[k][i] * q[i];
            }
            a[k] = sq / sy;
            for (size_t i = 0; i < n; ++i) q[i] -= a[k] * Y_[k][i];
        }
        double gamma = 1.0;
        if (!S_.empty()) {
            double sy = 0.0, yy = 0.0;
            for (size_t i = 0; i < n; ++i) {
                sy += S_.back()[i] * Y_.back()[i];
                yy += Y_.back()[i] * Y_.back()[i];
            }
            gamma = sy / yy;
        }
        for (size_t i = 0; i < n; ++i) q[i] *= gamma;
        for (size_t k = 0; k < S_.size(); ++k) {
            double sy = 0.0, yq = 0.0;
            for (size_t i = 0; i < n; ++i) {
                sy += S_[k][i] * Y_[k][i];
                yq += Y_[k][i] * q[i];
            }
            const double b = yq / sy;
            for (size_t i = 0; i < n; ++i) q[i] += (a[k] - b) * S_[k][i];
        }
        p_.assign(n, 0.0);
        slope_ = 0.0;
        double gmax = 0.0;
        for (size_t i = 0; i < n; ++i) {
            p_[i] = -q[i];
            slope_ += g_[i] * p_[i];
            gmax = std::max(gmax, fabs(g_[i]));
        }
        if (!(slope_ < 0.0)) {   // not a descent direction: fall back to the (projected) steepest descent
            S_.clear();
            Y_.clear();
            slope_ = 0.0;
            for (size_t i = 0; i < n; ++i) {
                double gi = g_[i];
                if ((x_[i] <= lo_[i] && gi > 0.0) || (x_[i] >= hi_[i] && gi < 0.0)) gi = 0.0;
                p_[i] = -gi;
                slope_ += g_[i] * p_[i];
            }
        }
        // first step of a fresh memory: move the most sensitive parameter by at most one e-fold
        alpha_ = S_.empty() ? std::min(1.0, 1.0 / std::max(gmax, 1e-12)) : 1.0;
        make_trial();
    }
    void make_trial()
    {
        trial_.resize(x_.size());
        for (size_t i = 0; i < x_.size(); ++i)
            trial_[i] = std::min(std::max(x_[i] + alpha_ * p_[i], lo_[i]), hi_[i]);
    }

    std::vector<double> x_, lo_, hi_, g_, p_, trial_;
    std::deque<std::vector<double>> S_, Y_;
    double f_ = INFINITY, alpha_ = 1.0, slope_ = 0.0, gtol_;
    bool started_ = false, done_ = false;
};

}  // namespace

}  // namespace r3

using namespace r3;

extern "C" {

r3_status_t r3_gp_refit(r3_gp_t* gp, const float* lengthscales, const float* signal_var, const float* noise_var,
                        void* cuda_stream)
{
    if (!gp || !lengthscales || !signal_var || !noise_var) {
        set_error("r3_gp_refit: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    const int B = gp->batch, d = gp->d;
    for (int g = 0; g < B; ++g) {
        if (!(signal_var[g] > 0.f) || !isfinite(signal_var[g]) || !(noise_var[g] >= 0.f) || !isfinite(noise_var[g])) {
            set_error("r3_gp_refit: GP %d needs signal_var > 0 and noise_var >= 0", g);
            return R3_ERR_INVALID_ARG;
        }
        for (int j = 0; j < d; ++j) {
            const float l = lengthscales[(size_t)g * d + j];
            if (!(l > 0.f) || !isfinite(l)) {
                set_error("r3_gp_refit: GP %d lengthscale %d must be positive and finite", g, j);
                return R3_ERR_INVALID_ARG;
            }
        }
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const std::vector<float> ell0 = gp->ell, sf0 = gp->sf2, sn0 = gp->sn2;
    gp->ell.assign(lengthscales, lengthscales + (size_t)B * d);
    gp->sf2.assign(signal_var, signal_var + B);
    gp->sn2.assign(noise_var, noise_var + B);
    int bits = 0, pivot = 0;
    r3_status_t st = refit_device(gp, stream, &bits, &pivot);
    if (st != R3_OK) return st;
    if (bits & DEV_NOT_PD) {
        gp->ell = ell0;
        gp->sf2 = sf0;
        gp->sn2 = sn0;
        st = refit_device(gp, stream, &bits);
        if (st == R3_OK) st = refresh_after_fit(gp, stream);
        if (st != R3_OK) return st;
        set_error("r3_gp_refit: K + noise*I is not positive definite with these hyper-parameters (pivot %d); the "
                  "previous ones were kept", pivot);
        return R3_ERR_NOT_PD;
    }
    return refresh_after_fit(gp, stream);
}

r3_status_t r3_gp_optimize(r3_gp_t* gp, int max_evals, double gtol, float* lengthscales, float* signal_var,
                           float* noise_var, double* lml, int* evals, void* cuda_stream)
{
    if (evals) *evals = 0;
    if (!gp) {
        set_error("r3_gp_optimize: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    if (max_evals < 1 || !(gtol > 0.0)) {
        set_error("r3_gp_optimize: need max_evals >= 1 and gtol > 0");
        return R3_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int B = gp->batch, d = gp->d, P = d + 2;
    std::vector<Lbfgs> opt;
    for (int g = 0; g < B; ++g) {
        std::vector<double> x(P), lo(P), hi(P);
        for (int j = 0; j < d; ++j) {
            lo[j] = log(1e-3);
            hi[j] = log(1e3);
            x[j] = log((double)gp->ell[(size_t)g * d + j]);
        }
        lo[d] = log(1e-6);
        hi[d] = log(1e6);
        x[d] = log((double)gp->sf2[g]);
        lo[d + 1] = log(1e-8);
        hi[d + 1] = log(1e2);
        x[d + 1] = log(std::max((double)gp->sn2[g], 1e-8));
        for (int j = 0; j < P; ++j) x[j] = std::min(std::max(x[j], lo[j]), hi[j]);
        opt.emplace_back(x, lo, hi, gtol);
    }
    auto load = [&](bool best) {
        for (int g = 0; g < B; ++g) {
            const std::vector<double>& x = (best || opt[g].done()) ? opt[g].best() : opt[g].ask();
            for (int j = 0; j < d; ++j) gp->ell[(size_t)g * d + j] = (float)exp(x[j]);
            gp->sf2[g] = (float)exp(x[d]);
            gp->sn2[g] = (float)exp(x[d + 1]);
        }
    };
    std::vector<double> out((size_t)B * (d + 3)), grad(P);
    int used = 0;
    r3_status_t st = R3_OK;
    while (used < max_evals) {
        bool any = false;
        for (int g = 0; g < B; ++g) any |= !opt[g].done();
        if (!any) break;
        load(false);
        int bits = 0;
        st = refit_device(gp, stream, &bits);
        if (st != R3_OK) return st;
        ++used;
        const bool ok = !(bits & (DEV_NOT_PD | DEV_NONFINITE));
        if (ok) {
            st = lml_device(gp, out.data(), stream);
            if (st != R3_OK) return st;
        }
        for (int g = 0; g < B; ++g) {
            if (opt[g].done()) continue;
            for (int j = 0; j < P; ++j) grad[j] = ok ? -out[(size_t)g * (d + 3) + 1 + j] : 0.0;
            opt[g].tell(ok, ok ? -out[(size_t)g * (d + 3)] : INFINITY, grad);
        }
    }
    // leave the handle at the best point of every GP
    load(true);
    int bits = 0;
    st = refit_device(gp, stream, &bits);
    if (st != R3_OK) return st;
    if (bits & (DEV_NOT_PD | DEV_NONFINITE)) {
        set_error("r3_gp_optimize: the starting hyper-parameters do not give a positive definite covariance matrix");
        return R3_ERR_NOT_PD;
    }
    st = refresh_after_fit(gp, stream);
    if (st != R3_OK) return st;
    for (int g = 0; g < B; ++g) {
        if (lengthscales)
            for (int j = 0; j < d; ++j) lengthscales[(size_t)g * d + j] = gp->ell[(size_t)g * d + j];
        if (signal_var) signal_var[g] = gp->sf2[g];
        if (noise_var) noise_var[g] = gp->sn2[g];
        if (lml) lml[g] = -opt[g].best_value();
    }
    if (evals) *evals = used;
    return R3_OK;
}

}  // extern "C"
