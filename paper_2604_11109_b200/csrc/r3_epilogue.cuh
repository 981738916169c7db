// Per-candidate epilogue shared by the scoring engines: variance, standard deviation and the
// closed-form Expected Improvement for minimisation, in FP64 (one evaluation per candidate, so the
// cost is negligible, and EI in the lower tail loses an order of magnitude to cancellation in FP32).
#pragma once

#include <cuda_runtime.h>

namespace r3 {

struct CandidateResult {
    float mu, sigma, ei;
};

__device__ __forceinline__ double ei_closed_form(double mu, double sd, double best)
{
    const double imp = best - mu;
    if (!(sd > 0.0)) return imp > 0.0 ? imp : 0.0;
    const double z = imp / sd;
    const double Phi = 0.5 * erfc(-z * 0.70710678118654752440);
    const double phi = exp(-0.5 * z * z) * 0.39894228040143267794;
    const double e = imp * Phi + sd * phi;
    return e > 0.0 ? e : 0.0;
}

// mu = k*.alpha and q = |W k*|^2 as the engine computed them; sf2 = signal variance, best = incumbent.
__device__ __forceinline__ CandidateResult finalize_candidate(double mu, double q, double sf2, double best)
{
    CandidateResult r;
    double var = sf2 - q;
    if (!(var > 0.0)) var = 0.0;
    const double sd = sqrt(var);
    r.mu = (float)mu;
    r.sigma = (float)sd;
    r.ei = (float)ei_closed_form(mu, sd, best);
    return r;
}

// First-order, random-sign estimates of the engine's own rounding error in mu and in q, from the
// per-entry relative error eps of k*:
//   d mu ~ 2 eps sqrt(sum_i (k*_i alpha_i)^2)
//   d q  ~ 2 eps |W|_2 sqrt(q sum_i k*_i^2)        (from dq = 2 V.(W dk*), |V|^2 = q)
// The flagging pass compares them with the accuracy contract once the pool's largest EI is known.
__device__ __forceinline__ float mu_error_estimate(double eps, double a2) { return (float)(2.0 * eps * sqrt(a2)); }
__device__ __forceinline__ float q_error_estimate(double eps, double wnorm, double q, double s2)
{
    return (float)(2.0 * eps * wnorm * sqrt(fmax(q, 0.0) * s2));
}

}  // namespace r3
