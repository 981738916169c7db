// Per-candidate epilogue shared by the scoring engines: variance, standard deviation and the
// closed-form Expected Improvement for minimisation, in FP64 (one evaluation per candidate, so the
// cost is negligible, and EI in the lower tail loses an order of magnitude to cancellation in FP32).
#pragma once

#include <cuda_runtime.h>

namespace r3 {

// A candidate whose variance is below this fraction of the signal variance is recomputed in FP64:
// sf2 - q cancels there and FP32-level q cannot give sigma to 1e-4 relative.
constexpr double kRescueFraction = 0.05;

struct CandidateResult {
    float mu, sigma, ei;
    bool needs_rescue;
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

// mu = k*.alpha, q = |W k*|^2 (both possibly FP32-accurate), sf2 = signal variance, best = incumbent.
__device__ __forceinline__ CandidateResult finalize_candidate(double mu, double q, double sf2, double best)
{
    CandidateResult r;
    double var = sf2 - q;
    r.needs_rescue = !(var >= kRescueFraction * sf2);  // also catches NaN
    if (!(var > 0.0)) var = 0.0;
    const double sd = sqrt(var);
    r.mu = (float)mu;
    r.sigma = (float)sd;
    r.ei = (float)ei_closed_form(mu, sd, best);
    return r;
}

}  // namespace r3
