/*
 * r3_oracle.c -- plain FP64 CPU oracle for GP-EI candidate scoring.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what the CUDA library must compute.  It shares no code, header, table or
 * constant with the CUDA path, and only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * What it follows.  The paper (Section IV, "replay server", and Section V-B,
 * "sampled point") states the inner problem only as Bayesian optimisation over
 * (pass configuration, launch parameters) -> runtime, to be minimised, and is
 * agnostic to the search strategy; it prints no equation for the surrogate.
 * The surrogate computed here is the textbook zero-mean Gaussian-process
 * posterior with an ARD Matern-5/2 covariance and the closed-form Expected
 * Improvement for minimisation.  Because the method reaches exactly (up to
 * rounding) a result with a plain definition, every function below is that
 * definition written out:
 *
 *   (1) r^2(x,z) = sum_j ((x_j - z_j)/l_j)^2            direct differences
 *       k(x,z)   = sf2 * (1 + s + s^2/3) * exp(-s),  s = sqrt(5) * sqrt(r^2)
 *   (2) K = k(X,X) + sn2 * I ;  K = L L^T (lower) ; error if a pivot <= 0
 *   (3) alpha = L^-T (L^-1 y) ;  best = min_i y_i
 *   (4) per candidate x*:  k*_i = k(x_i, x*);  mu = k* . alpha;
 *       v = L^-1 k* (forward substitution);  var = max(sf2 - v.v, 0);
 *       sigma = sqrt(var)                     (latent std, noise not added)
 *   (5) z = (best - mu)/sigma;  EI = (best - mu)*Phi(z) + sigma*phi(z),
 *       Phi(z) = erfc(-z/sqrt 2)/2,  phi(z) = exp(-z^2/2)/sqrt(2 pi);
 *       sigma == 0  ->  EI = max(best - mu, 0)
 *   (6) top-k = first k of the candidates ordered by (EI descending,
 *       index ascending).
 *
 * The only liberty taken with (4): the forward substitution is applied to a
 * small group of candidates at once (the same recurrence with a matrix right
 * hand side), so that one sweep over L serves the whole group; OpenMP threads
 * take different groups.  No other blocking, fusion or reordering.
 *
 * All inputs are the same FP32 arrays the GPU receives, widened to FP64 on
 * read; all arithmetic and all outputs are FP64.
 *
 * Pins (tests/test_oracle_pins.py): closed-form kernel and EI values, a
 * hand-derived n=1 and n=3 posterior, training-point identities, far-field
 * limits, invariances, duplicated-data equivalence, an independent
 * explicit-inverse posterior (oracle/brute_force.py) and a library GP.
 */
#define _USE_MATH_DEFINES
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define R3O_PI 3.14159265358979323846
#define R3O_GROUP 16 /* candidates per forward-substitution group */

/* (1) Matern-5/2 profile as a function of the squared scaled distance. */
double r3o_matern52(double r2)
{
    double s = sqrt(5.0) * sqrt(r2);
    return (1.0 + s + s * s / 3.0) * exp(-s);
}

/* (1) ARD covariance between two FP32 feature rows. */
double r3o_kernel(const float *x, const float *z, const float *ell, int d, double sf2)
{
    double r2 = 0.0;
    for (int j = 0; j < d; ++j) {
        double t = ((double)x[j] - (double)z[j]) / (double)ell[j];
        r2 += t * t;
    }
    return sf2 * r3o_matern52(r2);
}

/* (2) Gram matrix with the noise on the diagonal, full n x n, row-major. */
void r3o_gram(const float *X, const float *ell, double sf2, double sn2, int n, int d, double *K)
{
#pragma omp parallel for schedule(dynamic, 8)
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j)
            K[(size_t)i * n + j] =
                r3o_kernel(X + (size_t)i * d, X + (size_t)j * d, ell, d, sf2) + (i == j ? sn2 : 0.0);
}

/* (2) Cholesky factor, column by column (Cholesky-Crout).  A (n x n, row-major)
 * is overwritten: the lower triangle holds L, the strict upper triangle is
 * zeroed.  Returns 0, or j+1 if pivot j is not a positive finite number. */
int r3o_cholesky(double *A, int n)
{
    for (int j = 0; j < n; ++j) {
        double *Aj = A + (size_t)j * n;
        double diag = Aj[j];
        for (int k = 0; k < j; ++k) diag -= Aj[k] * Aj[k];
        if (!(diag > 0.0) || !isfinite(diag)) return j + 1;
        double ljj = sqrt(diag);
        Aj[j] = ljj;
#pragma omp parallel for schedule(static)
        for (int i = j + 1; i < n; ++i) {
            double *Ai = A + (size_t)i * n;
            double s = Ai[j];
            for (int k = 0; k < j; ++k) s -= Ai[k] * Aj[k];
            Ai[j] = s / ljj;
        }
    }
    for (int i = 0; i < n; ++i)
        for (int j = i + 1; j < n; ++j) A[(size_t)i * n + j] = 0.0;
    return 0;
}

/* (3) alpha = L^-T (L^-1 y): forward then backward substitution. */
void r3o_alpha(const double *L, const float *y, int n, double *alpha)
{
    for (int i = 0; i < n; ++i) {
        double s = (double)y[i];
        for (int k = 0; k < i; ++k) s -= L[(size_t)i * n + k] * alpha[k];
        alpha[i] = s / L[(size_t)i * n + i];
    }
    for (int i = n - 1; i >= 0; --i) {
        double s = alpha[i];
        for (int k = i + 1; k < n; ++k) s -= L[(size_t)k * n + i] * alpha[k];
        alpha[i] = s / L[(size_t)i * n + i];
    }
}

/* (2)+(3) fit one GP.  L (n*n) and alpha (n) are caller-allocated.
 * Returns 0, -1 on a non-finite input, or the 1-based index of a bad pivot. */
int r3o_fit(const float *X, const float *y, const float *ell, double sf2, double sn2, int n, int d,
            double *L, double *alpha, double *best)
{
    for (size_t i = 0; i < (size_t)n * d; ++i)
        if (!isfinite(X[i])) return -1;
    for (int i = 0; i < n; ++i)
        if (!isfinite(y[i])) return -1;
    r3o_gram(X, ell, sf2, sn2, n, d, L);
    int st = r3o_cholesky(L, n);
    if (st) return st;
    r3o_alpha(L, y, n, alpha);
    double b = (double)y[0];
    for (int i = 1; i < n; ++i)
        if ((double)y[i] < b) b = (double)y[i];
    *best = b;
    return 0;
}

/* (5) Expected Improvement for minimisation, closed form. */
double r3o_ei(double mu, double sigma, double best)
{
    double imp = best - mu;
    if (!(sigma > 0.0)) return imp > 0.0 ? imp : 0.0;
    double z = imp / sigma;
    double Phi = 0.5 * erfc(-z / sqrt(2.0));
    double phi = exp(-0.5 * z * z) / sqrt(2.0 * R3O_PI);
    return imp * Phi + sigma * phi;
}

/* (4)+(5) score m candidates against one fitted GP. */
void r3o_score(const float *X, const double *L, const double *alpha, double best, const float *ell,
               double sf2, int n, int d, const float *Xcand, long long m, double *mu, double *sigma,
               double *ei)
{
    long long groups = (m + R3O_GROUP - 1) / R3O_GROUP;
#pragma omp parallel
    {
        /* V[i][c]: row i of the right-hand side / solution for candidate c of the group */
        double *V = (double *)malloc((size_t)n * R3O_GROUP * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (long long g = 0; g < groups; ++g) {
            long long c0 = g * R3O_GROUP;
            int nc = (int)((m - c0) < R3O_GROUP ? (m - c0) : R3O_GROUP);
            double mean[R3O_GROUP], vv[R3O_GROUP];
            for (int c = 0; c < R3O_GROUP; ++c) mean[c] = vv[c] = 0.0;
            /* k* and the mean */
            for (int i = 0; i < n; ++i)
                for (int c = 0; c < R3O_GROUP; ++c) {
                    double kv = 0.0;
                    if (c < nc) kv = r3o_kernel(X + (size_t)i * d, Xcand + (size_t)(c0 + c) * d, ell, d, sf2);
                    V[(size_t)i * R3O_GROUP + c] = kv;
                    mean[c] += kv * alpha[i];
                }
            /* forward substitution L v = k*, all candidates of the group at once */
            for (int i = 0; i < n; ++i) {
                const double *Li = L + (size_t)i * n;
                double *Vi = V + (size_t)i * R3O_GROUP;
                for (int k = 0; k < i; ++k) {
                    double lik = Li[k];
                    const double *Vk = V + (size_t)k * R3O_GROUP;
                    for (int c = 0; c < R3O_GROUP; ++c) Vi[c] -= lik * Vk[c];
                }
                double inv = 1.0 / Li[i];
                for (int c = 0; c < R3O_GROUP; ++c) {
                    Vi[c] *= inv;
                    vv[c] += Vi[c] * Vi[c];
                }
            }
            for (int c = 0; c < nc; ++c) {
                double var = sf2 - vv[c];
                if (var < 0.0) var = 0.0;
                double sd = sqrt(var);
                mu[c0 + c] = mean[c];
                sigma[c0 + c] = sd;
                ei[c0 + c] = r3o_ei(mean[c], sd, best);
            }
        }
        free(V);
    }
}

/* (6) top-k by a full sort of (EI descending, index ascending). */
typedef struct { double v; long long i; } r3o_pair;
static int r3o_cmp(const void *a, const void *b)
{
    const r3o_pair *p = (const r3o_pair *)a, *q = (const r3o_pair *)b;
    if (p->v > q->v) return -1;
    if (p->v < q->v) return 1;
    return (p->i > q->i) - (p->i < q->i);
}
int r3o_topk(const double *ei, long long m, int k, long long *idx, double *val)
{
    if (k < 0 || k > m) return -1;
    r3o_pair *p = (r3o_pair *)malloc((size_t)m * sizeof(r3o_pair));
    if (!p) return -2;
    for (long long i = 0; i < m; ++i) { p[i].v = ei[i]; p[i].i = i; }
    qsort(p, (size_t)m, sizeof(r3o_pair), r3o_cmp);
    for (int j = 0; j < k; ++j) { idx[j] = p[j].i; if (val) val[j] = p[j].v; }
    free(p);
    return 0;
}

int r3o_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
