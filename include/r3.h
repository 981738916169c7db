/*
 * r3.h -- C ABI of libr3gp: Gaussian-process candidate scoring for the inner
 * Bayesian-optimisation loop of R^3 on one NVIDIA B200 (sm_100a).
 *
 * Where this sits in the paper.  Section IV: for every source candidate the
 * replay server runs a parallel Bayesian-optimisation search over compiler pass
 * configurations and launch parameters and keeps the best runtime.  Section
 * V-B: a sampled point is one replay experiment (pipeline + launch configuration
 * -> runtime), and the mechanism is agnostic to the search strategy.  The paper
 * prints no formula for the surrogate; this library implements the "propose the
 * next points" step with a zero-mean Gaussian process (ARD Matern-5/2
 * covariance), Expected Improvement for minimisation, and top-k selection:
 *
 *   history (X, y)  --r3_gp_fit-->  factor handle
 *   handle, pool    --r3_gp_score-> mu, sigma, EI per candidate
 *   EI              --r3_topk-->    the k pool members to replay next
 *
 * Conventions
 *   - Smaller y is better (y = log-runtime).  A maximiser negates y.
 *   - All matrices are row-major and dense.  "device" pointers are CUDA global
 *     memory of the current device; "host" pointers are ordinary memory.
 *   - The caller owns every array it passes; the library only reads or writes
 *     through the pointer during the call (asynchronously on `cuda_stream` where
 *     stated) and never frees it.  The library owns a handle until r3_gp_free.
 *   - `cuda_stream` is a cudaStream_t cast to void* (NULL = the default stream).
 *   - Every call returns a status and never aborts, throws or prints.  On error
 *     the outputs are unspecified, `*out` (if any) is NULL and r3_last_error()
 *     describes the failure (thread-local text).
 *   - There is no CPU fallback: without a CUDA device every compute entry point
 *     returns R3_ERR_CUDA.
 */
#ifndef R3_H
#define R3_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct r3_gp r3_gp_t; /* opaque; owns device memory */

typedef enum {
    R3_OK = 0,
    R3_ERR_INVALID_ARG = 1,    /* NULL pointer, size out of range, non-positive hyper-parameter */
    R3_ERR_NONFINITE = 2,      /* X, y or Xcand contains NaN/Inf (detected on the device) */
    R3_ERR_NOT_PD = 3,         /* a Cholesky pivot of K(X,X)+noise*I was not positive */
    R3_ERR_ALLOC = 4,          /* device or host allocation failed */
    R3_ERR_CUDA = 5,           /* a CUDA runtime call failed (no device, launch error, ...) */
    R3_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait ran out; results invalid */
    R3_ERR_UNSUPPORTED = 7     /* valid request outside the implemented limits */
} r3_status_t;

/* Scoring engines, for r3_gp_set_engine. */
typedef enum {
    R3_ENGINE_AUTO = 0,   /* tensor-core path where it applies, else SIMT */
    R3_ENGINE_SIMT = 1,   /* FP32 CUDA-core path (direct-difference distances) */
    R3_ENGINE_TENSOR = 2  /* tcgen05 path: FP16-split distance product + triangular contraction, FP32 accumulate */
} r3_engine_t;

/*
 * r3_gp_fit -- condition `batch` independent GPs on their histories.
 *
 * Computes, per GP and in FP64 on the device: K = k(X,X) + noise_var*I with
 *   k(x,z) = signal_var * (1 + s + s^2/3) * exp(-s),  s = sqrt(5) * r,
 *   r^2 = sum_j ((x_j - z_j)/lengthscale_j)^2            (ARD Matern-5/2),
 * its lower Cholesky factor L, the weights alpha = K^-1 y, the inverse factor
 * W = L^-1 used by the variance contraction, and best = min_i y_i.
 * (Inner BO search of Section IV; surrogate as stated above.)
 *
 *   X            device [batch][n][d]   observed configurations (feature rows)
 *   y            device [batch][n]      observed values
 *   lengthscales host   [batch][d]      > 0
 *   signal_var   host   [batch]         > 0
 *   noise_var    host   [batch]         >= 0
 *   batch >= 1, 1 <= n <= 8192, 1 <= d <= 256
 *   out          receives the handle (NULL on error)
 *
 * Synchronises `cuda_stream` before returning, so that R3_ERR_NOT_PD and
 * R3_ERR_NONFINITE are reported by this call.  No jitter is added: a
 * non-positive-definite K is an error, never silently repaired.
 */
r3_status_t r3_gp_fit(const float* X, const float* y, const float* lengthscales,
                      const float* signal_var, const float* noise_var, int batch, int n, int d,
                      void* cuda_stream, r3_gp_t** out);

/*
 * r3_gp_score -- posterior mean, latent standard deviation and Expected
 * Improvement of every candidate of every GP's pool.
 *
 *   k*_i  = k(x_i, x*),  mu = k* . alpha,
 *   sigma = sqrt(max(signal_var - |W k*|^2, 0))       (observation noise NOT added),
 *   z = (best - mu)/sigma,  EI = (best - mu)*Phi(z) + sigma*phi(z);
 *   sigma == 0  ->  EI = max(best - mu, 0).
 *
 *   Xcand  device [batch][m][d]      candidate pool of each GP, 1 <= m < 2^31
 *   mu, sigma, ei  device [batch][m] caller-allocated outputs (FP32)
 *
 * Asynchronous on `cuda_stream`; does not synchronise.  Device-side problems
 * (non-finite candidate, a bounded wait that ran out) are latched in the handle
 * and returned by r3_gp_check.  May grow the handle's private workspace (a
 * synchronising allocation) the first time a larger m is seen.
 */
r3_status_t r3_gp_score(r3_gp_t* gp, const float* Xcand, long long m, float* mu, float* sigma,
                        float* ei, void* cuda_stream);

/*
 * r3_topk -- indices of the k largest values of each row of `ei`.
 *
 *   ei   device [batch][m]
 *   idx  device [batch][k]  int32, sorted by value descending, ties by index ascending
 *   val  device [batch][k]  the selected values, or NULL
 *   1 <= k <= min(m, 1024).  NaN ranks below every number.
 *   scratch / scratch_bytes: device workspace of at least
 *   r3_topk_scratch_bytes(batch, m, k) bytes, or NULL/0 to let the call allocate
 *   and free one itself (which synchronises).
 *
 * Asynchronous on `cuda_stream` when a workspace is supplied.
 */
r3_status_t r3_topk(const float* ei, int batch, long long m, int k, int* idx, float* val,
                    void* scratch, unsigned long long scratch_bytes, void* cuda_stream);
unsigned long long r3_topk_scratch_bytes(int batch, long long m, int k);

/*
 * r3_topk_noalloc -- r3_topk for callers that must not allocate.  (The paper has no counterpart; this
 * entry point exists for the way the library gets embedded.)
 *
 * A replay server that proposes points from inside a latency-critical loop, a host whose device
 * memory is handed out once at start-up by another framework's arena, or any code running where
 * cudaMalloc is off limits (it synchronises the device and can fail late) cannot give r3_topk a
 * workspace sized at run time.  This variant keeps the workspace in a fixed array that is part of the
 * library image: 1 MiB of device memory on every GPU that loads the library, held until the process
 * exits.  The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 *
 *   Same arguments and results as r3_topk (idx/val sorted by value descending, ties by index
 *   ascending), without the scratch pair.
 *   Limit: batch * ceil(m / 4096) * k <= 65536 (e.g. one pool of 1,048,576 values with k <= 256, or
 *   64 pools of 65,536 values with k <= 64); larger requests return R3_ERR_UNSUPPORTED and say so.
 *   The first call on a device looks the array's device address up (once per device, cached); make
 *   that first call before any stream capture begins.
 *   Every call uses the same array and nothing in it needs to start at zero -- each level of the
 *   selection overwrites what the next one reads -- so the previous call's contents are harmless; but
 *   two calls that overlap on the GPU (different streams, no ordering between them) race on it.
 *   Order them, or use r3_topk with separate workspaces.
 * Asynchronous on `cuda_stream`.
 */
r3_status_t r3_topk_noalloc(const float* ei, int batch, long long m, int k, int* idx, float* val,
                            void* cuda_stream);

/*
 * r3_gp_score_topk -- r3_gp_score followed by r3_topk on the EI it produced, with
 * the handle's own workspace; asynchronous on `cuda_stream`.  This is the "one
 * BO proposal round" call: idx [batch][k] are the pool members to replay next.
 * The first level of the selection is taken by the accuracy guard's kernel, which
 * runs over the final EI anyway, so a step is four or five kernel launches.  Once
 * the workspace has its size (a first call with this m and k) the call only
 * enqueues work on `cuda_stream` and can be captured in a CUDA graph.
 */
r3_status_t r3_gp_score_topk(r3_gp_t* gp, const float* Xcand, long long m, int k, float* mu,
                             float* sigma, float* ei, int* idx, float* val, void* cuda_stream);

/*
 * Host-buffer convenience form of r3_gp_score_topk: Xcand and all outputs are
 * HOST arrays (pinned memory makes the copies asynchronous); the call stages
 * them through the handle's workspace, and synchronises the stream before
 * returning.  Any of mu, sigma, ei, val may be NULL to skip that copy.
 */
r3_status_t r3_gp_score_topk_host(r3_gp_t* gp, const float* Xcand_host, long long m, int k,
                                  float* mu_host, float* sigma_host, float* ei_host, int* idx_host,
                                  float* val_host, void* cuda_stream);

/* Synchronise `cuda_stream` and return (then clear) the handle's latched device status. */
r3_status_t r3_gp_check(r3_gp_t* gp, void* cuda_stream);

/*
 * Failure handling of the device-side waits (Section IV discards configurations that fail; the paper says
 * nothing about a surrogate step that fails, so this is the library's own).  Inside the tensor-core
 * scoring kernel the warp roles hand stages to one another through barriers, and every such wait gives
 * up after a limit: the kernel then raises a status bit, lets the copies in flight land, frees its
 * tensor memory and returns, r3_gp_check reports R3_ERR_DEVICE_TIMEOUT, the results of that call are
 * invalid and the handle stays usable.  r3_gp_set_wait_limit sets the limit in SM clock cycles
 * (default 4e9, about two seconds; at least 1e5).
 *
 * r3_gp_test_withhold is a testing aid for that path: on the next tensor-engine scoring call of this
 * handle (one call only) every thread block stops streaming the inverse factor before chunk `chunk`
 * (>= 0) of its own sequence, so that the consumer of that stage waits for data that never comes and
 * its wait runs out.  Nothing faults and nothing waits longer than the limit; use a short limit with it.
 */
r3_status_t r3_gp_set_wait_limit(r3_gp_t* gp, long long cycles);
r3_status_t r3_gp_test_withhold(r3_gp_t* gp, long long chunk);

/* Incumbent used by EI: defaults to min(y); may be overridden per GP.  host [batch]. */
r3_status_t r3_gp_get_best(const r3_gp_t* gp, float* best);
r3_status_t r3_gp_set_best(r3_gp_t* gp, const float* best);

/* Select the scoring engine (default R3_ENGINE_AUTO).  R3_ERR_UNSUPPORTED if the
 * requested engine cannot serve this handle's (n, d). */
r3_status_t r3_gp_set_engine(r3_gp_t* gp, r3_engine_t engine);
/* Engine that r3_gp_score will actually use for this handle. */
r3_engine_t r3_gp_engine(const r3_gp_t* gp);

/*
 * Diagnostics: the shape the tensor-core engine runs this handle in (all zero when it does not serve it).
 * info[0] NV   rows of the inverse factor per pass (columns of the accumulator in tensor memory)
 * info[1] P    passes per tile of 128 candidates (the chunks of k* are generated (P + 1) / 2 times on average)
 * info[2] DP   feature count padded to a multiple of 16 (depth of the distance product)
 * info[3] NP   history length padded to a multiple of NV
 * info[4] G    Matern warp groups;  info[5] W stages in shared memory;  info[6] 1: k* operand in tensor memory
 * info[7] 1: the cross terms of the variance product are FP8 MMAs (histories of eight passes and more)
 */
r3_status_t r3_gp_tensor_info(const r3_gp_t* gp, int* info /* host [8] */);

/*
 * Diagnostics: synchronises `cuda_stream` and returns how many candidates the last scoring call on
 * this handle recomputed in FP64 (summed over the first 64 GPs of the batch).  The scoring engines
 * work at FP32 level and hand to an FP64 pass every candidate whose estimated rounding error could
 * exceed the accuracy contract (candidates on top of observations, ill-conditioned histories).
 */
r3_status_t r3_gp_last_rescued(r3_gp_t* gp, void* cuda_stream, long long* total);

/*
 * Timing of the dominant scoring kernel (the variance contraction).  While enabled, every launch
 * of that kernel is bracketed by a CUDA event pair on the launching stream.  r3_gp_profile_read
 * waits for the recorded events, returns the summed kernel time in milliseconds and the number
 * of launches it covers, and clears the record.  Off by default; costs two event records per launch.
 */
r3_status_t r3_gp_profile(r3_gp_t* gp, int enable);
r3_status_t r3_gp_profile_read(r3_gp_t* gp, double* kernel_ms, long long* launches);

/*
 * r3_gp_lml -- log marginal likelihood of each GP's history under its current hyper-parameters, and
 * its gradient with respect to their logarithms: the objective of a hyper-parameter fit (the paper
 * passes lengthscales and variances in and says nothing about choosing them).
 *
 *   lml  = -1/2 y.alpha - 1/2 log|K| - n/2 log(2 pi),         K = k(X,X) + noise_var I, alpha = K^-1 y
 *   grad = 1/2 trace((alpha alpha^T - K^-1) dK/dtheta)  for theta = (log lengthscale_1..d,
 *          log signal_var, log noise_var), with dK/dlog lengthscale_j = signal_var e^-s (5/3)(1+s) u_j^2,
 *          u_j = (x_j - z_j)/lengthscale_j, s = sqrt(5 sum_j u_j^2).
 *
 *   lml   host [batch]  FP64            grad  host [batch][d + 2]  FP64, or NULL
 *
 * FP64 on the device from the factor the handle holds (K^-1 = W^T W costs n^3/3 multiply-adds);
 * synchronises `cuda_stream`; allocates temporary device memory.
 */
r3_status_t r3_gp_lml(r3_gp_t* gp, double* lml, double* grad, void* cuda_stream);

/*
 * r3_gp_refit -- condition the GPs of the handle on the same histories with other hyper-parameters
 * (arguments as for r3_gp_fit; the histories are the ones the handle holds, appended observations
 * included).  Synchronises.  On R3_ERR_NOT_PD the handle is refitted with its previous
 * hyper-parameters and stays usable.
 */
r3_status_t r3_gp_refit(r3_gp_t* gp, const float* lengthscales, const float* signal_var, const float* noise_var,
                        void* cuda_stream);

/*
 * r3_gp_optimize -- choose the hyper-parameters of every GP of the handle by maximising its log
 * marginal likelihood (r3_gp_lml) over theta = (log lengthscale_1..d, log signal_var, log noise_var),
 * starting from the handle's current values.  (The paper passes hyper-parameters in and gives no rule
 * for them; this is the usual type-II maximum likelihood.)
 *
 * Limited-memory BFGS (8 pairs) with a backtracking Armijo line search, one optimiser per GP, all GPs
 * evaluated together: an evaluation is one batched refit plus one r3_gp_lml.  theta is kept inside
 * lengthscale in [1e-3, 1e3], signal_var in [1e-6, 1e6], noise_var in [1e-8 , 1e2] by projection.
 * A GP stops when the largest projected gradient component falls below gtol or its line search
 * cannot improve; the call stops when every GP has stopped or after max_evals evaluations.  A trial
 * point at which some covariance matrix is not positive definite counts as a failed step for every GP
 * still searching (their steps are halved).
 *
 *   max_evals >= 1, gtol > 0
 *   lengthscales host [batch][d], signal_var host [batch], noise_var host [batch]   outputs (FP32), any may be NULL
 *   lml          host [batch]   the log marginal likelihood reached, or NULL
 *   evals        host [1]       evaluations used, or NULL
 *
 * On return the handle is fitted with the returned hyper-parameters (never worse than the start).
 * Synchronises.
 */
r3_status_t r3_gp_optimize(r3_gp_t* gp, int max_evals, double gtol, float* lengthscales, float* signal_var,
                           float* noise_var, double* lml, int* evals, void* cuda_stream);

/*
 * r3_gp_propose -- q distinct pool members to replay in parallel, chosen greedily by fantasies.
 *
 * Section IV runs a parallel search: several points are in flight at once.  The paper gives no rule
 * for choosing them; this is the usual sequential one.  q times: take the not-yet-picked candidate
 * of largest EI (incumbent fixed at the best observed value; ties to the lower index), then
 * condition the GP on it with a fantasised value rounded to FP32 -- its posterior mean
 * (lie = 0, "believer") or the incumbent (lie = 1, "liar").  The handle itself is not changed.
 *
 * Conditioning on one point is a rank-one update of every candidate's mean and variance, so the pool
 * is scored once (as r3_gp_score does) and the q picks run on a shortlist of the `shortlist` best
 * candidates of that scoring, recomputed in FP64.  With the believer's value EI can only drop from
 * pick to pick, so the shortlist loses nothing as long as every pick's EI stays above the best EI left
 * outside it: certified[g] = 1 says that this held for GP g (or that the shortlist was the whole
 * pool).  With lie = 1 a shortlist smaller than the pool is a heuristic and certified is 0.
 *
 *   Xcand      device [batch][m][d]
 *   q          1 <= q <= min(m, 256)
 *   shortlist  0 = automatic (max(8 q, 256), at most m and 1023), else q <= shortlist <= min(m, 1023)
 *   idx        device [batch][q] int32, in pick order
 *   ei_pick    device [batch][q] EI of each pick when it was picked, or NULL
 *   certified  host   [batch], or NULL
 *
 * Synchronises `cuda_stream`; allocates temporary device memory.
 */
r3_status_t r3_gp_propose(r3_gp_t* gp, const float* Xcand, long long m, int q, int shortlist, int lie, int* idx,
                          float* ei_pick, int* certified, void* cuda_stream);

/*
 * r3_gp_append -- add k observations to every GP of the handle without refactoring the history.
 *
 * One BO round ends with k replayed points; conditioning on them is a rank-k extension of the factor,
 * O(k n^2), instead of the O(n^3) of a new r3_gp_fit (the loop of Section IV: propose, replay, update).
 * With K' = [[K, B], [B^T, C]]:  L21 = (L^-1 B)^T,  L22 L22^T = C - L21 L21^T,  W' = L'^-1 by blocks,
 * alpha' = K'^-1 y'.  The handle afterwards equals, up to FP64 rounding, the one r3_gp_fit returns for
 * the concatenated history with the same hyper-parameters; best becomes min(y') (an incumbent set
 * with r3_gp_set_best is replaced) and the scoring engine is chosen again for the new size.  L21 is
 * formed with the stored inverse factor; when K is ill-conditioned (|L^-1|_2^2 (signal_var + noise_var)
 * above 1e8) one step of iterative refinement with L itself follows, so that the extension stays as
 * accurate as a fit there.
 *
 *   Xnew  device [batch][k][d]     ynew  device [batch][k]      1 <= k <= 128,  n + k <= 8192
 *
 * Synchronises `cuda_stream`.  On any error (R3_ERR_NONFINITE, R3_ERR_NOT_PD with the failing pivot in
 * r3_last_error, allocation failure) the handle is unchanged and still usable.
 */
r3_status_t r3_gp_append(r3_gp_t* gp, const float* Xnew, const float* ynew, int k, void* cuda_stream);

/* Number of observations per GP currently in the handle. */
int r3_gp_size(const r3_gp_t* gp);

/* Copy fit results to host arrays (diagnostics and tests): alpha [batch][n] FP64,
 * L [batch][n][n] FP64 lower-triangular (upper part zero).  Either may be NULL. */
r3_status_t r3_gp_get_factor(const r3_gp_t* gp, double* alpha, double* L);

/* Kernels launched by this library on the calling thread since the last reset. */
unsigned long long r3_launch_count(void);
void r3_launch_count_reset(void);

void r3_gp_free(r3_gp_t* gp);

/* ------------------------------------------------------------------------------------------------
 * The inner search as a whole (Section IV, the loop inside the replay server): fit the surrogate,
 * propose a batch of points to replay in parallel, replay them, discard the configurations that make
 * the kernel incorrect, add the rest to the history, repeat until a stopping rule fires, return the
 * best configuration found.  The three stopping rules are the paper's: a maximum number of
 * iterations, a maximum wall-clock time, a number of iterations without improvement.
 *
 * The replay itself is the caller's: `evaluate` gets q configurations (host, [q][d], rows of the pool)
 * and returns a value for each (smaller is better) and whether the kernel stayed correct (valid[i] != 0).
 * It returns 0 to go on, anything else to stop the search.
 */
typedef int (*r3_evaluate_fn)(const float* x, int q, int d, float* y, int* valid, void* user);

typedef struct {
    int q;               /* points proposed per round, 1..128 */
    int max_rounds;      /* stop after this many rounds, >= 1 */
    double max_seconds;  /* stop when this much wall-clock time has passed, <= 0: no limit */
    int patience;        /* stop after this many rounds in a row without a better value, <= 0: no limit */
    int optimize_every;  /* refit the hyper-parameters by r3_gp_optimize every this many rounds, <= 0: never; the noise
                            is then kept at or above 1e-6 signal_var, and raised tenfold (up to six times) if an
                            update meets a numerically singular matrix */
    int lie;             /* fantasised value of r3_gp_propose: 0 believer, 1 liar */
    int surrogate;       /* 0: Gaussian process (r3_gp_fit / r3_gp_propose / r3_gp_append);
                            1: Tree-Parzen estimator, the paper's choice (Section VII-C: parallel TPE): every round
                               r3_tpe_fit on the history so far, r3_tpe_score on the pool, the q best by r3_topk */
    const int* levels;   /* surrogate 1: kind of each feature as for r3_tpe_fit, host [d]; NULL = all ordinal */
    float gamma;         /* surrogate 1: good fraction, <= 0: 0.25 */
} r3_bo_options_t;

typedef enum {
    R3_BO_MAX_ROUNDS = 0, R3_BO_MAX_SECONDS = 1, R3_BO_NO_IMPROVEMENT = 2, R3_BO_POOL_EXHAUSTED = 3,
    R3_BO_HISTORY_FULL = 4, R3_BO_STOPPED_BY_CALLER = 5
} r3_bo_stop_t;

/*
 * r3_bo_run -- the loop above on one GP.
 *
 *   X0, y0     device [n0][d], [n0]   initial history (n0 >= 1)
 *   lengthscales host [d], signal_var, noise_var: starting hyper-parameters
 *   pool       device [m][d]          candidate configurations; the call works on a private copy from which
 *                                     every proposed row is removed, so no configuration is replayed twice
 *   best_x     host [d], best_y host [1]: the best valid configuration seen (initial history included)
 *   rounds, evaluated, discarded, stop_reason: host [1] each, any may be NULL
 *   gp_out     if not NULL receives the final handle (the caller frees it); otherwise it is freed
 *
 * With the GP every proposal is made by r3_gp_propose and every update by r3_gp_append; with the Parzen
 * estimator the hyper-parameter arguments are ignored, gp_out receives NULL and the history is refitted
 * every round (its fit is a few sorts).  Synchronises.
 */
r3_status_t r3_bo_run(const float* X0, const float* y0, int n0, int d, const float* lengthscales, float signal_var,
                      float noise_var, const float* pool, long long m, const r3_bo_options_t* options,
                      r3_evaluate_fn evaluate, void* user, float* best_x, float* best_y, int* rounds, int* evaluated,
                      int* discarded, int* stop_reason, r3_gp_t** gp_out, void* cuda_stream);

/* ------------------------------------------------------------------------------------------------
 * Tree-structured Parzen Estimator (TPE) candidate scoring.
 *
 * Section VII-C: inside the replay server the paper's experiments tune pass order and launch
 * parameters with parallel Tree Parzen Estimation for 30 iterations.  The paper prints no formula,
 * quantile, bandwidth rule or prior for it; the definition implemented here is this library's own
 * statement of the estimator, steps (T1)-(T4):
 *
 *   (T1) n_good = min(max(1, ceil(gamma*n)), n); sort the history by y ascending (ties: lower
 *        index); the first n_good observations are the "good" set, the rest the "bad" set.
 *   (T2) ordinal / continuous dimension (levels[j] == 0), per set with s values: a mixture of s + 1
 *        normal densities truncated to [0, 1] -- one per value (weight 1) and a prior (weight
 *        prior_weight, mean 1/2, sigma 1).  With the s + 1 means sorted ascending (the prior after
 *        equal values), a value's sigma is the larger gap to its neighbours, clipped to
 *        [1/min(100, s + 1), 1].
 *   (T3) categorical dimension (levels[j] == C, 2 <= C <= 64): level v = clamp(floor(x*(C-1) + 1/2),
 *        0, C-1) with the product and the sum each rounded to FP32;
 *        P(v) = (count_v + prior_weight/C) / (s + prior_weight).
 *   (T3g) ordinal dimension on a known grid (levels[j] == -L, 2 <= L <= 64; admissible values v/(L-1)):
 *        the mixture of (T2), evaluated at the candidate's nearest grid value (level as in (T3), value
 *        v/(L-1) rounded to FP32).  The L log-density ratios are tabulated by r3_tpe_fit, so such a
 *        dimension costs one look-up per candidate instead of n + 2 exponentials.
 *   (T4) score(x) = sum_j [ ln l_j(x_j) - ln g_j(x_j) ], l from the good set, g from the bad set.
 *        Larger is better; pass the scores to r3_topk to pick the next points.
 *
 * Features are expected in [0, 1] (normalised); values outside are evaluated with the same formulas.
 */
typedef struct r3_tpe r3_tpe_t; /* opaque; owns device memory */

/*
 * r3_tpe_fit -- steps (T1)-(T3) on the device: order of the history, mixtures and level tables.
 *
 *   X       device [n][d]   observed configurations, row-major
 *   y       device [n]      observed values (smaller is better)
 *   levels  host   [d]      0 = ordinal/continuous, C in [2, 64] = categorical with C levels,
 *                           -L in [-64, -2] = ordinal on the grid v/(L-1)
 *   1 <= n <= 4096, 1 <= d <= 256, 0 < gamma <= 1, prior_weight > 0
 *   out     receives the handle (NULL on error)
 *
 * Synchronises `cuda_stream` before returning; a NaN/Inf in X or y returns R3_ERR_NONFINITE.
 */
r3_status_t r3_tpe_fit(const float* X, const float* y, const int* levels, int n, int d, float gamma,
                       float prior_weight, void* cuda_stream, r3_tpe_t** out);

/*
 * r3_tpe_score -- step (T4) for every candidate of a pool.
 *
 *   Xcand  device [m][d], 1 <= m < 2^31        score  device [m] (FP32, caller-allocated)
 *
 * Asynchronous on `cuda_stream`; does not synchronise and does not allocate.  A non-finite candidate
 * is latched in the handle and reported by r3_tpe_check.
 */
r3_status_t r3_tpe_score(r3_tpe_t* tpe, const float* Xcand, long long m, float* score, void* cuda_stream);

/* Synchronises the stream and returns (and clears) the status latched by device code since the last
 * check: R3_OK or R3_ERR_NONFINITE. */
r3_status_t r3_tpe_check(r3_tpe_t* tpe, void* cuda_stream);

/*
 * r3_tpe_get_model -- copy the fitted model to host memory (for inspection and tests); synchronises.
 * Any output pointer may be NULL.
 *
 *   n_good  host [1]
 *   order   host [n]              history indices by y ascending
 *   comps   host [d][n + 2][4]    per dimension the good set's components from entry 0 and the bad set's
 *                                 from entry n_good + 1, each set sorted by mean:
 *                                 {mean, log2(e)/(2 sigma^2), log2(weight/(sigma Z sqrt(2 pi))), sigma}.
 *                                 Components of one set with the same mean and the same sigma (repeated
 *                                 values of a discrete feature) are stored once, with their weights
 *                                 summed; entries past a set's count are unspecified
 *   counts  host [d][2]           components stored for the good and the bad set (at most n_good + 1 and
 *                                 n - n_good + 1); zero for a categorical dimension
 *   table   host [d][64]          ln P_good(v) - ln P_bad(v) per level v of a categorical dimension,
 *                                 ln l(v/(L-1)) - ln g(v/(L-1)) per grid value of a grid dimension; zero elsewhere
 */
r3_status_t r3_tpe_get_model(r3_tpe_t* tpe, int* n_good, int* order, float* comps, int* counts, float* table);

/* Frees the handle and its device memory; NULL is allowed. */
void r3_tpe_free(r3_tpe_t* tpe);

/*
 * Device memory the library has freed is kept (per device, at most 2 GiB, blocks of 1 MiB and more) and
 * handed out again by later calls, because allocating and freeing the 100 MB arrays of a fit costs more
 * than the kernels of an append.  r3_trim_cache returns the kept blocks of the current device to the
 * driver; r3_cached_bytes reports how much is kept.
 */
void r3_trim_cache(void);
unsigned long long r3_cached_bytes(void);

/*
 * Testing aid for the allocation-failure paths (host side; no device is touched): the device
 * allocation number `after` from now on (0 = the very next one) made by the calling process through
 * this library fails once as if the device were out of memory, so that a caller can check that
 * r3_gp_fit returns R3_ERR_ALLOC without leaking and that r3_gp_append leaves its handle unchanged.
 * A negative value disarms it.  Returns how many allocations were counted since it was last armed.
 */
long long r3_test_fail_allocation(long long after);

const char* r3_status_string(r3_status_t status);
const char* r3_last_error(void);
int r3_version(void);

#ifdef __cplusplus
}
#endif
#endif /* R3_H */
