// Internal declarations shared by the translation units of libr3gp (CUDA, sm_100a).
// Nothing here is part of the public ABI; see include/r3.h for that.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "r3.h"

namespace r3 {

// ---------------------------------------------------------------------------------------------
// error text (thread-local) and launch accounting
void set_error(const char* fmt, ...);
extern thread_local unsigned long long g_launches;

#define R3_CUDA_TRY(expr)                                                                \
    do {                                                                                 \
        cudaError_t e__ = (expr);                                                        \
        if (e__ != cudaSuccess) {                                                        \
            r3::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__),       \
                          __FILE__, __LINE__);                                           \
            return e__ == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA;        \
        }                                                                                \
    } while (0)

// Launch a kernel, count it, and turn a launch error into a status.
#define R3_LAUNCH(kernel, grid, block, smem, stream, ...)                                \
    do {                                                                                 \
        kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);                      \
        ++r3::g_launches;                                                                \
        cudaError_t e__ = cudaGetLastError();                                            \
        if (e__ != cudaSuccess) {                                                        \
            r3::set_error("launch of %s failed: %s (%s:%d)", #kernel,                    \
                          cudaGetErrorString(e__), __FILE__, __LINE__);                  \
            return R3_ERR_CUDA;                                                          \
        }                                                                                \
    } while (0)

// Bits of the device status word (one int per handle, OR-ed by kernels).
enum : int {
    DEV_NONFINITE = 1,   // NaN/Inf met in an input
    DEV_NOT_PD = 2,      // non-positive Cholesky pivot
    DEV_TIMEOUT = 4,     // a bounded wait gave up
    DEV_BOUNDS = 8,      // an index check of the bounds-checking build failed (R3_BOUNDS_CHECK)
};

// Index checks of the bounds-checking build (python -m paper_2604_11109_b200.build --check; compute-sanitizer is
// not available where this library is developed).  R3_IDX(i, n, status) is i in the normal build.  In the
// checking build an index outside [0, n) raises DEV_BOUNDS in the handle's status word, leaves the source line
// of the check in the word after the pivot index, and is replaced by 0: the access goes to a valid element
// instead of faulting, control flow stays as it was (warp-wide instructions keep all their lanes), and
// r3_gp_check reports the line.
#ifdef R3_BOUNDS_CHECK
__device__ __forceinline__ long long checked_index(long long i, long long n, int* status, int line)
{
    if (i >= 0 && i < n) return i;
    atomicOr(status, DEV_BOUNDS);
    atomicMax(status + 2, line);
    return 0;
}
#define R3_IDX(i, n, status) r3::checked_index((long long)(i), (long long)(n), (status), __LINE__)
#else
#define R3_IDX(i, n, status) (i)
#endif

constexpr int kFitBlock = 32;   // Cholesky / inverse block size; n is padded to a multiple of it
constexpr int kMaxN = 8192;
constexpr int kMaxD = 256;
constexpr int kMaxK = 1024;
constexpr int kAppendMax = 128;   // observations per r3_gp_append call

// device-memory cache (r3_alloc.cu): cudaMalloc/cudaFree with freed blocks kept for reuse
cudaError_t dev_malloc_bytes(void** p, size_t bytes);
template <typename T>
inline cudaError_t dev_malloc(T** p, size_t bytes)
{
    return dev_malloc_bytes(reinterpret_cast<void**>(p), bytes);
}
void dev_free(void* p);
void trim_cache();
constexpr int kPinnedInts = 128;
int* pinned_word_acquire();          // kPinnedInts pinned host ints from a process-wide pool (nullptr on failure)
void pinned_word_release(int* w);
size_t cached_bytes();

inline int round_up(int a, int b) { return (a + b - 1) / b * b; }
inline long long round_up_ll(long long a, long long b) { return (a + b - 1) / b * b; }

}  // namespace r3

// A top-k that rides on the next scoring call of a handle: the guard kernel, which runs over the final EI
// anyway, leaves the k largest of each of its slices, and the selection's later levels follow at once.
struct TopkRequest {
    int k = 0;                 // 0: none
    int* idx = nullptr;        // device [batch][k]
    float* val = nullptr;      // device [batch][k] or nullptr
    void* ws = nullptr;        // at least guard_topk_workspace_bytes(batch, m, k)
    size_t ws_bytes = 0;
};

// The handle.  Device arrays are allocated at fit time and freed by r3_gp_free.
struct r3_gp {
    int batch = 0, n = 0, d = 0;
    int npad = 0;              // n rounded up to kFitBlock; padded rows/cols are identity / zero
    int device = 0;
    std::vector<float> ell, sf2, sn2, best;   // host copies [batch][d], [batch], [batch], [batch]
    std::vector<float> y_absmax;              // [batch] max |y|
    std::vector<double> wnorm;                // [batch] estimate of |L^-1|_2 (power iteration x 1.5)

    float* X = nullptr;        // [batch][n][d]   raw observations (FP32 as given)
    float* y = nullptr;        // [batch][n]      observed values as given (kept for r3_gp_append)
    float* ell_d = nullptr;    // [batch][d]      lengthscales as given
    float* inv_ell = nullptr;  // [batch][d]      1/lengthscale
    float* sn2_d = nullptr;    // [batch]
    float* sf2_d = nullptr;    // [batch]
    float* best_d = nullptr;   // [batch]
    float* yabs_d = nullptr;   // [batch] max |y|
    double* wnorm_d = nullptr; // [batch]
    double* L64 = nullptr;     // [batch][npad][npad] lower Cholesky factor (upper part zero)
    double* W64 = nullptr;     // [batch][npad][npad] W = L^-1, lower
    float* W32 = nullptr;      // [batch][npad][npad] W rounded to FP32
    double* alpha64 = nullptr; // [batch][npad]  (zero in the padding)
    float* alpha32 = nullptr;  // [batch][npad]
    int* status_d = nullptr;   // [4]: status bits, first bad pivot index, line of a failed index check, unused
    int* status_h = nullptr;   // pinned mirror of status_d
    int* rescued_h = nullptr;  // pinned [64]: candidates recomputed in FP64 by the last scoring call, per GP

    // tensor-core operands (built by fit when the tensor engine can serve (n, d))
    void* tc = nullptr;        // r3::TensorOperands*, see r3_score_tc.cu

    // grow-only private workspace used by scoring and top-k
    void* ws = nullptr;
    size_t ws_bytes = 0;

    r3_engine_t engine_req = R3_ENGINE_AUTO;
    TopkRequest topk_req;      // set by r3_gp_score_topk for the scoring call it makes, consumed by the guard

    // bounded device-side waits of the tensor engine: the limit in cycles, and the test aid that makes one run out
    long long wait_limit_cycles = 4000000000ll;   // about 2 s
    long long withhold_w = -1;

    // optional timing of the dominant scoring kernel: event pairs recorded around its launches
    bool profile = false;
    std::vector<cudaEvent_t> events;   // pairs (start, stop)
    size_t events_used = 0;

    // the host-buffer entry point copies the pool in pieces on a stream of its own while earlier pieces are scored
    cudaStream_t copy_stream = nullptr;
    std::vector<cudaEvent_t> copy_events;
};

namespace r3 {

// fit (r3_fit.cu)
r3_status_t fit_device(r3_gp* gp, const float* y, cudaStream_t stream);
// Appends k observations per GP (r3_gp_append): extends L, W, alpha, X, y in O(k n^2); synchronises.  On
// any error the handle is left as it was.
r3_status_t append_device(r3_gp* gp, const float* Xnew, const float* ynew, int k, cudaStream_t stream);

// SIMT scoring (r3_score_simt.cu)
size_t score_simt_workspace_bytes(const r3_gp* gp, long long m);
r3_status_t score_simt(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei,
                       void* ws, size_t ws_bytes, cudaStream_t stream);

// Accuracy guard and FP64 rescue (r3_rescue.cu).  The engines write their results and, per candidate,
// estimates of their own rounding error in mu (err_mu) and in q = |W k*|^2 (err_q); the guard then
// lists the candidates that may miss the accuracy contract and recomputes them in FP64.
struct GuardBuffers {
    float* err_mu;      // [batch][m]
    float* err_q;       // [batch][m]
    int* count;         // [batch]
    unsigned* maxbits;  // [batch] bit pattern of the largest EI
};
size_t guard_workspace_bytes(const r3_gp* gp, long long m);
// Zeroes the pool's maximum EI and the rescue counters; the engines call it before their first scoring kernel.
r3_status_t guard_begin(r3_gp* gp, const GuardBuffers& b, cudaStream_t stream);
// Key storage the guard kernel needs to leave the first level of a top-k of k (see TopkRequest).
size_t guard_topk_workspace_bytes(int batch, long long m, int k);
GuardBuffers guard_carve(const r3_gp* gp, long long m, void* ws);
// have_max: the engine's kernels have already raised maxbits to the pool's largest EI
r3_status_t guard_and_rescue(r3_gp* gp, const float* Xcand, long long m, const GuardBuffers& b, float* mu,
                             float* sigma, float* ei, bool have_max, cudaStream_t stream);

// tensor-core scoring (r3_score_tc.cu)
bool tc_supported(int n, int d);
r3_status_t tc_prepare(r3_gp* gp, cudaStream_t stream);
void tc_release(r3_gp* gp);
void tc_info(const r3_gp* gp, int* info);   // r3_gp_tensor_info
size_t score_tc_workspace_bytes(const r3_gp* gp, long long m);
r3_status_t score_tc(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei,
                     void* ws, size_t ws_bytes, cudaStream_t stream);
// The same in pieces, for a caller that overlaps the pool's copy with the scoring: tiles [tile_begin, tile_end) of
// the score_tc_tiles(gp, m) tiles of 128 candidates (tile_end < 0: all of them), the guard optionally left to
// one score_tc_guard call after the last piece.
long long score_tc_tiles(const r3_gp* gp, long long m);
bool score_tc_can_split(const r3_gp* gp);
r3_status_t score_tc_part(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                          size_t ws_bytes, long long tile_begin, long long tile_end, bool guard, cudaStream_t stream);
r3_status_t score_tc_guard(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                           cudaStream_t stream);

// top-k (r3_topk.cu)
size_t topk_workspace_bytes(int batch, long long m, int k);
r3_status_t topk_finish_from_keys(unsigned long long* keys_in, unsigned long long* keys_tmp, int batch, long long count,
                                  int k, const float* ei, long long m, int* idx, float* val, cudaStream_t stream);
r3_status_t topk_device(const float* ei, int batch, long long m, int k, int* idx, float* val, void* ws,
                        size_t ws_bytes, cudaStream_t stream);

// log marginal likelihood and gradient (r3_lml.cu): out_h host [batch][d + 3]
r3_status_t lml_device(r3_gp* gp, double* out_h, cudaStream_t stream);

// greedy batch proposal on a shortlist (r3_propose.cu)
size_t propose_workspace_bytes(int batch, int npad, int R, int q);
r3_status_t propose_shortlist(r3_gp* gp, const float* Xcand, long long m, const int* sidx, int Rk, int R, int q, int liar,
                              int* idx_out, float* ei_out, void* ws, cudaStream_t stream);

// fixed (never allocated) key storage for r3_topk_noalloc
r3_status_t topk_static_scratch(void** ptr);
size_t topk_static_capacity_keys();
size_t topk_static_capacity_bytes();

r3_status_t ensure_workspace(r3_gp* gp, size_t bytes);

// Event pair around one launch of the dominant kernel (no-ops unless profiling is on).
void prof_begin(r3_gp* gp, cudaStream_t stream);
void prof_end(r3_gp* gp, cudaStream_t stream);

}  // namespace r3
