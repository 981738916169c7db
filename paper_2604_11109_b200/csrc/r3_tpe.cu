// Tree-structured Parzen Estimator: fit (order of the history, per-dimension mixtures and level
// tables) and candidate scoring (log-density ratio), steps (T1)-(T4) of the definition in r3.h.
//
// Fit is small (n <= 4096): one block sorts the history by y, then one block per dimension sorts each
// set's values (bitonic network in shared memory), derives the bandwidths from the neighbour gaps in
// FP64 and stores every component as {mean, a, b, sigma} with
//     a = log2(e) / (2 sigma^2),   b = log2( weight / (sum of weights * sigma * Z * sqrt(2 pi)) ),
// so that the scoring kernel evaluates a component as exp2(b - a (x - mean)^2): one subtraction, one
// multiplication, one fused multiply-add, one MUFU.EX2 and one addition per (candidate, component).
// Scoring is bound by the MUFU unit (16 results per clock per SM); the components of a dimension are
// staged through shared memory and every thread carries one or two candidates.
#include <math.h>
#include <stdlib.h>

#include <algorithm>
#include <new>
#include <vector>

#include "r3_internal.cuh"

struct r3_tpe {
    int n = 0, d = 0, n_good = 0, device = 0;
    float prior_weight = 1.f;
    std::vector<int> levels;
    int* levels_d = nullptr;   // [d]
    int* order_d = nullptr;    // [n] history indices by y ascending
    float4* comps_d = nullptr; // [d][n + 2]: good set's components from 0, the bad set's from n_good + 1
    int* counts_d = nullptr;   // [d][2]: components of each set after merging equal ones
    // a model small enough for shared memory is also kept packed: set (j, s) at [offs[2j + s], offs[2j + s + 1])
    int total = 0;             // components kept over all dimensions and sets
    bool resident = false;     // the packed model is in use
    float4* packed_d = nullptr;
    int* offs_d = nullptr;     // [2d + 1]
    char* arena_d = nullptr;   // the one allocation all device pointers of the handle point into
    float* table_d = nullptr;  // [d][64] ln P_good - ln P_bad per level
    int* status_d = nullptr;   // status bits
    int* status_h = nullptr;   // pinned mirror
};

namespace r3 {

namespace {

constexpr int kTpeMaxN = 4096;
constexpr int kTpeMaxLevels = 64;
constexpr int kSortThreads = 1024;
constexpr int kScoreThreads = 256;
constexpr int kStage = 512;   // components per shared-memory stage
constexpr size_t kResidentBytes = 72 * 1024;   // largest model a scoring block keeps whole in shared memory

// Unsigned integer with the same order as the float (-0 and +0 equal).
__device__ __forceinline__ unsigned ordered_bits(float v)
{
    if (v == 0.0f) v = 0.0f;
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(unsigned u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// Ascending bitonic sort of `count` (a power of two) 64-bit keys in shared memory.
__device__ void bitonic_sort_asc(unsigned long long* s, int count)
{
    for (int size = 2; size <= count; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < count / 2; t += blockDim.x) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool asc = ((lo & size) == 0);
                const unsigned long long a = s[lo], b = s[hi];
                if ((a > b) == asc) {
                    s[lo] = b;
                    s[hi] = a;
                }
            }
        }
    }
    __syncthreads();
}

__device__ __forceinline__ int pow2_at_least(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// (T1) order[i] = index of the i-th smallest y, ties by lower index.
__global__ void __launch_bounds__(kSortThreads) tpe_order_kernel(const float* __restrict__ y, int n,
                                                                 int* __restrict__ order, int* __restrict__ status)
{
    __shared__ unsigned long long keys[kTpeMaxN];
    const int count = pow2_at_least(n);
    bool bad = false;
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        unsigned long long k = ~0ull;
        if (i < n) {
            const float v = y[i];
            bad |= !isfinite(v);
            k = ((unsigned long long)ordered_bits(v) << 32) | (unsigned)i;
        }
        keys[i] = k;
    }
    if (bad) atomicOr(status, DEV_NONFINITE);
    bitonic_sort_asc(keys, count);
    for (int i = threadIdx.x; i < n; i += blockDim.x) order[i] = (int)(keys[i] & 0xFFFFFFFFull);
}

// (T2), (T3): one block per (dimension, set).  The log-probabilities (categorical) or log-densities (grid) of a
// set go to lnp[j][set][v]; tpe_table_kernel subtracts the two sets afterwards.
__global__ void __launch_bounds__(kSortThreads) tpe_mixture_kernel(const float* __restrict__ X,
                                                                   const int* __restrict__ order, int n, int d,
                                                                   int n_good, const int* __restrict__ levels,
                                                                   double prior_weight, float4* __restrict__ comps,
                                                                   int* __restrict__ n_comps, double* __restrict__ lnp_out,
                                                                   int* __restrict__ status)
{
    extern __shared__ unsigned long long keys[];   // pow2 >= n + 1 keys, then (grid dimensions) 2 (n + 1) doubles
    __shared__ int counts[kTpeMaxLevels];
    __shared__ double wsum_s[32];
    const int j = blockIdx.x >> 1;
    const int code = levels[j];
    const int C = code > 0 ? code : 0;      // categorical levels
    const int G = code < 0 ? -code : 0;     // grid values of an ordinal dimension
    bool bad = false;
    double* lnp_set = lnp_out + ((size_t)j * 2 + (blockIdx.x & 1)) * kTpeMaxLevels;
    for (int set = blockIdx.x & 1; set == (int)(blockIdx.x & 1); set += 2) {
        const int s = set == 0 ? n_good : n - n_good;
        const int first = set == 0 ? 0 : n_good;            // position in `order`
        float4* out = comps + (size_t)j * (n + 2) + (set == 0 ? 0 : n_good + 1);
        if (C > 0) {
            // ---- (T3) smoothed level frequencies
            for (int v = threadIdx.x; v < kTpeMaxLevels; v += blockDim.x) counts[v] = 0;
            __syncthreads();
            for (int i = threadIdx.x; i < s; i += blockDim.x) {
                const float x = X[(size_t)order[first + i] * d + j];
                bad |= !isfinite(x);
                const float lv = floorf(__fadd_rn(__fmul_rn(x, (float)(C - 1)), 0.5f));
                const int v = (int)fminf(fmaxf(lv, 0.f), (float)(C - 1));
                atomicAdd(&counts[isfinite(x) ? v : 0], 1);
            }
            __syncthreads();
            for (int v = threadIdx.x; v < C; v += blockDim.x) {
                lnp_set[v] = log(((double)counts[v] + prior_weight / C) / ((double)s + prior_weight));
            }
            if (threadIdx.x == 0) n_comps[2 * j + set] = 0;
            __syncthreads();
            continue;
        }
        // ---- (T2) sort the s values and the prior mean; the prior (index s) goes after equal values
        const int count = pow2_at_least(s + 1);
        for (int i = threadIdx.x; i < count; i += blockDim.x) {
            unsigned long long k = ~0ull;
            if (i < s) {
                const float x = X[(size_t)order[first + i] * d + j];
                bad |= !isfinite(x);
                k = ((unsigned long long)ordered_bits(isfinite(x) ? x : 0.f) << 32) | (unsigned)i;
            } else if (i == s) {
                k = ((unsigned long long)ordered_bits(0.5f) << 32) | (unsigned)s;
            }
            keys[i] = k;
        }
        bitonic_sort_asc(keys, count);
        const double sigma_lo = 1.0 / fmin(100.0, (double)s + 1.0);
        const double wsum = (double)s + prior_weight;
        for (int t = threadIdx.x; t <= s; t += blockDim.x) {
            const unsigned long long k = keys[t];
            const bool is_prior = (int)(k & 0xFFFFFFFFull) == s;
            const double mu = (double)from_ordered_bits((unsigned)(k >> 32));
            double sigma = 1.0;
            if (!is_prior) {
                double gap = -1.0;
                if (t > 0) gap = fmax(gap, mu - (double)from_ordered_bits((unsigned)(keys[t - 1] >> 32)));
                if (t < s) gap = fmax(gap, (double)from_ordered_bits((unsigned)(keys[t + 1] >> 32)) - mu);
                sigma = fmin(fmax(gap, sigma_lo), 1.0);
            }
            const double w = is_prior ? prior_weight : 1.0;
            const double Z = 0.5 * erfc(-(1.0 - mu) / sigma * 0.70710678118654752440) -
                             0.5 * erfc(-(0.0 - mu) / sigma * 0.70710678118654752440);
            double* par = reinterpret_cast<double*>(keys + count);
            par[2 * t] = sigma;
            par[2 * t + 1] = w / (wsum * sigma * Z * 2.5066282746310005024);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            // Components with the same mean and bandwidth (repeated values of a discrete feature) are one
            // component with the summed coefficient: the density is the same sum, with far fewer terms.
            // Equal means are neighbours in the sorted order; among them a run of equal values has one
            // bandwidth inside and one at each end, so a handful of open slots per mean is enough (a full
            // set of slots emits its oldest one, which only costs a missed merge).
            constexpr int kSlots = 4;
            const double* par = reinterpret_cast<const double*>(keys + count);
            int c = 0, open = 0;
            unsigned run_mu = 0;
            double slot_sigma[kSlots], slot_coef[kSlots];
            auto emit = [&](int i) {
                const double a = 1.4426950408889634074 / (2.0 * slot_sigma[i] * slot_sigma[i]);
                out[c++] = make_float4(from_ordered_bits(run_mu), (float)a, (float)log2(slot_coef[i]), (float)slot_sigma[i]);
            };
            for (int t = 0; t <= s; ++t) {
                const unsigned mu_bits = (unsigned)(keys[t] >> 32);
                if (mu_bits != run_mu) {
                    for (int i = 0; i < open; ++i) emit(i);
                    open = 0;
                    run_mu = mu_bits;
                }
                const double sigma = par[2 * t], coef = par[2 * t + 1];
                int hit = -1;
                for (int i = 0; i < open; ++i)
                    if (slot_sigma[i] == sigma) hit = i;
                if (hit >= 0) {
                    slot_coef[hit] += coef;
                    continue;
                }
                if (open == kSlots) {
                    emit(0);
                    for (int i = 1; i < kSlots; ++i) slot_sigma[i - 1] = slot_sigma[i], slot_coef[i - 1] = slot_coef[i];
                    --open;
                }
                slot_sigma[open] = sigma;
                slot_coef[open++] = coef;
            }
            for (int i = 0; i < open; ++i) emit(i);
            n_comps[2 * j + set] = c;
        }
        __syncthreads();
        if (G > 0) {
            // (T3g) the mixture at each of the G grid values, in FP64; the warps' sums are added in order
            const double* par = reinterpret_cast<const double*>(keys + count);
            for (int v = 0; v < G; ++v) {
                const double xg = (double)(float)((double)v / (double)(G - 1));
                double acc = 0.0;
                for (int t = threadIdx.x; t <= s; t += blockDim.x) {
                    const double z = (xg - (double)from_ordered_bits((unsigned)(keys[t] >> 32))) / par[2 * t];
                    acc += par[2 * t + 1] * exp(-0.5 * z * z);
                }
                for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if ((threadIdx.x & 31) == 0) wsum_s[threadIdx.x / 32] = acc;
                __syncthreads();
                if (threadIdx.x == 0) {
                    double tot = 0.0;
                    for (int w = 0; w < (int)blockDim.x / 32; ++w) tot += wsum_s[w];
                    lnp_set[v] = log(tot);
                }
                __syncthreads();
            }
        }
    }
    if (bad) atomicOr(status, DEV_NONFINITE);
}

// (T3), (T3g): table[j][v] = ln l_j(v) - ln g_j(v) for the tabulated dimensions, zero elsewhere
__global__ void tpe_table_kernel(const int* __restrict__ levels, const double* __restrict__ lnp, int d,
                                 float* __restrict__ table)
{
    const int j = blockIdx.x, v = threadIdx.x;
    const int code = levels[j];
    const int cnt = code < 0 ? -code : code;
    const double* l = lnp + (size_t)j * 2 * kTpeMaxLevels;
    table[(size_t)j * kTpeMaxLevels + v] = v < cnt ? (float)(l[v] - l[kTpeMaxLevels + v]) : 0.f;
}

__device__ __forceinline__ float ex2_fast(float x)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float lg2_fast(float x)
{
    float r;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// sum over `count` components of exp2(b - a (x - mean)^2) for R candidates at once.  The components are
// staged through shared memory by the whole block (all of its threads must call this together): one
// broadcast LDS.128 per component instead of a global load per thread was worth 14 % on the full pool.
template <int R>
__device__ __forceinline__ void mixture_sums_staged(const float4* __restrict__ comp, int count, const float (&x)[R],
                                                    float (&sum)[R], float4* stage)
{
    // four partial sums per candidate: independent add chains, and half the rounding of one long sum
    float part[4][R];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int r = 0; r < R; ++r) part[u][r] = 0.f;
    for (int c0 = 0; c0 < count; c0 += kStage) {
        const int nc = min(kStage, count - c0);
        __syncthreads();
        for (int i = threadIdx.x; i < nc; i += kScoreThreads) stage[i] = __ldg(comp + c0 + i);
        __syncthreads();
        int c = 0;
        for (; c + 4 <= nc; c += 4) {
            float4 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) q[u] = stage[c + u];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float t = x[r] - q[u].x;
                    part[u][r] += ex2_fast(fmaf(-t, t * q[u].y, q[u].z));
                }
            }
        }
        for (; c < nc; ++c) {
            const float4 q = stage[c];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float t = x[r] - q.x;
                part[c & 3][r] += ex2_fast(fmaf(-t, t * q.y, q.z));
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) sum[r] = (part[0][r] + part[1][r]) + (part[2][r] + part[3][r]);
}

// (T4) score of every candidate.  A block covers R * blockDim.x consecutive candidates; thread t holds
// candidates t, t + blockDim.x, ... of the block's range so that the result stores coalesce.
template <int R>
__global__ void __launch_bounds__(kScoreThreads) tpe_score_kernel(const float* __restrict__ Xc, long long m, int n,
                                                                  int d, int n_good, const int* __restrict__ levels,
                                                                  const float4* __restrict__ comps,
                                                                  const int* __restrict__ counts,
                                                                  const float* __restrict__ table,
                                                                  float* __restrict__ score, int* __restrict__ status)
{
    const long long tiles = (m + (long long)R * kScoreThreads - 1) / ((long long)R * kScoreThreads);
    bool bad = false;
    __shared__ float4 stage[kStage];
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long base = tile * (long long)R * kScoreThreads + threadIdx.x;
        const float* row[R];
        bool valid[R];
        float acc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const long long cand = base + (long long)r * kScoreThreads;
            valid[r] = cand < m;
            row[r] = Xc + (size_t)(valid[r] ? cand : 0) * d;
            acc[r] = 0.f;
        }
        for (int j = 0; j < d; ++j) {
            float x[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r] = row[r][j];
                bad |= valid[r] && !isfinite(x[r]);
            }
            const int code = __ldg(levels + j);
            const int C = code < 0 ? -code : code;   // categorical levels, or grid values of an ordinal dimension
            if (C > 0) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float lv = floorf(__fadd_rn(__fmul_rn(x[r], (float)(C - 1)), 0.5f));
                    const int v = isfinite(x[r]) ? (int)fminf(fmaxf(lv, 0.f), (float)(C - 1)) : 0;
                    acc[r] += __ldg(table + (size_t)j * kTpeMaxLevels + v);
                }
            } else {
                const float4* cj = comps + (size_t)j * (n + 2);
                float sl[R], sg[R];
                mixture_sums_staged<R>(cj, __ldg(counts + 2 * j), x, sl, stage);
                mixture_sums_staged<R>(cj + n_good + 1, __ldg(counts + 2 * j + 1), x, sg, stage);
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] += 0.69314718f * (lg2_fast(sl[r]) - lg2_fast(sg[r]));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (valid[r]) score[base + (long long)r * kScoreThreads] = acc[r];
    }
    if (bad) atomicOr(status, DEV_NONFINITE);
}

// One (dimension, set) per block: copy its kept components to their place in the packed model.
__global__ void __launch_bounds__(256) tpe_pack_kernel(const float4* __restrict__ comps, int n, int n_good,
                                                       const int* __restrict__ offs, float4* __restrict__ packed)
{
    const int j = blockIdx.x >> 1, set = blockIdx.x & 1;
    const float4* src = comps + (size_t)j * (n + 2) + (set ? n_good + 1 : 0);
    const int lo = offs[blockIdx.x], hi = offs[blockIdx.x + 1];
    for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) packed[i] = src[i - lo];
}

// sum over components [lo, hi) of a model held in shared memory, for R candidates at once
template <int R>
__device__ __forceinline__ void mixture_sums_resident(const float4* __restrict__ model, int lo, int hi,
                                                      const float (&x)[R], float (&sum)[R])
{
    float part[4][R];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int r = 0; r < R; ++r) part[u][r] = 0.f;
    int c = lo;
    for (; c + 4 <= hi; c += 4) {
        float4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) q[u] = model[c + u];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float t = x[r] - q[u].x;
                part[u][r] += ex2_fast(fmaf(-t, t * q[u].y, q[u].z));
            }
        }
    }
    for (; c < hi; ++c) {
        const float4 q = model[c];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float t = x[r] - q.x;
            part[(c - lo) & 3][r] += ex2_fast(fmaf(-t, t * q.y, q.z));
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) sum[r] = (part[0][r] + part[1][r]) + (part[2][r] + part[3][r]);
}

// (T4) for a model that fits shared memory (discrete features leave a few components per admissible value):
// every block loads the packed model once and then walks its tiles without a block-wide barrier.  (Reading
// four or eight features of a row per load, with the feature loop unrolled to match, measured 10-30 % slower:
// the kernel is bound by instruction issue, not by the row reads.)
template <int R>
__global__ void __launch_bounds__(kScoreThreads) tpe_score_resident_kernel(
    const float* __restrict__ Xc, long long m, int d, const int* __restrict__ levels, const int* __restrict__ offs,
    const float4* __restrict__ packed, int total, const float* __restrict__ table, float* __restrict__ score,
    int* __restrict__ status)
{
    extern __shared__ float4 model[];   // [total] components, then [2d + 1] offsets, then [d] level codes
    int* offs_s = reinterpret_cast<int*>(model + total);
    int* code_s = offs_s + 2 * d + 1;
    for (int i = threadIdx.x; i < total; i += kScoreThreads) model[i] = __ldg(packed + i);
    for (int i = threadIdx.x; i <= 2 * d; i += kScoreThreads) offs_s[i] = __ldg(offs + i);
    for (int i = threadIdx.x; i < d; i += kScoreThreads) code_s[i] = __ldg(levels + i);
    __syncthreads();
    const long long tiles = (m + (long long)R * kScoreThreads - 1) / ((long long)R * kScoreThreads);
    bool bad = false;
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long base = tile * (long long)R * kScoreThreads + threadIdx.x;
        const float* row[R];
        bool valid[R];
        float acc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const long long cand = base + (long long)r * kScoreThreads;
            valid[r] = cand < m;
            row[r] = Xc + (size_t)(valid[r] ? cand : 0) * d;
            acc[r] = 0.f;
        }
        for (int j = 0; j < d; ++j) {
            float x[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                x[r] = row[r][j];
                bad |= valid[r] && !isfinite(x[r]);
            }
            const int code = code_s[j];
            const int C = code < 0 ? -code : code;
            if (C > 0) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float lv = floorf(__fadd_rn(__fmul_rn(x[r], (float)(C - 1)), 0.5f));
                    const int v = isfinite(x[r]) ? (int)fminf(fmaxf(lv, 0.f), (float)(C - 1)) : 0;
                    acc[r] += __ldg(table + (size_t)j * kTpeMaxLevels + v);
                }
            } else {
                float sl[R], sg[R];
                mixture_sums_resident<R>(model, offs_s[2 * j], offs_s[2 * j + 1], x, sl);
                mixture_sums_resident<R>(model, offs_s[2 * j + 1], offs_s[2 * j + 2], x, sg);
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] += 0.69314718f * (lg2_fast(sl[r]) - lg2_fast(sg[r]));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (valid[r]) score[base + (long long)r * kScoreThreads] = acc[r];
    }
    if (bad) atomicOr(status, DEV_NONFINITE);
}

// (T4) when every dimension is tabulated (categorical or grid) and d is a multiple of 4: the score is
// d look-ups per candidate and the kernel is a streaming read of the pool.  LPC lanes share a candidate
// (each takes every LPC-th group of four features, a 16-byte load), so that a warp reads whole rows
// contiguously; their partial sums meet by shuffles.  A lane always serves the same features, so the block
// keeps a copy of the tables laid out by lane -- entry (iteration, feature-in-group, level) of lane l at
// word ((it*4 + e)*64 + level)*32 + l -- which makes every look-up conflict-free.  Four candidates per
// lane group are in flight.
template <int LPC>
__global__ void __launch_bounds__(256) tpe_table_score_kernel(const float* __restrict__ Xc, long long m, int d,
                                                              const int* __restrict__ levels,
                                                              const float* __restrict__ table,
                                                              float* __restrict__ score, int* __restrict__ status)
{
    constexpr int CPW = 32 / LPC;          // candidates per warp and step
    constexpr int UNROLL = 4;
    extern __shared__ float tsm[];         // [iters][4][64][32] tables by lane, then [iters][4][32] level scales
    const int d4 = d / 4;
    const int iters = (d4 + LPC - 1) / LPC;
    float* scale_sm = tsm + (size_t)iters * 4 * kTpeMaxLevels * 32;
    for (int w = threadIdx.x; w < iters * 4 * kTpeMaxLevels * 32; w += blockDim.x) {
        const int l = w % 32, v = (w / 32) % kTpeMaxLevels, e = (w / (32 * kTpeMaxLevels)) % 4;
        const int it = w / (32 * kTpeMaxLevels * 4);
        const int j4 = l % LPC + it * LPC;
        tsm[w] = j4 < d4 ? table[(size_t)(4 * j4 + e) * kTpeMaxLevels + v] : 0.f;
    }
    for (int w = threadIdx.x; w < iters * 4 * 32; w += blockDim.x) {
        const int l = w % 32, e = (w / 32) % 4, it = w / 128;
        const int j4 = l % LPC + it * LPC;
        const int code = j4 < d4 ? levels[4 * j4 + e] : 2;
        scale_sm[w] = (float)((code < 0 ? -code : code) - 1);
    }
    __syncthreads();
    const int lane = threadIdx.x % 32, sub = lane % LPC;
    const long long warp = (long long)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const long long nwarps = (long long)gridDim.x * (blockDim.x / 32);
    bool bad = false;
    for (long long c0 = warp * CPW * UNROLL; c0 < m; c0 += nwarps * CPW * UNROLL) {
        float acc[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) acc[u] = 0.f;
        for (int it = 0; it < iters; ++it) {
            const int j4 = sub + it * LPC;
            float4 x[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const long long cand = c0 + u * CPW + lane / LPC;
                x[u] = (cand < m && j4 < d4) ? __ldcs(reinterpret_cast<const float4*>(Xc + (size_t)cand * d) + j4)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float cm1 = scale_sm[(it * 4 + e) * 32 + lane];
                const float* tl = tsm + (size_t)(it * 4 + e) * kTpeMaxLevels * 32 + lane;
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const float xe = e == 0 ? x[u].x : (e == 1 ? x[u].y : (e == 2 ? x[u].z : x[u].w));
                    bad |= !isfinite(xe);
                    const float lv = floorf(__fadd_rn(__fmul_rn(xe, cm1), 0.5f));
                    const int v = isfinite(xe) ? (int)fminf(fmaxf(lv, 0.f), cm1) : 0;
                    acc[u] += tl[v * 32];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
#pragma unroll
            for (int o = LPC / 2; o > 0; o >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], o);
            const long long cand = c0 + u * CPW + lane / LPC;
            if (sub == 0 && cand < m) score[cand] = acc[u];
        }
    }
    if (bad) atomicOr(status, DEV_NONFINITE);
}

size_t resident_bytes(int total, int d) { return sizeof(float4) * (size_t)total + sizeof(int) * (3 * (size_t)d + 1); }

void tpe_destroy(r3_tpe* t)
{
    if (!t) return;
    dev_free(t->arena_d);
    pinned_word_release(t->status_h);
    delete t;
}

r3_status_t tpe_fit_impl(r3_tpe* t, const float* X, const float* y, cudaStream_t stream)
{
    const int n = t->n, d = t->d;
    R3_CUDA_TRY(cudaGetDevice(&t->device));
    // one block of device memory for the whole model (the library's cache hands it back to the next fit)
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t b_comps = up(sizeof(float4) * (size_t)d * (n + 2)), b_packed = up(kResidentBytes),
                 b_table = up(sizeof(float) * (size_t)d * kTpeMaxLevels), b_order = up(sizeof(int) * n),
                 b_levels = up(sizeof(int) * d), b_counts = up(sizeof(int) * 2 * (size_t)d),
                 b_offs = up(sizeof(int) * (2 * (size_t)d + 1)), b_status = 256,
                 b_lnp = up(sizeof(double) * 2 * (size_t)d * kTpeMaxLevels);
    char* base = nullptr;
    if (dev_malloc(&base, b_comps + b_packed + b_table + b_order + b_levels + b_counts + b_offs + b_status + b_lnp) !=
        cudaSuccess) {
        cudaGetLastError();
        set_error("r3_tpe_fit: out of device memory");
        return R3_ERR_ALLOC;
    }
    t->arena_d = base;
    t->comps_d = reinterpret_cast<float4*>(base); base += b_comps;
    t->packed_d = reinterpret_cast<float4*>(base); base += b_packed;
    t->table_d = reinterpret_cast<float*>(base); base += b_table;
    t->order_d = reinterpret_cast<int*>(base); base += b_order;
    t->levels_d = reinterpret_cast<int*>(base); base += b_levels;
    t->counts_d = reinterpret_cast<int*>(base); base += b_counts;
    t->offs_d = reinterpret_cast<int*>(base); base += b_offs;
    t->status_d = reinterpret_cast<int*>(base); base += b_status;
    double* lnp_d = reinterpret_cast<double*>(base);   // scratch of the fit
    t->status_h = pinned_word_acquire();
    if (!t->status_h) {
        set_error("r3_tpe_fit: no pinned host memory");
        return R3_ERR_ALLOC;
    }
    R3_CUDA_TRY(cudaMemcpyAsync(t->levels_d, t->levels.data(), sizeof(int) * d, cudaMemcpyHostToDevice, stream));
    R3_CUDA_TRY(cudaMemsetAsync(t->status_d, 0, sizeof(int), stream));
    R3_LAUNCH(tpe_order_kernel, 1, kSortThreads, 0, stream, y, n, t->order_d, t->status_d);
    int count = 1;
    while (count < n + 1) count <<= 1;
    const size_t smem = sizeof(unsigned long long) * (size_t)count + sizeof(double) * 2 * ((size_t)n + 2);
    if (smem > 48 * 1024)
        R3_CUDA_TRY(cudaFuncSetAttribute(tpe_mixture_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    R3_LAUNCH(tpe_mixture_kernel, 2 * d, kSortThreads, smem, stream, X, t->order_d, n, d, t->n_good, t->levels_d,
              (double)t->prior_weight, t->comps_d, t->counts_d, lnp_d, t->status_d);
    R3_LAUNCH(tpe_table_kernel, d, kTpeMaxLevels, 0, stream, t->levels_d, lnp_d, d, t->table_d);
    R3_CUDA_TRY(cudaMemcpyAsync(t->status_h, t->status_d, sizeof(int), cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));
    if (*t->status_h & DEV_NONFINITE) {
        set_error("r3_tpe_fit: X or y contains NaN or Inf");
        return R3_ERR_NONFINITE;
    }
    // pack a model that a scoring block can hold in shared memory
    std::vector<int> counts(2 * (size_t)d), offs(2 * (size_t)d + 1, 0);
    R3_CUDA_TRY(cudaMemcpy(counts.data(), t->counts_d, sizeof(int) * 2 * (size_t)d, cudaMemcpyDeviceToHost));
    for (int i = 0; i < 2 * d; ++i) offs[i + 1] = offs[i] + counts[i];
    t->total = offs[2 * d];
    t->resident = t->total > 0 && resident_bytes(t->total, d) <= kResidentBytes;
    if (t->resident) {
        R3_CUDA_TRY(cudaMemcpyAsync(t->offs_d, offs.data(), sizeof(int) * offs.size(), cudaMemcpyHostToDevice, stream));
        R3_LAUNCH(tpe_pack_kernel, 2 * d, 256, 0, stream, t->comps_d, n, t->n_good, t->offs_d, t->packed_d);
        R3_CUDA_TRY(cudaStreamSynchronize(stream));   // `offs` leaves scope
    }
    return R3_OK;
}

}  // namespace

}  // namespace r3

using namespace r3;

extern "C" {

r3_status_t r3_tpe_fit(const float* X, const float* y, const int* levels, int n, int d, float gamma,
                       float prior_weight, void* cuda_stream, r3_tpe_t** out)
{
    if (out) *out = nullptr;
    if (!X || !y || !levels || !out) {
        set_error("r3_tpe_fit: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (n < 1 || n > kTpeMaxN || d < 1 || d > kMaxD) {
        set_error("r3_tpe_fit: need 1 <= n <= %d and 1 <= d <= %d (got n=%d, d=%d)", kTpeMaxN, kMaxD, n, d);
        return R3_ERR_INVALID_ARG;
    }
    if (!(gamma > 0.f && gamma <= 1.f) || !(prior_weight > 0.f) || !isfinite(prior_weight)) {
        set_error("r3_tpe_fit: need 0 < gamma <= 1 and a finite prior_weight > 0");
        return R3_ERR_INVALID_ARG;
    }
    for (int j = 0; j < d; ++j)
        if (levels[j] != 0 && (abs(levels[j]) < 2 || abs(levels[j]) > kTpeMaxLevels)) {
            set_error("r3_tpe_fit: levels[%d] = %d; allowed are 0, 2..%d and -%d..-2", j, levels[j], kTpeMaxLevels,
                      kTpeMaxLevels);
            return R3_ERR_INVALID_ARG;
        }
    r3_tpe* t = new (std::nothrow) r3_tpe;
    if (!t) {
        set_error("r3_tpe_fit: out of host memory");
        return R3_ERR_ALLOC;
    }
    t->n = n;
    t->d = d;
    t->prior_weight = prior_weight;
    const long long ng = (long long)ceil((double)gamma * (double)n);
    t->n_good = (int)(ng < 1 ? 1 : (ng > n ? n : ng));
    t->levels.assign(levels, levels + d);
    const r3_status_t st = tpe_fit_impl(t, X, y, (cudaStream_t)cuda_stream);
    if (st != R3_OK) {
        tpe_destroy(t);
        return st;
    }
    *out = t;
    return R3_OK;
}

r3_status_t r3_tpe_score(r3_tpe_t* tpe, const float* Xcand, long long m, float* score, void* cuda_stream)
{
    if (!tpe || !Xcand || !score) {
        set_error("r3_tpe_score: NULL argument");
        return R3_ERR_INVALID_ARG;
    }
    if (m < 1 || m >= (1ll << 31)) {
        set_error("r3_tpe_score: need 1 <= m < 2^31 (got %lld)", m);
        return R3_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    bool all_tables = (tpe->d % 4) == 0 && (reinterpret_cast<uintptr_t>(Xcand) % 16) == 0;
    for (int j = 0; j < tpe->d && all_tables; ++j) all_tables = tpe->levels[j] != 0;
    if (all_tables) {
        // every dimension is a look-up: stream the pool with whole-row loads
        const int d4 = tpe->d / 4;
#define R3_TPE_TABLE(LPC)                                                                                      \
    do {                                                                                                       \
        const int iters = (d4 + LPC - 1) / LPC;                                                                \
        const size_t smem = sizeof(float) * (size_t)iters * 4 * 32 * (kTpeMaxLevels + 1);                      \
        if (smem > 48 * 1024)                                                                                  \
            R3_CUDA_TRY(cudaFuncSetAttribute(tpe_table_score_kernel<LPC>,                                      \
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));         \
        const unsigned grid = 148 * (smem > 56 * 1024 ? 2 : 4);                                                \
        R3_LAUNCH(tpe_table_score_kernel<LPC>, grid, 256, smem, stream, Xcand, m, tpe->d, tpe->levels_d,       \
                  tpe->table_d, score, tpe->status_d);                                                         \
    } while (0)
        if (d4 >= 32) R3_TPE_TABLE(32);
        else if (d4 >= 16) R3_TPE_TABLE(16);
        else if (d4 >= 8) R3_TPE_TABLE(8);
        else if (d4 >= 4) R3_TPE_TABLE(4);
        else if (d4 >= 2) R3_TPE_TABLE(2);
        else R3_TPE_TABLE(1);
#undef R3_TPE_TABLE
        return R3_OK;
    }
    if (tpe->resident) {
        // the whole model in shared memory.  Sixteen blocks per SM's worth of grid (several waves of short
        // blocks) measured up to 8 % faster than one resident wave walking the tiles: the model is a small
        // read from L2 and the finer grain balances the SMs better.
        const size_t smem = resident_bytes(tpe->total, tpe->d);
        const long long tiles2 = (m + 2ll * kScoreThreads - 1) / (2ll * kScoreThreads);
        const long long tiles1 = (m + kScoreThreads - 1) / kScoreThreads;
#define R3_TPE_RESIDENT(R, TILES)                                                                              \
    do {                                                                                                       \
        if (smem > 48 * 1024)                                                                                  \
            R3_CUDA_TRY(cudaFuncSetAttribute(tpe_score_resident_kernel<R>,                                     \
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));         \
        const unsigned grid = (unsigned)std::min<long long>(TILES, 148ll * 16);                                \
        R3_LAUNCH(tpe_score_resident_kernel<R>, grid, kScoreThreads, smem, stream, Xcand, m, tpe->d,           \
                  tpe->levels_d, tpe->offs_d, tpe->packed_d, tpe->total, tpe->table_d, score, tpe->status_d);  \
    } while (0)
        if (tiles2 >= 148ll * 8)
            R3_TPE_RESIDENT(2, tiles2);
        else
            R3_TPE_RESIDENT(1, tiles1);
#undef R3_TPE_RESIDENT
        return R3_OK;
    }
    // Two candidates per thread (one shared-memory read serves both) when that still gives every SM
    // several blocks; one per thread for small pools.  More per thread measured slower on the full pool
    // (fewer, longer blocks balance worse over the 148 SMs).
    const long long tiles2 = (m + 2ll * kScoreThreads - 1) / (2ll * kScoreThreads);
    if (tiles2 >= 148ll * 4) {
        const unsigned grid = (unsigned)(tiles2 < 148ll * 64 ? tiles2 : 148ll * 64);
        R3_LAUNCH(tpe_score_kernel<2>, grid, kScoreThreads, 0, stream, Xcand, m, tpe->n, tpe->d, tpe->n_good,
                  tpe->levels_d, tpe->comps_d, tpe->counts_d, tpe->table_d, score, tpe->status_d);
    } else {
        const long long tiles1 = (m + kScoreThreads - 1) / kScoreThreads;
        R3_LAUNCH(tpe_score_kernel<1>, (unsigned)tiles1, kScoreThreads, 0, stream, Xcand, m, tpe->n, tpe->d,
                  tpe->n_good, tpe->levels_d, tpe->comps_d, tpe->counts_d, tpe->table_d, score, tpe->status_d);
    }
    return R3_OK;
}

r3_status_t r3_tpe_check(r3_tpe_t* tpe, void* cuda_stream)
{
    if (!tpe) {
        set_error("r3_tpe_check: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    R3_CUDA_TRY(cudaMemcpyAsync(tpe->status_h, tpe->status_d, sizeof(int), cudaMemcpyDeviceToHost, stream));
    R3_CUDA_TRY(cudaMemsetAsync(tpe->status_d, 0, sizeof(int), stream));
    R3_CUDA_TRY(cudaStreamSynchronize(stream));
    if (*tpe->status_h & DEV_NONFINITE) {
        set_error("r3_tpe_score: a candidate contains NaN or Inf");
        return R3_ERR_NONFINITE;
    }
    return R3_OK;
}

r3_status_t r3_tpe_get_model(r3_tpe_t* tpe, int* n_good, int* order, float* comps, int* counts, float* table)
{
    if (!tpe) {
        set_error("r3_tpe_get_model: NULL handle");
        return R3_ERR_INVALID_ARG;
    }
    R3_CUDA_TRY(cudaDeviceSynchronize());
    if (n_good) *n_good = tpe->n_good;
    if (order) R3_CUDA_TRY(cudaMemcpy(order, tpe->order_d, sizeof(int) * tpe->n, cudaMemcpyDeviceToHost));
    if (comps)
        R3_CUDA_TRY(cudaMemcpy(comps, tpe->comps_d, sizeof(float4) * (size_t)tpe->d * (tpe->n + 2),
                               cudaMemcpyDeviceToHost));
    if (counts) R3_CUDA_TRY(cudaMemcpy(counts, tpe->counts_d, sizeof(int) * 2 * (size_t)tpe->d, cudaMemcpyDeviceToHost));
    if (table)
        R3_CUDA_TRY(cudaMemcpy(table, tpe->table_d, sizeof(float) * (size_t)tpe->d * kTpeMaxLevels,
                               cudaMemcpyDeviceToHost));
    return R3_OK;
}

void r3_tpe_free(r3_tpe_t* tpe) { tpe_destroy(tpe); }

}  // extern "C"
