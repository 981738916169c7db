// Device pieces of the top-k selection shared by r3_topk.cu (selection on its own) and r3_rescue.cu (the
// guard kernel leaves the partial top-k of its slice of candidates): the 64-bit key and the block-wide
// "k largest of a chunk" in shared memory.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace r3 {

// A value and its index in one 64-bit key whose unsigned order is (value ascending, index descending): the
// float is mapped to an order-preserving unsigned integer in the high word and the low word holds ~index, so
// "larger key" means "larger value, or equal value and smaller index".  Key 0 is below every real key.
__device__ __forceinline__ unsigned long long topk_make_key(float v, unsigned idx)
{
    unsigned u;
    if (v != v) {
        u = 0u;  // NaN ranks below every number
    } else {
        if (v == 0.0f) v = 0.0f;  // -0 and +0 tie
        u = __float_as_uint(v);
        u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
        if (u == 0u) u = 1u;  // keep 0 for NaN / padding (only -NaN patterns map here)
    }
    return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}

__device__ __forceinline__ unsigned topk_key_index(unsigned long long key)
{
    return 0xFFFFFFFFu - (unsigned)(key & 0xFFFFFFFFull);
}

// Shared-memory scratch of block_select_desc for a selection of K keys: K keys, K ranks, a 256-bin histogram
// and eight words of state (8-byte aligned).
constexpr int kRankSortMaxK = 256;   // above this many survivors a sorting network is cheaper than K^2 comparisons
__host__ __device__ inline int topk_pow2_at_least(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}
__host__ __device__ inline size_t topk_select_scratch_bytes(int K)
{
    const size_t Kc = K > kRankSortMaxK ? (size_t)topk_pow2_at_least(K) : (size_t)K;   // the network sorts a power of two
    return sizeof(unsigned long long) * Kc + sizeof(unsigned) * (Kc + 256 + 8);
}

// The K largest of the n keys s[0..n) end up in s[0..K), sorted descending; the rest of s is scratch.
// 1 <= K <= n; blockDim.x is a multiple of 32; all threads of the block call it.
//
// Radix selection, then a rank sort of the K survivors -- no sorting network over the n keys:
//  1. the K-th largest key is found digit by digit from the top (8 bits per step): a histogram of the digit
//     over the keys that match the digits found so far (lanes that share a digit with the warp's first active lane add once, so a
//     pool whose values share their exponent does not serialise on one bin), a walk over the 256 bins from the top by one
//     warp; it stops as soon as the chosen bin holds one key, typically after three or four steps;
//  2. the keys above that bin, and as many of the bin's as are still wanted (more than one only for the
//     duplicated padding key 0), are gathered: exactly K;
//  3. every survivor counts the survivors that precede it (K^2 comparisons spread over the block, operands
//     read as broadcasts) and is written to that position; more than 256 survivors go through a bitonic
//     network instead.
// About n / blockDim.x key reads per thread and step and four barriers per step, against the roughly
// (log2 n)^2 / 2 barrier-separated sweeps of a sorting network.
__device__ __forceinline__ void block_select_desc(unsigned long long* s, int n, int K, void* scratch)
{
    const int Kc = K > kRankSortMaxK ? topk_pow2_at_least(K) : K;
    unsigned long long* tmp = reinterpret_cast<unsigned long long*>(scratch);   // [Kc] survivors, unordered
    unsigned* rank = reinterpret_cast<unsigned*>(tmp + Kc);                     // [Kc]
    unsigned* hist = rank + K;                                                  // [256]
    unsigned* sel = hist + 256;   // [0] chosen digit, [1] rank wanted inside its bin, [2] keys in that bin,
                                  // [4], [5] fill counters of the gather
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    for (int i = tid; i < K; i += T) rank[i] = 0u;
    if (tid == 0) sel[4] = sel[5] = 0u;
    if (K >= n) {
        for (int i = tid; i < n; i += T) tmp[i] = s[i];
    } else {
        unsigned long long prefix = 0ull;   // the digits of the K-th largest key found so far, in place
        unsigned want = (unsigned)K;        // its rank among the keys that share them
        int shift = 56;
        const int n_up = (n + 31) & ~31;    // whole warps take part in the vote below
        for (;; shift -= 8) {
            for (int b = tid; b < 256; b += T) hist[b] = 0u;
            __syncthreads();
            const unsigned long long himask = shift == 56 ? 0ull : (~0ull << (shift + 8));
            for (int i = tid; i < n_up; i += T) {
                const unsigned long long key = i < n ? s[i] : 0ull;
                const bool act = i < n && (key & himask) == prefix;
                const unsigned dgt = (unsigned)(key >> shift) & 255u;
                // the lanes that share the first active lane's digit add once (pools whose values share their
                // exponent would otherwise serialise on one bin); the others add for themselves
                const unsigned active = __ballot_sync(0xffffffffu, act);
                if (active) {
                    const int first = __ffs(active) - 1;
                    const unsigned d0 = __shfl_sync(0xffffffffu, dgt, first);
                    const unsigned same = __ballot_sync(0xffffffffu, act && dgt == d0);
                    if (lane == first) atomicAdd(&hist[d0], (unsigned)__popc(same));
                    else if (act && dgt != d0) atomicAdd(&hist[dgt], 1u);
                }
            }
            __syncthreads();
            if (tid < 32) {   // bins from the top: lane l owns bins 255 - 8 l - j, j = 0..7
                unsigned c[8], sum = 0u;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    c[j] = hist[255 - 8 * lane - j];
                    sum += c[j];
                }
                unsigned incl = sum;
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                unsigned acc = incl - sum;
                if (acc < want && want <= incl) {   // exactly one lane: the wanted rank falls among its bins
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (acc < want && want <= acc + c[j]) {
                            sel[0] = (unsigned)(255 - 8 * lane - j);
                            sel[1] = want - acc;
                            sel[2] = c[j];
                        }
                        acc += c[j];
                    }
                }
            }
            __syncthreads();
            prefix |= (unsigned long long)sel[0] << shift;
            want = sel[1];
            if (sel[2] == 1u || shift == 0) break;
        }
        // gather: the keys above the chosen bin (K - want of them), then `want` keys of the bin
        const unsigned long long ph = prefix >> shift;
        for (int i = tid; i < n_up; i += T) {
            const unsigned long long key = i < n ? s[i] : 0ull, hi = key >> shift;
            const bool above = i < n && hi > ph;
            const unsigned votes = __ballot_sync(0xffffffffu, above);   // one counter update per warp
            if (votes) {
                unsigned base = 0u;
                if (lane == __ffs(votes) - 1) base = atomicAdd(&sel[4], (unsigned)__popc(votes));
                base = __shfl_sync(0xffffffffu, base, __ffs(votes) - 1);
                if (above) tmp[base + __popc(votes & ((1u << lane) - 1u))] = key;
            }
            if (i < n && hi == ph) {
                const unsigned r = atomicAdd(&sel[5], 1u);
                if (r < want) tmp[K - 1 - (int)r] = key;
            }
        }
    }
    const int k_cap = K < n ? K : n;
    if (k_cap > kRankSortMaxK) {
        // many survivors: bitonic network over the next power of two (padding key 0 sorts last)
        for (int i = k_cap + tid; i < Kc; i += T) tmp[i] = 0ull;
        for (int size = 2; size <= Kc; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                __syncthreads();
                for (int t = tid; t < Kc / 2; t += T) {
                    const int lo = 2 * t - (t & (stride - 1));
                    const int hi = lo + stride;
                    const bool desc = (lo & size) == 0;
                    const unsigned long long a = tmp[lo], b = tmp[hi];
                    if ((a < b) == desc) {
                        tmp[lo] = b;
                        tmp[hi] = a;
                    }
                }
            }
        }
        __syncthreads();
        for (int i = tid; i < k_cap; i += T) s[i] = tmp[i];
        __syncthreads();
        return;
    }
    __syncthreads();
    // rank sort of tmp[0..K) into s[0..K): position = number of keys that come first (equal keys -- only the
    // padding key repeats -- keep their order in tmp)
    if (k_cap <= T) {
        const int parts = T / k_cap, part = tid / k_cap, i = tid - part * k_cap;
        if (part < parts) {
            const unsigned long long key = tmp[i];
            const int j0 = (int)((long long)part * k_cap / parts), j1 = (int)((long long)(part + 1) * k_cap / parts);
            unsigned before = 0u;
            for (int j = j0; j < j1; ++j) {
                const unsigned long long o = tmp[j];
                before += (o > key || (o == key && j < i)) ? 1u : 0u;
            }
            if (parts == 1) rank[i] = before;
            else if (before) atomicAdd(&rank[i], before);
        }
    } else {
        for (int i = tid; i < k_cap; i += T) {
            const unsigned long long key = tmp[i];
            unsigned before = 0u;
            for (int j = 0; j < k_cap; ++j) {
                const unsigned long long o = tmp[j];
                before += (o > key || (o == key && j < i)) ? 1u : 0u;
            }
            rank[i] = before;
        }
    }
    __syncthreads();
    for (int i = tid; i < k_cap; i += T) s[rank[i]] = tmp[i];
    __syncthreads();
}

}  // namespace r3
