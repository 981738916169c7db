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

// The K largest of the n keys s[0..n) end up in s[0..K), sorted descending; the rest of s is scratch.
// n and K are powers of two, K <= n, n <= 8 * blockDim.x * 2 (a thread stages at most 8 keys in registers).
// All threads of the block call it.  Blocks of K keys are sorted first (bitonic network), then pairs of
// sorted blocks are reduced to the K largest of their union -- max(a[i], b[K-1-i]) is a bitonic sequence
// that holds exactly those -- and re-sorted with the log2(K) merge steps, halving the data each round:
// about (log2 K)^2 / 2 + 2 log2(K) sweeps over the chunk instead of the (log2 n)^2 / 2 of a full sort.
__device__ __forceinline__ void block_topk_desc(unsigned long long* s, int n, int K)
{
    const int T = blockDim.x, tid = threadIdx.x;
    // sort every block of K keys descending
    for (int size = 2; size <= K; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = tid; t < n / 2; t += T) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool desc = size == K ? true : ((lo & size) == 0);
                const unsigned long long a = s[lo], b = s[hi];
                if ((a < b) == desc) {
                    s[lo] = b;
                    s[hi] = a;
                }
            }
        }
    }
    for (int len = n; len > K; len >>= 1) {
        const int half = len >> 1;
        unsigned long long keep[8];
        __syncthreads();
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = tid + u * T;
            if (e < half) {
                const int blk = e / K, i = e % K;
                const unsigned long long a = s[(2 * blk) * K + i], b = s[(2 * blk + 1) * K + (K - 1 - i)];
                keep[u] = a > b ? a : b;
            }
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = tid + u * T;
            if (e < half) s[e] = keep[u];
        }
        for (int stride = K >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = tid; t < half / 2; t += T) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const unsigned long long a = s[lo], b = s[hi];
                if (a < b) {
                    s[lo] = b;
                    s[hi] = a;
                }
            }
        }
    }
    __syncthreads();
}

__host__ __device__ inline int topk_pow2_at_least(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

}  // namespace r3
