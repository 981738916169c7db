// Top-k selection: the k largest EI of each GP's pool, ties to the lower index.
//
// A value and its index are packed in one 64-bit key whose unsigned order is exactly
// (value descending-friendly, index ascending): the float is mapped to an order-preserving unsigned
// integer in the high word and the low word holds ~index, so "larger key" means "larger value, or
// equal value and smaller index".  A block sorts a chunk of keys in shared memory (bitonic network)
// and emits its k largest; levels repeat until one chunk is left, whose k largest are the answer.
// The first level reads the EI array once (4 bytes per candidate); later levels touch k keys per
// chunk of the level before.
#include <mutex>

#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr int CHUNK = 4096;      // keys sorted per block
constexpr int THREADS = 1024;

__device__ __forceinline__ unsigned long long make_key(float v, unsigned idx)
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

// Sort CHUNK keys descending in shared memory.
__device__ __forceinline__ void bitonic_sort_desc(unsigned long long* s)
{
    for (int size = 2; size <= CHUNK; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < CHUNK / 2; t += THREADS) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool desc = ((lo & size) == 0);
                const unsigned long long a = s[lo], b = s[hi];
                if ((a < b) == desc) {
                    s[lo] = b;
                    s[hi] = a;
                }
            }
        }
    }
    __syncthreads();
}

// Level 0: keys from the EI array.  grid = (chunks, batch).
__global__ void __launch_bounds__(THREADS) topk_from_values_kernel(const float* __restrict__ ei, long long m,
                                                                   int k, unsigned long long* __restrict__ out)
{
    __shared__ unsigned long long s[CHUNK];
    const int g = blockIdx.y;
    const long long base = (long long)blockIdx.x * CHUNK;
    const float* e = ei + (size_t)g * m;
    for (int t = threadIdx.x; t < CHUNK; t += THREADS) {
        const long long i = base + t;
        s[t] = (i < m) ? make_key(e[i], (unsigned)i) : 0ull;
    }
    bitonic_sort_desc(s);
    unsigned long long* o = out + ((size_t)g * gridDim.x + blockIdx.x) * k;
    for (int t = threadIdx.x; t < k; t += THREADS) o[t] = s[t];
}

// Later levels: keys from the level before.  count = keys per GP in `in`.
__global__ void __launch_bounds__(THREADS) topk_from_keys_kernel(const unsigned long long* __restrict__ in,
                                                                 long long count, int k,
                                                                 unsigned long long* __restrict__ out)
{
    __shared__ unsigned long long s[CHUNK];
    const int g = blockIdx.y;
    const long long base = (long long)blockIdx.x * CHUNK;
    const unsigned long long* src = in + (size_t)g * count;
    for (int t = threadIdx.x; t < CHUNK; t += THREADS) {
        const long long i = base + t;
        s[t] = (i < count) ? src[i] : 0ull;
    }
    bitonic_sort_desc(s);
    unsigned long long* o = out + ((size_t)g * gridDim.x + blockIdx.x) * k;
    for (int t = threadIdx.x; t < k; t += THREADS) o[t] = s[t];
}

__global__ void topk_write_kernel(const unsigned long long* __restrict__ keys, const float* __restrict__ ei,
                                  long long m, int k, int* __restrict__ idx, float* __restrict__ val)
{
    const int g = blockIdx.y;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= k) return;
    const unsigned i = 0xFFFFFFFFu - (unsigned)(keys[(size_t)g * k + t] & 0xFFFFFFFFull);
    idx[(size_t)g * k + t] = (int)i;
    if (val) val[(size_t)g * k + t] = ((long long)i < m) ? ei[(size_t)g * m + i] : __int_as_float(0x7fc00000);
}

long long chunks_of(long long count) { return (count + CHUNK - 1) / CHUNK; }

// Fixed key storage of r3_topk_noalloc: two ping-pong buffers of kStaticKeys keys each, resident in
// every device that loads the library until the process exits (1 MiB, plus the 64 bytes of slack the
// workspace size formula carries).
constexpr size_t kStaticKeys = 65536;
static __device__ __align__(256) unsigned long long g_topk_static_keys[2 * kStaticKeys + 8];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};   // device address of g_topk_static_keys, per device ordinal

}  // namespace

// Device address of the static key array on the current device.  The array's name is only a host-side
// handle: the address a kernel can use has to be asked for, once per device, with that device current.
r3_status_t topk_static_scratch(void** ptr)
{
    int dev = 0;
    R3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error("r3_topk_noalloc: device ordinal %d outside [0, %d)", dev, kMaxDevices);
        return R3_ERR_UNSUPPORTED;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        R3_CUDA_TRY(cudaGetSymbolAddress(&p, g_topk_static_keys));
        g_static_ptr[dev] = p;
    }
    *ptr = g_static_ptr[dev];
    return R3_OK;
}

size_t topk_static_capacity_keys() { return kStaticKeys; }
size_t topk_static_capacity_bytes() { return sizeof(unsigned long long) * (2 * kStaticKeys + 8); }

size_t topk_workspace_bytes(int batch, long long m, int k)
{
    // two ping-pong key buffers, each large enough for the first level's output
    const size_t level0 = (size_t)batch * chunks_of(m) * k;
    return 2 * level0 * sizeof(unsigned long long) + 64;
}

r3_status_t topk_device(const float* ei, int batch, long long m, int k, int* idx, float* val, void* ws,
                        size_t ws_bytes, cudaStream_t stream)
{
    if (ws_bytes < topk_workspace_bytes(batch, m, k)) {
        set_error("top-k workspace too small: %zu < %zu", ws_bytes, topk_workspace_bytes(batch, m, k));
        return R3_ERR_INVALID_ARG;
    }
    const size_t level0 = (size_t)batch * chunks_of(m) * k;
    unsigned long long* buf[2] = {(unsigned long long*)ws, (unsigned long long*)ws + level0};
    long long chunks = chunks_of(m);
    R3_LAUNCH(topk_from_values_kernel, dim3((unsigned)chunks, batch), THREADS, 0, stream, ei, m, k, buf[0]);
    int cur = 0;
    long long count = chunks * k;
    while (chunks > 1) {
        chunks = chunks_of(count);
        R3_LAUNCH(topk_from_keys_kernel, dim3((unsigned)chunks, batch), THREADS, 0, stream, buf[cur], count, k,
                  buf[cur ^ 1]);
        cur ^= 1;
        count = chunks * k;
    }
    R3_LAUNCH(topk_write_kernel, dim3((k + 255) / 256, batch), 256, 0, stream, buf[cur], ei, m, k, idx, val);
    return R3_OK;
}

}  // namespace r3
