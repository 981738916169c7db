// Top-k selection: the k largest EI of each GP's pool, ties to the lower index.
//
// A value and its index are packed in one 64-bit key (r3_topk.cuh) whose unsigned order is exactly "larger
// value, or equal value and smaller index".  A block takes a chunk of 4096 keys into shared memory and keeps
// its k largest (block_select_desc: radix selection of the k-th largest, then a rank sort of the k survivors);
// levels repeat until one chunk is left, and the block that handles it writes the indices and values.  The first level
// reads the EI array once (4 bytes per candidate); later levels touch k keys per chunk of the level before.
// When the scoring call asked for a top-k, the accuracy guard's kernel has already left the first level's keys
// (r3_rescue.cu), and only the later levels run here.
#include <mutex>

#include "r3_internal.cuh"
#include "r3_topk.cuh"

namespace r3 {

namespace {

constexpr int CHUNK = 4096;      // keys per block
constexpr int THREADS = 1024;
constexpr int kMaxK = 1024;      // the interface's limit on k
constexpr size_t kSelectBytes = sizeof(unsigned long long) * kMaxK + sizeof(unsigned) * (kMaxK + 256 + 8);

// The last level writes the answer instead of keys: idx (and val, read back from the EI array) are non-null.
__device__ __forceinline__ void emit(const unsigned long long* s, int k, unsigned long long* out_keys,
                                     const float* __restrict__ ei, long long m, int* __restrict__ idx,
                                     float* __restrict__ val)
{
    const int g = blockIdx.y;
    if (idx) {
        for (int t = threadIdx.x; t < k; t += blockDim.x) {
            const unsigned i = topk_key_index(s[t]);
            idx[(size_t)g * k + t] = (int)i;
            if (val) val[(size_t)g * k + t] = ((long long)i < m) ? ei[(size_t)g * m + i] : __int_as_float(0x7fc00000);
        }
    } else {
        unsigned long long* o = out_keys + ((size_t)g * gridDim.x + blockIdx.x) * k;
        for (int t = threadIdx.x; t < k; t += blockDim.x) o[t] = s[t];
    }
}

// Level 0: keys from the EI array.  grid = (chunks, batch).
__global__ void __launch_bounds__(THREADS) topk_from_values_kernel(const float* __restrict__ ei, long long m,
                                                                   int k, unsigned long long* __restrict__ out,
                                                                   int* __restrict__ idx, float* __restrict__ val)
{
    __shared__ unsigned long long s[CHUNK];
    __shared__ unsigned long long scratch[kSelectBytes / 8];
    const int g = blockIdx.y;
    const long long base = (long long)blockIdx.x * CHUNK;
    const float* e = ei + (size_t)g * m;
    for (int t = threadIdx.x; t < CHUNK; t += THREADS) {
        const long long i = base + t;
        s[t] = (i < m) ? topk_make_key(e[i], (unsigned)i) : 0ull;
    }
    block_select_desc(s, CHUNK, k, scratch);
    emit(s, k, out, ei, m, idx, val);
}

// Later levels: keys from the level before.  count = keys per GP in `in`.
__global__ void __launch_bounds__(THREADS) topk_from_keys_kernel(const unsigned long long* __restrict__ in,
                                                                 long long count, int k,
                                                                 unsigned long long* __restrict__ out,
                                                                 const float* __restrict__ ei, long long m,
                                                                 int* __restrict__ idx, float* __restrict__ val)
{
    __shared__ unsigned long long s[CHUNK];
    __shared__ unsigned long long scratch[kSelectBytes / 8];
    const int g = blockIdx.y;
    const long long base = (long long)blockIdx.x * CHUNK;
    const unsigned long long* src = in + (size_t)g * count;
    for (int t = threadIdx.x; t < CHUNK; t += THREADS) {
        const long long i = base + t;
        s[t] = (i < count) ? src[i] : 0ull;
    }
    block_select_desc(s, CHUNK, k, scratch);
    emit(s, k, out, ei, m, idx, val);
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

// The levels after the first: `count` keys per GP in keys_in (k per block of the level before), ping-pong
// through keys_tmp, indices and values out.  count == k means a single block produced them, sorted: only the
// write is left, and the last level's kernel does it all the same (one chunk).
r3_status_t topk_finish_from_keys(unsigned long long* keys_in, unsigned long long* keys_tmp, int batch, long long count,
                                  int k, const float* ei, long long m, int* idx, float* val, cudaStream_t stream)
{
    unsigned long long* buf[2] = {keys_in, keys_tmp};
    int cur = 0;
    while (true) {
        const long long chunks = chunks_of(count);
        const bool last = chunks == 1;
        R3_LAUNCH(topk_from_keys_kernel, dim3((unsigned)chunks, batch), THREADS, 0, stream, buf[cur], count, k,
                  buf[cur ^ 1], ei, m, last ? idx : nullptr, last ? val : nullptr);
        if (last) break;
        cur ^= 1;
        count = chunks * k;
    }
    return R3_OK;
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
    const long long chunks = chunks_of(m);
    const bool last = chunks == 1;
    R3_LAUNCH(topk_from_values_kernel, dim3((unsigned)chunks, batch), THREADS, 0, stream, ei, m, k, buf[0],
              last ? idx : nullptr, last ? val : nullptr);
    if (last) return R3_OK;
    return topk_finish_from_keys(buf[0], buf[1], batch, chunks * k, k, ei, m, idx, val, stream);
}

}  // namespace r3
