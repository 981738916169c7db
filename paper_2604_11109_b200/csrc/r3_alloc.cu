// Device-memory cache of the library.
//
// A BO round frees and allocates the same few large arrays again and again (a refit, an append, a
// larger pool): cudaMalloc and cudaFree of 100 MB blocks cost milliseconds each -- more than the
// kernels of an append -- so freed blocks are kept, per device, and handed out again.  Sizes are
// rounded up to five significant bits so that neighbouring sizes (a history that grew by a few
// rows) share a bin; blocks below 1 MiB -- a small history's fit is two dozen of them, and their cudaMalloc and
// cudaFree calls were most of its time -- are rounded up to a multiple of 512 bytes and kept as well.  dev_free waits for the device like cudaFree does, which makes the block safe to
// reuse at once.  The cache holds at most kCacheLimit bytes per device; r3_trim_cache() returns
// everything to the driver.
#include <map>
#include <mutex>
#include <vector>

#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr size_t kCacheLimit = 2ull << 30;
constexpr size_t kSmall = 1 << 20;   // below 1 MiB: bins of 512 bytes
constexpr size_t kCacheBlocks = 4096;   // at most this many kept blocks per device

struct DeviceCache {
    std::multimap<size_t, void*> free_blocks;   // bin size -> block
    std::map<void*, size_t> live;               // block -> bin size (only blocks handed out by dev_malloc)
    size_t cached_bytes = 0;
};

std::mutex g_mutex;
std::map<int, DeviceCache> g_cache;

// r3_test_fail_allocation: allocations counted since arming, and the one that is to fail (-1: none)
long long g_alloc_seen = 0, g_alloc_fail_at = -1;

size_t bin_of(size_t bytes)
{
    if (bytes < kSmall) return (bytes + 511) & ~(size_t)511;
    size_t top = bytes;
    int shift = 0;
    while (top >= 32) {   // keep five leading bits: bins are at most 1/16 apart
        top >>= 1;
        ++shift;
    }
    size_t bin = top << shift;
    if (bin < bytes) bin = (top + 1) << shift;
    return bin;
}

}  // namespace

cudaError_t dev_malloc_bytes(void** p, size_t bytes)
{
    *p = nullptr;
    if (bytes == 0) bytes = 1;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const size_t bin = bin_of(bytes);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (g_alloc_seen++ == g_alloc_fail_at) {   // test aid: this allocation is refused
            g_alloc_fail_at = -1;
            return cudaErrorMemoryAllocation;
        }
        DeviceCache& c = g_cache[dev];
        auto it = c.free_blocks.find(bin);
        if (it != c.free_blocks.end()) {
            *p = it->second;
            c.free_blocks.erase(it);
            c.cached_bytes -= bin;
            c.live[*p] = bin;
            return cudaSuccess;
        }
    }
    e = cudaMalloc(p, bin);
    if (e == cudaErrorMemoryAllocation) {
        // give the cache back to the driver and try once more
        cudaGetLastError();
        trim_cache();
        e = cudaMalloc(p, bin);
    }
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_cache[dev].live[*p] = bin;
    return cudaSuccess;
}

void dev_free(void* p)
{
    if (!p) return;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaFree(p);
        return;
    }
    size_t bin = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        DeviceCache& c = g_cache[dev];
        auto it = c.live.find(p);
        if (it != c.live.end()) {
            bin = it->second;
            c.live.erase(it);
        }
    }
    if (bin == 0) {   // not ours: plain free
        cudaFree(p);
        return;
    }
    cudaDeviceSynchronize();   // as cudaFree would: nothing in flight may still use the block
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCache& c = g_cache[dev];
    if (c.cached_bytes + bin > kCacheLimit || c.free_blocks.size() >= kCacheBlocks) {
        cudaFree(p);
        return;
    }
    c.free_blocks.emplace(bin, p);
    c.cached_bytes += bin;
}

void trim_cache()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return;
    std::vector<void*> blocks;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        DeviceCache& c = g_cache[dev];
        for (auto& kv : c.free_blocks) blocks.push_back(kv.second);
        c.free_blocks.clear();
        c.cached_bytes = 0;
    }
    for (void* b : blocks) cudaFree(b);
}

// Pinned host blocks of kPinnedInts ints for status read-backs: cudaMallocHost costs far more than the kernels
// of a small fit, so released blocks are kept for the life of the process.
namespace {
std::vector<int*> g_pinned_words;
}

int* pinned_word_acquire()
{
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_pinned_words.empty()) {
            int* w = g_pinned_words.back();
            g_pinned_words.pop_back();
            return w;
        }
    }
    int* w = nullptr;
    if (cudaMallocHost(&w, sizeof(int) * kPinnedInts) != cudaSuccess) return nullptr;
    return w;
}

void pinned_word_release(int* w)
{
    if (!w) return;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_pinned_words.push_back(w);
}

size_t cached_bytes()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    return g_cache[dev].cached_bytes;
}

}  // namespace r3

extern "C" {

void r3_trim_cache(void) { r3::trim_cache(); }

long long r3_test_fail_allocation(long long after)
{
    std::lock_guard<std::mutex> lock(r3::g_mutex);
    const long long seen = r3::g_alloc_seen;
    r3::g_alloc_seen = 0;
    r3::g_alloc_fail_at = after < 0 ? -1 : after;
    return seen;
}
unsigned long long r3_cached_bytes(void) { return r3::cached_bytes(); }

}  // extern "C"
