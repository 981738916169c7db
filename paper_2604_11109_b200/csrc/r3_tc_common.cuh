// Shared pieces of the tensor-core scoring kernels (sm_100a): constants, operand descriptors of the
// handle, kernel parameters, inline-PTX wrappers (mbarrier, bulk copy, tcgen05), the FP16 split and the
// cold close-pair refinement.  Included by the translation units that hold tcgen05 kernels; everything
// here has internal linkage.
#pragma once

#include <cuda_fp16.h>
#include <math.h>
#include <stdint.h>

#include "r3_internal.cuh"

namespace r3 {

struct TensorOperands {
    int NV = 0, G = 0, KD = 0, DP = 0, NP = 0, P = 0, ws = 0;
    bool kt = false;           // k* buffers in TMEM
    bool f8 = false;           // cross terms of the variance product as FP8 MMAs
    int nbk = 0;               // number of k* buffers (== G: one per group; smaller: a shared ring)
    size_t smem_bytes = 0;
    size_t wt_gp_stride = 0;   // halves per GP in wt
    float* centre = nullptr;   // [B][DP]  column means of X (zero padded)
    float* scale = nullptr;    // [B][DP]  1/lengthscale (zero padded)
    __half* xt = nullptr;      // [B][NP/KD][2][DP/8][KD][8]  scaled observations, FP16 hi/lo planes
    float* xs32 = nullptr;     // [B][NP][DP]  scaled observations in FP32 (refinement of close pairs)
    float* xnorm = nullptr;    // [B][NP]  |x~_k|^2
    float* xnmax = nullptr;    // [B]      max_k |x~_k|^2
    float* alpha = nullptr;    // [B][NP]  weights, zero padded
    __half* wt = nullptr;      // [B][tile(p,c)][2][KC/8][NV][8]  chunks of 2^eW W, FP16 hi/lo planes; with f8 the
                               // second plane is two 8-bit planes [2][KC/16][NV][16]: hi parts (E4M3), then lo parts (E5M2)
    float* kscale = nullptr;   // [B]  2^eK, applied to k* before its split
    double* vinv2 = nullptr;   // [B]  2^(-2 (eK + eW)): scales sum V^2 back
};

struct TcParams {
    const float* xcand;
    long long m;
    int batch, d;
    float *mu, *sigma, *ei, *err_mu, *err_q;
    const float *centre, *scale, *xs32, *xnorm, *xnmax, *alpha, *kscale;
    const __half *xt, *wt;
    const double* vinv2;
    size_t wt_gp_stride;
    const float *sf2, *best;
    const double* wnorm;
    int DP, NP, P, ws;
    int* status;
    long long tiles_per_gp, total_tiles;   // total_tiles: one past the last tile of this launch
    long long tile_begin;                  // first tile of this launch (the single-CTA kernel; 0 for a whole pool)
    long long* trace;   // optional [grid][4 roles][8] cycle counters (diagnostics)
    long long wait_limit;   // cycles after which a device-side wait gives up (r3_gp_set_wait_limit)
    long long withhold_w;   // >= 0: every CTA's stream of W stops before that chunk of its own sequence, so that the
                            // consumer's wait runs out (r3_gp_test_withhold, one call); -1 otherwise
};

// paired (two-CTA cluster) form of the tensor kernel, r3_score_tc2.cu
bool tc_pair_fits(const TensorOperands* t, int* ws_out);
r3_status_t launch_tc_pair(const TensorOperands* t, TcParams prm, int sms, cudaStream_t stream);

namespace {

constexpr int KC = 32;        // observations per chunk of the variance product
constexpr int TILE_M = 128;   // candidates per CTA tile
constexpr int XS = 2;         // stages of scaled observations
constexpr int MAX_STAGES = 6; // stages of W

// Scaled coordinates are x^ = (x - centre) * sqrt(5) log2(e) / lengthscale, so that u = |z^ - x^| is the
// Matern argument in base-2 units: s = sqrt(5) r = u ln 2, exp(-s) = 2^-u, 1 + s + s^2/3 = 1 + c1 u + c2 u^2.
constexpr double kCoordScale = 2.23606797749978969641 * 1.44269504088896340736;
constexpr float kPolyC1 = 0.69314718055994530942f;               // ln 2
constexpr float kPolyC2 = 0.16015101049403078f;                  // (ln 2)^2 / 3
// relative error of one k* entry: eps0 + eps1 * (|z^|^2 + max|x^|^2) / sqrt(d)  (distance by split GEMM)
constexpr double kEpsTc0 = 2.5e-7;
constexpr double kEpsTc1 = 5.0e-8 / (kCoordScale * kCoordScale);
// A pair (candidate, observation) whose k*/sf2 (|z^|^2 + |x^|^2) exceeds kRefine has its squared distance
// recomputed by direct differences: r^2 from the norm expansion loses (|z~|^2 + |x~|^2) / r^2 digits, and
// the close pairs are the ones that carry the posterior.
constexpr float kRefine = 2.0f * (float)(kCoordScale * kCoordScale);
// scaled coordinates beyond this do not fit the FP16 planes of the distance product
constexpr float kMaxScaled = 16384.f;
// operands of the variance product are scaled to at most 2^kScaleExp before the FP16 split
constexpr int kScaleExp = 14;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand from TMEM (lane = row, one 32-bit column = two consecutive FP16 k-elements)
__device__ __forceinline__ void tc_mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                              uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// kind::f8f6f4, K = 32; the instruction descriptor is the FP16 one plus the operands' format codes
// (instr_desc_f8)
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand from TMEM (lane = row, one 32-bit column = four consecutive 8-bit k-elements)
__device__ __forceinline__ void tc_mma_f8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t* r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// The same load without the wait: several can be in flight; tc_wait_ld32 ends them.
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, float* v)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]),
          "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
        : "r"(taddr)
        : "memory");
}
// Wait for the loads in flight.  The 32 destination registers are operands of the wait (and of an empty
// statement after it) so that no use of them can be scheduled ahead of it.
__device__ __forceinline__ void tc_wait_ld32(float* a, float* b)
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7]),
                   "+f"(a[8]), "+f"(a[9]), "+f"(a[10]), "+f"(a[11]), "+f"(a[12]), "+f"(a[13]), "+f"(a[14]), "+f"(a[15])
                 :
                 : "memory");
    asm volatile(""
                 : "+f"(b[0]), "+f"(b[1]), "+f"(b[2]), "+f"(b[3]), "+f"(b[4]), "+f"(b[5]), "+f"(b[6]), "+f"(b[7]),
                   "+f"(b[8]), "+f"(b[9]), "+f"(b[10]), "+f"(b[11]), "+f"(b[12]), "+f"(b[13]), "+f"(b[14]), "+f"(b[15])
                 :
                 : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t* r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ uint64_t pack64(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ float sqrt_approx(float x)
{
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float exp2_approx(float x)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// (a, b) -> FP16 hi parts and FP16 low parts, each packed as half2
__device__ __forceinline__ void split2(float a, float b, __half2& hi, __half2& lo)
{
    hi = __floats2half2_rn(a, b);
    const float2 back = __half22float2(hi);
    lo = __floats2half2_rn(a - back.x, b - back.y);
}

// Cross terms of the variance product in FP8.  With x = hi + lo (hi = fp16(x)) the product W k* is
// W_hi k_hi + W_hi k_lo + W_lo k_hi; the two cross terms are 2^-11 of the first, so 8-bit factors leave them with a
// relative error of 2^-3 to 2^-4 and the sum with about 2^-15 -- enough wherever q = |W k*|^2 is a modest part of
// the signal variance, and the accuracy guard recomputes the rest in FP64.
// Formats: the parts of k* are E5M2, taken from the FP16 hi part and the FP32 remainder as they are (hi parts
// below 2^14, lo parts below 2^3: both inside E5M2's range, no scaling -- the conversion is all the Matern warps
// pay, and with E4M3 the two multiplications per element that brought the parts into its range were a tenth of
// their instructions); W is scaled to below 2^8 for these histories, so that its hi parts fit E4M3 unscaled
// (three mantissa bits where it costs nothing: W is converted once per fit) and its lo parts, below 2^-3, go to
// E5M2 for the range.
constexpr int kScaleExpF8 = 8;   // |scaled W| < 2^8 when the cross terms are FP8 (E4M3 holds up to 448)
// (a, b, c, d) -> four E4M3 bytes, a in the lowest
__device__ __forceinline__ uint32_t e4m3x4(float a, float b, float c, float d)
{
    uint16_t lo16, hi16;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo16) : "f"(b), "f"(a));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi16) : "f"(d), "f"(c));
    return (uint32_t)lo16 | ((uint32_t)hi16 << 16);
}
// (a, b, c, d) -> four E5M2 bytes, a in the lowest
__device__ __forceinline__ uint32_t e5m2x4(float a, float b, float c, float d)
{
    uint16_t lo16, hi16;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(lo16) : "f"(b), "f"(a));
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(hi16) : "f"(d), "f"(c));
    return (uint32_t)lo16 | ((uint32_t)hi16 << 16);
}
// two packed halves -> two E5M2 bytes (the lower half in the lower byte)
__device__ __forceinline__ uint32_t e5m2x2_of_half2(uint32_t h2)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e5m2x2.f16x2 %0, %1;" : "=h"(r) : "r"(h2));
    return (uint32_t)r;
}
// four values -> FP16 hi parts (two half2), and the E5M2 forms of the hi parts and of the remainders
__device__ __forceinline__ void split4_f8(const float* v, uint32_t& h01, uint32_t& h23, uint32_t& hi8, uint32_t& lo8)
{
    const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
    const float2 fa = __half22float2(a), fb = __half22float2(b);
    h01 = *reinterpret_cast<const uint32_t*>(&a);
    h23 = *reinterpret_cast<const uint32_t*>(&b);
    hi8 = e5m2x2_of_half2(h01) | (e5m2x2_of_half2(h23) << 16);
    lo8 = e5m2x4(v[0] - fa.x, v[1] - fa.y, v[2] - fb.x, v[3] - fb.y);
}
// relative error of one cross product in that form (root mean square over rounding positions), added to the
// per-entry error of k* in the estimate of the error of q
constexpr double kEpsF8 = 2.9e-5;

// Shared-memory matrix descriptors are the no-swizzle K-major form: bits 0-13 start address >> 4,
// bits 16-29 the byte distance between the two 16-byte k-slices of one MMA >> 4, bits 32-45 the byte
// distance between 8-row groups (128) >> 4, bit 46 the descriptor version.
constexpr uint32_t kDescHi = (128u >> 4) | (1u << 14);
// Start-address field of a descriptor: the CTA-local 18-bit shared-memory offset >> 4.  Inside a cluster a
// shared-memory address carries the CTA's rank in its upper bits, which must not leak into the next field.
__device__ __forceinline__ uint32_t desc_addr(uint32_t saddr) { return (saddr & 0x3FFFFu) >> 4; }
// Instruction descriptor: FP32 accumulate, FP16 x FP16 (format code 0), both K-major, M = 128, N = n.
__device__ __forceinline__ constexpr uint32_t instr_desc_f16(uint32_t n)
{
    return (1u << 4) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
// kind::f8f6f4: format code of A in bits 7-9 and of B in bits 10-12 (0 = E4M3, 1 = E5M2)
constexpr uint32_t kFmtE4M3 = 0u, kFmtE5M2 = 1u;
__device__ __forceinline__ constexpr uint32_t instr_desc_f8(uint32_t n, uint32_t a_fmt, uint32_t b_fmt)
{
    return instr_desc_f16(n) | (a_fmt << 7) | (b_fmt << 10);
}

// Out-of-line (cold) path of the Matern warps: for the pairs whose (scaled) k* exceeds v_thresh, replace it by the value
// computed from r^2 = sum_j (z~_j - x~_j)^2, with z~ = hi + lo read back from the TMEM planes at z_taddr
// and x~ in FP32 from global memory.  Called by all 32 lanes of a warp together (TMEM loads are
// warp-wide); a lane without marked pairs only takes part in the loads.
// Refined values are kept for the later passes of the same tile (k* chunks are regenerated for every pass, and this
// path is what a regeneration costs most: the warp that takes it holds up its group and then the MMA issuer).
// `slots`: the candidate row's kCacheSlots direct-mapped entries (key << 32 | value bits) in shared memory, or
// nullptr; key0 + i identifies (tile, observation) of kv[i]; `lookup`: earlier passes may have left the values.
// An overwritten slot is a miss, and a miss is recomputed.
constexpr uint32_t kCacheSlots = 4;
__device__ __forceinline__ uint32_t cache_slot(uint32_t key) { return (key + (key >> 4)) & (kCacheSlots - 1); }
template <bool CACHE>
__device__ __noinline__ void refine_close_pairs(float* kv, float v_thresh, float kvscale, uint32_t z_taddr, int DP,
                                                const float* __restrict__ xrow0, unsigned long long* slots,
                                                uint32_t key0, bool lookup)
{
    uint32_t close = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) close |= (kv[i] > v_thresh) ? (1u << i) : 0u;
    if (CACHE && lookup) {
        uint32_t missing = 0;
        for (uint32_t rest = close; rest; rest &= rest - 1) {
            const int i = __ffs(rest) - 1;
            const unsigned long long e = slots[cache_slot(key0 + i)];
            if ((uint32_t)(e >> 32) == key0 + i)
                kv[i] = __uint_as_float((uint32_t)e);
            else
                missing |= 1u << i;
        }
        if (!__any_sync(0xffffffffu, missing != 0)) return;
        close = missing;
    }
    float r2x[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) r2x[i] = 0.f;
    for (int j16 = 0; j16 < DP / 16; ++j16) {
        uint32_t zh[8], zl[8];
        tc_ld8(z_taddr + j16 * 8, zh);
        tc_ld8(z_taddr + DP / 2 + j16 * 8, zl);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        float z[16];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&zh[e]));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&zl[e]));
            z[2 * e] = a.x + b.x;
            z[2 * e + 1] = a.y + b.y;
        }
        for (uint32_t rest = close; rest; rest &= rest - 1) {
            const int i = __ffs(rest) - 1;
            const float4* xp = reinterpret_cast<const float4*>(xrow0 + (size_t)i * DP + j16 * 16);
            float acc = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float4 x4 = __ldg(xp + e);
                float df = z[4 * e] - x4.x;
                acc = fmaf(df, df, acc);
                df = z[4 * e + 1] - x4.y;
                acc = fmaf(df, df, acc);
                df = z[4 * e + 2] - x4.z;
                acc = fmaf(df, df, acc);
                df = z[4 * e + 3] - x4.w;
                acc = fmaf(df, df, acc);
            }
            r2x[i] += acc;
        }
    }
    for (uint32_t rest = close; rest; rest &= rest - 1) {
        const int i = __ffs(rest) - 1;
        const float u = sqrtf(r2x[i]);
        kv[i] = kvscale * fmaf(u, fmaf(u, kPolyC2, kPolyC1), 1.f) * exp2f(-u);
        if (CACHE) slots[cache_slot(key0 + i)] = ((unsigned long long)(key0 + i) << 32) | __float_as_uint(kv[i]);
    }
}

// Per-role cycle accounting, compiled in only with -DR3_TC_TRACE (it costs issue slots on the hot path).
#ifndef R3_TC_TRACE
#define TICK(cat) do { } while (0)
#define LOGEV(ev, tt) do { } while (0)
#else
// event log of the first CTA: clock of event `ev` for global chunk number tt in [kLogT0, kLogT0 + kLogN)
constexpr long long kLogT0 = 1088 + 600, kLogN = 128;
#define LOGEV(ev, tt)                                                                                         \
    do {                                                                                                      \
        if (prm.trace && blockIdx.x == 0 && (tt) >= kLogT0 && (tt) < kLogT0 + kLogN)                          \
            prm.trace[(size_t)gridDim.x * 32 + (ev) * kLogN + ((tt) - kLogT0)] = clock64();                   \
    } while (0)
#ifdef R3_TC_TRACE_EVENTS_ONLY
#define TICK(cat) do { } while (0)
#else
#define TICK(cat)                                                                          \
    do {                                                                                   \
        if (prm.trace) {                                                                   \
            const long long now__ = clock64();                                             \
            tacc[cat] += now__ - tlast;                                                    \
            tlast = now__;                                                                 \
        }                                                                                  \
    } while (0)
#endif
#endif

}  // namespace

}  // namespace r3
