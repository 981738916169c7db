// Tensor-core scoring engine for sm_100a: tcgen05 MMAs (kind::tf32, 3xTF32 split) with TMEM
// accumulators, operands staged by bulk asynchronous copies, everything fused in one kernel so that
// the cross-covariance k* never leaves the SM.
//
// One CTA owns a tile of 128 candidates; a TMEM lane IS a candidate.  For that tile it walks the rows
// of W = L^-1 in passes of NV rows (the V accumulator: 128 lanes x NV TMEM columns) and, inside a pass,
// the observations in chunks of KC = 16:
//
//   distance MMA   D[cand][k] = z~ . x~_k   (A = scaled candidates, B = scaled observations, depth d)
//   Matern warps   r^2 = |z~|^2 + |x~_k|^2 - 2 D, k* = sf2 M52(r): read D from TMEM, write k* (hi/lo
//                  TF32 planes) as the next A operand into shared memory; mu += k* alpha on the way
//   variance MMA   V[cand][i] += k*[cand][k] W[i][k]   (B = pre-tiled chunk of W, hi/lo planes)
//   end of pass    q += sum_i V[cand][i]^2 read back from TMEM; after the last pass sigma, EI, outputs
//
// Each product is three MMAs (hi*hi + hi*lo + lo*hi) accumulating in FP32, which restores FP32-level
// accuracy from TF32 operands.  W is lower-triangular, so pass p only needs k < (p+1) NV; k* chunks are
// regenerated for every pass they take part in instead of being stored.
//
// Warp roles: warp 0 streams chunks of scaled observations, warp 1 streams chunks of W, warp 2 issues
// every MMA (one thread) and owns the TMEM allocation, warps 4.. form G Matern/epilogue groups of four
// warps (one warp per TMEM lane quarter); group g takes every G-th chunk with its own distance and k*
// buffers, so G chunks are in flight between the two MMA streams.  Stages are handed over through mbarriers; every wait is
// bounded: when a limit is hit the CTA raises a status bit, all roles leave their loops, in-flight
// copies and MMAs are drained (bounded again), TMEM is freed and the kernel returns.
//
// Operand layouts are the no-swizzle K-major "core matrix" form: 8 rows x 16 bytes contiguous, 8-row
// groups 128 bytes apart, 16-byte k-slices one full panel apart.  W and the observations are stored
// in global memory already tiled that way by the fit, so a stage is one contiguous bulk copy.
#include "r3_epilogue.cuh"
#include "r3_internal.cuh"

namespace r3 {

namespace {

constexpr int KC = 16;        // observations per chunk
constexpr int TILE_M = 128;   // candidates per CTA tile
constexpr int MAX_STAGES = 4;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;  // ~2 s

// relative error of one k* entry: eps0 + eps1 * (|z~|^2 + max|x~|^2) / sqrt(d)  (distance by 3xTF32 GEMM)
constexpr double kEpsTc0 = 2.5e-7;
constexpr double kEpsTc1 = 2.0e-7;

struct TensorOperands {
    int NV = 0, G = 0, DP = 0, NP = 0, P = 0, xs = 0, ws = 0, tmem_cols = 0;
    size_t smem_bytes = 0;
    size_t wt_gp_stride = 0;   // floats per GP in wt
    float* centre = nullptr;   // [B][DP]  column means of X (zero padded)
    float* scale = nullptr;    // [B][DP]  1/lengthscale (zero padded)
    float* xt = nullptr;       // [B][NP/KC][2][DP/4][KC][4]  scaled observations, hi/lo planes
    float* xnorm = nullptr;    // [B][NP]  |x~_k|^2
    float* xnmax = nullptr;    // [B]      max_k |x~_k|^2
    float* alpha = nullptr;    // [B][NP]  weights, zero padded
    float* wt = nullptr;       // [B][tile(p,c)][2][KC/4][NV][4]  W chunks, hi/lo planes
};

struct TcParams {
    const float* xcand;
    long long m;
    int batch, d;
    float *mu, *sigma, *ei, *err_mu, *err_q;
    const float *centre, *scale, *xt, *xnorm, *xnmax, *alpha, *wt;
    size_t wt_gp_stride;
    const float *sf2, *best;
    const double* wnorm;
    int DP, NP, P, xs, ws;
    int* status;
    long long tiles_per_gp, total_tiles;
};

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
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
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
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
__device__ __forceinline__ float tf32_hi(float x)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

// Shared-memory matrix descriptors are the no-swizzle K-major form: bits 0-13 start address >> 4,
// bits 16-29 the byte distance between the two 16-byte k-slices of one MMA >> 4, bits 32-45 the byte
// distance between 8-row groups >> 4, bit 46 the descriptor version.
// Instruction descriptor: FP32 accumulate, TF32 x TF32, both K-major, M = 128, N = n.
__device__ __forceinline__ constexpr uint32_t instr_desc(uint32_t n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// shared-memory map (byte offsets from a 1024-aligned base)
struct SmemMap {
    uint32_t z, k, x, w, bar;
    uint32_t x_stage, w_stage;
};
__host__ __device__ inline SmemMap smem_map(int DP, int NV, int G, int xs, int ws)
{
    SmemMap s;
    s.z = 0;                                       // 2 planes x [DP/4][128][4] floats
    s.k = s.z + 2u * DP * 512u;                    // G buffers x 2 planes x [KC/4][128][4]
    s.x = s.k + (uint32_t)G * 16384u;              // xs stages x 2 planes x [DP/4][KC][4]
    s.x_stage = 2u * DP * KC * 4u;
    s.w = s.x + (uint32_t)xs * s.x_stage;          // ws stages x 2 planes x [KC/4][NV][4]
    s.w_stage = 2u * KC * NV * 4u;
    s.bar = s.w + (uint32_t)ws * s.w_stage;
    return s;
}
constexpr uint32_t kBarBytes = 1024;   // barriers, flags, TMEM slot, candidate norms

// barrier slots (8 bytes each) inside the barrier block
enum : uint32_t {
    BAR_X_FULL = 0, BAR_X_EMPTY = 4, BAR_W_FULL = 8, BAR_W_EMPTY = 12, BAR_D_FULL = 16, BAR_D_EMPTY = 20,
    BAR_K_FULL = 24, BAR_K_EMPTY = 28, BAR_V_FULL = 32, BAR_V_EMPTY = 33, BAR_Z_READY = 34, BAR_MMA_DONE = 35,
    BAR_RED_READY = 36, BAR_COUNT = 37
};
constexpr uint32_t kFlagOffset = BAR_COUNT * 8;       // int abort, int drain-abort, uint32 tmem base
constexpr uint32_t kZnOffset = 512;                   // float[128] squared norms of the scaled candidates

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

// NV: rows of W per pass (TMEM columns of the V accumulator).  G: number of Matern warp groups; group
// g owns items t = g (mod G) of the chunk sequence together with distance buffer g and k* buffer g.
template <int NV, int G>
__global__ void __launch_bounds__(128 + 128 * G, 1) score_tc_kernel(const TcParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const SmemMap map = smem_map(prm.DP, NV, G, prm.xs, prm.ws);
    const uint32_t bars = base + map.bar;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + map.bar + kFlagOffset);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + map.bar + kFlagOffset + 8);
    float* zn_s = reinterpret_cast<float*>(sm + map.bar + kZnOffset);
    auto bar = [&](uint32_t slot) { return bars + slot * 8u; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int CPP = NV / KC;                  // chunks per pass width
    constexpr uint32_t TMEM_COLS = (NV + G * KC) <= 256 ? 256u : 512u;
    const int DP = prm.DP, P = prm.P, xs = prm.xs, ws = prm.ws;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(bar(BAR_X_FULL + i), 1);
            mbar_init(bar(BAR_X_EMPTY + i), 1);
            mbar_init(bar(BAR_W_FULL + i), 1);
            mbar_init(bar(BAR_W_EMPTY + i), 1);
            mbar_init(bar(BAR_D_FULL + i), 1);
            mbar_init(bar(BAR_D_EMPTY + i), 128);
            mbar_init(bar(BAR_K_FULL + i), 128);
            mbar_init(bar(BAR_K_EMPTY + i), 1);
        }
        mbar_init(bar(BAR_V_FULL), 1);
        mbar_init(bar(BAR_V_EMPTY), 128 * G);
        mbar_init(bar(BAR_Z_READY), 128);
        mbar_init(bar(BAR_MMA_DONE), 1);
        mbar_init(bar(BAR_RED_READY), 128 * G);
        abort_flag[0] = 0;
        abort_flag[1] = 0;   // private flag of the bounded drain waits
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32((const void*)tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
    const long long first_tile = blockIdx.x, tile_step = gridDim.x;
    const int items_per_tile = CPP * P * (P + 1) / 2;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------ producer: scaled observations
        const uint32_t bytes = map.x_stage;
        long long t = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const float* src = prm.xt + (size_t)g * (prm.NP / KC) * (bytes / 4);
            for (int p = 0; ok && p < P; ++p)
                for (int c = 0; c < (p + 1) * CPP; ++c, ++t) {
                    const int s = (int)(t % xs);
                    if (!(ok = mbar_wait(bar(BAR_X_EMPTY + s), (uint32_t)(((t / xs) & 1) ^ 1), abort_flag))) break;
                    mbar_arrive_expect_tx(bar(BAR_X_FULL + s), bytes);
                    bulk_g2s(base + map.x + s * bytes, src + (size_t)c * (bytes / 4), bytes, bar(BAR_X_FULL + s));
                }
        }
        if (!ok)  // aborting: let the copies still in flight land before the CTA goes away
            for (long long u = (t > xs ? t - xs : 0); u < t; ++u)
                mbar_wait(bar(BAR_X_FULL + (int)(u % xs)), (uint32_t)((u / xs) & 1), abort_flag + 1);
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------ producer: chunks of W
        const uint32_t bytes = map.w_stage;
        long long t = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const float* src = prm.wt + (size_t)g * prm.wt_gp_stride;
            for (int p = 0; ok && p < P; ++p) {
                const float* psrc = src + (size_t)(CPP * p * (p + 1) / 2) * (bytes / 4);
                for (int c = 0; c < (p + 1) * CPP; ++c, ++t) {
                    const int s = (int)(t % ws);
                    if (!(ok = mbar_wait(bar(BAR_W_EMPTY + s), (uint32_t)(((t / ws) & 1) ^ 1), abort_flag))) break;
                    mbar_arrive_expect_tx(bar(BAR_W_FULL + s), bytes);
                    bulk_g2s(base + map.w + s * bytes, psrc + (size_t)c * (bytes / 4), bytes, bar(BAR_W_FULL + s));
                }
            }
        }
        if (!ok)
            for (long long u = (t > ws ? t - ws : 0); u < t; ++u)
                mbar_wait(bar(BAR_W_FULL + (int)(u % ws)), (uint32_t)((u / ws) & 1), abort_flag + 1);
    } else if (warp == 2 && lane == 0) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t IDESC_D = instr_desc(KC);
        constexpr uint32_t IDESC_V = instr_desc(NV);
        // descriptor words: lo = start>>4 | (lbo>>4)<<16, hi = sbo>>4 | version bit
        constexpr uint32_t HI = (128u >> 4) | (1u << 14);
        const uint32_t zH_lo = ((base + map.z) >> 4) | ((2048u >> 4) << 16);
        const uint32_t zL_lo = zH_lo + (((uint32_t)DP * 512u) >> 4);
        const uint32_t x_lo0 = ((base + map.x) >> 4) | (((KC * 16u) >> 4) << 16);
        const uint32_t k_lo0 = ((base + map.k) >> 4) | ((2048u >> 4) << 16);
        const uint32_t w_lo0 = ((base + map.w) >> 4) | (((NV * 16u) >> 4) << 16);
        const int ksteps_d = DP / 8;
        long long t = 0;      // item counter (rings)
        long long pv = 0;     // pass counter (V accumulator hand-over)
        long long tile_iter = 0;
        bool ok = true;

        auto issue_distance = [&](long long tu) -> bool {
            const int s = (int)(tu % xs), b = (int)(tu % G);
            const long long j = tu / G;
            if (!mbar_wait(bar(BAR_X_FULL + s), (uint32_t)((tu / xs) & 1), abort_flag)) return false;
            if (!mbar_wait(bar(BAR_D_EMPTY + b), (uint32_t)((j & 1) ^ 1), abort_flag)) return false;
            tc_fence_after();
            const uint32_t xH_lo = x_lo0 + ((s * map.x_stage) >> 4), xL_lo = xH_lo + (((uint32_t)DP * KC * 4u) >> 4);
            const uint32_t dcol = tmem + NV + b * KC;
            uint32_t acc = 0;
#pragma unroll
            for (int combo = 0; combo < 3; ++combo) {
                const uint32_t a0 = combo == 2 ? zL_lo : zH_lo, b0 = combo == 1 ? xL_lo : xH_lo;
                for (int jj = 0; jj < ksteps_d; ++jj) {
                    tc_mma_tf32(dcol, pack64(a0 + jj * (4096u >> 4), HI), pack64(b0 + jj * ((2u * KC * 16u) >> 4), HI),
                                IDESC_D, acc);
                    acc = 1;
                }
            }
            tc_commit(bar(BAR_X_EMPTY + s));
            tc_commit(bar(BAR_D_FULL + b));
            return true;
        };

        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            if (!(ok = mbar_wait(bar(BAR_Z_READY), (uint32_t)(tile_iter & 1), abort_flag))) break;
            tc_fence_after();
            const long long t_tile0 = t;
            for (int u = 0; ok && u < G && u < items_per_tile; ++u) ok = issue_distance(t_tile0 + u);
            for (int p = 0; ok && p < P; ++p) {
                const int nchunk = (p + 1) * CPP;
                for (int c = 0; ok && c < nchunk; ++c, ++t) {
                    const int b = (int)(t % G), s = (int)(t % ws);
                    const long long j = t / G;
                    if (c == 0) {
                        if (!(ok = mbar_wait(bar(BAR_V_EMPTY), (uint32_t)((pv & 1) ^ 1), abort_flag))) break;
                    }
                    if (!(ok = mbar_wait(bar(BAR_K_FULL + b), (uint32_t)(j & 1), abort_flag))) break;
                    if (!(ok = mbar_wait(bar(BAR_W_FULL + s), (uint32_t)((t / ws) & 1), abort_flag))) break;
                    tc_fence_after();
                    const uint32_t aH = k_lo0 + ((b * 16384u) >> 4), aL = aH + (8192u >> 4);
                    const uint32_t bH = w_lo0 + ((s * map.w_stage) >> 4), bL = bH + (((uint32_t)KC * NV * 4u) >> 4);
#pragma unroll
                    for (int combo = 0; combo < 3; ++combo) {
                        const uint32_t a0 = combo == 2 ? aL : aH, b0 = combo == 1 ? bL : bH;
#pragma unroll
                        for (int jj = 0; jj < KC / 8; ++jj)
                            tc_mma_tf32(tmem, pack64(a0 + jj * (4096u >> 4), HI),
                                        pack64(b0 + jj * ((2u * NV * 16u) >> 4), HI), IDESC_V,
                                        (c > 0 || combo > 0 || jj > 0) ? 1u : 0u);
                    }
                    tc_commit(bar(BAR_W_EMPTY + s));
                    tc_commit(bar(BAR_K_EMPTY + b));
                    if (c == nchunk - 1) {
                        tc_commit(bar(BAR_V_FULL));
                        ++pv;
                    }
                    const long long ahead = t + G;
                    if (ahead - t_tile0 < items_per_tile) ok = issue_distance(ahead);
                }
            }
        }
        // every MMA issued so far must have completed before TMEM is freed
        tc_commit(bar(BAR_MMA_DONE));
        mbar_wait(bar(BAR_MMA_DONE), 0, abort_flag + 1);
    } else if (warp >= 4) {
        // ------------------------------------------------------------ Matern / epilogue warp groups
        const int grp = (warp - 4) >> 2;         // 0..G-1
        const int q4 = warp & 3;                 // TMEM lane quarter == warp % 4
        const int row = q4 * 32 + lane;          // candidate row in the tile == TMEM lane
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        long long t = grp;                       // next own item (global numbering)
        long long t_tile0 = 0;                   // first item of the current tile
        long long pv = 0, tile_iter = 0;
        bool ok = true;
        bool bad = false;
        // scratch for the end-of-tile reduction lives in k* buffer 0 (dead once the last pass is done)
        double* red = reinterpret_cast<double*>(sm + map.k);
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const long long cand = (tile % prm.tiles_per_gp) * TILE_M + row;
            const bool valid = cand < prm.m;
            const float sf2 = prm.sf2[g];
            if (grp == G - 1) {
                // ---- scale the candidate, split it, store it as the A operand of the distance MMA
                float zn = 0.f;
                const float* zrow = prm.xcand + ((size_t)g * prm.m + (valid ? cand : 0)) * prm.d;
                const float* cen = prm.centre + (size_t)g * DP;
                const float* scl = prm.scale + (size_t)g * DP;
                const bool vec = (prm.d % 4) == 0;
                for (int j4 = 0; j4 < DP / 4; ++j4) {
                    float z[4];
                    if (vec && 4 * j4 < prm.d) {
                        const float4 v = *reinterpret_cast<const float4*>(zrow + 4 * j4);
                        z[0] = v.x; z[1] = v.y; z[2] = v.z; z[3] = v.w;
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) z[e] = (4 * j4 + e < prm.d) ? zrow[4 * j4 + e] : 0.f;
                    }
                    const float4 c4 = __ldg(reinterpret_cast<const float4*>(cen + 4 * j4));
                    const float4 s4 = __ldg(reinterpret_cast<const float4*>(scl + 4 * j4));
                    const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
                    float hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        bad |= !isfinite(z[e]);
                        const float zt = valid ? (z[e] - cc[e]) * ss[e] : 0.f;
                        zn = fmaf(zt, zt, zn);
                        hi[e] = tf32_hi(zt);
                        lo[e] = zt - hi[e];
                    }
                    *reinterpret_cast<float4*>(sm + map.z + (uint32_t)j4 * 2048u + row * 16) =
                        make_float4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<float4*>(sm + map.z + (uint32_t)DP * 512u + (uint32_t)j4 * 2048u + row * 16) =
                        make_float4(lo[0], lo[1], lo[2], lo[3]);
                }
                zn_s[row] = zn;
                fence_proxy_async();
                mbar_arrive(bar(BAR_Z_READY));
            }
            ok = mbar_wait(bar(BAR_Z_READY), (uint32_t)(tile_iter & 1), abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const float zn = zn_s[row];

            const float* xn_g = prm.xnorm + (size_t)g * prm.NP;
            const float* al_g = prm.alpha + (size_t)g * prm.NP;
            double mu_acc = 0.0, a2_acc = 0.0, s2_acc = 0.0, q_acc = 0.0;
            int pass_base = 0;   // items of this tile before pass p
            for (int p = 0; ok && p < P; ++p) {
                const int nchunk = (p + 1) * CPP;
                // own items of this pass: global t with t - t_tile0 - pass_base in [0, nchunk)
                while (t - t_tile0 - pass_base < nchunk) {
                    const int c = (int)(t - t_tile0 - pass_base);
                    const long long j = t / G;
                    // the next own chunk's norms and weights: pull them towards L1 while this one is worked on
                    if (lane < 2) {
                        const int cn = c + G < nchunk ? c + G : (c + G - nchunk);
                        const float* pf = (lane == 0 ? xn_g : al_g) + cn * KC;
                        asm volatile("prefetch.global.L1 [%0];" ::"l"(pf));
                    }
                    ok = mbar_wait(bar(BAR_D_FULL + grp), (uint32_t)(j & 1), abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    float dot[KC];
                    tc_ld16(lane_addr + NV + grp * KC, dot);
                    tc_fence_before();
                    mbar_arrive(bar(BAR_D_EMPTY + grp));
                    const bool fresh = c >= p * CPP;   // first time this chunk is generated for the tile
                    float kv[KC];
                    float mpart = 0.f, apart = 0.f, spart = 0.f;
#pragma unroll
                    for (int q = 0; q < KC / 4; ++q) {
                        const float4 xn4 = __ldg(reinterpret_cast<const float4*>(xn_g + c * KC + 4 * q));
                        const float4 al4 = __ldg(reinterpret_cast<const float4*>(al_g + c * KC + 4 * q));
                        const float xn[4] = {xn4.x, xn4.y, xn4.z, xn4.w}, al[4] = {al4.x, al4.y, al4.z, al4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float r2 = fmaxf(fmaf(-2.f, dot[4 * q + e], zn + xn[e]), 0.f);
                            const float s = sqrt_approx(5.f * r2);
                            const float v = sf2 * fmaf(s, fmaf(s, 1.f / 3.f, 1.f), 1.f) * __expf(-s);
                            kv[4 * q + e] = v;
                            const float va = v * al[e];
                            mpart += va;
                            apart = fmaf(va, va, apart);
                            spart = fmaf(v, v, spart);
                        }
                    }
                    if (fresh) {
                        mu_acc += (double)mpart;
                        a2_acc += (double)apart;
                        s2_acc += (double)spart;
                    }
                    ok = mbar_wait(bar(BAR_K_EMPTY + grp), (uint32_t)((j & 1) ^ 1), abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    uint8_t* kb = sm + map.k + grp * 16384u + row * 16;
#pragma unroll
                    for (int q = 0; q < KC / 4; ++q) {
                        float hi[4], lo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            hi[e] = tf32_hi(kv[4 * q + e]);
                            lo[e] = kv[4 * q + e] - hi[e];
                        }
                        *reinterpret_cast<float4*>(kb + q * 2048u) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<float4*>(kb + 8192u + q * 2048u) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                    }
                    fence_proxy_async();
                    mbar_arrive(bar(BAR_K_FULL + grp));
                    t += G;
                }
                if (!ok) break;
                pass_base += nchunk;
                // ---- end of pass: q += sum_i V^2 over this group's share of the columns
                ok = mbar_wait(bar(BAR_V_FULL), (uint32_t)(pv & 1), abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int c0 = grp * 16; c0 < NV; c0 += 16 * G) {
                    float v[16];
                    tc_ld16(lane_addr + c0, v);
                    float part = 0.f;
#pragma unroll
                    for (int i = 0; i < 16; ++i) part = fmaf(v[i], v[i], part);
                    q_acc += (double)part;
                }
                tc_fence_before();
                mbar_arrive(bar(BAR_V_EMPTY));
                ++pv;
            }
            if (!ok) break;
            t_tile0 += items_per_tile;
            // ---- combine the groups' partial sums; group 0 finishes the candidate
            if (G > 1) {
                double* mine = red + ((size_t)grp * TILE_M + row) * 4;
                mine[0] = mu_acc; mine[1] = a2_acc; mine[2] = s2_acc; mine[3] = q_acc;
                mbar_arrive(bar(BAR_RED_READY));
                if (grp == 0) {   // only the finishing group waits; the others move on to the next tile
                    ok = mbar_wait(bar(BAR_RED_READY), (uint32_t)(tile_iter & 1), abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
            }
            if (grp == 0 && valid) {
                if (G > 1) {
                    mu_acc = a2_acc = s2_acc = q_acc = 0.0;
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) {
                        const double* o = red + ((size_t)gg * TILE_M + row) * 4;
                        mu_acc += o[0]; a2_acc += o[1]; s2_acc += o[2]; q_acc += o[3];
                    }
                }
                const size_t f = (size_t)g * prm.m + cand;
                const CandidateResult res = finalize_candidate(mu_acc, q_acc, (double)sf2, (double)prm.best[g]);
                prm.mu[f] = res.mu;
                prm.sigma[f] = res.sigma;
                prm.ei[f] = res.ei;
                const double eps = kEpsTc0 + kEpsTc1 * (double)(zn + prm.xnmax[g]) * rsqrt((double)DP);
                prm.err_mu[f] = mu_error_estimate(eps, a2_acc);
                prm.err_q[f] = q_error_estimate(eps, prm.wnorm[g], q_acc, s2_acc);
            }
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(prm.status, DEV_NONFINITE);
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, DEV_TIMEOUT);
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// operand preparation (fit time)
__global__ void centre_kernel(const float* __restrict__ X, const float* __restrict__ inv_ell, int n, int d, int DP,
                              float* __restrict__ centre, float* __restrict__ scale)
{
    __shared__ double s[256];
    const int g = blockIdx.y, j = blockIdx.x;
    double acc = 0.0;
    if (j < d)
        for (int i = threadIdx.x; i < n; i += 256) acc += (double)X[((size_t)g * n + i) * d + j];
    s[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        centre[(size_t)g * DP + j] = (j < d) ? (float)(s[0] / n) : 0.f;
        scale[(size_t)g * DP + j] = (j < d) ? inv_ell[(size_t)g * d + j] : 0.f;
    }
}

// One block per (chunk, GP): scaled observations as hi/lo planes in the MMA's B-operand layout,
// their squared norms, and the padded weights.
__global__ void xt_build_kernel(const float* __restrict__ X, const float* __restrict__ centre,
                                const float* __restrict__ scale, const float* __restrict__ alpha32, int n, int d,
                                int npad_fit, int DP, int NP, float* __restrict__ xt, float* __restrict__ xnorm,
                                float* __restrict__ alpha)
{
    const int g = blockIdx.y, c = blockIdx.x;
    float* blob = xt + ((size_t)g * (NP / KC) + c) * (2 * DP * KC);
    const float* cen = centre + (size_t)g * DP;
    const float* scl = scale + (size_t)g * DP;
    for (int e = threadIdx.x; e < DP * KC; e += blockDim.x) {
        const int r = e % KC, j = e / KC;
        const int k = c * KC + r;
        float xv = 0.f;
        if (k < n && j < d) xv = (float)(((double)X[((size_t)g * n + k) * d + j] - (double)cen[j]) * (double)scl[j]);
        // round to nearest on the 13 dropped mantissa bits, as cvt.rna.tf32 does
        const float h = __uint_as_float((__float_as_uint(xv) + 0x1000u) & 0xFFFFE000u);
        const size_t off = ((size_t)(j / 4) * KC + r) * 4 + (j % 4);
        blob[off] = h;
        blob[(size_t)DP * KC + off] = xv - h;
    }
    for (int r = threadIdx.x; r < KC; r += blockDim.x) {
        const int k = c * KC + r;
        double nrm = 0.0;
        if (k < n)
            for (int j = 0; j < d; ++j) {
                const float xv = (float)(((double)X[((size_t)g * n + k) * d + j] - (double)cen[j]) * (double)scl[j]);
                nrm += (double)xv * (double)xv;
            }
        xnorm[(size_t)g * NP + k] = (float)nrm;
        alpha[(size_t)g * NP + k] = (k < n) ? alpha32[(size_t)g * npad_fit + k] : 0.f;
    }
}

__global__ void xnmax_kernel(const float* __restrict__ xnorm, int NP, float* __restrict__ xnmax)
{
    __shared__ float s[256];
    float v = 0.f;
    for (int i = threadIdx.x; i < NP; i += 256) v = fmaxf(v, xnorm[(size_t)blockIdx.x * NP + i]);
    s[threadIdx.x] = v;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] = fmaxf(s[threadIdx.x], s[threadIdx.x + o]);
        __syncthreads();
    }
    if (threadIdx.x == 0) xnmax[blockIdx.x] = s[0];
}

// One block per (chunk c, pass p, GP): the KC x NV block of W (rows p NV.., columns c KC..) as hi/lo
// planes in the B-operand layout; zero outside the lower triangle and outside n.
__global__ void wt_build_kernel(const double* __restrict__ W64, int n, int npad_fit, int NV, size_t gp_stride,
                                float* __restrict__ wt)
{
    const int c = blockIdx.x, p = blockIdx.y, g = blockIdx.z;
    const int CPP = NV / KC;
    if (c >= (p + 1) * CPP) return;
    const size_t tile = (size_t)CPP * p * (p + 1) / 2 + c;
    float* dst = wt + (size_t)g * gp_stride + tile * (2 * KC * NV);
    const double* Wg = W64 + (size_t)g * npad_fit * npad_fit;
    for (int e = threadIdx.x; e < KC * NV; e += blockDim.x) {
        const int kk = e % KC, r = e / KC;   // consecutive threads walk k: coalesced reads of a W row
        const int i = p * NV + r, k = c * KC + kk;
        float w = 0.f;
        if (i < n && k <= i) w = (float)Wg[(size_t)i * npad_fit + k];
        const uint32_t u = __float_as_uint(w);
        const float h = __uint_as_float((u + 0x1000u) & 0xFFFFE000u);
        const size_t off = ((size_t)(kk / 4) * NV + r) * 4 + (kk % 4);
        dst[off] = h;
        dst[(size_t)KC * NV + off] = w - h;
    }
}

TensorOperands* ops_of(const r3_gp* gp) { return static_cast<TensorOperands*>(gp->tc); }

}  // namespace

bool tc_supported(int n, int d) { return n >= 1 && n <= kMaxN && d >= 1 && d <= 128; }

void tc_release(r3_gp* gp)
{
    TensorOperands* t = ops_of(gp);
    if (!t) return;
    cudaFree(t->centre);
    cudaFree(t->scale);
    cudaFree(t->xt);
    cudaFree(t->xnorm);
    cudaFree(t->xnmax);
    cudaFree(t->alpha);
    cudaFree(t->wt);
    delete t;
    gp->tc = nullptr;
}

r3_status_t tc_prepare(r3_gp* gp, cudaStream_t stream)
{
    const int B = gp->batch, n = gp->n, d = gp->d;
    TensorOperands* t = new (std::nothrow) TensorOperands;
    if (!t) {
        set_error("out of host memory");
        return R3_ERR_ALLOC;
    }
    gp->tc = t;
    t->DP = round_up(d, 8);
    t->NV = (t->DP <= 64 && n > 128) ? 256 : 128;
    t->NP = round_up(n, t->NV);
    t->P = t->NP / t->NV;
    t->xs = 2;
    t->G = t->NV == 256 ? 3 : 2;
    const size_t budget = 227 * 1024 - 1024 - kBarBytes;
    for (t->ws = MAX_STAGES; t->ws >= 2; --t->ws) {
        const SmemMap mp = smem_map(t->DP, t->NV, t->G, t->xs, t->ws);
        if (mp.bar <= budget) break;
    }
    if (t->ws < 2) {
        tc_release(gp);   // does not fit: the SIMT engine serves this shape
        return R3_OK;
    }
    t->smem_bytes = smem_map(t->DP, t->NV, t->G, t->xs, t->ws).bar + kBarBytes + 1024;
    t->tmem_cols = (t->NV + t->G * KC) <= 256 ? 256 : 512;
    const int CPP = t->NV / KC;
    const size_t tiles = (size_t)CPP * t->P * (t->P + 1) / 2;
    t->wt_gp_stride = tiles * (2 * (size_t)KC * t->NV);
    auto fail = [&](const char* what, cudaError_t e) {
        set_error("%s failed: %s", what, cudaGetErrorString(e));
        tc_release(gp);
        return e == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA;
    };
    cudaError_t e;
    if ((e = cudaMalloc(&t->centre, sizeof(float) * B * t->DP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->scale, sizeof(float) * B * t->DP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->xt, sizeof(float) * B * (size_t)(t->NP / KC) * 2 * t->DP * KC)) != cudaSuccess)
        return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->xnorm, sizeof(float) * B * t->NP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->xnmax, sizeof(float) * B)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->alpha, sizeof(float) * B * t->NP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = cudaMalloc(&t->wt, sizeof(float) * B * t->wt_gp_stride)) != cudaSuccess) return fail("cudaMalloc", e);

    centre_kernel<<<dim3(t->DP, B), 256, 0, stream>>>(gp->X, gp->inv_ell, n, d, t->DP, t->centre, t->scale);
    xt_build_kernel<<<dim3(t->NP / KC, B), 256, 0, stream>>>(gp->X, t->centre, t->scale, gp->alpha32, n, d, gp->npad,
                                                             t->DP, t->NP, t->xt, t->xnorm, t->alpha);
    xnmax_kernel<<<B, 256, 0, stream>>>(t->xnorm, t->NP, t->xnmax);
    wt_build_kernel<<<dim3(t->P * CPP, t->P, B), 256, 0, stream>>>(gp->W64, n, gp->npad, t->NV, t->wt_gp_stride, t->wt);
    g_launches += 4;
    if ((e = cudaGetLastError()) != cudaSuccess) return fail("operand preparation launch", e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return fail("operand preparation", e);
    if (t->NV == 256)
        e = cudaFuncSetAttribute(score_tc_kernel<256, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t->smem_bytes);
    else
        e = cudaFuncSetAttribute(score_tc_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t->smem_bytes);
    if (e != cudaSuccess) return fail("cudaFuncSetAttribute", e);
    return R3_OK;
}

size_t score_tc_workspace_bytes(const r3_gp* gp, long long m) { return guard_workspace_bytes(gp, m); }

r3_status_t score_tc(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                     size_t ws_bytes, cudaStream_t stream)
{
    TensorOperands* t = ops_of(gp);
    if (!t) {
        set_error("the tensor-core engine does not serve this handle");
        return R3_ERR_UNSUPPORTED;
    }
    if (ws_bytes < score_tc_workspace_bytes(gp, m)) {
        set_error("internal: tensor workspace too small");
        return R3_ERR_INVALID_ARG;
    }
    const GuardBuffers gb = guard_carve(gp, m, ws);
    TcParams prm;
    prm.xcand = Xcand;
    prm.m = m;
    prm.batch = gp->batch;
    prm.d = gp->d;
    prm.mu = mu;
    prm.sigma = sigma;
    prm.ei = ei;
    prm.err_mu = gb.err_mu;
    prm.err_q = gb.err_q;
    prm.centre = t->centre;
    prm.scale = t->scale;
    prm.xt = t->xt;
    prm.xnorm = t->xnorm;
    prm.xnmax = t->xnmax;
    prm.alpha = t->alpha;
    prm.wt = t->wt;
    prm.wt_gp_stride = t->wt_gp_stride;
    prm.sf2 = gp->sf2_d;
    prm.best = gp->best_d;
    prm.wnorm = gp->wnorm_d;
    prm.DP = t->DP;
    prm.NP = t->NP;
    prm.P = t->P;
    prm.xs = t->xs;
    prm.ws = t->ws;
    prm.status = gp->status_d;
    prm.tiles_per_gp = (m + TILE_M - 1) / TILE_M;
    prm.total_tiles = prm.tiles_per_gp * gp->batch;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, gp->device);
    const unsigned grid = (unsigned)(prm.total_tiles < sms ? prm.total_tiles : sms);
    prof_begin(gp, stream);
    if (t->NV == 256)
        R3_LAUNCH((score_tc_kernel<256, 3>), grid, 128 + 128 * 3, t->smem_bytes, stream, prm);
    else
        R3_LAUNCH((score_tc_kernel<128, 2>), grid, 128 + 128 * 2, t->smem_bytes, stream, prm);
    prof_end(gp, stream);
    return guard_and_rescue(gp, Xcand, m, gb, mu, sigma, ei, stream);
}

}  // namespace r3
