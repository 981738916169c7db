// Tensor-core scoring engine for sm_100a: tcgen05 MMAs (kind::f16 on two-term FP16 splits, FP32
// accumulation in TMEM), operands staged by bulk asynchronous copies, everything fused in one kernel
// so that the cross-covariance k* never leaves the SM.
//
// One CTA owns a tile of 128 candidates; a TMEM lane IS a candidate.  For that tile it walks the rows
// of W = L^-1 in passes of NV rows (the V accumulator: 128 lanes x NV TMEM columns) and, inside a pass,
// the observations in chunks of KC = 32:
//
//   distance MMA   D[cand][k] = z~ . x~_k   (A = scaled candidates, kept in TMEM for the whole tile;
//                  B = scaled observations, depth d), for KD observations at a time
//   Matern warps   r^2 = |z~|^2 + |x~_k|^2 - 2 D, k* = sf2 M52(r): read D from TMEM, write k* (scaled,
//                  FP16 hi/lo planes) as the next A operand into TMEM or shared memory; mu += k* alpha
//                  on the way
//   variance MMA   V[cand][i] += k*[cand][k] W[i][k]   (B = pre-tiled chunk of W, scaled FP16 hi/lo planes)
//   end of pass    q += sum_i V[cand][i]^2 read back from TMEM; after the last pass sigma, EI, outputs
//
// Precision.  Every product is three MMAs (hi*hi + hi*lo + lo*hi): x = hi + lo with hi = fp16(x) and
// lo = fp16(x - hi) carries 22 significant bits, and the tensor core accumulates in FP32, so the
// result is FP32-grade at twice the TF32 rate and half the operand bytes.  k* and W are multiplied by
// powers of two before the split (so that the low parts stay normal numbers) and the accumulator is
// scaled back exactly.  The scaled coordinates of the distance product must fit FP16's range; a
// history that does not is left to the SIMT engine and a candidate that does not is recomputed in FP64.
//
// W is lower-triangular, so pass p only needs k < (p+1) NV; k* chunks are regenerated for every pass
// they take part in instead of being stored.
//
// Warp roles: warp 0 streams the operands (lane 0: scaled observations, lane 1: chunks of W), warp 1
// issues the distance MMAs, warp 2 issues the variance MMAs and owns the TMEM allocation (one thread
// each), warps 4.. form G Matern/epilogue groups of four warps (one warp per TMEM lane quarter); group
// g takes every G-th chunk; the k* buffers are one per group (shared memory) or a ring of two shared by
// the groups (TMEM, where columns are scarce; a group that has computed its chunk keeps it in registers
// until its slot is free).  Stages are handed over through mbarriers; every wait is bounded: when a limit is hit the
// CTA raises a status bit, all roles leave their loops, in-flight copies and MMAs are drained (bounded
// again), TMEM is freed and the kernel returns.
//
// Operand layouts are the no-swizzle K-major "core matrix" form: 8 rows x 16 bytes contiguous, 8-row
// groups 128 bytes apart, 16-byte k-slices one full panel apart.  W and the observations are stored
// in global memory already tiled that way by the fit, so a stage is one contiguous bulk copy.
#include <algorithm>
#include <cuda_fp16.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include "r3_epilogue.cuh"
#include "r3_internal.cuh"
#include "r3_tc_common.cuh"

namespace r3 {

namespace {

// shared-memory map (byte offsets from a 1024-aligned base)
struct SmemMap {
    uint32_t z, k, x, w, zs, bar;   // z: reduction scratch; k: k* buffers (absent when k* lives in TMEM); zs: see kZsStride
    uint32_t x_stage, w_stage;
};
// With at most 16 (padded) features the scaled candidates of the tile are also kept in FP32 in shared memory,
// 128 rows of kZsStride floats (the odd stride keeps a warp's 32 rows on 32 banks): close pairs then get their
// squared distance from direct differences inline, without the out-of-line refinement and its round trips.
constexpr uint32_t kZsStride = 17;
constexpr int kZsMaxDP = 16;
// Registers per thread after the roles have parted: the kernel starts with the register file split evenly
// (128 per thread for 512 threads, 168 for 384); the four control warps, whose loops are short, give theirs back
// and the Matern groups, whose chunk loop does not fit 128 without spills, take them.
constexpr int kRegsControl = 80;
__host__ __device__ constexpr int regs_matern(int G) { return G == 3 ? 144 : 208; }
__host__ __device__ inline SmemMap smem_map(int DP, int NV, int G, int KD, int ws, bool kt)
{
    SmemMap s;
    s.z = 0;                                       // end-of-tile reduction scratch: G x 128 rows x 4 doubles
    s.k = (uint32_t)G * 4096u;                     // k* in shared memory: G buffers x 2 planes x [KC/8][128][8] halves
    s.x = s.k + (kt ? 0u : (uint32_t)G * 16384u);  // XS stages x 2 planes x [DP/8][KD][8] halves
    s.x_stage = 2u * DP * KD * 2u;
    s.w = s.x + (uint32_t)XS * s.x_stage;          // ws stages x 2 planes x [KC/8][NV][8] halves
    s.w_stage = 2u * KC * NV * 2u;
    s.zs = s.w + (uint32_t)ws * s.w_stage;
    s.bar = s.zs + (DP <= kZsMaxDP ? TILE_M * kZsStride * 4u : 0u);
    return s;
}
// barriers, flags, TMEM slot, candidate norms; then the tile's cache of refined close pairs
constexpr uint32_t kCacheOffset = 1024;
constexpr uint32_t kBarBytes = kCacheOffset + TILE_M * kCacheSlots * 8;

// barrier slots (8 bytes each) inside the barrier block
enum : uint32_t {
    BAR_X_FULL = 0, BAR_X_EMPTY = 2, BAR_W_FULL = 4, BAR_W_EMPTY = 10, BAR_D_FULL = 16, BAR_D_EMPTY = 18,
    BAR_K_FULL = 20, BAR_K_EMPTY = 24, BAR_V_FULL = 28, BAR_V_EMPTY = 29, BAR_Z_READY = 30, BAR_RED_READY = 31,
    BAR_MMA_DONE = 32,  // two slots: distance issuer, variance issuer
    BAR_COUNT = 34
};
constexpr uint32_t kFlagOffset = BAR_COUNT * 8;       // int abort, int drain-abort, uint32 tmem base
constexpr uint32_t kZnOffset = 512;                   // float[128] squared norms of the scaled candidates


// NV: rows of W per pass (TMEM columns of the V accumulator).  G: number of Matern warp groups; group
// g owns chunks t = g (mod G) and k* buffer g.  KD: observations per distance product.  KT: the k*
// buffers (A operand of the variance product) live in TMEM instead of shared memory: shared memory then
// only feeds the B operands, which is what keeps its 128 B/clk from becoming the limit.
// NBK: number of k* buffers.  NBK == G: group g owns buffer g.  NBK < G (k* in TMEM, where columns are
// scarce): the buffers form a ring shared by the groups, chunk t uses buffer t mod NBK; a group that has
// computed its chunk keeps it in registers until the ring slot is free, so the groups still run ahead.
// F8: the two cross terms of the variance product (W_hi k_lo, W_lo k_hi) are single FP8 MMAs of depth 32
// instead of two FP16 MMAs of depth 16 each: four MMAs per chunk instead of six.
// PUTOFF: a pass's epilogue (read the accumulator back, hand it over) is put off until the group's first chunk of
// the next pass is on its way, when that chunk can be handed over without the accumulator's release (its k* slot is
// freed by chunks of the old pass): the MMA issuer then finds the new pass's first chunks waiting when the
// accumulator is released, instead of waiting for them to be computed after it.  With few passes per tile the
// refill after a hand-over is a visible part of a tile (4-6 % on histories of two to four passes); with many it is
// not, and the loop structure it needs costs the long histories more than it saves, hence a kernel variant.
// ZS: the feature count is at most 16: close pairs are refined inline from the FP32 copy of the scaled tile in
// shared memory (pools of few features are full of close pairs: on the 16-feature workload 98 % of a warp's
// 16-entry blocks hold one, and the out-of-line refinement was most of the kernel's time).
template <int NV, int G, int KD, bool KT, int NBK = G, bool F8 = false, bool PUTOFF = false, bool ZS = false>
__global__ void __launch_bounds__(128 + 128 * G, 1) score_tc_kernel(const TcParams prm)
{
    static_assert(NBK == G || (KT && NBK >= 2 && NBK < G), "ring of k* buffers: TMEM only");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const SmemMap map = smem_map(prm.DP, NV, G, KD, prm.ws, KT);
    const uint32_t bars = base + map.bar;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + map.bar + kFlagOffset);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + map.bar + kFlagOffset + 8);
    float* zn_s = reinterpret_cast<float*>(sm + map.bar + kZnOffset);
    unsigned long long* pair_cache = reinterpret_cast<unsigned long long*>(sm + map.bar + kCacheOffset);
    float* zs_s = reinterpret_cast<float*>(sm + map.zs);
    auto bar = [&](uint32_t slot) { return bars + slot * 8u; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int CPP = NV / KC;                  // chunks per pass width
    constexpr int SL = KD / KC;                   // chunks per distance product
    // TMEM columns: V accumulator [0, NV), two distance buffers [NV, NV + 2 KD), scaled candidates
    // (FP16 hi plane, then lo plane, DP/2 columns each) from NV + 2 KD, then (KT) G k* buffers of
    // 2 planes x KC/2 columns
    constexpr uint32_t TMEM_COLS = 512u;
    constexpr uint32_t ZCOL = NV + 2 * KD;
    const uint32_t KCOL = ZCOL + (uint32_t)prm.DP;
    const int DP = prm.DP, P = prm.P, ws = prm.ws;
    const long long wl = prm.wait_limit;

    if (threadIdx.x == 0) {
        for (int i = 0; i < XS; ++i) {
            mbar_init(bar(BAR_X_FULL + i), 1);
            mbar_init(bar(BAR_X_EMPTY + i), 1);
            mbar_init(bar(BAR_D_FULL + i), 1);
            mbar_init(bar(BAR_D_EMPTY + i), 128 * SL);
        }
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(bar(BAR_W_FULL + i), 1);
            mbar_init(bar(BAR_W_EMPTY + i), 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar(BAR_K_FULL + i), 128);
            mbar_init(bar(BAR_K_EMPTY + i), 1);
        }
        mbar_init(bar(BAR_V_FULL), 1);
        mbar_init(bar(BAR_V_EMPTY), 128 * G);
        mbar_init(bar(BAR_Z_READY), 128);
        mbar_init(bar(BAR_RED_READY), 128 * G);
        mbar_init(bar(BAR_MMA_DONE), 1);
        mbar_init(bar(BAR_MMA_DONE + 1), 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;   // private flag of the bounded drain waits
    }
    if (threadIdx.x < TILE_M * kCacheSlots / 4) {   // no entry yet: a key that no (tile, observation) forms
        for (int i = 0; i < 4; ++i) pair_cache[threadIdx.x * 4 + i] = ~0ull;
    }
    if (threadIdx.x == 0) {
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
    const long long first_tile = prm.tile_begin + blockIdx.x, tile_step = gridDim.x;
    const int items_per_tile = CPP * P * (P + 1) / 2;
    long long tacc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long tlast = prm.trace ? clock64() : 0;

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsControl));
    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------ producer: scaled observations
        const uint32_t bytes = map.x_stage;
        long long issued = 0;
        int st = 0;
        uint32_t ph = 0;   // stage ring: (stage, phase) advance together, no divisions in the loop
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const __half* src = prm.xt + (size_t)g * (prm.NP / KD) * (bytes / 2);
            for (int p = 0; ok && p < P; ++p)
                for (int c = 0; c < (p + 1) * (NV / KD); ++c, ++issued) {
                    if (!(ok = mbar_wait(bar(BAR_X_EMPTY + st), ph ^ 1u, abort_flag, wl))) break;
                    mbar_arrive_expect_tx(bar(BAR_X_FULL + st), bytes);
                    bulk_g2s(base + map.x + (uint32_t)R3_IDX(st, XS, prm.status) * bytes,
                             src + (size_t)R3_IDX(c, prm.NP / KD, prm.status) * (bytes / 2), bytes, bar(BAR_X_FULL + st));
                    if (++st == XS) { st = 0; ph ^= 1u; }
                }
        }
        if (!ok) {  // aborting: let the copies still in flight land before the CTA goes away
            const int pending = (int)(issued < XS ? issued : XS);
            for (int u = 0; u < pending; ++u) {
                if (--st < 0) { st = XS - 1; ph ^= 1u; }
                mbar_wait(bar(BAR_X_FULL + st), ph, abort_flag + 1, wl);
            }
        }
    } else if (warp == 0 && lane == 1) {
        // ------------------------------------------------------------ producer: chunks of W
        const uint32_t bytes = map.w_stage;
        long long issued = 0;
        int st = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const __half* src = prm.wt + (size_t)g * prm.wt_gp_stride;
            for (int p = 0; ok && p < P; ++p) {
                const __half* psrc = src + (size_t)(CPP * p * (p + 1) / 2) * (bytes / 2);
                for (int c = 0; c < (p + 1) * CPP; ++c, ++issued) {
                    if (issued == prm.withhold_w) { ok = false; break; }   // test aid: the stream of W stops here
                    if (!(ok = mbar_wait(bar(BAR_W_EMPTY + st), ph ^ 1u, abort_flag, wl))) break;
                    mbar_arrive_expect_tx(bar(BAR_W_FULL + st), bytes);
                    (void)R3_IDX(CPP * p * (p + 1) / 2 + c, CPP * P * (P + 1) / 2, prm.status);   // chunk of W within the GP's tiles
                    bulk_g2s(base + map.w + (uint32_t)R3_IDX(st, ws, prm.status) * bytes, psrc + (size_t)c * (bytes / 2), bytes,
                             bar(BAR_W_FULL + st));
                    if (++st == ws) { st = 0; ph ^= 1u; }
                }
            }
        }
        if (!ok) {
            const int pending = (int)(issued < ws ? issued : ws);
            for (int u = 0; u < pending; ++u) {
                if (--st < 0) { st = ws - 1; ph ^= 1u; }
                mbar_wait(bar(BAR_W_FULL + st), ph, abort_flag + 1, wl);
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------ MMA issuer: distance products
        constexpr uint32_t IDESC_D = instr_desc_f16(KD);
        // descriptor low word = start >> 4 | (k-slice distance >> 4) << 16
        const uint32_t zH = tmem + ZCOL, zL = zH + (uint32_t)DP / 2;
        const uint32_t x_lo0 = desc_addr(base + map.x) | (((KD * 16u) >> 4) << 16);
        const int ksteps = DP / 16;
        long long tile_iter = 0;
        int st = 0, db = 0;
        uint32_t ph = 0, d_ph = 0;   // X stage ring; parity of the distance-buffer pair
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            TICK(7);
            if (!(ok = mbar_wait(bar(BAR_Z_READY), (uint32_t)(tile_iter & 1), abort_flag, wl))) break;
            TICK(3);
            tc_fence_after();
            for (int u = 0; u < items_per_tile / SL; ++u) {
                TICK(7);
                if (!(ok = mbar_wait(bar(BAR_X_FULL + st), ph, abort_flag, wl))) break;
                TICK(0);
                if (!(ok = mbar_wait(bar(BAR_D_EMPTY + db), d_ph ^ 1u, abort_flag, wl))) break;
                TICK(1);
                LOGEV(8, (long long)(tile_iter * (items_per_tile / SL) + u) * SL);
                tc_fence_after();
                const uint32_t xH_lo = x_lo0 + ((st * map.x_stage) >> 4), xL_lo = xH_lo + (((uint32_t)DP * KD * 2u) >> 4);
                const uint32_t dcol = tmem + NV + db * KD;
                uint32_t acc = 0;
#pragma unroll
                for (int combo = 0; combo < 3; ++combo) {
                    const uint32_t a0 = combo == 2 ? zL : zH, b0 = combo == 1 ? xL_lo : xH_lo;
                    for (int jj = 0; jj < ksteps; ++jj) {
                        tc_mma_f16_ts(dcol, a0 + jj * 8u, pack64(b0 + jj * ((2u * KD * 16u) >> 4), kDescHi), IDESC_D, acc);
                        acc = 1;
                    }
                }
                tc_commit(bar(BAR_X_EMPTY + st));
                tc_commit(bar(BAR_D_FULL + db));
                TICK(2);
                LOGEV(7, (long long)(tile_iter * (items_per_tile / SL) + u) * SL);
                if (++st == XS) { st = 0; ph ^= 1u; }
                if (++db == 2) { db = 0; d_ph ^= 1u; }
            }
        }
        // every MMA issued by this thread must have completed before TMEM is freed
        tc_commit(bar(BAR_MMA_DONE));
        mbar_wait(bar(BAR_MMA_DONE), 0, abort_flag + 1, wl);
        if (prm.trace)
            for (int i = 0; i < 8; ++i) prm.trace[((size_t)blockIdx.x * 4 + 3) * 8 + i] = tacc[i];
    } else if (warp == 2 && lane == 0) {
        // ------------------------------------------------------------ MMA issuer: variance product
        const uint32_t k_lo0 = desc_addr(base + map.k) | ((2048u >> 4) << 16);
        const uint32_t w_lo0 = desc_addr(base + map.w) | (((NV * 16u) >> 4) << 16);
        uint32_t v_ph = 0;    // parity of the pass counter (V accumulator hand-over)
        int w_s = 0, k_s = 0, e_s = 0;   // e_s: chunk number mod 4 (ring mode: which "consumed" barrier)
        uint32_t w_ph = 0, k_ph = 0;
        bool ok = true;
        // whether the next chunk's k* and W were already seen complete (tested between this chunk's MMAs, while
        // the pipe has work queued, so that nothing but the commits sits between two chunks' MMAs)
        bool k_seen = false, w_seen = false;
        long long tv = 0;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            for (int p = 0; ok && p < P; ++p) {
                const int nchunk = (p + 1) * CPP;
                for (int c = 0; ok && c < nchunk; ++c) {
                    const int b = k_s, s = w_s;
                    TICK(7);
                    if (c == 0) {
                        if (!(ok = mbar_wait(bar(BAR_V_EMPTY), v_ph ^ 1u, abort_flag, wl))) break;
                    }
                    TICK(3);
                    if (!k_seen && !(ok = mbar_wait(bar(BAR_K_FULL + b), k_ph, abort_flag, wl))) break;
                    TICK(4);
                    LOGEV(0, tv);
                    if (!w_seen && !(ok = mbar_wait(bar(BAR_W_FULL + s), w_ph, abort_flag, wl))) break;
                    LOGEV(1, tv);
                    if (++k_s == NBK) { k_s = 0; k_ph ^= 1u; }
                    if (++w_s == ws) { w_s = 0; w_ph ^= 1u; }
                    TICK(5);
                    tc_fence_after();
                    // In the pass's diagonal block the rows of W above the chunk's columns are zero (W is lower
                    // triangular): the MMAs start at the first row that can be non-zero and get narrower.
                    (void)R3_IDX(s, ws, prm.status);
                    (void)R3_IDX(b, NBK, prm.status);
                    const uint32_t skip = c > p * CPP ? (uint32_t)R3_IDX((c - p * CPP) * KC, NV, prm.status) : 0u;
                    const uint32_t idesc_v = instr_desc_f16(NV - skip);
                    const uint32_t vcol = tmem + skip;
                    const uint32_t bH = w_lo0 + ((s * map.w_stage) >> 4) + skip, bL = bH + (((uint32_t)KC * NV * 2u) >> 4);
                    if (F8) {
                        // main term: FP16 hi x hi, two MMAs of depth 16; cross terms: one FP8 MMA of depth 32 each
                        // (planes after the FP16 hi plane: scaled hi parts, then scaled lo parts)
                        const uint32_t first = c > 0 ? 1u : 0u;
                        const uint32_t b8H = bH + (((uint32_t)KC * NV * 2u) >> 4), b8L = b8H + (((uint32_t)KC * NV) >> 4);
                        // k* parts are E5M2; W's hi parts E4M3, its lo parts E5M2
                        const uint32_t idesc_hl = instr_desc_f8(NV - skip, kFmtE5M2, kFmtE5M2);   // k*_hi x W_lo
                        const uint32_t idesc_lh = instr_desc_f8(NV - skip, kFmtE5M2, kFmtE4M3);   // k*_lo x W_hi
                        if (KT) {
                            const uint32_t aH = tmem + KCOL + (uint32_t)b * KC;
                            tc_mma_f16_ts(vcol, aH, pack64(bH, kDescHi), idesc_v, first);
                            tc_mma_f16_ts(vcol, aH + 8u, pack64(bH + ((2u * NV * 16u) >> 4), kDescHi), idesc_v, 1u);
                            tc_mma_f8_ts(vcol, aH + KC / 2, pack64(b8L, kDescHi), idesc_hl, 1u);
                            k_seen = mbar_try_wait(bar(BAR_K_FULL + k_s), k_ph);
                            w_seen = mbar_try_wait(bar(BAR_W_FULL + w_s), w_ph);
                            tc_mma_f8_ts(vcol, aH + KC / 2 + KC / 4, pack64(b8H, kDescHi), idesc_lh, 1u);
                        } else {
                            const uint32_t aH = k_lo0 + ((b * 16384u) >> 4), a8H = aH + (8192u >> 4), a8L = a8H + (4096u >> 4);
                            tc_mma_f16(vcol, pack64(aH, kDescHi), pack64(bH, kDescHi), idesc_v, first);
                            tc_mma_f16(vcol, pack64(aH + (4096u >> 4), kDescHi), pack64(bH + ((2u * NV * 16u) >> 4), kDescHi),
                                       idesc_v, 1u);
                            tc_mma_f8(vcol, pack64(a8H, kDescHi), pack64(b8L, kDescHi), idesc_hl, 1u);
                            k_seen = mbar_try_wait(bar(BAR_K_FULL + k_s), k_ph);
                            w_seen = mbar_try_wait(bar(BAR_W_FULL + w_s), w_ph);
                            tc_mma_f8(vcol, pack64(a8L, kDescHi), pack64(b8H, kDescHi), idesc_lh, 1u);
                        }
                    } else if (KT) {
                        const uint32_t aH = tmem + KCOL + (uint32_t)b * KC, aL = aH + KC / 2;
#pragma unroll
                        for (int combo = 0; combo < 3; ++combo) {
                            const uint32_t a0 = combo == 2 ? aL : aH, b0 = combo == 1 ? bL : bH;
#pragma unroll
                            for (int jj = 0; jj < KC / 16; ++jj)
                                tc_mma_f16_ts(vcol, a0 + jj * 8u, pack64(b0 + jj * ((2u * NV * 16u) >> 4), kDescHi), idesc_v,
                                              (c > 0 || combo > 0 || jj > 0) ? 1u : 0u);
                            if (combo == 1) {
                                k_seen = mbar_try_wait(bar(BAR_K_FULL + k_s), k_ph);
                                w_seen = mbar_try_wait(bar(BAR_W_FULL + w_s), w_ph);
                            }
                        }
                    } else {
                        const uint32_t aH = k_lo0 + ((b * 16384u) >> 4), aL = aH + (8192u >> 4);
#pragma unroll
                        for (int combo = 0; combo < 3; ++combo) {
                            const uint32_t a0 = combo == 2 ? aL : aH, b0 = combo == 1 ? bL : bH;
#pragma unroll
                            for (int jj = 0; jj < KC / 16; ++jj)
                                tc_mma_f16(vcol, pack64(a0 + jj * (4096u >> 4), kDescHi),
                                           pack64(b0 + jj * ((2u * NV * 16u) >> 4), kDescHi), idesc_v,
                                           (c > 0 || combo > 0 || jj > 0) ? 1u : 0u);
                            if (combo == 1) {
                                k_seen = mbar_try_wait(bar(BAR_K_FULL + k_s), k_ph);
                                w_seen = mbar_try_wait(bar(BAR_W_FULL + w_s), w_ph);
                            }
                        }
                    }
                    tc_commit(bar(BAR_W_EMPTY + s));
                    tc_commit(bar(BAR_K_EMPTY + (NBK == G ? b : e_s)));
                    e_s = (e_s + 1) & 3;
                    if (c == nchunk - 1) {
                        tc_commit(bar(BAR_V_FULL));
                        v_ph ^= 1u;
                    }
                    TICK(6);
                    LOGEV(2, tv);
                    ++tv;
                }
            }
        }
        tc_commit(bar(BAR_MMA_DONE + 1));
        mbar_wait(bar(BAR_MMA_DONE + 1), 0, abort_flag + 1, wl);
        if (prm.trace)
            for (int i = 0; i < 8; ++i) prm.trace[((size_t)blockIdx.x * 4 + 0) * 8 + i] = tacc[i];
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(regs_matern(G)));
        // ------------------------------------------------------------ Matern / epilogue warp groups
        const int grp = (warp - 4) >> 2;         // 0..G-1
        const int q4 = warp & 3;                 // TMEM lane quarter == warp % 4
        const int row = q4 * 32 + lane;          // candidate row in the tile == TMEM lane
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        long long t = grp;                       // next own chunk (global numbering)
        long long t_tile0 = 0;                   // first chunk of the current tile
        uint32_t own_ph = 0;                     // parity of this group's own-chunk count
        uint32_t v_ph = 0;                       // parity of the pass counter
        long long tile_iter = 0;
        bool ok = true;
        bool bad = false;
        double* red = reinterpret_cast<double*>(sm + map.z);   // scratch of the end-of-tile reduction
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const long long cand = (tile % prm.tiles_per_gp) * TILE_M + row;
            const bool valid = cand < prm.m;
            const float sf2 = prm.sf2[g];
            const float kvscale = prm.kscale[g] * sf2;   // k* = sf2 * (k*/sf2), scaled for its FP16 split
            if (grp == G - 1) {
                // ---- scale the candidate, split it, store it as the A operand of the distance MMA
                float zn = 0.f;
                bool far = false;
                const float* zrow =
                    prm.xcand + (size_t)R3_IDX((long long)g * prm.m + (valid ? cand : 0), (long long)prm.batch * prm.m, prm.status) * prm.d;
                {
                    // the row this thread will need for the CTA's next tile: start it on its way to L2 now
                    const long long nt = tile + tile_step;
                    if (nt < prm.total_tiles) {
                        const long long nc = (nt % prm.tiles_per_gp) * TILE_M + row;
                        if (nc < prm.m) {
                            const char* pf = reinterpret_cast<const char*>(
                                prm.xcand + ((size_t)(nt / prm.tiles_per_gp) * prm.m + nc) * prm.d);
                            for (int off = 0; off < prm.d * 4; off += 128)
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + off));
                        }
                    }
                }
                const float* cen = prm.centre + (size_t)g * DP;
                const float* scl = prm.scale + (size_t)g * DP;
                const bool vec = (prm.d % 4) == 0 && (reinterpret_cast<uintptr_t>(prm.xcand) & 15) == 0;
                // Two forms of the same loop over the row's features.  The long-history kernel keeps the plain one: its
                // chunk loop sits at the register limit, and the pipelined form, although it runs once per tile, costs
                // that loop registers (config 5: 45.9 ms to 47.9 ms per pool); everywhere else the row's loads overlap
                // (config 3: 5.74 ms to 5.52 ms).
                if constexpr (F8) {
                    uint32_t zh[8], zl[8];
                    for (int j8 = 0; j8 < DP / 8; ++j8) {
                        __half2 hi2[4], lo2[4];
    #pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int j4 = 2 * j8 + h;
                            float z[4];
                            if (vec && 4 * j4 < prm.d) {
                                // read once: streaming load, so that the pool does not push W out of L2
                                const float4 v = __ldcs(reinterpret_cast<const float4*>(zrow + 4 * j4));
                                z[0] = v.x; z[1] = v.y; z[2] = v.z; z[3] = v.w;
                            } else {
    #pragma unroll
                                for (int e = 0; e < 4; ++e) z[e] = (4 * j4 + e < prm.d) ? __ldcs(zrow + 4 * j4 + e) : 0.f;
                            }
                            const float4 c4 = __ldg(reinterpret_cast<const float4*>(cen + R3_IDX(4 * j4, DP - 3, prm.status)));
                            const float4 s4 = __ldg(reinterpret_cast<const float4*>(scl + R3_IDX(4 * j4, DP - 3, prm.status)));
                            const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
                            float zt[4];
    #pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                bad |= !isfinite(z[e]);
                                float v = valid ? (z[e] - cc[e]) * ss[e] : 0.f;
                                if (fabsf(v) > kMaxScaled) {   // outside the FP16 planes' range: clamp, and have it recomputed
                                    v = copysignf(kMaxScaled, v);
                                    far = true;
                                }
                                zt[e] = v;
                                zn = fmaf(v, v, zn);
                            }
                            split2(zt[0], zt[1], hi2[2 * h], lo2[2 * h]);
                            split2(zt[2], zt[3], hi2[2 * h + 1], lo2[2 * h + 1]);
                            if (ZS) {
    #pragma unroll
                                for (int e = 0; e < 4; ++e) zs_s[row * kZsStride + 4 * j4 + e] = zt[e];
                            }
                        }
                        // 8 features = 4 columns of each plane; two such groups make one 8-column store
                        if (j8 & 1) {
    #pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                zh[4 + e] = *reinterpret_cast<const uint32_t*>(&hi2[e]);
                                zl[4 + e] = *reinterpret_cast<const uint32_t*>(&lo2[e]);
                            }
                            // candidate planes: columns [ZCOL, ZCOL + DP) of the 512
                            (void)R3_IDX(ZCOL + DP / 2 + (j8 >> 1) * 8 + 7, min((int)TMEM_COLS, (int)ZCOL + DP), prm.status);
                            tc_st8(lane_addr + ZCOL + (uint32_t)(j8 >> 1) * 8u, zh);
                            tc_st8(lane_addr + ZCOL + (uint32_t)DP / 2 + (uint32_t)(j8 >> 1) * 8u, zl);
                        } else {
    #pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                zh[e] = *reinterpret_cast<const uint32_t*>(&hi2[e]);
                                zl[e] = *reinterpret_cast<const uint32_t*>(&lo2[e]);
                            }
                        }
                    }
                } else {
                    // 16 features per step (one 8-column store to each plane); the next step's four loads are under way
                    // while this one is scaled and split, so that the row costs one trip to L2 or HBM and not DP / 8
                    auto load4 = [&](int j4) {
                        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (vec && 4 * j4 < prm.d) {
                            // read once: streaming load, so that the pool does not push W out of L2
                            v = __ldcs(reinterpret_cast<const float4*>(zrow + 4 * j4));
                        } else if (4 * j4 < prm.d) {
                            v.x = __ldcs(zrow + 4 * j4);
                            v.y = (4 * j4 + 1 < prm.d) ? __ldcs(zrow + 4 * j4 + 1) : 0.f;
                            v.z = (4 * j4 + 2 < prm.d) ? __ldcs(zrow + 4 * j4 + 2) : 0.f;
                            v.w = (4 * j4 + 3 < prm.d) ? __ldcs(zrow + 4 * j4 + 3) : 0.f;
                        }
                        return v;
                    };
                    float4 nxt[4];
    #pragma unroll
                    for (int h = 0; h < 4; ++h) nxt[h] = load4(h);
                    for (int j16 = 0; j16 < DP / 16; ++j16) {
                        float4 cur[4];
    #pragma unroll
                        for (int h = 0; h < 4; ++h) cur[h] = nxt[h];
                        if (j16 + 1 < DP / 16) {
    #pragma unroll
                            for (int h = 0; h < 4; ++h) nxt[h] = load4(4 * (j16 + 1) + h);
                        }
                        uint32_t zh[8], zl[8];
    #pragma unroll
                        for (int h = 0; h < 4; ++h) {
                            const int j4 = 4 * j16 + h;
                            const float z[4] = {cur[h].x, cur[h].y, cur[h].z, cur[h].w};
                            const float4 c4 = __ldg(reinterpret_cast<const float4*>(cen + R3_IDX(4 * j4, DP - 3, prm.status)));
                            const float4 s4 = __ldg(reinterpret_cast<const float4*>(scl + R3_IDX(4 * j4, DP - 3, prm.status)));
                            const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
                            float zt[4];
    #pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                bad |= !isfinite(z[e]);
                                float v = valid ? (z[e] - cc[e]) * ss[e] : 0.f;
                                if (fabsf(v) > kMaxScaled) {   // outside the FP16 planes' range: clamp, and have it recomputed
                                    v = copysignf(kMaxScaled, v);
                                    far = true;
                                }
                                zt[e] = v;
                                zn = fmaf(v, v, zn);
                            }
                            __half2 hi0, lo0, hi1, lo1;
                            split2(zt[0], zt[1], hi0, lo0);
                            split2(zt[2], zt[3], hi1, lo1);
                            zh[2 * h] = *reinterpret_cast<const uint32_t*>(&hi0);
                            zh[2 * h + 1] = *reinterpret_cast<const uint32_t*>(&hi1);
                            zl[2 * h] = *reinterpret_cast<const uint32_t*>(&lo0);
                            zl[2 * h + 1] = *reinterpret_cast<const uint32_t*>(&lo1);
                            if (ZS) {
    #pragma unroll
                                for (int e = 0; e < 4; ++e) zs_s[row * kZsStride + 4 * j4 + e] = zt[e];
                            }
                        }
                        // candidate planes: columns [ZCOL, ZCOL + DP) of the 512
                        (void)R3_IDX(ZCOL + DP / 2 + j16 * 8 + 7, min((int)TMEM_COLS, (int)ZCOL + DP), prm.status);
                        tc_st8(lane_addr + ZCOL + (uint32_t)j16 * 8u, zh);
                        tc_st8(lane_addr + ZCOL + (uint32_t)DP / 2 + (uint32_t)j16 * 8u, zl);
                    }
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                zn_s[R3_IDX(row, TILE_M, prm.status)] = far ? -zn : zn;   // the sign carries the out-of-range mark
                tc_fence_before();
                mbar_arrive(bar(BAR_Z_READY));
            }
            ok = mbar_wait(bar(BAR_Z_READY), (uint32_t)(tile_iter & 1), abort_flag, wl);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const bool far_cand = zn_s[row] < 0.f;
            const float zn = fabsf(zn_s[row]);

            const float* xs_g = prm.xs32 + (size_t)g * prm.NP * DP;
            const float v_thresh = far_cand ? INFINITY : kvscale * kRefine / (zn + prm.xnmax[g]);
            const float pc0 = kvscale, pc1 = kvscale * kPolyC1, pc2 = kvscale * kPolyC2;
            const float inv_kscale = 1.f / prm.kscale[g];   // scaled k* -> k*
            const float* xn_g = prm.xnorm + (size_t)g * prm.NP;
            const float* al_g = prm.alpha + (size_t)g * prm.NP;
            double mu_acc = 0.0, a2_acc = 0.0, s2_acc = 0.0, q_acc = 0.0;
            int pass_base = 0;   // chunks of this tile before pass p
            // one chunk of this group: chunk c of pass p (which has nchunk chunks); clears ok when the CTA aborts
            auto do_chunk = [&](const int c, const int p, const int nchunk) {
                {
                    const long long U = t / SL;       // distance product and the slice of its buffer
                    const int db = (int)(U & 1), slice = (int)(t % SL);
                    // the next own chunk's norms and weights: pull them towards L1 while this one is worked on
                    if (lane < 2) {
                        const int cn = c + G < nchunk ? c + G : (c + G - nchunk);
                        const float* pf = (lane == 0 ? xn_g : al_g) + cn * KC;
                        asm volatile("prefetch.global.L1 [%0];" ::"l"(pf));
                    }
                    TICK(7);
                    ok = mbar_wait(bar(BAR_D_FULL + db), (uint32_t)((U >> 1) & 1), abort_flag, wl);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) return;
                    TICK(0);
                    if (threadIdx.x % 128 == 0) LOGEV(3, t);
                    tc_fence_after();
                    const bool fresh = c >= p * CPP;   // first time this chunk is generated for the tile
                    // k* buffer and the parity of its hand-over: the group's own buffer, or slot t mod NBK of the ring
                    const int kbuf = NBK == G ? grp : (int)(t % NBK);
                    const uint32_t kpar = NBK == G ? own_ph : (uint32_t)((t / NBK) & 1);
                    uint8_t* kb = sm + map.k + (uint32_t)R3_IDX(kbuf, NBK, prm.status) * 16384u + row * 16;
                    if (KT) (void)R3_IDX(KCOL + kbuf * KC + KC - 1, TMEM_COLS, prm.status);   // the slot's columns in tensor memory
                    uint32_t kh[KC / 16][8], kl[KC / 16][8];
                    // both halves of the chunk's dot products in one round trip to TMEM, then the buffer is free
                    float dots[KC / 16][16];
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h)
                        tc_ld16_issue(lane_addr + NV + (uint32_t)R3_IDX(db * KD + slice * KC + h * 16, 2 * KD - 15, prm.status), dots[h]);
                    tc_wait_ld32(dots[0], dots[1]);
                    tc_fence_before();
                    mbar_arrive(bar(BAR_D_EMPTY + db));
                    TICK(1);
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h) {
                        const float* dot = dots[h];
                        float kv[16];   // k* times kvscale (the power of two of its FP16 split)
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 xn4 =
                                __ldg(reinterpret_cast<const float4*>(xn_g + R3_IDX(c * KC + h * 16 + 4 * q, prm.NP - 3, prm.status)));
                            const float xn[4] = {xn4.x, xn4.y, xn4.z, xn4.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // |.|: a slightly negative r^2 (rounding) is a tiny distance either way
                                const float u = sqrt_approx(fabsf(fmaf(-2.f, dot[4 * q + e], zn + xn[e])));
                                kv[4 * q + e] = fmaf(u, fmaf(u, pc2, pc1), pc0) * exp2_approx(-u);
                            }
                        }
                        // largest of the sixteen in eight three-input maxima
                        const float vmax = max3(max3(max3(kv[0], kv[1], kv[2]), max3(kv[3], kv[4], kv[5]), max3(kv[6], kv[7], kv[8])),
                                                max3(max3(kv[9], kv[10], kv[11]), max3(kv[12], kv[13], kv[14]), kv[15]), 0.f);
                        if (ZS) {
                            if (vmax > v_thresh) {   // close pairs of this candidate: direct differences, inline
                                uint32_t marked = 0;
#pragma unroll
                                for (int i = 0; i < 16; ++i) marked |= (kv[i] > v_thresh) ? (1u << i) : 0u;
                                const float* zr = zs_s + row * kZsStride;
                                for (; marked; marked &= marked - 1) {
                                    const uint32_t i = (uint32_t)__ffs(marked) - 1u;
                                    const float4* xp = reinterpret_cast<const float4*>(
                                        xs_g + (size_t)R3_IDX(c * KC + h * 16 + (int)i, prm.NP, prm.status) * kZsMaxDP);
                                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        const float4 x4 = __ldg(xp + e);
                                        float df = zr[4 * e] - x4.x;
                                        acc0 = fmaf(df, df, acc0);
                                        df = zr[4 * e + 1] - x4.y;
                                        acc1 = fmaf(df, df, acc1);
                                        df = zr[4 * e + 2] - x4.z;
                                        acc0 = fmaf(df, df, acc0);
                                        df = zr[4 * e + 3] - x4.w;
                                        acc1 = fmaf(df, df, acc1);
                                    }
                                    const float u = sqrtf(acc0 + acc1);
                                    const float val = kvscale * fmaf(u, fmaf(u, kPolyC2, kPolyC1), 1.f) * exp2f(-u);
#pragma unroll
                                    for (int e2 = 0; e2 < 16; ++e2) kv[e2] = (uint32_t)e2 == i ? val : kv[e2];
                                }
                            }
                        } else
                        if (__any_sync(0xffffffffu, vmax > v_thresh)) {
                            // rare: close pairs.  Values refined in an earlier pass of this tile come back from the
                            // cache without a call; what is left goes to the out-of-line refinement through a local
                            // array, so that the hot path keeps kv in registers.
                            const uint32_t key0 = (((uint32_t)tile_iter & 0x3ffffu) << 13) | (uint32_t)(c * KC + h * 16);
                            unsigned long long* slots = P > 1 ? pair_cache + R3_IDX(row, TILE_M, prm.status) * kCacheSlots : nullptr;
                            (void)R3_IDX(c * KC + h * 16 + 15, prm.NP, prm.status);   // rows of the FP32 observations the refinement reads
                            bool need = vmax > v_thresh;
                            if (need && slots && !fresh) {
                                uint32_t marked = 0;
#pragma unroll
                                for (int i = 0; i < 16; ++i) marked |= (kv[i] > v_thresh) ? (1u << i) : 0u;
                                need = false;
                                for (; marked; marked &= marked - 1) {
                                    const uint32_t i = (uint32_t)__ffs(marked) - 1u;
                                    const unsigned long long e = slots[cache_slot(key0 + i)];
                                    if ((uint32_t)(e >> 32) != key0 + i) {
                                        need = true;
                                        break;
                                    }
                                    const float val = __uint_as_float((uint32_t)e);
#pragma unroll
                                    for (int e2 = 0; e2 < 16; ++e2) kv[e2] = (uint32_t)e2 == i ? val : kv[e2];
                                }
                            }
                            if (__any_sync(0xffffffffu, need)) {
                                float tmp[16];
#pragma unroll
                                for (int i = 0; i < 16; ++i) tmp[i] = kv[i];
                                if (slots)
                                    refine_close_pairs<true>(tmp, v_thresh, kvscale, lane_addr + ZCOL, DP,
                                                             xs_g + (size_t)(c * KC + h * 16) * DP, slots, key0, !fresh);
                                else
                                    refine_close_pairs<false>(tmp, v_thresh, kvscale, lane_addr + ZCOL, DP,
                                                              xs_g + (size_t)(c * KC + h * 16) * DP, nullptr, 0u, false);
#pragma unroll
                                for (int i = 0; i < 16; ++i) kv[i] = tmp[i];
                            }
                        }
                        if (fresh) {   // warp-uniform: the mean and the error scales see every observation once
                            float mpart = 0.f, apart = 0.f, spart = 0.f;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float4 al4 =
                                    __ldg(reinterpret_cast<const float4*>(al_g + R3_IDX(c * KC + h * 16 + 4 * q, prm.NP - 3, prm.status)));
                                const float al[4] = {al4.x, al4.y, al4.z, al4.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float v = kv[4 * q + e], va = v * al[e];
                                    mpart += va;
                                    apart = fmaf(va, va, apart);
                                    spart = fmaf(v, v, spart);
                                }
                            }
                            mu_acc += (double)(mpart * inv_kscale);
                            a2_acc += (double)(apart * inv_kscale * inv_kscale);
                            s2_acc += (double)(spart * inv_kscale * inv_kscale);
                        }
                        // split into the two FP16 planes; the stores wait until the whole chunk is computed
                        // so that the arithmetic does not sit between the buffer's release and its refill
                        if (F8) {
                            // kl[h][0..3]: the 16 hi parts as E5M2, kl[h][4..7]: the 16 lo parts
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                split4_f8(kv + 4 * e, kh[h][2 * e], kh[h][2 * e + 1], kl[h][e], kl[h][4 + e]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                __half2 hi, lo;
                                split2(kv[2 * e], kv[2 * e + 1], hi, lo);
                                kh[h][e] = *reinterpret_cast<const uint32_t*>(&hi);
                                kl[h][e] = *reinterpret_cast<const uint32_t*>(&lo);
                            }
                        }
                    }
                    TICK(2);
                    if (threadIdx.x % 128 == 0) LOGEV(4, t);
                    if (NBK == G) {
                        ok = mbar_wait(bar(BAR_K_EMPTY + kbuf), kpar ^ 1u, abort_flag, wl);
                    } else if (t >= NBK) {
                        // Ring shorter than the number of groups: slot t mod NBK is free once chunk t - NBK has
                        // been consumed.  A parity wait is only valid at most one phase behind, and with one
                        // barrier per slot this group could be two uses of its slot ahead of the issuer, or the
                        // issuer two ahead of the group.  The "consumed" barriers are therefore indexed by the
                        // chunk number mod 4: the chunks 4 apart that share a barrier are never both pending.
                        const long long te = t - NBK;
                        ok = mbar_wait(bar(BAR_K_EMPTY + (int)(te & 3)), (uint32_t)((te >> 2) & 1), abort_flag, wl);
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) return;
                    TICK(3);
                    if (threadIdx.x % 128 == 0) LOGEV(5, t);
                    if (F8) {
                        if (KT) {
                            // FP16 hi plane: 16 columns; then the chunk's 32 E5M2 hi parts (8 columns) and lo parts (8)
                            uint32_t p8[8];
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC, kh[0]);
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC + 8, kh[1]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) { p8[e] = kl[0][e]; p8[4 + e] = kl[1][e]; }
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC + KC / 2, p8);
#pragma unroll
                            for (int e = 0; e < 4; ++e) { p8[e] = kl[0][4 + e]; p8[4 + e] = kl[1][4 + e]; }
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC + KC / 2 + KC / 4, p8);
                        } else {
#pragma unroll
                            for (int h = 0; h < KC / 16; ++h) {
#pragma unroll
                                for (int sl = 0; sl < 2; ++sl)
                                    *reinterpret_cast<uint4*>(kb + (2 * h + sl) * 2048u) =
                                        make_uint4(kh[h][4 * sl], kh[h][4 * sl + 1], kh[h][4 * sl + 2], kh[h][4 * sl + 3]);
                                // one 16-byte k-slice of each 8-bit plane per 16 observations
                                *reinterpret_cast<uint4*>(kb + 8192u + h * 2048u) = make_uint4(kl[h][0], kl[h][1], kl[h][2], kl[h][3]);
                                *reinterpret_cast<uint4*>(kb + 12288u + h * 2048u) = make_uint4(kl[h][4], kl[h][5], kl[h][6], kl[h][7]);
                            }
                        }
                    } else
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h) {
                        if (KT) {
                            // 16 columns = 8 packed TMEM columns of each plane
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC + h * 8, kh[h]);
                            tc_st8(lane_addr + KCOL + (uint32_t)kbuf * KC + KC / 2 + h * 8, kl[h]);
                        } else {
                            // 16 columns = two 16-byte k-slices of the A operand, hi and lo planes
#pragma unroll
                            for (int sl = 0; sl < 2; ++sl) {
                                *reinterpret_cast<uint4*>(kb + (2 * h + sl) * 2048u) =
                                    make_uint4(kh[h][4 * sl], kh[h][4 * sl + 1], kh[h][4 * sl + 2], kh[h][4 * sl + 3]);
                                *reinterpret_cast<uint4*>(kb + 8192u + (2 * h + sl) * 2048u) =
                                    make_uint4(kl[h][4 * sl], kl[h][4 * sl + 1], kl[h][4 * sl + 2], kl[h][4 * sl + 3]);
                            }
                        }
                    }
                    if (!ok) return;
                    if (KT) {
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                        tc_fence_before();
                    } else {
                        fence_proxy_async();
                    }
                    mbar_arrive(bar(BAR_K_FULL + kbuf));
                    TICK(4);
                    if (threadIdx.x % 128 == 0) LOGEV(6, t);
                    t += G;
                    own_ph ^= 1u;
                }
            };
            // end of a pass: q += sum_i V^2 over this group's share of the columns, then the accumulator is free
            auto do_epilogue = [&]() {
                TICK(7);
                ok = mbar_wait(bar(BAR_V_FULL), v_ph, abort_flag, wl);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return;
                TICK(5);
                tc_fence_after();
#pragma unroll 1
                for (int c0 = grp * 16; c0 < NV; c0 += 32 * G) {   // two column blocks per round trip to TMEM
                    const int c1 = c0 + 16 * G;
                    (void)R3_IDX(c0 + 15, NV, prm.status);
                    float v[16], w[16];
                    float part0 = 0.f, part1 = 0.f;
                    if (c1 < NV) {
                        tc_ld16_issue(lane_addr + c0, v);
                        tc_ld16_issue(lane_addr + c1, w);
                        tc_wait_ld32(v, w);
#pragma unroll
                        for (int i = 0; i < 16; ++i) part1 = fmaf(w[i], w[i], part1);
                    } else {
                        tc_ld16(lane_addr + c0, v);
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) part0 = fmaf(v[i], v[i], part0);
                    q_acc += (double)part0;
                    q_acc += (double)part1;
                }
                tc_fence_before();
                mbar_arrive(bar(BAR_V_EMPTY));
                TICK(6);
                v_ph ^= 1u;
            };
            if constexpr (!PUTOFF) {
                for (int p = 0; ok && p < P; ++p) {
                    const int nchunk = (p + 1) * CPP;
                    // own chunks of this pass: global t with t - t_tile0 - pass_base in [0, nchunk)
                    while (ok && t - t_tile0 - pass_base < nchunk) do_chunk((int)(t - t_tile0 - pass_base), p, nchunk);
                    if (!ok) break;
                    pass_base += nchunk;
                    do_epilogue();
                }
            } else {
                // one loop over the group's chunks of the tile, pass after pass, the epilogues in between
                int p = 0, nchunk = CPP, epilogues_due = 0;
                while (ok) {
                    bool first_of_pass = false;
                    if (t - t_tile0 - pass_base >= nchunk) {   // this group's chunks of pass p are done
                        pass_base += nchunk;
                        ++p;
                        nchunk += CPP;
                        ++epilogues_due;
                        first_of_pass = true;
                    }
                    const int c = (int)(t - t_tile0 - pass_base);
                    const bool put_off = first_of_pass && p < P && (NBK == G || c < NBK);
                    for (int run = epilogues_due - (put_off ? 1 : 0); ok && run > 0; --run) {
                        --epilogues_due;
                        do_epilogue();
                    }
                    if (!ok || p >= P) break;
                    do_chunk(c, p, nchunk);
                }
            }
            if (!ok) break;
            t_tile0 += items_per_tile;
            // ---- combine the groups' partial sums; group 0 finishes the candidate
            double* mine = red + (size_t)R3_IDX(grp * TILE_M + row, G * TILE_M, prm.status) * 4;
            mine[0] = mu_acc; mine[1] = a2_acc; mine[2] = s2_acc; mine[3] = q_acc;
            mbar_arrive(bar(BAR_RED_READY));
            if (grp == 0) {   // only the finishing group waits; the others move on to the next tile
                ok = mbar_wait(bar(BAR_RED_READY), (uint32_t)(tile_iter & 1), abort_flag, wl);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (valid) {
                    mu_acc = a2_acc = s2_acc = q_acc = 0.0;
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) {
                        const double* o = red + ((size_t)gg * TILE_M + row) * 4;
                        mu_acc += o[0]; a2_acc += o[1]; s2_acc += o[2]; q_acc += o[3];
                    }
                    q_acc *= prm.vinv2[g];   // undo the power-of-two scaling of k* and W
                    const size_t f = (size_t)R3_IDX((long long)g * prm.m + cand, (long long)prm.batch * prm.m, prm.status);
                    const CandidateResult res = finalize_candidate(mu_acc, q_acc, (double)sf2, (double)prm.best[R3_IDX(g, prm.batch, prm.status)]);
                    __stcs(prm.mu + f, res.mu);
                    __stcs(prm.sigma + f, res.sigma);
                    __stcs(prm.ei + f, res.ei);
                    const double eps =
                        far_cand ? 1.0 : kEpsTc0 + kEpsTc1 * (double)(zn + prm.xnmax[g]) * rsqrt((double)DP);
                    prm.err_mu[f] = mu_error_estimate(eps, a2_acc);
                    prm.err_q[f] = q_error_estimate(F8 && !far_cand ? eps + kEpsF8 : eps, prm.wnorm[g], q_acc, s2_acc);
                }
            }
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(prm.status, DEV_NONFINITE);
        if (prm.trace && q4 == 0 && lane == 0 && grp < 2)
            for (int i = 0; i < 8; ++i) prm.trace[((size_t)blockIdx.x * 4 + 1 + grp) * 8 + i] = tacc[i];
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
        scale[(size_t)g * DP + j] = (j < d) ? (float)((double)inv_ell[(size_t)g * d + j] * kCoordScale) : 0.f;
    }
}

// One block per (distance product, GP): scaled observations as FP16 hi/lo planes in the MMA's
// B-operand layout, their squared norms (of the FP32 values the planes represent), the padded weights,
// and the largest scaled coordinate (the FP16 planes have a limited range).
__global__ void xt_build_kernel(const float* __restrict__ X, const float* __restrict__ centre,
                                const float* __restrict__ scale, const float* __restrict__ alpha32, int n, int d,
                                int npad_fit, int DP, int NP, int KD, __half* __restrict__ xt,
                                float* __restrict__ xs32, float* __restrict__ xnorm, float* __restrict__ alpha, unsigned* __restrict__ xamax_bits)
{
    const int g = blockIdx.y, c = blockIdx.x;
    __half* blob = xt + ((size_t)g * (NP / KD) + c) * (2 * DP * KD);
    const float* cen = centre + (size_t)g * DP;
    const float* scl = scale + (size_t)g * DP;
    float amax = 0.f;
    for (int e = threadIdx.x; e < DP * KD; e += blockDim.x) {
        const int r = e % KD, j = e / KD;
        const int k = c * KD + r;
        float xv = 0.f;
        if (k < n && j < d) xv = (float)(((double)X[((size_t)g * n + k) * d + j] - (double)cen[j]) * (double)scl[j]);
        amax = fmaxf(amax, fabsf(xv));
        xs32[((size_t)g * NP + k) * DP + j] = xv;
        const __half h = __float2half_rn(xv);
        const size_t off = ((size_t)(j / 8) * KD + r) * 8 + (j % 8);
        blob[off] = h;
        blob[(size_t)DP * KD + off] = __float2half_rn(xv - __half2float(h));
    }
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) atomicMax(xamax_bits, __float_as_uint(amax));
    for (int r = threadIdx.x; r < KD; r += blockDim.x) {
        const int k = c * KD + r;
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

// Largest |W| entry of each GP (bit pattern of a non-negative float, so atomicMax orders it).
__global__ void wmax_kernel(const double* __restrict__ W64, int n, int npad_fit, unsigned* __restrict__ wmax_bits)
{
    const int g = blockIdx.y;
    const double* Wg = W64 + (size_t)g * npad_fit * npad_fit;
    float v = 0.f;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < (size_t)n * n; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / n), k = (int)(e % n);
        if (k <= i) v = fmaxf(v, fabsf((float)Wg[(size_t)i * npad_fit + k]));
    }
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) atomicMax(&wmax_bits[g], __float_as_uint(v));
}

// One block per (chunk c, pass p, GP): the KC x NV block of 2^eW W (rows p NV.., columns c KC..) as
// FP16 hi/lo planes in the B-operand layout; zero outside the lower triangle and outside n.
// With f8 the second plane holds, instead of the FP16 lo parts, two 8-bit planes in the 8-bit form of the same
// layout (16 k-elements per 16-byte slice): the hi parts as E4M3 (|2^eW W| < 2^8 for these histories), then the
// lo parts as E5M2.
__global__ void wt_build_kernel(const double* __restrict__ W64, int n, int npad_fit, int NV, size_t gp_stride,
                                const float* __restrict__ wscale, __half* __restrict__ wt, bool f8)
{
    const int c = blockIdx.x, p = blockIdx.y, g = blockIdx.z;
    const int CPP = NV / KC;
    if (c >= (p + 1) * CPP) return;
    const size_t tile = (size_t)CPP * p * (p + 1) / 2 + c;
    __half* dst = wt + (size_t)g * gp_stride + tile * (2 * KC * NV);
    const double* Wg = W64 + (size_t)g * npad_fit * npad_fit;
    const double sc = (double)wscale[g];
    for (int e = threadIdx.x; e < KC * NV; e += blockDim.x) {
        const int kk = e % KC, r = e / KC;   // consecutive threads walk k: coalesced reads of a W row
        const int i = p * NV + r, k = c * KC + kk;
        float w = 0.f;
        if (i < n && k <= i) w = (float)(Wg[(size_t)i * npad_fit + k] * sc);
        const __half h = __float2half_rn(w);
        const size_t off = ((size_t)(kk / 8) * NV + r) * 8 + (kk % 8);
        dst[off] = h;
        if (f8) {
            uint8_t* d8 = reinterpret_cast<uint8_t*>(dst + (size_t)KC * NV);
            const size_t off8 = ((size_t)(kk / 16) * NV + r) * 16 + (kk % 16);
            const float hf = __half2float(h);
            d8[off8] = (uint8_t)(e4m3x4(hf, 0.f, 0.f, 0.f) & 0xffu);
            d8[(size_t)KC * NV + off8] = (uint8_t)(e5m2x4(w - hf, 0.f, 0.f, 0.f) & 0xffu);
        } else {
            dst[(size_t)KC * NV + off] = __float2half_rn(w - __half2float(h));
        }
    }
}

TensorOperands* ops_of(const r3_gp* gp) { return static_cast<TensorOperands*>(gp->tc); }

void (*kernel_for(int NV, int G, bool kt, int nbk, bool f8, bool putoff, bool zs))(const TcParams)
{
    if (zs && kt && nbk == 2 && G == 3 && !f8) {   // at most 16 features, in the preferred shape
        if (NV == 128) return score_tc_kernel<128, 3, 64, true, 2, false, false, true>;
        return putoff ? score_tc_kernel<256, 3, 64, true, 2, false, true, true> : score_tc_kernel<256, 3, 64, true, 2, false, false, true>;
    }
    if (putoff && !f8 && NV == 256 && G == 3) {   // histories of two to seven passes in the two preferred shapes
        if (kt && nbk == 2) return score_tc_kernel<256, 3, 64, true, 2, false, true>;
        if (!kt && nbk == 3) return score_tc_kernel<256, 3, 64, false, 3, false, true>;
    }
    if (f8) {   // offered for the shapes of long histories only (tc_prepare)
        if (kt && nbk == 2 && G == 3) return score_tc_kernel<256, 3, 64, true, 2, true>;
        if (kt) return G == 3 ? score_tc_kernel<256, 3, 64, true, 3, true> : score_tc_kernel<256, 2, 64, true, 2, true>;
        return G == 3 ? score_tc_kernel<256, 3, 64, false, 3, true> : score_tc_kernel<256, 2, 64, false, 2, true>;
    }
    if (kt && nbk == 2 && G == 3)
        return NV == 256 ? score_tc_kernel<256, 3, 64, true, 2> : score_tc_kernel<128, 3, 64, true, 2>;
    if (kt) {
        if (NV == 256) return G == 3 ? score_tc_kernel<256, 3, 64, true> : score_tc_kernel<256, 2, 64, true>;
        return G == 3 ? score_tc_kernel<128, 3, 64, true> : score_tc_kernel<128, 2, 64, true>;
    }
    if (NV == 256) return G == 3 ? score_tc_kernel<256, 3, 64, false> : score_tc_kernel<256, 2, 64, false>;
    return G == 3 ? score_tc_kernel<128, 3, 64, false> : score_tc_kernel<128, 2, 64, false>;
}

constexpr int kF8MinPasses = 8;   // n > 1792: below that the guard hands more candidates to the FP64 pass than the cheaper MMAs save

int env_int(const char* name, int fallback)
{
    const char* v = getenv(name);
    return v ? atoi(v) : fallback;
}

}  // namespace

bool tc_supported(int n, int d) { return n >= 1 && n <= kMaxN && d >= 1 && d <= 128; }

void tc_release(r3_gp* gp)
{
    TensorOperands* t = ops_of(gp);
    if (!t) return;
    dev_free(t->centre);
    dev_free(t->scale);
    dev_free(t->xt);
    dev_free(t->xs32);
    dev_free(t->xnorm);
    dev_free(t->xnmax);
    dev_free(t->alpha);
    dev_free(t->wt);
    dev_free(t->kscale);
    dev_free(t->vinv2);
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
    t->DP = round_up(d, 16);
    t->NV = n > 128 ? 256 : 128;
    t->NP = round_up(n, t->NV);
    t->P = t->NP / t->NV;
    // Shape, in order of preference (measured on the largest workload: the first two are within 1 %):
    // k* in shared memory with three Matern groups and at least three W stages; k* in TMEM (needs
    // V accumulator + two distance buffers + candidates + G k* buffers <= 512 columns), which frees
    // shared memory for W stages; then whatever fits with two W stages.
    const size_t budget = 227 * 1024 - 1024 - kBarBytes;
    const int want_kt = env_int("R3_TC_KT", -1), want_g = env_int("R3_TC_G", 0);
    t->KD = 64;
    bool found = false;
    static const struct { bool kt; int G, min_ws, nbk; } prefs[] = {
        {true, 3, 3, 2},  {false, 3, 3, 3}, {true, 3, 3, 3}, {true, 2, 3, 2},
        {false, 2, 3, 2}, {false, 3, 2, 3}, {true, 2, 2, 2}, {false, 2, 2, 2}};
    const int want_nbk = env_int("R3_TC_NBK", 0);
    // Stages of W: four by default although shared memory would hold up to six for few features.  Measured, the
    // fifth and sixth buy nothing on any workload and cost the short histories 3-5 % (256 observations, 16
    // features: 0.241 ms to 0.228 ms per pool; 512 and 32: 5.79 ms to 5.63 ms; 1024 and 4096 observations:
    // unchanged down to three).  R3_TC_MAXWS = 2..6 overrides.
    const int max_ws = std::min(std::max(env_int("R3_TC_MAXWS", 4), 2), MAX_STAGES);
    for (const auto& pr : prefs) {
        if (found) break;
        t->kt = pr.kt;
        t->G = pr.G;
        t->nbk = pr.nbk;
        if (want_kt >= 0 && (int)t->kt != want_kt) continue;
        if (want_g && t->G != want_g) continue;
        if (want_nbk && t->nbk != want_nbk) continue;
        if (t->NV + 2 * t->KD + t->DP + (t->kt ? t->nbk * KC : 0) > 512) continue;
        for (t->ws = max_ws; t->ws >= 2; --t->ws)
            if (smem_map(t->DP, t->NV, t->G, t->KD, t->ws, t->kt).bar <= budget) break;
        found = t->ws >= pr.min_ws;
    }
    if (!found) {
        tc_release(gp);   // does not fit: the SIMT engine serves this shape
        return R3_OK;
    }
    t->smem_bytes = smem_map(t->DP, t->NV, t->G, t->KD, t->ws, t->kt).bar + kBarBytes + 1024;
    // FP8 cross terms: R3_TC_F8 = 0/1 decides; by default histories of at least kF8MinPasses passes take them
    const int want_f8 = env_int("R3_TC_F8", -1);
    t->f8 = t->NV == 256 && (want_f8 >= 0 ? want_f8 != 0 : t->P >= kF8MinPasses);
    const int CPP = t->NV / KC;
    const size_t tiles = (size_t)CPP * t->P * (t->P + 1) / 2;
    t->wt_gp_stride = tiles * (2 * (size_t)KC * t->NV);
    unsigned* wmax_bits = nullptr;
    float* wscale_d = nullptr;
    auto fail = [&](const char* what, cudaError_t e) {
        set_error("%s failed: %s", what, cudaGetErrorString(e));
        dev_free(wmax_bits);
        dev_free(wscale_d);
        tc_release(gp);
        return e == cudaErrorMemoryAllocation ? R3_ERR_ALLOC : R3_ERR_CUDA;
    };
    auto decline = [&]() {   // the SIMT engine serves this history
        dev_free(wmax_bits);
        dev_free(wscale_d);
        tc_release(gp);
        return R3_OK;
    };
    cudaError_t e;
    if ((e = dev_malloc(&t->centre, sizeof(float) * B * t->DP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->scale, sizeof(float) * B * t->DP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->xt, sizeof(__half) * B * (size_t)(t->NP / t->KD) * 2 * t->DP * t->KD)) != cudaSuccess)
        return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->xs32, sizeof(float) * B * (size_t)t->NP * t->DP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->xnorm, sizeof(float) * B * t->NP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->xnmax, sizeof(float) * (B > 2 ? B : 2))) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->alpha, sizeof(float) * B * t->NP)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->wt, sizeof(__half) * B * t->wt_gp_stride)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->kscale, sizeof(float) * B)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&t->vinv2, sizeof(double) * B)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&wmax_bits, sizeof(unsigned) * B)) != cudaSuccess) return fail("cudaMalloc", e);
    if ((e = dev_malloc(&wscale_d, sizeof(float) * B)) != cudaSuccess) return fail("cudaMalloc", e);

    // scaled observations (their largest coordinate decides whether the FP16 planes can hold them) and
    // the largest |W| of each GP (it decides the power-of-two scale of its W planes)
    unsigned* xamax_bits = reinterpret_cast<unsigned*>(t->xnmax);   // borrowed until xnmax_kernel overwrites it
    if ((e = cudaMemsetAsync(xamax_bits, 0, sizeof(unsigned), stream)) != cudaSuccess) return fail("cudaMemsetAsync", e);
    if ((e = cudaMemsetAsync(wmax_bits, 0, sizeof(unsigned) * B, stream)) != cudaSuccess) return fail("cudaMemsetAsync", e);
    centre_kernel<<<dim3(t->DP, B), 256, 0, stream>>>(gp->X, gp->inv_ell, n, d, t->DP, t->centre, t->scale);
    xt_build_kernel<<<dim3(t->NP / t->KD, B), 256, 0, stream>>>(gp->X, t->centre, t->scale, gp->alpha32, n, d, gp->npad,
                                                                t->DP, t->NP, t->KD, t->xt, t->xs32, t->xnorm, t->alpha, xamax_bits);
    wmax_kernel<<<dim3(296, B), 256, 0, stream>>>(gp->W64, n, gp->npad, wmax_bits);
    g_launches += 3;
    float xamax = 0.f;
    std::vector<float> wmax(B);
    if ((e = cudaMemcpyAsync(&xamax, xamax_bits, sizeof(float), cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return fail("cudaMemcpyAsync", e);
    if ((e = cudaMemcpyAsync(wmax.data(), wmax_bits, sizeof(float) * B, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return fail("cudaMemcpyAsync", e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return fail("operand preparation", e);
    if (!(xamax <= kMaxScaled)) return decline();   // scaled coordinates beyond the FP16 planes
    std::vector<float> wscale(B), kscale(B);
    std::vector<double> vinv2(B);
    for (int g = 0; g < B; ++g) {
        int ew = 0, ek = 0;
        frexp((double)wmax[g], &ew);               // wmax < 2^ew
        frexp((double)gp->sf2[g], &ek);            // sf2  < 2^ek  (k* <= sf2)
        const int sw = (t->f8 ? kScaleExpF8 : kScaleExp) - ew, sk = kScaleExp - ek;
        if (!(wmax[g] > 0.f) || sw < -60 || sw > 60 || sk < -60 || sk > 60) return decline();   // degenerate scales
        wscale[g] = (float)ldexp(1.0, sw);
        kscale[g] = (float)ldexp(1.0, sk);
        vinv2[g] = ldexp(1.0, -2 * (sw + sk));
    }
    if ((e = cudaMemcpyAsync(wscale_d, wscale.data(), sizeof(float) * B, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail("cudaMemcpyAsync", e);
    if ((e = cudaMemcpyAsync(t->kscale, kscale.data(), sizeof(float) * B, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail("cudaMemcpyAsync", e);
    if ((e = cudaMemcpyAsync(t->vinv2, vinv2.data(), sizeof(double) * B, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail("cudaMemcpyAsync", e);
    xnmax_kernel<<<B, 256, 0, stream>>>(t->xnorm, t->NP, t->xnmax);
    wt_build_kernel<<<dim3(t->P * CPP, t->P, B), 256, 0, stream>>>(gp->W64, n, gp->npad, t->NV, t->wt_gp_stride,
                                                                   wscale_d, t->wt, t->f8);
    g_launches += 2;
    if ((e = cudaGetLastError()) != cudaSuccess) return fail("operand preparation launch", e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return fail("operand preparation", e);
    dev_free(wmax_bits);
    dev_free(wscale_d);
    wmax_bits = nullptr;
    wscale_d = nullptr;
    // The cap on dynamic shared memory belongs to the kernel, not to the handle, and handles with different
    // feature counts share an instantiation with different sizes: raise it to the device's limit (the kernel
    // has no static shared memory), so that no handle's preparation lowers it for another.
    int smem_optin = 0;
    if ((e = cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, gp->device)) != cudaSuccess)
        return fail("cudaDeviceGetAttribute", e);
    if ((size_t)smem_optin < t->smem_bytes) return decline();
    e = cudaFuncSetAttribute(kernel_for(t->NV, t->G, t->kt, t->nbk, t->f8, t->P >= 2 && t->P < kF8MinPasses, t->DP <= kZsMaxDP), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             smem_optin);
    if (e != cudaSuccess) return fail("cudaFuncSetAttribute", e);
    return R3_OK;
}

void tc_info(const r3_gp* gp, int* info)
{
    const TensorOperands* t = ops_of(gp);
    for (int i = 0; i < 8; ++i) info[i] = 0;
    if (!t) return;
    info[0] = t->NV; info[1] = t->P; info[2] = t->DP; info[3] = t->NP;
    info[4] = t->G; info[5] = t->ws; info[6] = t->kt ? 1 : 0; info[7] = t->f8 ? 1 : 0;
}

size_t score_tc_workspace_bytes(const r3_gp* gp, long long m) { return guard_workspace_bytes(gp, m); }

r3_status_t score_tc(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                     size_t ws_bytes, cudaStream_t stream)
{
    return score_tc_part(gp, Xcand, m, mu, sigma, ei, ws, ws_bytes, 0, -1, true, stream);
}

long long score_tc_tiles(const r3_gp* gp, long long m) { return (m + TILE_M - 1) / TILE_M * gp->batch; }

bool score_tc_can_split(const r3_gp* gp) { return ops_of(gp) != nullptr && env_int("R3_TC_PAIR", 0) == 0; }

r3_status_t score_tc_guard(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                           cudaStream_t stream)
{
    return guard_and_rescue(gp, Xcand, m, guard_carve(gp, m, ws), mu, sigma, ei, false, stream);
}

r3_status_t score_tc_part(r3_gp* gp, const float* Xcand, long long m, float* mu, float* sigma, float* ei, void* ws,
                          size_t ws_bytes, long long tile_begin, long long tile_end, bool guard, cudaStream_t stream)
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
    prm.xs32 = t->xs32;
    prm.xnorm = t->xnorm;
    prm.xnmax = t->xnmax;
    prm.alpha = t->alpha;
    prm.wt = t->wt;
    prm.kscale = t->kscale;
    prm.vinv2 = t->vinv2;
    prm.wt_gp_stride = t->wt_gp_stride;
    prm.sf2 = gp->sf2_d;
    prm.best = gp->best_d;
    prm.wnorm = gp->wnorm_d;
    prm.DP = t->DP;
    prm.NP = t->NP;
    prm.P = t->P;
    prm.ws = t->ws;
    prm.status = gp->status_d;
    prm.tiles_per_gp = (m + TILE_M - 1) / TILE_M;
    prm.total_tiles = prm.tiles_per_gp * gp->batch;
    prm.tile_begin = 0;
    prm.wait_limit = gp->wait_limit_cycles;
    prm.withhold_w = gp->withhold_w;
    gp->withhold_w = -1;   // one call only
    if (tile_end >= 0) {   // a range of the pool's tiles (the caller runs the guard once, after the last range)
        prm.tile_begin = tile_begin;
        prm.total_tiles = tile_end < prm.total_tiles ? tile_end : prm.total_tiles;
    }
    const long long launch_tiles = prm.total_tiles - prm.tile_begin;
    if (launch_tiles <= 0) return R3_OK;
    if (prm.tile_begin == 0) {   // the pool's first (or only) piece: the rescue counters start at zero
        const r3_status_t st0 = guard_begin(gp, gb, stream);
        if (st0 != R3_OK) return st0;
    }
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, gp->device);
    const unsigned grid = (unsigned)(launch_tiles < sms ? launch_tiles : sms);
    // R3_TC_TRACE=1 prints, for the first CTA, the cycles each role spent per wait / issue category
    prm.trace = nullptr;
    if (getenv("R3_TC_TRACE")) {
        if (dev_malloc(&prm.trace, sizeof(long long) * (grid * 32 + 32 * 128)) != cudaSuccess) prm.trace = nullptr;
        if (prm.trace) cudaMemset(prm.trace, 0, sizeof(long long) * (grid * 32 + 32 * 128));
    }
    // The paired kernel (two CTAs of a cluster share a tile and the k* chunks) serves histories with at least
    // two passes; R3_TC_PAIR=0/1 overrides the choice.
    int pair_ws = 0;
    const bool pair = tile_end < 0 && !t->f8 && env_int("R3_TC_PAIR", 0) != 0 && tc_pair_fits(t, &pair_ws);
    prof_begin(gp, stream);
    if (pair) {
        const r3_status_t st = launch_tc_pair(t, prm, sms, stream);
        if (st != R3_OK) return st;
    } else {
        void (*kernel)(const TcParams) = kernel_for(t->NV, t->G, t->kt, t->nbk, t->f8, t->P >= 2 && t->P < kF8MinPasses, t->DP <= kZsMaxDP);
        R3_LAUNCH(kernel, grid, 128 + 128 * t->G, t->smem_bytes, stream, prm);
    }
    prof_end(gp, stream);
    if (prm.trace) {
        std::vector<long long> h((size_t)grid * 32 + 32 * 128);
        cudaMemcpy(h.data(), prm.trace, sizeof(long long) * h.size(), cudaMemcpyDeviceToHost);
        for (int i = 0; i < 128; ++i) {
            fprintf(stderr, "ev %d:", i);
            for (int e = 0; e < 24; ++e) fprintf(stderr, " %lld", h[(size_t)grid * 32 + e * 128 + i] - h[(size_t)grid * 32 + 128 * 12]);
            fprintf(stderr, "\n");
        }
        dev_free(prm.trace);
        const char* names[4] = {"mmaV", "matern0", "matern1", "mmaD"};
        fprintf(stderr, "trace shape NV=%d G=%d KD=%d kt=%d ws=%d DP=%d P=%d smem=%zu\n", t->NV, t->G, t->KD, (int)t->kt, t->ws,
                t->DP, t->P, t->smem_bytes);
        for (int cta = 0; cta < (pair ? 2 : 1); ++cta)
            for (int r = 0; r < 4; ++r) {
                fprintf(stderr, "trace cta%d %s:", cta, names[r]);
                for (int i = 0; i < 8; ++i) fprintf(stderr, " %lld", h[((size_t)cta * 4 + r) * 8 + i]);
                fprintf(stderr, "\n");
            }
    }
    if (!guard) return R3_OK;
    return guard_and_rescue(gp, Xcand, m, gb, mu, sigma, ei, false, stream);
}

}  // namespace r3
