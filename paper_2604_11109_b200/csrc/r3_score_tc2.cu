// Tensor-core scoring, paired form: a cluster of two CTAs (two SMs) shares one tile of 128 candidates.
//
// The single-CTA kernel (r3_score_tc.cu) regenerates the cross-covariance chunks k* for every pass over
// the rows of W, (P+1)/2 times on average, and each regeneration costs distance MMAs and Matern
// arithmetic that compete with the variance product for the tensor pipe and the issue slots.  Here the
// two CTAs of a cluster take consecutive passes (CTA r owns passes 2j + r, with its own V accumulator, W
// stream and MMA issuer) and consume the SAME sequence of k* chunks: each chunk is generated once, by one
// of the two CTAs (they alternate by distance product), and written into both CTAs' k* rings -- the local
// one with ordinary shared-memory stores, the peer's with one 16 KB bulk copy from shared memory to the
// peer's shared memory (per-thread remote stores were four times slower than the arithmetic they
// followed).  Per SM the generation work drops to about a quarter; the variance product is unchanged.
//
// Hand-over of a k* buffer b (ring of four per CTA, same ring position in both CTAs):
//   K_FULL[b]   one arrival per CTA.  The generating group's threads fence their stores towards the async
//               proxy and meet at a named barrier; one thread then arrives on the local barrier, arrives
//               with a 16 KB transaction count on the peer's, and issues the bulk copy whose bytes
//               complete that count.  The consumer waits with cluster-scope acquire.
//   K_EMPTY[b]  two arrivals, one per CTA: tcgen05.commit multicast to both CTAs after the MMAs that read
//               it (or plain arrives from a CTA whose pass does not use that chunk).
// Everything else (operand streams, distance products, V hand-over) is local to a CTA and works as in the
// single-CTA kernel.  At the end of a tile CTA 1 sends its partial sums to CTA 0, which runs the epilogue.
// All waits are bounded; the two CTAs meet at a cluster barrier before they exit, so that no
// distributed-shared-memory access can target a CTA that has already gone.
#include <stdio.h>
#include <stdlib.h>

#include "r3_epilogue.cuh"
#include "r3_tc_common.cuh"

namespace r3 {

namespace {

#ifndef R3_TC_TRACE
#define LOGEV2(ev, tt) do { } while (0)
#else
// event log of the first cluster: clock of event `ev` (0..7) of CTA `rank` for stream chunk tt in the window
constexpr long long kLog2T0 = 576 + 300;
#define LOGEV2(ev, tt)                                                                                        \
    do {                                                                                                      \
        if (prm.trace && blockIdx.x < 2 && (tt) >= kLog2T0 && (tt) < kLog2T0 + kLogN)                         \
            prm.trace[(size_t)gridDim.x * 32 + (blockIdx.x * 12 + (ev)) * kLogN + ((tt) - kLog2T0)] = clock64(); \
    } while (0)
#endif

constexpr int NV2 = 256;      // rows of W per pass
constexpr int KD2 = 64;       // observations per distance product
constexpr int SL2 = KD2 / KC; // chunks per distance product == Matern groups per CTA
constexpr int G2 = SL2;       // group g generates the g-th chunk of each product its CTA owns
constexpr int NB = 4;         // k* ring buffers per CTA
constexpr int CPP2 = NV2 / KC;
constexpr int MAX_WS2 = 6;

struct PairMap {
    uint32_t red, k, x, w, bar, x_stage, w_stage;
};
__host__ __device__ inline PairMap pair_map(int DP, int ws)
{
    PairMap s;
    s.red = 0;                                   // (G2 + 1) x 128 rows x 4 doubles: local groups, peer slot
    s.k = (uint32_t)(G2 + 1) * 4096u;            // NB buffers x 2 planes x [KC/8][128][8] halves
    s.x = s.k + (uint32_t)NB * 16384u;           // XS stages x 2 planes x [DP/8][KD][8] halves
    s.x_stage = 2u * DP * KD2 * 2u;
    s.w = s.x + (uint32_t)XS * s.x_stage;        // ws stages x 2 planes x [KC/8][NV][8] halves
    s.w_stage = 2u * KC * NV2 * 2u;
    s.bar = s.w + (uint32_t)ws * s.w_stage;
    return s;
}
constexpr uint32_t kPairBarBytes = 1024;
enum : uint32_t {
    PB_X_FULL = 0, PB_X_EMPTY = 2, PB_W_FULL = 4, PB_W_EMPTY = 10, PB_D_FULL = 16, PB_D_EMPTY = 18,
    PB_K_FULL = 20, PB_K_EMPTY = 24, PB_V_FULL = 28, PB_V_EMPTY = 29, PB_Z_READY = 30, PB_RED_READY = 31,
    PB_RED_PEER = 32, PB_MMA_DONE = 33, PB_COUNT = 35
};
constexpr uint32_t kPairFlagOffset = PB_COUNT * 8;
constexpr uint32_t kPairZnOffset = 512;

// ---- cluster-scope PTX
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes)
                 : "memory");
}

// Bulk copy from this CTA's shared memory into the peer's; the bytes are counted on the peer's barrier.
__device__ __forceinline__ void bulk_s2peer(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t cluster_bar)
{
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster),
                 "r"(src_cta), "r"(bytes), "r"(cluster_bar)
                 : "memory");
}

__device__ __forceinline__ void st_cluster_f64(uint32_t cluster_addr, double v)
{
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(cluster_addr), "d"(v) : "memory");
}
// arrive on the same barrier of both CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// chunks of super-pass j (passes 2j and 2j+1; a lone last pass when P is odd)
__device__ __forceinline__ int superpass_chunks(int j, int P) { return (2 * j + 2 < P ? 2 * j + 2 : P) * CPP2; }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128 + 128 * G2, 1) score_tc_pair_kernel(const TcParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const PairMap map = pair_map(prm.DP, prm.ws);
    const uint32_t bars = base + map.bar;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + map.bar + kPairFlagOffset);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + map.bar + kPairFlagOffset + 8);
    float* zn_s = reinterpret_cast<float*>(sm + map.bar + kPairZnOffset);
    auto bar = [&](uint32_t slot) { return bars + slot * 8u; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(), peer = rank ^ 1u;
    const int DP = prm.DP, P = prm.P, ws = prm.ws;
    const long long wl = prm.wait_limit;
    const int NSP = (P + 1) / 2;                       // super-passes per tile
    constexpr uint32_t TMEM_COLS = 512u;
    constexpr uint32_t ZCOL = NV2 + 2 * KD2;

    if (threadIdx.x == 0) {
        for (int i = 0; i < XS; ++i) {
            mbar_init(bar(PB_X_FULL + i), 1);
            mbar_init(bar(PB_X_EMPTY + i), 1);
            mbar_init(bar(PB_D_FULL + i), 1);
            mbar_init(bar(PB_D_EMPTY + i), 128 * SL2);
        }
        for (int i = 0; i < MAX_WS2; ++i) {
            mbar_init(bar(PB_W_FULL + i), 1);
            mbar_init(bar(PB_W_EMPTY + i), 1);
        }
        for (int i = 0; i < NB; ++i) {
            mbar_init(bar(PB_K_FULL + i), 1);
            mbar_init(bar(PB_K_EMPTY + i), 2);
        }
        mbar_init(bar(PB_V_FULL), 1);
        mbar_init(bar(PB_V_EMPTY), 128 * G2);
        mbar_init(bar(PB_Z_READY), 128);
        mbar_init(bar(PB_RED_READY), 128 * G2);
        mbar_init(bar(PB_RED_PEER), 128);
        mbar_init(bar(PB_MMA_DONE), 1);
        mbar_init(bar(PB_MMA_DONE + 1), 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
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
    cluster_sync_all();   // both CTAs' barriers exist before anyone arrives on the peer's
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const long long first_tile = blockIdx.x >> 1, tile_step = gridDim.x >> 1;
    long long tacc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long tlast = prm.trace ? clock64() : 0;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------ producer: scaled observations (own products)
        const uint32_t bytes = map.x_stage;
        long long issued = 0, Ug = 0;
        int st = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const __half* src = prm.xt + (size_t)g * (prm.NP / KD2) * (bytes / 2);
            for (int j = 0; ok && j < NSP; ++j) {
                const int nprod = superpass_chunks(j, P) / SL2;
                for (int u = 0; u < nprod; ++u, ++Ug) {
                    if ((uint32_t)(Ug & 1) != rank) continue;
                    if (!(ok = mbar_wait(bar(PB_X_EMPTY + st), ph ^ 1u, abort_flag, wl))) break;
                    mbar_arrive_expect_tx(bar(PB_X_FULL + st), bytes);
                    bulk_g2s(base + map.x + st * bytes, src + (size_t)u * (bytes / 2), bytes, bar(PB_X_FULL + st));
                    ++issued;
                    if (++st == XS) { st = 0; ph ^= 1u; }
                }
            }
        }
        if (!ok) {
            const int pending = (int)(issued < XS ? issued : XS);
            for (int u = 0; u < pending; ++u) {
                if (--st < 0) { st = XS - 1; ph ^= 1u; }
                mbar_wait(bar(PB_X_FULL + st), ph, abort_flag + 1, wl);
            }
        }
    } else if (warp == 0 && lane == 1) {
        // ------------------------------------------------------------ producer: chunks of W (own passes)
        const uint32_t bytes = map.w_stage;
        long long issued = 0;
        int st = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const __half* src = prm.wt + (size_t)g * prm.wt_gp_stride;
            for (int j = 0; ok && j < NSP; ++j) {
                const int p = 2 * j + (int)rank;
                if (p >= P) continue;
                const __half* psrc = src + (size_t)(CPP2 * p * (p + 1) / 2) * (bytes / 2);
                for (int c = 0; c < (p + 1) * CPP2; ++c, ++issued) {
                    if (issued == prm.withhold_w) { ok = false; break; }   // test aid: the stream of W stops here
                    if (!(ok = mbar_wait(bar(PB_W_EMPTY + st), ph ^ 1u, abort_flag, wl))) break;
                    mbar_arrive_expect_tx(bar(PB_W_FULL + st), bytes);
                    bulk_g2s(base + map.w + st * bytes, psrc + (size_t)c * (bytes / 2), bytes, bar(PB_W_FULL + st));
                    if (++st == ws) { st = 0; ph ^= 1u; }
                }
            }
        }
        if (!ok) {
            const int pending = (int)(issued < ws ? issued : ws);
            for (int u = 0; u < pending; ++u) {
                if (--st < 0) { st = ws - 1; ph ^= 1u; }
                mbar_wait(bar(PB_W_FULL + st), ph, abort_flag + 1, wl);
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------ MMA issuer: distance products (own)
        constexpr uint32_t IDESC_D = instr_desc_f16(KD2);
        const uint32_t zH = tmem + ZCOL, zL = zH + (uint32_t)DP / 2;
        const uint32_t x_lo0 = desc_addr(base + map.x) | (((KD2 * 16u) >> 4) << 16);
        const int ksteps = DP / 16;
        long long tile_iter = 0, Ug = 0;
        int st = 0, db = 0;
        uint32_t ph = 0, d_ph = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            if (!(ok = mbar_wait(bar(PB_Z_READY), (uint32_t)(tile_iter & 1), abort_flag, wl))) break;
            tc_fence_after();
            for (int j = 0; ok && j < NSP; ++j) {
                const int nprod = superpass_chunks(j, P) / SL2;
                for (int u = 0; u < nprod; ++u, ++Ug) {
                    if ((uint32_t)(Ug & 1) != rank) continue;
                    if (!(ok = mbar_wait(bar(PB_X_FULL + st), ph, abort_flag, wl))) break;
                    if (!(ok = mbar_wait(bar(PB_D_EMPTY + db), d_ph ^ 1u, abort_flag, wl))) break;
                    tc_fence_after();
                    const uint32_t xH_lo = x_lo0 + ((st * map.x_stage) >> 4), xL_lo = xH_lo + (((uint32_t)DP * KD2 * 2u) >> 4);
                    const uint32_t dcol = tmem + NV2 + db * KD2;
                    uint32_t acc = 0;
#pragma unroll
                    for (int combo = 0; combo < 3; ++combo) {
                        const uint32_t a0 = combo == 2 ? zL : zH, b0 = combo == 1 ? xL_lo : xH_lo;
                        for (int jj = 0; jj < ksteps; ++jj) {
                            tc_mma_f16_ts(dcol, a0 + jj * 8u, pack64(b0 + jj * ((2u * KD2 * 16u) >> 4), kDescHi), IDESC_D, acc);
                            acc = 1;
                        }
                    }
                    tc_commit(bar(PB_X_EMPTY + st));
                    tc_commit(bar(PB_D_FULL + db));
                    if (++st == XS) { st = 0; ph ^= 1u; }
                    if (++db == 2) { db = 0; d_ph ^= 1u; }
                }
            }
        }
        tc_commit(bar(PB_MMA_DONE));
        mbar_wait(bar(PB_MMA_DONE), 0, abort_flag + 1, wl);
    } else if (warp == 2 && lane == 0) {
        // ------------------------------------------------------------ MMA issuer: variance product (own passes)
        const uint32_t k_lo0 = desc_addr(base + map.k) | ((2048u >> 4) << 16);
        const uint32_t w_lo0 = desc_addr(base + map.w) | (((NV2 * 16u) >> 4) << 16);
        const uint32_t k_empty_peer0 = map_to_cta(bar(PB_K_EMPTY), peer);
        uint32_t v_ph = 0;
        int w_s = 0, k_s = 0;
        uint32_t w_ph = 0, k_ph = 0;
        bool ok = true;
        long long tv = 0;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step) {
            for (int j = 0; ok && j < NSP; ++j) {
                const int p = 2 * j + (int)rank;
                const int mine = p < P ? (p + 1) * CPP2 : 0;   // chunks of this super-pass that my pass uses
                const int nchunk = superpass_chunks(j, P);
                for (int c = 0; ok && c < nchunk; ++c, ++tv) {
                    const int b = k_s;
                    TICK(7);
                    if (c < mine) {
                        const int s = w_s;
                        if (c == 0) {
                            if (!(ok = mbar_wait(bar(PB_V_EMPTY), v_ph ^ 1u, abort_flag, wl))) break;
                        }
                        TICK(3);
                        if (!(ok = mbar_wait(bar(PB_K_FULL + b), k_ph, abort_flag, wl))) break;
                        TICK(4);
                        LOGEV2(0, tv);
                        if (!(ok = mbar_wait(bar(PB_W_FULL + s), w_ph, abort_flag, wl))) break;
                        TICK(5);
                        LOGEV2(1, tv);
                        if (++w_s == ws) { w_s = 0; w_ph ^= 1u; }
                        // (the writers of a k* buffer fence their stores towards the async proxy before they arrive,
                        // and the peer's copy arrives through the async proxy: no proxy fence on this side)
                        tc_fence_after();
                        LOGEV2(7, tv);
                        // In the pass's diagonal block the rows of W above the chunk's columns are zero (W is lower
                        // triangular): the MMAs start at the first row that can be non-zero and get narrower.
                        const uint32_t skip = c > p * CPP2 ? (uint32_t)(c - p * CPP2) * KC : 0u;
                        const uint32_t idesc_v = instr_desc_f16(NV2 - skip);
                        const uint32_t vcol = tmem + skip;
                        const uint32_t aH = k_lo0 + ((b * 16384u) >> 4), aL = aH + (8192u >> 4);
                        const uint32_t bH = w_lo0 + ((s * map.w_stage) >> 4) + skip, bL = bH + (((uint32_t)KC * NV2 * 2u) >> 4);
#pragma unroll
                        for (int combo = 0; combo < 3; ++combo) {
                            const uint32_t a0 = combo == 2 ? aL : aH, b0 = combo == 1 ? bL : bH;
#pragma unroll
                            for (int jj = 0; jj < KC / 16; ++jj)
                                tc_mma_f16(vcol, pack64(a0 + jj * (4096u >> 4), kDescHi),
                                           pack64(b0 + jj * ((2u * NV2 * 16u) >> 4), kDescHi), idesc_v,
                                           (c > 0 || combo > 0 || jj > 0) ? 1u : 0u);
                        }
                        LOGEV2(8, tv);
                        tc_commit(bar(PB_W_EMPTY + s));
                        LOGEV2(9, tv);
                        tc_commit_pair(bar(PB_K_EMPTY + b));
                        LOGEV2(10, tv);
                        if (c == mine - 1) {
                            tc_commit(bar(PB_V_FULL));
                            v_ph ^= 1u;
                        }
                        TICK(6);
                        LOGEV2(2, tv);
                    } else {
                        // my pass does not use this chunk: release the buffer on both CTAs once it has been filled
                        if (!(ok = mbar_wait(bar(PB_K_FULL + b), k_ph, abort_flag, wl))) break;
                        mbar_arrive(bar(PB_K_EMPTY + b));
                        mbar_arrive_cluster(k_empty_peer0 + (uint32_t)b * 8u);
                        TICK(0);
                    }
                    if (++k_s == NB) { k_s = 0; k_ph ^= 1u; }
                }
            }
        }
        tc_commit(bar(PB_MMA_DONE + 1));
        mbar_wait(bar(PB_MMA_DONE + 1), 0, abort_flag + 1, wl);
        if (prm.trace)
            for (int i = 0; i < 8; ++i) prm.trace[((size_t)blockIdx.x * 4 + 0) * 8 + i] = tacc[i];
#ifdef R3_TC_TRACE
    } else if (warp == 3 && lane == 0) {
        // observer (trace builds only): when each k* buffer became full in this CTA
        long long tv = 0;
        bool ok = true;
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step)
            for (int j = 0; ok && j < NSP; ++j)
                for (int c = 0; ok && c < superpass_chunks(j, P); ++c, ++tv) {
                    ok = mbar_wait(bar(PB_K_FULL + (int)(tv % NB)), (uint32_t)((tv / NB) & 1), abort_flag, wl);
                    LOGEV2(11, tv);
                }
#endif
    } else if (warp >= 4) {
        // ------------------------------------------------------------ Matern / epilogue warp groups
        const int grp = (warp - 4) >> 2;         // 0..G2-1: which chunk of each own product
        const int q4 = warp & 3;
        const int row = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t k_full_peer0 = map_to_cta(bar(PB_K_FULL), peer);
        const uint32_t kbuf_peer0 = map_to_cta(base + map.k, peer);
        long long Ug = 0;                        // global product counter (same sequence in both CTAs)
        long long tg = 0;                        // global chunk counter at the start of the current super-pass
        long long own = 0;                       // own products so far (distance-buffer ring)
        uint32_t v_ph = 0;
        long long tile_iter = 0;
        bool ok = true, bad = false;
        double* red = reinterpret_cast<double*>(sm + map.red);
        for (long long tile = first_tile; ok && tile < prm.total_tiles; tile += tile_step, ++tile_iter) {
            const int g = (int)(tile / prm.tiles_per_gp);
            const long long cand = (tile % prm.tiles_per_gp) * TILE_M + row;
            const bool valid = cand < prm.m;
            const float sf2 = prm.sf2[g];
            const float kvscale = prm.kscale[g] * sf2;
            if (grp == G2 - 1) {
                // The candidate planes and norms of the previous tile may still be read by the other group's
                // close-pair refinement until that group has handed in its partial sums.
                if (tile_iter > 0) {
                    ok = mbar_wait(bar(PB_RED_READY), (uint32_t)((tile_iter - 1) & 1), abort_flag, wl);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                // ---- scale the candidate, split it, keep it in TMEM as the A operand of the distance MMAs
                float zn = 0.f;
                bool far = false;
                const float* zrow = prm.xcand + ((size_t)g * prm.m + (valid ? cand : 0)) * prm.d;
                const float* cen = prm.centre + (size_t)g * DP;
                const float* scl = prm.scale + (size_t)g * DP;
                const bool vec = (prm.d % 4) == 0 && (reinterpret_cast<uintptr_t>(prm.xcand) & 15) == 0;
                uint32_t zh[8], zl[8];
                for (int j8 = 0; j8 < DP / 8; ++j8) {
                    __half2 hi2[4], lo2[4];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int j4 = 2 * j8 + h;
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
                        float zt[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            bad |= !isfinite(z[e]);
                            float v = valid ? (z[e] - cc[e]) * ss[e] : 0.f;
                            if (fabsf(v) > kMaxScaled) {
                                v = copysignf(kMaxScaled, v);
                                far = true;
                            }
                            zt[e] = v;
                            zn = fmaf(v, v, zn);
                        }
                        split2(zt[0], zt[1], hi2[2 * h], lo2[2 * h]);
                        split2(zt[2], zt[3], hi2[2 * h + 1], lo2[2 * h + 1]);
                    }
                    const int o = (j8 & 1) * 4;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        zh[o + e] = *reinterpret_cast<const uint32_t*>(&hi2[e]);
                        zl[o + e] = *reinterpret_cast<const uint32_t*>(&lo2[e]);
                    }
                    if (j8 & 1) {
                        tc_st8(lane_addr + ZCOL + (uint32_t)(j8 >> 1) * 8u, zh);
                        tc_st8(lane_addr + ZCOL + (uint32_t)DP / 2 + (uint32_t)(j8 >> 1) * 8u, zl);
                    }
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                zn_s[row] = far ? -zn : zn;
                tc_fence_before();
                mbar_arrive(bar(PB_Z_READY));
            }
            ok = mbar_wait(bar(PB_Z_READY), (uint32_t)(tile_iter & 1), abort_flag, wl);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const bool far_cand = zn_s[row] < 0.f;
            const float zn = fabsf(zn_s[row]);
            const float* xs_g = prm.xs32 + (size_t)g * prm.NP * DP;
            const float v_thresh = far_cand ? INFINITY : kvscale * kRefine / (zn + prm.xnmax[g]);
            const float pc0 = kvscale, pc1 = kvscale * kPolyC1, pc2 = kvscale * kPolyC2;
            const float inv_kscale = 1.f / prm.kscale[g];
            const float* xn_g = prm.xnorm + (size_t)g * prm.NP;
            const float* al_g = prm.alpha + (size_t)g * prm.NP;
            double mu_acc = 0.0, a2_acc = 0.0, s2_acc = 0.0, q_acc = 0.0;
            // End of a super-pass: q += sum_i V^2 over this group's share of my pass's columns.  It runs only
            // after the group has generated its first chunk of the NEXT super-pass (the ring has one slot per
            // group of the pair), so that the variance MMAs find k* waiting when the accumulator is free again.
            bool epilogue_due = false;
            auto pass_epilogue = [&]() {
                TICK(7);
                ok = mbar_wait(bar(PB_V_FULL), v_ph, abort_flag, wl);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return;
                TICK(5);
                tc_fence_after();
#pragma unroll 1
                for (int c0 = grp * 16; c0 < NV2; c0 += 32 * G2) {   // two column blocks per round trip to TMEM
                    const int c1 = c0 + 16 * G2;
                    float v[16], w[16];
                    float part0 = 0.f, part1 = 0.f;
                    tc_ld16_issue(lane_addr + c0, v);
                    tc_ld16_issue(lane_addr + c1, w);
                    tc_wait_ld32(v, w);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        part0 = fmaf(v[i], v[i], part0);
                        part1 = fmaf(w[i], w[i], part1);
                    }
                    q_acc += (double)part0;
                    q_acc += (double)part1;
                }
                tc_fence_before();
                mbar_arrive(bar(PB_V_EMPTY));
                v_ph ^= 1u;
                TICK(6);
            };
            for (int j = 0; ok && j < NSP; ++j) {
                const int nchunk = superpass_chunks(j, P);
                const int nprod = nchunk / SL2;
                for (int u = 0; u < nprod; ++u, ++Ug) {
                    if ((uint32_t)(Ug & 1) != rank) continue;
                    const int c = u * SL2 + grp;            // my chunk of this product, within the super-pass
                    const long long t = tg + c;             // global chunk number: ring position and phase
                    const int b = (int)(t % NB);
                    const uint32_t k_par = (uint32_t)((t / NB) & 1);
                    const int db = (int)(own & 1);
                    TICK(7);
                    ok = mbar_wait(bar(PB_D_FULL + db), (uint32_t)((own >> 1) & 1), abort_flag, wl);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    TICK(0);
                    if (q4 == 0 && lane == 0) LOGEV2(3, t);
                    ++own;
                    tc_fence_after();
                    const bool fresh = c >= 2 * j * CPP2;   // first super-pass that generates this chunk
                    uint8_t* kb = sm + map.k + b * 16384u + row * 16;
                    uint32_t kh[KC / 16][8], kl[KC / 16][8];
                    // both halves of the chunk's dot products in one round trip to TMEM, then the buffer is free
                    float dots[KC / 16][16];
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h) tc_ld16_issue(lane_addr + NV2 + db * KD2 + grp * KC + h * 16, dots[h]);
                    tc_wait_ld32(dots[0], dots[1]);
                    tc_fence_before();
                    mbar_arrive(bar(PB_D_EMPTY + db));
                    TICK(1);
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h) {
                        const float* dot = dots[h];
                        float kv[16];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 xn4 = __ldg(reinterpret_cast<const float4*>(xn_g + c * KC + h * 16 + 4 * q));
                            const float xn[4] = {xn4.x, xn4.y, xn4.z, xn4.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float uu = sqrt_approx(fabsf(fmaf(-2.f, dot[4 * q + e], zn + xn[e])));
                                kv[4 * q + e] = fmaf(uu, fmaf(uu, pc2, pc1), pc0) * exp2_approx(-uu);
                            }
                        }
                        float vmax = fmaxf(fmaxf(kv[0], kv[1]), fmaxf(kv[2], kv[3]));
#pragma unroll
                        for (int i = 4; i < 16; i += 4)
                            vmax = fmaxf(vmax, fmaxf(fmaxf(kv[i], kv[i + 1]), fmaxf(kv[i + 2], kv[i + 3])));
                        if (__any_sync(0xffffffffu, vmax > v_thresh)) {
                            float tmp[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) tmp[i] = kv[i];
                            refine_close_pairs<false>(tmp, v_thresh, kvscale, lane_addr + ZCOL, DP, xs_g + (size_t)(c * KC + h * 16) * DP, nullptr, 0u, false);
#pragma unroll
                            for (int i = 0; i < 16; ++i) kv[i] = tmp[i];
                        }
                        if (fresh) {
                            float mpart = 0.f, apart = 0.f, spart = 0.f;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float4 al4 = __ldg(reinterpret_cast<const float4*>(al_g + c * KC + h * 16 + 4 * q));
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
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            __half2 hi, lo;
                            split2(kv[2 * e], kv[2 * e + 1], hi, lo);
                            kh[h][e] = *reinterpret_cast<const uint32_t*>(&hi);
                            kl[h][e] = *reinterpret_cast<const uint32_t*>(&lo);
                        }
                    }
                    // both CTAs must have finished with the previous chunk in this ring position
                    TICK(2);
                    if (q4 == 0 && lane == 0) LOGEV2(4, t);
                    ok = mbar_wait_cluster(bar(PB_K_EMPTY + b), k_par ^ 1u, abort_flag, wl);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    TICK(3);
                    if (q4 == 0 && lane == 0) LOGEV2(5, t);
                    // the peer's barrier learns of the 16 KB to come now: the remote arrive takes hundreds of cycles,
                    // which pass while this group stores the chunk
                    if (q4 == 1 && lane == 0) mbar_arrive_expect_tx_cluster(k_full_peer0 + (uint32_t)b * 8u, 16384u);
#pragma unroll
                    for (int h = 0; h < KC / 16; ++h) {
#pragma unroll
                        for (int sl = 0; sl < 2; ++sl) {
                            *reinterpret_cast<uint4*>(kb + (2 * h + sl) * 2048u) =
                                make_uint4(kh[h][4 * sl], kh[h][4 * sl + 1], kh[h][4 * sl + 2], kh[h][4 * sl + 3]);
                            *reinterpret_cast<uint4*>(kb + 8192u + (2 * h + sl) * 2048u) =
                                make_uint4(kl[h][4 * sl], kl[h][4 * sl + 1], kl[h][4 * sl + 2], kl[h][4 * sl + 3]);
                        }
                    }
                    if (!ok) break;
                    // The chunk is complete in this CTA's buffer: publish it here, and send a copy to the
                    // same ring position of the peer with one bulk copy that completes the peer's barrier.
                    if (q4 == 0 && lane == 0) LOGEV2(7, t);
                    fence_proxy_async();
                    if (q4 == 0 && lane == 0) LOGEV2(8, t);
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory");
                    if (q4 == 0 && lane == 0) {
                        LOGEV2(9, t);
                        mbar_arrive(bar(PB_K_FULL + b));
                        const uint32_t peer_bar = k_full_peer0 + (uint32_t)b * 8u;
                        LOGEV2(10, t);
                        bulk_s2peer(kbuf_peer0 + b * 16384u, base + map.k + b * 16384u, 16384u, peer_bar);
                        LOGEV2(6, t);
                    }
                    TICK(4);
                    if (epilogue_due) {   // the previous super-pass's accumulator, now that the next k* is on its way
                        epilogue_due = false;
                        pass_epilogue();
                        if (!ok) break;
                    }
                }
                if (!ok) break;
                tg += nchunk;
                epilogue_due = 2 * j + (int)rank < P;
            }
            if (ok && epilogue_due) pass_epilogue();
            if (!ok) break;
            // ---- combine: groups within the CTA, then CTA 1 -> CTA 0, which finishes the candidate
            double* mine = red + ((size_t)grp * TILE_M + row) * 4;
            mine[0] = mu_acc; mine[1] = a2_acc; mine[2] = s2_acc; mine[3] = q_acc;
            mbar_arrive(bar(PB_RED_READY));
            if (grp == 0) {
                ok = mbar_wait(bar(PB_RED_READY), (uint32_t)(tile_iter & 1), abort_flag, wl);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                mu_acc = a2_acc = s2_acc = q_acc = 0.0;
#pragma unroll
                for (int gg = 0; gg < G2; ++gg) {
                    const double* o = red + ((size_t)gg * TILE_M + row) * 4;
                    mu_acc += o[0]; a2_acc += o[1]; s2_acc += o[2]; q_acc += o[3];
                }
                if (rank == 1) {
                    const uint32_t slot = map_to_cta(base + map.red + (uint32_t)((G2 * TILE_M + row) * 32), 0);
                    st_cluster_f64(slot, mu_acc);
                    st_cluster_f64(slot + 8, a2_acc);
                    st_cluster_f64(slot + 16, s2_acc);
                    st_cluster_f64(slot + 24, q_acc);
                    mbar_arrive_cluster(map_to_cta(bar(PB_RED_PEER), 0));
                } else {
                    ok = mbar_wait_cluster(bar(PB_RED_PEER), (uint32_t)(tile_iter & 1), abort_flag, wl);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    if (valid) {
                        const double* o = red + ((size_t)G2 * TILE_M + row) * 4;
                        mu_acc += o[0]; a2_acc += o[1]; s2_acc += o[2]; q_acc += o[3];
                        q_acc *= prm.vinv2[g];
                        const size_t f = (size_t)g * prm.m + cand;
                        const CandidateResult res = finalize_candidate(mu_acc, q_acc, (double)sf2, (double)prm.best[g]);
                        prm.mu[f] = res.mu;
                        prm.sigma[f] = res.sigma;
                        prm.ei[f] = res.ei;
                        const double eps =
                            far_cand ? 1.0 : kEpsTc0 + kEpsTc1 * (double)(zn + prm.xnmax[g]) * rsqrt((double)DP);
                        prm.err_mu[f] = mu_error_estimate(eps, a2_acc);
                        prm.err_q[f] = q_error_estimate(eps, prm.wnorm[g], q_acc, s2_acc);
                    }
                }
            }
        }
        if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(prm.status, DEV_NONFINITE);
        if (prm.trace && q4 == 0 && lane == 0)
            for (int i = 0; i < 8; ++i) prm.trace[((size_t)blockIdx.x * 4 + 1 + grp) * 8 + i] = tacc[i];
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(prm.status, DEV_TIMEOUT);
    cluster_sync_all();   // the peer may still be writing into this CTA's shared memory until it gets here
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

// Whether the paired kernel serves this handle: at least two passes, and a shape that fits.
bool tc_pair_fits(const TensorOperands* t, int* ws_out)
{
    if (t->NV != NV2 || t->KD != KD2 || t->P < 2) return false;
    if (NV2 + 2 * KD2 + t->DP > 512) return false;
    const size_t budget = 227 * 1024 - 1024 - kPairBarBytes;
    int ws;
    for (ws = MAX_WS2; ws >= 2; --ws)
        if (pair_map(t->DP, ws).bar <= budget) break;
    if (ws < 2) return false;
    *ws_out = ws;
    return true;
}

r3_status_t launch_tc_pair(const TensorOperands* t, TcParams prm, int sms, cudaStream_t stream)
{
    int ws = 0;
    if (!tc_pair_fits(t, &ws)) {
        set_error("internal: paired tensor kernel does not fit this shape");
        return R3_ERR_UNSUPPORTED;
    }
    prm.ws = ws;
    const size_t smem = pair_map(t->DP, ws).bar + kPairBarBytes + 1024;
    R3_CUDA_TRY(cudaFuncSetAttribute(score_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long clusters = sms / 2;
    if (clusters > prm.total_tiles) clusters = prm.total_tiles;
    if (clusters < 1) clusters = 1;
    score_tc_pair_kernel<<<(unsigned)(2 * clusters), 128 + 128 * G2, smem, stream>>>(prm);
    ++g_launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("launch of score_tc_pair_kernel failed: %s", cudaGetErrorString(e));
        return R3_ERR_CUDA;
    }
    return R3_OK;
}

}  // namespace r3
