// Accuracy guard, FP64 rescue pass and the first level of the pool's top-k, in one kernel.
//
// The scoring engines work at FP32 level.  That is enough for almost every candidate of a
// well-conditioned GP, but not where the posterior variance sf2 - |W k*|^2 is a small difference of
// two numbers close to sf2 (a candidate on top of an observation), nor where mu = k*.alpha cancels
// heavily (an ill-conditioned history with large weights).  Each engine therefore writes, next to
// its results, an estimate of its own rounding error in mu and in q, and raises the pool's largest EI
// (the EI tolerance is relative to it) with one atomic maximum per warp.  Once the whole pool is scored,
// guard_kernel gives every block a slice of candidates, and the block
//   flags    the candidates of its slice whose estimated error exceeds half of the accuracy contract
//            (1e-4 relative on mu and sigma with absolute floors, 1e-5 max(EI) on EI),
//   rescues  them: recomputes them from the raw inputs entirely in FP64 -- direct-difference distances with
//            FP64 reciprocal lengthscales, FP64 weights and the FP64 inverse factor -- and overwrites
//            their mu, sigma and EI,
//   selects  (when the call asked for a top-k) the k largest final EI of its slice as 64-bit keys: the first
//            level of the selection, taken while the slice's values are at hand; r3_topk.cu finishes it.
#include "r3_epilogue.cuh"
#include "r3_internal.cuh"
#include "r3_topk.cuh"

namespace r3 {

namespace {

constexpr int RESCUE_GROUP = 4;   // candidates recomputed together (they share every read of W)

struct GuardArgs {
    const float *X, *ell, *sf2v, *bestv, *yabsv, *Xcand;
    const double *alpha64, *W64;
    int n, d, npad;
    long long m;
    int slice;                    // candidates per block, a power of two in [32, 4096]
    float *mu, *sigma, *ei;
    const float *err_mu, *err_q;
    const unsigned* maxbits;      // [batch] bit pattern of the pool's largest EI
    int* count;                   // [batch] candidates recomputed (diagnostics)
    int* status;                  // the handle's status words (index checks of the bounds-checking build)
    int k, K2;                    // top-k request (k = 0: none); K2 = min(k, slice): keys a block selects
    unsigned select_offset;       // byte offset of the selection's scratch in the dynamic shared memory
    unsigned long long* keys;     // [batch][blocks][k]
};

// The pool's largest EI for an engine whose scoring kernel does not raise it itself (the tensor-core kernel's
// registers are spoken for).
__global__ void max_ei_kernel(const float* __restrict__ ei, long long m, unsigned* __restrict__ maxbits)
{
    const int g = blockIdx.y;
    const float* e = ei + (size_t)g * m;
    float v = 0.f;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x)
        v = fmaxf(v, e[i]);  // EI >= 0; NaN is ignored by fmaxf
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) atomicMax(&maxbits[g], __float_as_uint(v));  // order-preserving for v >= 0
}

template <int R>
__global__ void __launch_bounds__(256) guard_kernel(const GuardArgs a)
{
    extern __shared__ double smem[];
    // rescue: ks [R][npad], zs [R][d], ls [d]; afterwards the same bytes hold the slice's keys
    double* ks = smem;
    double* zs = smem + (size_t)R * a.npad;
    double* ls = zs + (size_t)R * a.d;   // [d] reciprocal lengthscales
    __shared__ double red[2][R][8];
    __shared__ int nflag_s;
    const int g = blockIdx.y;
    const int t = threadIdx.x, lane = t % 32, warp = t / 32;
    const long long m = a.m;
    const long long c_begin = (long long)blockIdx.x * a.slice;
    const long long c_end = c_begin + a.slice < m ? c_begin + a.slice : m;
    // the list of flagged candidates sits after the larger of the two uses of the dynamic region
    size_t region = sizeof(double) * ((size_t)R * a.npad + (size_t)R * a.d + a.d);
    if (region < sizeof(unsigned long long) * (size_t)a.slice) region = sizeof(unsigned long long) * (size_t)a.slice;
    int* list = reinterpret_cast<int*>(reinterpret_cast<char*>(smem) + region);
    if (t == 0) nflag_s = 0;
    __syncthreads();

    // ---- flag
    {
        const float sf2 = a.sf2v[g], best = a.bestv[g];
        const float tol_ei = 1e-5f * __uint_as_float(a.maxbits[g]);
        const float mu_floor = 1e-6f * a.yabsv[g], sd_floor = 1e-6f * sqrtf(sf2);
        for (long long i = c_begin + t; i < c_end; i += 256) {
            const size_t f = (size_t)g * m + i;
            const float mu_i = a.mu[f], sd = a.sigma[f], dmu = a.err_mu[f], dq = a.err_q[f];
            // d sigma = dq / (2 sigma); with sigma -> 0 every rounding error in q matters
            const float dsd = (sd > 0.f) ? dq / (2.f * sd) : ((dq > 0.f) ? INFINITY : 0.f);
            const float tol_mu = 1e-4f * fabsf(mu_i) + mu_floor;
            const float tol_sd = 1e-4f * sd + sd_floor;
            bool flag = !(dmu <= 0.5f * tol_mu) || !(dsd <= 0.5f * tol_sd);
            // EI: dEI = Phi(z) dmu + phi(z) dsigma against 1e-5 of the pool's largest EI
            const float z = (sd > 0.f) ? (best - mu_i) / sd : 0.f;
            const float Phi = 0.5f * erfcf(-z * 0.70710678f);
            const float phi = expf(-0.5f * z * z) * 0.39894228f;
            if (isfinite(dsd)) flag |= !(Phi * dmu + phi * dsd <= 0.5f * tol_ei);
            flag |= !(sd * sd >= 1e-3f * sf2);   // deep cancellation: do not trust the estimates either
            if (flag) list[R3_IDX(atomicAdd(&nflag_s, 1), a.slice, a.status)] = (int)i;
        }
    }
    __syncthreads();
    const int total = nflag_s;
    if (t == 0 && total > 0) atomicAdd(&a.count[g], total);

    // ---- rescue
    if (total > 0) {
        const float* Xg = a.X + (size_t)g * a.n * a.d;
        const double* Wg = a.W64 + (size_t)g * a.npad * a.npad;
        const double* ag = a.alpha64 + (size_t)g * a.npad;
        const double sf2 = (double)a.sf2v[g];
        const int n = a.n, d = a.d, npad = a.npad;
        // reciprocal lengthscales in FP64: one rounding of 2^-53 per difference against an FP64 division per
        // difference (the divisions were most of a rescue's time at d = 128)
        for (int j = t; j < d; j += 256) ls[j] = 1.0 / (double)a.ell[(size_t)g * d + j];
        for (int e0 = 0; e0 < total; e0 += R) {
            const int nr = min(R, total - e0);
            __syncthreads();
            for (int e = t; e < R * d; e += 256) {
                const int r = e / d, j = e % d;
                const int c = list[R3_IDX(e0 + min(r, nr - 1), a.slice, a.status)];
                zs[e] = (double)a.Xcand[(size_t)R3_IDX((long long)g * m + c, (long long)gridDim.y * m, a.status) * d + j];
            }
            __syncthreads();
            double mu_part[R];
#pragma unroll
            for (int r = 0; r < R; ++r) mu_part[r] = 0.0;
            for (int i = t; i < n; i += 256) {
                double r2[R];
#pragma unroll
                for (int r = 0; r < R; ++r) r2[r] = 0.0;
                for (int j = 0; j < d; ++j) {
                    const double x = (double)Xg[(size_t)i * d + j], il = ls[j];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double df = (x - zs[r * d + j]) * il;
                        r2[r] += df * df;
                    }
                }
                const double al = ag[i];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const double sq = sqrt(5.0) * sqrt(r2[r]);
                    const double kv = sf2 * (1.0 + sq + sq * sq / 3.0) * exp(-sq);
                    ks[(size_t)R3_IDX((long long)r * npad + i, (long long)R * npad, a.status)] = kv;
                    mu_part[r] += kv * al;
                }
            }
            __syncthreads();
            double q_part[R];
#pragma unroll
            for (int r = 0; r < R; ++r) q_part[r] = 0.0;
            for (int i = warp; i < n; i += 8) {
                const double* Wr = Wg + (size_t)i * npad;
                double v[R];
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = 0.0;
                for (int kk = lane; kk <= i; kk += 32) {
                    const double w = Wr[kk];
#pragma unroll
                    for (int r = 0; r < R; ++r) v[r] += w * ks[(size_t)r * npad + kk];
                }
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    for (int o = 16; o > 0; o >>= 1) v[r] += __shfl_xor_sync(0xffffffffu, v[r], o);
                    q_part[r] += v[r] * v[r];  // identical in every lane; lane 0's copy is used
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                for (int o = 16; o > 0; o >>= 1) mu_part[r] += __shfl_xor_sync(0xffffffffu, mu_part[r], o);
                if (lane == 0) {
                    red[0][r][warp] = mu_part[r];
                    red[1][r][warp] = q_part[r];
                }
            }
            __syncthreads();
            if (t < nr) {
                double mu_s = 0.0, q = 0.0;
                for (int w = 0; w < 8; ++w) {
                    mu_s += red[0][t][w];
                    q += red[1][t][w];
                }
                const size_t f = (size_t)R3_IDX((long long)g * m + list[e0 + t], (long long)gridDim.y * m, a.status);
                const CandidateResult res = finalize_candidate(mu_s, q, sf2, (double)a.bestv[g]);
                a.mu[f] = res.mu;
                a.sigma[f] = res.sigma;
                a.ei[f] = res.ei;
            }
        }
    }
    if (a.k == 0) return;

    // ---- the k largest final EI of the slice (the rescued values were written by this block)
    __syncthreads();
    unsigned long long* keys_s = reinterpret_cast<unsigned long long*>(smem);
    const float* e = a.ei + (size_t)g * m;
    for (int i = t; i < a.slice; i += 256) {
        const long long c = c_begin + i;
        keys_s[i] = (c < m) ? topk_make_key(e[c], (unsigned)c) : 0ull;
    }
    block_select_desc(keys_s, a.slice, a.K2, reinterpret_cast<char*>(smem) + a.select_offset);
    unsigned long long* out = a.keys + ((size_t)g * gridDim.x + blockIdx.x) * a.k;
    for (int i = t; i < a.k; i += 256) out[i] = i < a.slice ? keys_s[R3_IDX(i, a.slice, a.status)] : 0ull;
}

}  // namespace

size_t guard_workspace_bytes(const r3_gp* gp, long long m)
{
    const size_t bm = (size_t)gp->batch * m;
    return 2 * bm * sizeof(float) + 2 * (size_t)gp->batch * sizeof(int) + 256;
}

GuardBuffers guard_carve(const r3_gp* gp, long long m, void* ws)
{
    GuardBuffers b;
    const size_t bm = (size_t)gp->batch * m;
    char* p = (char*)ws;
    b.err_mu = (float*)p;
    p += bm * sizeof(float);
    b.err_q = (float*)p;
    p += bm * sizeof(float);
    b.count = (int*)p;
    p += (size_t)gp->batch * sizeof(int);
    b.maxbits = (unsigned*)p;
    return b;
}

// Candidates per block of the guard kernel: enough blocks to fill the GPU on a large pool, small slices on a
// small one (a power of two: the slice is also the chunk of the first top-k level).
int guard_slice(long long m, int k)
{
    long long s = k > 32 ? 128 : 32;   // small pools: many blocks (the rescues of a block run one after another)
    while (s < 4096 && s * 148 < m) s <<= 1;
    return (int)s;
}

size_t guard_topk_workspace_bytes(int batch, long long m, int k)
{
    const long long blocks = (m + guard_slice(m, k) - 1) / guard_slice(m, k);
    return 2 * (size_t)batch * blocks * k * sizeof(unsigned long long) + 64;
}

r3_status_t guard_begin(r3_gp* gp, const GuardBuffers& b, cudaStream_t stream)
{
    R3_CUDA_TRY(cudaMemsetAsync(b.count, 0, 2 * (size_t)gp->batch * sizeof(int), stream));  // count and maxbits
    return R3_OK;
}

r3_status_t guard_and_rescue(r3_gp* gp, const float* Xcand, long long m, const GuardBuffers& b, float* mu,
                             float* sigma, float* ei, bool have_max, cudaStream_t stream)
{
    const int B = gp->batch;
    if (!have_max) {
        const unsigned gx = (unsigned)((m + 1023) / 1024);
        R3_LAUNCH(max_ei_kernel, dim3(gx < 592u ? gx : 592u, B), 256, 0, stream, ei, m, b.maxbits);
    }
    const TopkRequest req = gp->topk_req;
    gp->topk_req = TopkRequest();
    GuardArgs a;
    a.X = gp->X; a.ell = gp->ell_d; a.sf2v = gp->sf2_d; a.bestv = gp->best_d; a.yabsv = gp->yabs_d; a.Xcand = Xcand;
    a.alpha64 = gp->alpha64; a.W64 = gp->W64;
    a.n = gp->n; a.d = gp->d; a.npad = gp->npad;
    a.m = m;
    a.slice = guard_slice(m, req.k);
    a.mu = mu; a.sigma = sigma; a.ei = ei;
    a.err_mu = b.err_mu; a.err_q = b.err_q;
    a.maxbits = b.maxbits;
    a.count = b.count;
    a.status = gp->status_d;
    a.k = req.k;
    a.K2 = req.k > 0 ? std::min(req.k, a.slice) : 1;   // keys a block selects
    a.keys = (unsigned long long*)req.ws;
    const long long blocks = (m + a.slice - 1) / a.slice;
    if (req.k > 0 && req.ws_bytes < guard_topk_workspace_bytes(B, m, req.k)) {
        set_error("internal: top-k workspace of the guard too small");
        return R3_ERR_INVALID_ARG;
    }
    const int R = gp->npad <= 4096 ? RESCUE_GROUP : 1;
    size_t region = sizeof(double) * ((size_t)R * gp->npad + (size_t)R * gp->d + gp->d);
    region = std::max(region, sizeof(unsigned long long) * (size_t)a.slice);
    // after the flag list (unused by then, but kept apart): the scratch of the slice's top-k selection
    a.select_offset = (unsigned)((region + sizeof(int) * (size_t)a.slice + 7) & ~(size_t)7);
    const size_t smem = a.select_offset + (req.k > 0 ? topk_select_scratch_bytes(a.K2) : 0);
    if (R == RESCUE_GROUP) {
        if (smem + 1024 > 48 * 1024)   // the kernel's static shared memory counts against the same limit
            R3_CUDA_TRY(cudaFuncSetAttribute(guard_kernel<RESCUE_GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        R3_LAUNCH(guard_kernel<RESCUE_GROUP>, dim3((unsigned)blocks, B), 256, smem, stream, a);
    } else {
        if (smem + 1024 > 48 * 1024)   // the kernel's static shared memory counts against the same limit
            R3_CUDA_TRY(cudaFuncSetAttribute(guard_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        R3_LAUNCH(guard_kernel<1>, dim3((unsigned)blocks, B), 256, smem, stream, a);
    }
    R3_CUDA_TRY(cudaMemcpyAsync(gp->rescued_h, b.count, sizeof(int) * (B < 64 ? B : 64), cudaMemcpyDeviceToHost,
                                stream));
    if (req.k == 0) return R3_OK;
    unsigned long long* keys = (unsigned long long*)req.ws;
    return topk_finish_from_keys(keys, keys + (size_t)B * blocks * req.k, B, blocks * req.k, req.k, ei, m, req.idx,
                                 req.val, stream);
}

}  // namespace r3
