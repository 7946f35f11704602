// Tensor-core path of libdarkattn: bf16 operands, fp32 accumulation, tcgen05.mma with TMEM accumulators,
// operands staged by TMA (128-byte swizzle), exponentials fused into the TMEM read-out.
//
// Work decomposition. Features are cut into slabs of 128; one CTA owns one (batch, head, slab). Every
// quantity of the attention is a sum over features, so a slab CTA produces, for its 128 features, the
// partial numerator rows, the partial normaliser and the exponent its rows were scaled by; a small
// combine kernel adds the slabs. Per 128-token tile a slab CTA computes
//     U = X Omega_slab^T            Omega = log2(e) s W M folded once per call (u = w.(sMx) = (sM^T w).x)
//     phi(Q) = 2^(U - rowmax U)     any per-row factor cancels in O, including exp(-|Mq|^2/2)
//     phi(K) = 2^(U - n - c)        n = log2(e) |sMk|^2/2 per key (from the norms kernel), c per slab
// and then, causal:   P = tril(phi(Q) phi(K)^T),  O = P V + phi(Q) S_prev,  S += phi(K)^T V,  z += phi(K)^T 1
// with the state S (128 x dv, fp32) resident in TMEM across the chunks of the sequence;
// non-causal: a key pass accumulates S and z over all keys, a query pass applies them.
#include "common.cuh"
#include "tc_common.cuh"

#include <math.h>
#include <string.h>

namespace darkattn {

using namespace tc;

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxNsplit = 64;

// ------------------------------------------------------------------ small helpers
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// ------------------------------------------------------------------ prologue kernels (SIMT, tiny)
// Omega[h,l,c] = log2(e) * s * sum_a W[l,a] M[h,a,c]  (bf16);  one block per (h, l).
__global__ void fold_omega_kernel(const __nv_bfloat16 *W, const __nv_bfloat16 *M, __nv_bfloat16 *Om, int m, int r, int d,
                                  int w_per_head, float coef)
{
    const int h = blockIdx.y, l = blockIdx.x;
    const __nv_bfloat16 *w = W + ((size_t)(w_per_head ? h : 0) * m + l) * r;
    const __nv_bfloat16 *Mh = M + (size_t)h * r * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float acc = 0.f;
        for (int a = 0; a < r; ++a) acc = fmaf(__bfloat162float(w[a]), __bfloat162float(Mh[(size_t)a * d + c]), acc);
        Om[((size_t)h * m + l) * d + c] = __float2bfloat16_rn(coef * acc);
    }
}

// Key-side shift of a slab, in log2 units: c = log2(e) * max(0, max_l |w_l|^2/2 - 40).
// u - n <= |w_l|^2 / 2 for every key (complete the square), so phi(K) <= e^40 whatever the data.
// One block per (bh, slab), 128 threads.
__global__ void slab_shift_kernel(const __nv_bfloat16 *W, float *cs, int H, int m, int r, int nslab, int w_per_head)
{
    const int bh = blockIdx.x / nslab, slab = blockIdx.x % nslab, h = bh % H;
    const __nv_bfloat16 *w = W + ((size_t)(w_per_head ? h : 0) * m + (size_t)slab * 128 + threadIdx.x) * r;
    float acc = 0.f;
    for (int a = 0; a < r; ++a) { const float v = __bfloat162float(w[a]); acc = fmaf(v, v, acc); }
    acc *= 0.5f;
    __shared__ float red[128];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 64; o; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + o]); __syncthreads(); }
    if (threadIdx.x == 0) cs[blockIdx.x] = kLog2e * fmaxf(0.f, red[0] - 40.f);
}

// ------------------------------------------------------------------ key norms: n[bh,j] = coef * |M_h k_j|^2
struct NormParams {
    CUtensorMap mapK, mapM;
    float *nK;
    int *status;
    int N, H, T, nsplit, r;
    float coef;   // log2(e) * s^2 / 2
};

template <int D>
__global__ void __launch_bounds__(160, 1) tc_key_norms_kernel(const __grid_constant__ NormParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kTile = 128 * D * 2;
    unsigned char *sM = smem, *sK = smem + kTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 2 * kTile);
    uint64_t *bar_m = bars, *bar_k = bars + 1, *bar_u = bars + 2, *bar_e = bars + 3;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 5);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    if (tid == 0) {
        mbar_init(bar_m, 1); mbar_init(bar_k, 1); mbar_init(bar_u, 1); mbar_init(bar_e, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(tmem_slot, 128); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (*abort_flag) { if (tid == 0) atomicExch(p.status, (int)DARKATTN_ERR_CUDA); }
    else if (warp == 4) {
        if ((tid & 31) == 0 && t1 > t0) {
            mbar_expect_tx(bar_m, kTile);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sM + a * 16384, &p.mapM, bar_m, a * 64, h * p.r);
            mbar_expect_tx(bar_k, kTile);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sK + a * 16384, &p.mapK, bar_k, a * 64, bh * p.N + t0 * 128);
            const uint32_t idesc = make_idesc(128, p.r, 0, 0);
            bool ok = wait_or_abort(bar_m, 0, p.status, abort_flag);
            for (int t = t0; t < t1 && ok; ++t) {
                const uint32_t ph = (t - t0) & 1;
                ok = wait_or_abort(bar_k, ph, p.status, abort_flag);
                if (ok && t > t0) ok = wait_or_abort(bar_e, ph ^ 1, p.status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k)
                    mma_ss(tmem, make_sdesc(smem_u32(sK) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024),
                           make_sdesc(smem_u32(sM) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024), idesc, k > 0);
                mma_commit(bar_u);
                if (t + 1 < t1) {
                    ok = wait_or_abort(bar_u, ph, p.status, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar_k, kTile);
                    for (int a = 0; a < D / 64; ++a)
                        tma_load_2d(sK + a * 16384, &p.mapK, bar_k, a * 64, bh * p.N + (t + 1) * 128);
                }
            }
        }
    } else {
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        for (int t = t0; t < t1; ++t) {
            const uint32_t ph = (t - t0) & 1;
            if (!wait_or_abort(bar_u, ph, p.status, abort_flag)) break;
            tc_fence_after();
            float acc = 0.f;
            for (int c0 = 0; c0 < p.r; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) { const float x = __uint_as_float(v[j]); acc = fmaf(x, x, acc); }
            }
            tc_fence_before();
            mbar_arrive(bar_e);
            p.nK[(size_t)bh * p.N + (size_t)t * 128 + tid] = p.coef * acc;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 128);
}

// ------------------------------------------------------------------ the main kernel
struct MainParams {
    CUtensorMap mapQ, mapK, mapV, mapOm, mapSb, mapPN;
    const float *nK;     // [BH, N]      key norms in log2 units
    const float *cs;     // [BH, nslab]  key-side shift per slab (log2 units)
    float *pdr;          // [nslab, BH*N, 2]  partial normaliser and the exponent the partial is scaled by
    float *Sacc;         // [BH, m, DV]  fp32 state sums (non-causal key pass, atomics)
    float *zacc;         // [BH, m]
    int *status;
    int N, H, BH, m, nslab, T, nsplit;
};

enum { MODE_CAUSAL = 0, MODE_KEYS = 1, MODE_QUERIES = 2 };

template <int D, int DV, int MODE>
struct SmemLayout {
    static constexpr int kOm = 0;
    static constexpr int kQ = kOm + 128 * D * 2;
    static constexpr int kK = kQ + 128 * D * 2;                                  // also the masked P tile (causal)
    static constexpr int kKBytes = (MODE == MODE_CAUSAL && D < 128) ? 32768 : 128 * D * 2;
    static constexpr int kV = kK + kKBytes;
    static constexpr int kFQ = kV + 128 * DV * 2;                                // also the output staging tile
    static constexpr int kFK = kFQ + 32768;
    static constexpr int kSb = kFK + 32768;
    static constexpr int kOnes = kSb + 128 * DV * 2;
    static constexpr int kZ = kOnes + 2048;
    static constexpr int kBars = kZ + 512;
    static constexpr int kTotal = kBars + 192;
};

// TMEM columns (512 allocated): state S at 0 (DV columns), z at DV (16), R1 at 256, R2 at 384 (128 each).
constexpr uint32_t kColS = 0, kColR1 = 256, kColR2 = 384;

template <int D, int DV, int MODE>
__global__ void __launch_bounds__(160, 1) tc_attn_kernel(const __grid_constant__ MainParams p)
{
    using L = SmemLayout<D, DV, MODE>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sQ = smem + L::kQ, *sK = smem + L::kK, *sV = smem + L::kV;
    unsigned char *sFQ = smem + L::kFQ, *sFK = smem + L::kFK, *sSb = smem + L::kSb, *sOnes = smem + L::kOnes;
    unsigned char *sP = sK, *sStage = sFQ;
    float *sZ = reinterpret_cast<float *>(smem + L::kZ);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint64_t *bar_om = bars + 0, *bar_q = bars + 1, *bar_k = bars + 2, *bar_v = bars + 3, *bar_uq = bars + 4,
             *bar_uk = bars + 5, *bar_p = bars + 6, *bar_o = bars + 7, *bar_s = bars + 8, *bar_eq = bars + 9,
             *bar_ek = bars + 10, *bar_ep = bars + 11, *bar_eo = bars + 12, *bar_es = bars + 13;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 14);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 15);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit;
    const int bh = unit / p.nslab, slab = unit % p.nslab, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    const int row0 = bh * p.N;                    // first row of this (b,h) in the [BH*N, *] views

    if (tid == 0) {
        for (int i = 0; i < 9; ++i) mbar_init(bars + i, 1);
        for (int i = 9; i < 14; ++i) mbar_init(bars + i, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) {   // 2 KB of bf16 ones: B operand of the z += phi(K)^T 1 MMAs
        *reinterpret_cast<uint4 *>(sOnes + tid * 16) = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
        fence_async_smem();
    }
    if (warp == 4) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (t1 <= t0) {
        // nothing to do for this split
    } else if (warp == 4) {
        // ============================== control thread: TMA loads and MMA issue
        if ((tid & 31) == 0) {
            constexpr uint32_t kXBytes = 128 * D * 2, kVBytes = 128 * DV * 2;
            auto load_x = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int t) {
                mbar_expect_tx(bar, kXBytes);
                for (int a = 0; a < D / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, row0 + t * 128);
            };
            auto load_v = [&](int t) {
                mbar_expect_tx(bar_v, kVBytes);
                for (int a = 0; a < DV / 64; ++a) tma_load_2d(sV + a * 16384, &p.mapV, bar_v, a * 64, row0 + t * 128);
            };
            // K-major operand with K split over 64-element atoms: step k of 16 elements
            auto kdesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024); };
            // MN-major operand: 16 K-rows per step, 64-element blocks along M/N are 16 KB apart
            auto mndesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + k * 2048, 16384, 1024); };
            const uint32_t id_u = make_idesc(128, 128, 0, 0);     // U = X Omega^T, P = phi(Q) phi(K)^T
            const uint32_t id_o = make_idesc(128, DV, 0, 1);      // O += A[K-major] B[MN-major]
            const uint32_t id_s = make_idesc(128, DV, 1, 1);      // S += phi(K)^T V
            const uint32_t id_z = make_idesc(128, 16, 1, 1);      // z += phi(K)^T 1

            mbar_expect_tx(bar_om, 128 * D * 2 + (MODE == MODE_QUERIES ? 128 * DV * 2 : 0));
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sOm + a * 16384, &p.mapOm, bar_om, a * 64, h * p.m + slab * 128);
            if (MODE == MODE_QUERIES)
                for (int a = 0; a < DV / 64; ++a) tma_load_2d(sSb + a * 16384, &p.mapSb, bar_om, a * 64, bh * p.m + slab * 128);
            if (MODE != MODE_KEYS) load_x(sQ, &p.mapQ, bar_q, t0);
            if (MODE != MODE_QUERIES) { load_x(sK, &p.mapK, bar_k, t0); load_v(t0); }

            bool ok = wait_or_abort(bar_om, 0, status, abort_flag);
            for (int t = t0; t < t1 && ok; ++t) {
                const uint32_t ph = (t - t0) & 1;
                const bool first = (t == t0), last = (t + 1 == t1);
                if (MODE != MODE_KEYS) {            // U_Q -> R1
                    ok = wait_or_abort(bar_q, ph, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int k = 0; k < D / 16; ++k) mma_ss(tmem + kColR1, kdesc(sQ, k), kdesc(sOm, k), id_u, k > 0);
                    mma_commit(bar_uq);
                }
                if (MODE != MODE_QUERIES) {         // U_K -> R2
                    if (MODE == MODE_CAUSAL && !first) ok = wait_or_abort(bar_eo, ph ^ 1, status, abort_flag);
                    if (ok) ok = wait_or_abort(bar_k, ph, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int k = 0; k < D / 16; ++k) mma_ss(tmem + kColR2, kdesc(sK, k), kdesc(sOm, k), id_u, k > 0);
                    mma_commit(bar_uk);
                }
                if (MODE != MODE_KEYS) {            // the query tile is free once U_Q has run: prefetch the next
                    ok = wait_or_abort(bar_uq, ph, status, abort_flag);
                    if (!ok) break;
                    if (!last) load_x(sQ, &p.mapQ, bar_q, t + 1);
                }
                if (MODE == MODE_KEYS) {            // the key tile is free once U_K has run
                    ok = wait_or_abort(bar_uk, ph, status, abort_flag);
                    if (!ok) break;
                    if (!last) load_x(sK, &p.mapK, bar_k, t + 1);
                }
                if (MODE != MODE_KEYS) { ok = wait_or_abort(bar_eq, ph, status, abort_flag); if (!ok) break; }
                if (MODE != MODE_QUERIES) { ok = wait_or_abort(bar_ek, ph, status, abort_flag); if (!ok) break; }
                tc_fence_after();
                if (MODE == MODE_CAUSAL) {          // P = phi(Q) phi(K)^T -> R1
                    for (int k = 0; k < 8; ++k) mma_ss(tmem + kColR1, kdesc(sFQ, k), kdesc(sFK, k), id_u, k > 0);
                    mma_commit(bar_p);
                }
                bool o_started = false;
                if (MODE == MODE_QUERIES || (MODE == MODE_CAUSAL && !first)) {   // O = phi(Q) S_prev -> R2
                    if (MODE == MODE_CAUSAL) ok = wait_or_abort(bar_es, ph ^ 1, status, abort_flag);
                    if (MODE == MODE_QUERIES && !first) ok = wait_or_abort(bar_eo, ph ^ 1, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int k = 0; k < 8; ++k) mma_ss(tmem + kColR2, kdesc(sFQ, k), mndesc(sSb, k), id_o, k > 0);
                    o_started = true;
                }
                if (MODE == MODE_QUERIES) mma_commit(bar_o);
                if (MODE != MODE_QUERIES) {         // S += phi(K)^T V ; z += phi(K)^T 1
                    ok = wait_or_abort(bar_v, ph, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int k = 0; k < 8; ++k) mma_ss(tmem + kColS, mndesc(sFK, k), mndesc(sV, k), id_s, (!first) || k > 0);
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tmem + kColS + DV, mndesc(sFK, k), make_sdesc(smem_u32(sOnes), 16384, 1024), id_z, (!first) || k > 0);
                    mma_commit(bar_s);
                }
                if (MODE == MODE_CAUSAL) {          // O += P V
                    ok = wait_or_abort(bar_ep, ph, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int k = 0; k < 8; ++k) mma_ss(tmem + kColR2, kdesc(sP, k), mndesc(sV, k), id_o, o_started || k > 0);
                    mma_commit(bar_o);
                }
                if (MODE != MODE_QUERIES && !last) { // key (causal) and value tiles are free: load the next
                    if (MODE == MODE_CAUSAL) ok = wait_or_abort(bar_o, ph, status, abort_flag);
                    if (ok) ok = wait_or_abort(bar_s, ph, status, abort_flag);
                    if (!ok) break;
                    if (MODE == MODE_CAUSAL) load_x(sK, &p.mapK, bar_k, t + 1);
                    load_v(t + 1);
                }
            }
        }
    } else {
        // ============================== epilogue threads: thread = TMEM lane = tile row
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const float cshift = p.cs[bh * p.nslab + slab];
        const size_t prow0 = ((size_t)slab * p.BH + bh) * p.N;       // first row of this CTA's partial
        bool ok = true;
        if (MODE == MODE_QUERIES) sZ[tid] = p.zacc[(size_t)bh * p.m + slab * 128 + tid];
        if (MODE == MODE_CAUSAL) sZ[tid] = 0.f;
        for (int t = t0; t < t1 && ok; ++t) {
            const uint32_t ph = (t - t0) & 1;
            const bool first = (t == t0), last = (t + 1 == t1);
            float rmax = -INFINITY, dz = 0.f, rowsum = 0.f;
            // ---------------- phi(Q)
            if (MODE != MODE_KEYS) {
                ok = wait_or_abort(bar_uq, ph, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColR1 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) rmax = fmaxf(rmax, __uint_as_float(v[j]));
                }
                if (tid == 0) tma_store_wait_read();      // the staging tile (same memory) has been read out
                epi_bar_sync();                            // also: z of the previous chunk is visible
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t v[32], pk[16];
                    tmem_ld32(lane_addr + kColR1 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float f0 = ex2f(__uint_as_float(v[j]) - rmax), f1 = ex2f(__uint_as_float(v[j + 1]) - rmax);
                        dz = fmaf(f0, sZ[c0 + j], dz);
                        dz = fmaf(f1, sZ[c0 + j + 1], dz);
                        pk[j / 2] = pack_bf16(f0, f1);
                    }
                    unsigned char *atom = sFQ + (c0 / 64) * 16384;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(atom + swz128(tid, (c0 % 64) / 8 + q)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar_eq);
            }
            // ---------------- phi(K)
            if (MODE != MODE_QUERIES) {
                const float nk = p.nK[(size_t)bh * p.N + (size_t)t * 128 + tid] + cshift;
                if (MODE == MODE_KEYS && !first) ok = wait_or_abort(bar_s, ph ^ 1, status, abort_flag);
                if (ok) ok = wait_or_abort(bar_uk, ph, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t v[32], pk[16];
                    tmem_ld32(lane_addr + kColR2 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 2)
                        pk[j / 2] = pack_bf16(ex2f(__uint_as_float(v[j]) - nk), ex2f(__uint_as_float(v[j + 1]) - nk));
                    unsigned char *atom = sFK + (c0 / 64) * 16384;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(atom + swz128(tid, (c0 % 64) / 8 + q)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar_ek);
            }
            // ---------------- P = tril(phi(Q) phi(K)^T) as bf16 operand, and its row sums
            if (MODE == MODE_CAUSAL) {
                ok = wait_or_abort(bar_p, ph, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t v[32], pk[16];
                    tmem_ld32(lane_addr + kColR1 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float x0 = (c0 + j <= tid) ? __uint_as_float(v[j]) : 0.f;
                        const float x1 = (c0 + j + 1 <= tid) ? __uint_as_float(v[j + 1]) : 0.f;
                        rowsum += x0 + x1;
                        pk[j / 2] = pack_bf16(x0, x1);
                    }
                    unsigned char *atom = sP + (c0 / 64) * 16384;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(atom + swz128(tid, (c0 % 64) / 8 + q)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar_ep);
            }
            // ---------------- partial output rows
            if (MODE != MODE_KEYS) {
                ok = wait_or_abort(bar_o, ph, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int c0 = 0; c0 < DV; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColR2 + c0, v);
                    tmem_wait_ld();
                    unsigned char *atom = sStage + (c0 / 64) * 16384;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(atom + swz128(tid, (c0 % 64) / 8 + q)) =
                            make_uint4(pack_bf16(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1])),
                                       pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                       pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                       pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar_eo);
                epi_bar_sync();
                if (tid == 0) {
                    for (int a = 0; a < DV / 64; ++a) tma_store_2d(&p.mapPN, sStage + a * 16384, a * 64, (int)(prow0 + (size_t)t * 128));
                    tma_store_commit();
                }
                const float den = rowsum + dz;
                if (!(den > 0.f) || !isfinite(den)) atomicCAS(status, 0, (int)DARKATTN_ERR_NONFINITE);
                *reinterpret_cast<float2 *>(p.pdr + 2 * (prow0 + (size_t)t * 128 + tid)) = make_float2(den, rmax + cshift);
            }
            // ---------------- bf16 copy of the state for the next chunk's phi(Q) S_prev
            if (MODE == MODE_CAUSAL && !last) {
                ok = wait_or_abort(bar_s, ph, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int c0 = 0; c0 < DV; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColS + c0, v);
                    tmem_wait_ld();
                    unsigned char *atom = sSb + (c0 / 64) * 16384;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(atom + swz128(tid, (c0 % 64) / 8 + q)) =
                            make_uint4(pack_bf16(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1])),
                                       pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                       pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                       pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
                }
                {
                    uint32_t v[16];
                    tmem_ld16(lane_addr + kColS + DV, v);
                    tmem_wait_ld();
                    sZ[tid] = __uint_as_float(v[0]);
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar_es);
            }
        }
        if (MODE == MODE_KEYS && ok) {        // add this CTA's state to the global sums
            ok = wait_or_abort(bar_s, (t1 - 1 - t0) & 1, status, abort_flag);
            if (ok) {
                tc_fence_after();
                float *dst = p.Sacc + ((size_t)bh * p.m + slab * 128 + tid) * DV;
                for (int c0 = 0; c0 < DV; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColS + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) atomicAdd(dst + c0 + j, __uint_as_float(v[j]));
                }
                uint32_t v[16];
                tmem_ld16(lane_addr + kColS + DV, v);
                tmem_wait_ld();
                atomicAdd(p.zacc + (size_t)bh * p.m + slab * 128 + tid, __uint_as_float(v[0]));
            }
        }
        if (MODE != MODE_KEYS && tid == 0) tma_store_wait_all();
    }
    if (*abort_flag) __nanosleep(200000);   // error path only: let copies and MMAs in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// Sb[bh,l,:] = bf16(Sacc[bh,l,:])  (operand of the query pass)
__global__ void state_to_bf16_kernel(const float *S, __nv_bfloat16 *Sb, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        Sb[i] = __float2bfloat16_rn(S[i]);
}

// O[row,:] = sum_s num_s[row,:] 2^(rho_s - rho) / sum_s den_s 2^(rho_s - rho), rho = max_s rho_s.
// One thread per 8 output columns.
// The combined normaliser and rho are also written to sv (and to sv2 when given) for the backward pass.
__global__ void combine_kernel(const __nv_bfloat16 *pnum, const float *pdr, __nv_bfloat16 *O, float2 *sv, float2 *sv2,
                               long long rows, int dv, int nslab)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const int per_row = dv / 8;
    if (i >= rows * per_row) return;
    const long long row = i / per_row;
    const int c0 = (int)(i % per_row) * 8;
    float rho = -INFINITY;
    for (int s = 0; s < nslab; ++s) rho = fmaxf(rho, pdr[2 * ((size_t)s * rows + row) + 1]);
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, den = 0.f;
    for (int s = 0; s < nslab; ++s) {
        const float2 dr = *reinterpret_cast<const float2 *>(pdr + 2 * ((size_t)s * rows + row));
        const float w = exp2f(dr.y - rho);
        den = fmaf(dr.x, w, den);
        const uint4 raw = *reinterpret_cast<const uint4 *>(pnum + ((size_t)s * rows + row) * dv + c0);
        const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 f = __bfloat1622float2(h2[q]);
            acc[2 * q] = fmaf(f.x, w, acc[2 * q]);
            acc[2 * q + 1] = fmaf(f.y, w, acc[2 * q + 1]);
        }
    }
    if (c0 == 0) {
        sv[row] = make_float2(den, rho);
        if (sv2) sv2[row] = make_float2(den, rho);
    }
    const float inv = 1.f / den;
    uint4 out;
    out.x = pack_bf16(acc[0] * inv, acc[1] * inv); out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    out.z = pack_bf16(acc[4] * inv, acc[5] * inv); out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
    *reinterpret_cast<uint4 *>(O + (size_t)row * dv + c0) = out;
}

size_t take(size_t &off, size_t bytes)
{
    const size_t at = off;
    off += (bytes + 255) / 256 * 256;
    return at;
}

template <int D, int DV, int MODE>
cudaError_t launch_main(const MainParams &P, int grid, cudaStream_t st)
{
    using L = SmemLayout<D, DV, MODE>;
    static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
    cudaError_t e = cudaFuncSetAttribute(tc_attn_kernel<D, DV, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    tc_attn_kernel<D, DV, MODE><<<grid, 160, L::kTotal, st>>>(P);
    return cudaGetLastError();
}

template <int MODE>
cudaError_t launch_main_shape(int d, int dv, const MainParams &P, int grid, cudaStream_t st)
{
    if (d == 64 && dv == 64) return launch_main<64, 64, MODE>(P, grid, st);
    if (d == 128 && dv == 128) return launch_main<128, 128, MODE>(P, grid, st);
    if (d == 64 && dv == 128) return launch_main<64, 128, MODE>(P, grid, st);
    if (d == 128 && dv == 64) return launch_main<128, 64, MODE>(P, grid, st);
    return cudaErrorInvalidValue;
}

}  // namespace

// Shapes the tensor kernels cover: bf16, d and dv in {64, 128}, m and N multiples of 128, chunk 128,
// r a multiple of 16 up to 128.
bool tensor_supported(const darkattn_plan_s *plan)
{
    const Dims &D = plan->dims;
    if (!D.bf16) return false;
    if (!(D.d == 64 || D.d == 128) || !(D.dv == 64 || D.dv == 128)) return false;
    if (D.m % 128 || D.m < 128 || D.N % 128) return false;
    if (D.r % 16 || D.r < 16 || D.r > 128) return false;
    if (D.causal && D.C != 128) return false;
    if ((long long)D.BH * D.N * (D.m / 128) >= (1ll << 31)) return false;
    return true;
}

void tensor_make_layout(darkattn_plan_s *plan)
{
    const Dims &D = plan->dims;
    TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N, m = D.m, d = D.d, dv = D.dv;
    Y.nslab = D.m / 128;
    Y.T = D.N / 128;
    int nsplit = 1;
    if (!D.causal) {
        const long long units = (long long)BH * Y.nslab;
        nsplit = (int)((148ll * 4 + units - 1) / units);
        if (nsplit > Y.T) nsplit = Y.T;
        if (nsplit > kMaxNsplit) nsplit = kMaxNsplit;
        if (nsplit < 1) nsplit = 1;
    }
    Y.nsplit = nsplit;
    size_t off = 0;
    Y.status = take(off, 256);
    Y.Om = take(off, (size_t)D.H * m * d * 2);
    Y.cs = take(off, BH * Y.nslab * 4);
    Y.nK = take(off, BH * N * 4);
    Y.pnum = take(off, (size_t)Y.nslab * BH * N * dv * 2);
    Y.pdr = take(off, (size_t)Y.nslab * BH * N * 8);
    Y.Sacc = take(off, BH * m * dv * 4);
    Y.zacc = take(off, BH * m * 4);
    Y.Sb = take(off, BH * m * dv * 2);
    Y.sv = take(off, BH * N * 8);
    plan->launches_fwd = D.causal ? 5 : 7;
    plan->saved_bytes = BH * N * 8;
    if (D.causal) {       // tensor-core backward (the non-causal backward runs on the FP32 path)
        Y.Oscr = take(off, BH * N * dv * 2);
        Y.delta = take(off, BH * N * 4);
        Y.rhoc = take(off, BH * (size_t)Y.T * m * 4);
        Y.pdQ = take(off, (size_t)Y.nslab * BH * N * d * 2);
        Y.pdK = take(off, (size_t)Y.nslab * BH * N * d * 2);
        Y.pdV = take(off, (size_t)Y.nslab * BH * N * dv * 2);
        Y.espart = take(off, (size_t)4 * Y.nslab * BH * N * 4);
        Y.Tacc = take(off, (size_t)D.H * m * d * 4);
        Y.dMn = take(off, (size_t)D.H * D.r * d * 4);
        plan->launches_bwd = 3 + 1 + 2 + 3 + 1;   // prologue, delta, two scan kernels, three combines, dM
    }
    Y.total_bytes = off;
    if (Y.total_bytes > plan->workspace_bytes) plan->workspace_bytes = Y.total_bytes;
}

cudaError_t tensor_prologue(const darkattn_plan_s *plan, const void *K, const void *M, const void *W, char *ws,
                            cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16 *>(ws + off); };
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    NormParams NP;
    memset(&NP, 0, sizeof(NP));
    if (!make_map(&NP.mapK, K, BH * N, D.d, 128) || !make_map(&NP.mapM, M, (size_t)D.H * D.r, D.d, 128))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaSuccess;
    auto chk = [&]() { cudaError_t x = cudaGetLastError(); if (x != cudaSuccess && e == cudaSuccess) e = x; };

    timer_mark(plan, st, "fold_omega_kernel");
    fold_omega_kernel<<<dim3(D.m, D.H), 128, 0, st>>>((const __nv_bfloat16 *)W, (const __nv_bfloat16 *)M, bf(Y.Om), D.m, D.r, D.d,
                                                      D.w_per_head, kLog2e * D.s);
    chk();
    timer_mark(plan, st, "slab_shift_kernel");
    slab_shift_kernel<<<(unsigned)(BH * Y.nslab), 128, 0, st>>>((const __nv_bfloat16 *)W, fl(Y.cs), D.H, D.m, D.r, Y.nslab, D.w_per_head);
    chk();

    NP.nK = fl(Y.nK); NP.status = reinterpret_cast<int *>(ws + Y.status);
    NP.N = D.N; NP.H = D.H; NP.T = Y.T; NP.r = D.r;
    NP.nsplit = (int)((148 * 2 + BH - 1) / BH);
    if (NP.nsplit > Y.T) NP.nsplit = Y.T;
    NP.coef = kLog2e * 0.5f * D.s * D.s;
    const int smem_bytes = 2 * 128 * D.d * 2 + 64;
    timer_mark(plan, st, "tc_key_norms_kernel");
    if (D.d == 64) {
        cudaFuncSetAttribute(tc_key_norms_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        tc_key_norms_kernel<64><<<(unsigned)(BH * NP.nsplit), 160, smem_bytes, st>>>(NP);
    } else {
        cudaFuncSetAttribute(tc_key_norms_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        tc_key_norms_kernel<128><<<(unsigned)(BH * NP.nsplit), 160, smem_bytes, st>>>(NP);
    }
    chk();
    return e;
}

darkattn_status_t tensor_forward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                 const void *M, const void *W, void *O, void *saved, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16 *>(ws + off); };
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    if (!encode_fn()) { set_cuda_error(cudaErrorNotSupported, "tensor_forward: cuTensorMapEncodeTiled unavailable"); return DARKATTN_ERR_CUDA; }

    MainParams P;
    memset(&P, 0, sizeof(P));
    bool ok = make_map(&P.mapQ, Q, BH * N, D.d, 128) && make_map(&P.mapK, K, BH * N, D.d, 128) &&
              make_map(&P.mapV, V, BH * N, D.dv, 128) && make_map(&P.mapOm, bf(Y.Om), (size_t)D.H * D.m, D.d, 128) &&
              make_map(&P.mapSb, bf(Y.Sb), BH * D.m, D.dv, 128) &&
              make_map(&P.mapPN, bf(Y.pnum), (size_t)Y.nslab * BH * N, D.dv, 128);
    if (!ok) { set_cuda_error(cudaErrorInvalidValue, "tensor_forward: tensor map encode"); return DARKATTN_ERR_CUDA; }

    cudaError_t e = tensor_prologue(plan, K, M, W, ws, st);
    auto chk = [&]() { cudaError_t x = cudaGetLastError(); if (x != cudaSuccess && e == cudaSuccess) e = x; };

    P.nK = fl(Y.nK); P.cs = fl(Y.cs); P.pdr = fl(Y.pdr); P.Sacc = fl(Y.Sacc); P.zacc = fl(Y.zacc);
    P.status = reinterpret_cast<int *>(ws + Y.status);
    P.N = D.N; P.H = D.H; P.BH = D.BH; P.m = D.m; P.nslab = Y.nslab; P.T = Y.T; P.nsplit = Y.nsplit;
    const int units = (int)(BH * Y.nslab);
    if (D.causal) {
        P.nsplit = 1;
        timer_mark(plan, st, "tc_attn_kernel<causal>");
        cudaError_t x = launch_main_shape<MODE_CAUSAL>(D.d, D.dv, P, units, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
    } else {
        e = (e == cudaSuccess) ? cudaMemsetAsync(ws + Y.Sacc, 0, (Y.Sb - Y.Sacc), st) : e;   // S and z sums
        timer_mark(plan, st, "tc_attn_kernel<keys>");
        cudaError_t x = launch_main_shape<MODE_KEYS>(D.d, D.dv, P, units * Y.nsplit, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
        const long long n = (long long)BH * D.m * D.dv;
        timer_mark(plan, st, "state_to_bf16_kernel");
        state_to_bf16_kernel<<<(unsigned)((n + 1023) / 1024), 256, 0, st>>>(fl(Y.Sacc), bf(Y.Sb), n);
        chk();
        timer_mark(plan, st, "tc_attn_kernel<queries>");
        x = launch_main_shape<MODE_QUERIES>(D.d, D.dv, P, units * Y.nsplit, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
    }
    {
        const long long rows = (long long)BH * N, threads = rows * (D.dv / 8);
        timer_mark(plan, st, "combine_kernel");
        combine_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(bf(Y.pnum), fl(Y.pdr), (__nv_bfloat16 *)O,
                                                                          reinterpret_cast<float2 *>(ws + Y.sv),
                                                                          reinterpret_cast<float2 *>(saved), rows, D.dv, Y.nslab);
        chk();
    }
    if (e != cudaSuccess) { set_cuda_error(e, "tensor_forward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

}  // namespace darkattn
