// Tensor-core path of libdarkattn: bf16 operands, fp32 accumulation, tcgen05.mma with TMEM accumulators,
// operands staged by TMA (128-byte swizzle), exponentials fused into the TMEM read-out.
//
// Work decomposition. Features are cut into slabs of 128; one CTA owns one (batch, head, slab). Every
// quantity of the attention is a sum over features, so a slab CTA produces, for its 128 features, the
// partial numerator rows, the partial normaliser and the exponent its rows were scaled by; a small
// combine kernel adds the slabs. Per 128-token tile a slab CTA computes
//     U = X Omega_slab^T            Omega = log2(e) s W M folded once per call (u = w.(sMx) = (sM^T w).x), kept as the
//                                   sum of two bf16 matrices (its rounding and what the rounding left out), so that the
//                                   exponent's argument is as accurate as its fp32 accumulation
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
// The key features are scaled so that the largest one of a (batch, head, slab) is 2^kShiftHeadroom rather than 1: fp32 and
// bf16 reach down to 2^-126, so keys up to 190 binary orders below the largest keep a nonzero feature (causal prefixes see
// only some of the keys), while sums over 2^17 keys of products with values and query features (<= 1) stay far from 2^127.
constexpr float kShiftHeadroom = 64.f;

// ------------------------------------------------------------------ small helpers

// ------------------------------------------------------------------ prologue kernels (SIMT, tiny)
// Omega[h,l,c] = log2(e) * s * sum_a W[l,a] M[h,a,c], stored as its bf16 rounding Om and the bf16 rounding Oml of what
// that left out (Om + Oml carries 16 bits of Omega). One block per (head, 16 rows l); its four warps split the sum over a and add up through
// shared memory; d / 32 columns per lane: a thread's 16 x d/32 tile of outputs takes one broadcast load of four W values per
// 4 d/32 products.
template <int TC>
__global__ void __launch_bounds__(128) fold_omega_kernel(const __nv_bfloat16 *W, const __nv_bfloat16 *M, __nv_bfloat16 *Om, __nv_bfloat16 *Oml,
                                                         int m, int r, int w_per_head, float coef)
{
    constexpr int R = 16, d = 32 * TC;
    __shared__ __align__(16) float sw[R][128];
    __shared__ float part[3][R * TC][32];           // the partial sums of warps 1..3
    const int h = blockIdx.y, l0 = blockIdx.x * R, lane = threadIdx.x & 31, wq = threadIdx.x >> 5;
    const __nv_bfloat16 *w = W + ((size_t)(w_per_head ? h : 0) * m + l0) * r;
    for (int i = threadIdx.x; i < R * r; i += 128) sw[i / r][i % r] = __bfloat162float(w[i]);
    __syncthreads();
    const __nv_bfloat16 *Mh = M + (size_t)h * r * d + lane;
    float acc[R][TC];
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
        for (int q = 0; q < TC; ++q) acc[i][q] = 0.f;
#pragma unroll 2
    for (int a0 = 4 * wq; a0 < r; a0 += 16) {       // r is a multiple of 16: warp wq takes a = 4 wq .. 4 wq + 3 of every 16
        float x[4][TC];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int q = 0; q < TC; ++q) x[jj][q] = __bfloat162float(Mh[(size_t)(a0 + jj) * d + 32 * q]);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const float4 wv = *reinterpret_cast<const float4 *>(&sw[i][a0]);
#pragma unroll
            for (int q = 0; q < TC; ++q)
                acc[i][q] = fmaf(wv.x, x[0][q], fmaf(wv.y, x[1][q], fmaf(wv.z, x[2][q], fmaf(wv.w, x[3][q], acc[i][q]))));
        }
    }
    if (wq > 0) {
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int q = 0; q < TC; ++q) part[wq - 1][i * TC + q][lane] = acc[i][q];
    }
    __syncthreads();
    if (wq == 0) {
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int q = 0; q < TC; ++q) {
                const float om = coef * (acc[i][q] + part[0][i * TC + q][lane] + part[1][i * TC + q][lane] + part[2][i * TC + q][lane]);
                const __nv_bfloat16 hi = __float2bfloat16_rn(om);
                const size_t o = ((size_t)h * m + l0 + i) * d + lane + 32 * q;
                Om[o] = hi;
                Oml[o] = __float2bfloat16_rn(om - __bfloat162float(hi));
            }
    }
}

// Start value of the key-side shifts, which tc_key_prepass_kernel raises to the maximum over the keys: the smallest order key.
__global__ void shift_init_kernel(int *cs, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) cs[i] = (int)0x80000000u;
}

// ------------------------------------------------------------------ key prepass: norms and key-side shifts in one pass over K
//   n[bh,j]     = coef * |M_h k_j|^2                                   (log2 units; written by the CTAs of the first slab pair)
//   c[bh,slab]  = max_j max_{l in slab} (u_jl - n_j) - kShiftHeadroom   u = K Omega_hi^T
// The stabiliser of the key features is the largest exponent any key of the (batch, head) reaches in the slab, taken
// from the data (with it the largest key feature is 2^kShiftHeadroom, whatever the norms of the keys); being one constant per
// (batch, head, slab) it cancels in O. One CTA per (batch, head, pair of slabs, piece of the sequence): K tiles by TMA into
// two buffers, x~ = K M^T and U = K Omega_slab^T on the tensor cores, squared norms and row maxima read out of tensor memory
// by four warps (x~ of tile t + 1 is computed while U of tile t is read), the piece's maxima by atomicMax on order keys.
struct PrepassParams {
    CUtensorMap mapK, mapM, mapOm;
    float *nK;           // [BH, N] key norms, log2 units
    int *cs;             // [BH, nslab] order keys of the shifts
    int *status;
    int N, H, Hkv, T, m, r, nslab, npair, nsplit;
    float coef;          // log2(e) * s^2 / 2
};

enum PBars { PB_M, PB_K0, PB_K1, PMX, PMU, PEX, PEU, PNBARS };

template <int D>
__global__ void __launch_bounds__(160, 1) tc_key_prepass_kernel(const __grid_constant__ PrepassParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kTile = 128 * D * 2;
    unsigned char *sM = smem, *sOm = smem + kTile, *sK = smem + 3 * kTile;       // M, two slabs of Omega, two K buffers
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 5 * kTile);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + PNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + PNBARS + 1);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit;
    const int bh = unit / p.npair, pair = unit % p.npair, h = bh % p.H;
    const int slab0 = 2 * pair, ns = (slab0 + 1 < p.nslab) ? 2 : 1;           // this CTA's one or two slabs
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    const int rowk0 = kv_row0(bh, p.H, p.Hkv, p.N);
    if (tid == 0) {
        for (int i = 0; i < PEX; ++i) mbar_init(bars + i, 1);
        mbar_init(bars + PEX, 128); mbar_init(bars + PEU, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t kColX = 0, kColU = 128;      // x~ at 0, U of the two slabs at 128 and 256
    if (*abort_flag) { if (tid == 0) atomicExch(p.status, (int)DARKATTN_ERR_CUDA); }
    else if (warp == 4) {
        if ((tid & 31) == 0 && t1 > t0) {
            auto load_k = [&](int t) {
                const int b = (t - t0) & 1;
                mbar_expect_tx(bars + PB_K0 + b, kTile);
                for (int a = 0; a < D / 64; ++a) tma_load_2d(sK + b * kTile + a * 16384, &p.mapK, bars + PB_K0 + b, a * 64, rowk0 + t * 128);
            };
            mbar_expect_tx(bars + PB_M, kTile * (1 + ns));
            for (int a = 0; a < D / 64; ++a) {
                tma_load_2d(sM + a * 16384, &p.mapM, bars + PB_M, a * 64, h * p.r);
                for (int s = 0; s < ns; ++s) tma_load_2d(sOm + s * kTile + a * 16384, &p.mapOm, bars + PB_M, a * 64, h * p.m + (slab0 + s) * 128);
            }
            load_k(t0);
            if (t0 + 1 < t1) load_k(t0 + 1);
            const TileDesc tM(sM), tOm0(sOm), tOm1(sOm + kTile), tK0(sK), tK1(sK + kTile);
            const uint32_t id_x = make_idesc(128, p.r, 0, 0), id_u = make_idesc(128, 128, 0, 0);
            bool ok = wait_or_abort(bars + PB_M, 0, p.status, abort_flag);
            for (int t = t0; t < t1 && ok; ++t) {
                const int i = t - t0, b = i & 1;
                const uint32_t ph = i & 1, phk = (i >> 1) & 1;
                const TileDesc &tK = b ? tK1 : tK0;
                ok = wait_or_abort(bars + PB_K0 + b, phk, p.status, abort_flag);
                if (ok && i > 0) ok = wait_or_abort(bars + PEX, ph ^ 1, p.status, abort_flag);       // x~ of the tile before has been read
                if (!ok) break;
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(tmem + kColX, kdesc(tK, k), kdesc(tM, k), id_x, k > 0);
                mma_commit(bars + PMX);
                if (i > 0) { ok = wait_or_abort(bars + PEU, ph ^ 1, p.status, abort_flag); if (!ok) break; }      // U of the tile before has been read
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(tmem + kColU, kdesc(tK, k), kdesc(tOm0, k), id_u, k > 0);
                if (ns == 2)
                    _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(tmem + kColU + 128, kdesc(tK, k), kdesc(tOm1, k), id_u, k > 0);
                mma_commit(bars + PMU);
                if (t + 2 < t1) {       // this tile's buffer is free once its MMAs are done
                    ok = wait_or_abort(bars + PMU, ph, p.status, abort_flag);
                    if (!ok) break;
                    load_k(t + 2);
                }
            }
        }
    } else {
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        float best0 = -INFINITY, best1 = -INFINITY;
        bool ok = true;
        for (int t = t0; t < t1; ++t) {
            const uint32_t ph = (t - t0) & 1;
            ok = __all_sync(0xffffffffu, wait_or_abort(bars + PMX, ph, p.status, abort_flag));
            if (!ok) break;
            tc_fence_after();
            float acc = 0.f;
            for (int c0 = 0; c0 < p.r; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + kColX + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) { const float x = __uint_as_float(v[j]); acc = fmaf(x, x, acc); }
            }
            tc_fence_before();
            mbar_arrive(bars + PEX);
            const float nk = p.coef * acc;
            if (pair == 0) p.nK[(size_t)bh * p.N + (size_t)t * 128 + tid] = nk;
            ok = __all_sync(0xffffffffu, wait_or_abort(bars + PMU, ph, p.status, abort_flag));
            if (!ok) break;
            tc_fence_after();
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + kColU + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) mx0 = fmaxf(mx0, __uint_as_float(v[j]));
            }
            if (ns == 2) {
#pragma unroll
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColU + 128 + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) mx1 = fmaxf(mx1, __uint_as_float(v[j]));
                }
            }
            tc_fence_before();
            mbar_arrive(bars + PEU);
            best0 = fmaxf(best0, mx0 - nk);
            best1 = fmaxf(best1, mx1 - nk);
        }
        if (ok && t1 > t0) {
            for (int o = 16; o; o >>= 1) {
                best0 = fmaxf(best0, __shfl_xor_sync(0xffffffffu, best0, o));
                best1 = fmaxf(best1, __shfl_xor_sync(0xffffffffu, best1, o));
            }
            if ((tid & 31) == 0) {
                atomicMax(p.cs + bh * p.nslab + slab0, float_order_key(best0 - kShiftHeadroom));
                if (ns == 2) atomicMax(p.cs + bh * p.nslab + slab0 + 1, float_order_key(best1 - kShiftHeadroom));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ the main kernel
struct MainParams {
    CUtensorMap mapQ, mapK, mapV, mapOm, mapOml, mapSb, mapPN;
    CUtensorMap mapSst;  // causal, when stash_S: S before every chunk as [BH*T*m, dv] bf16, for the backward pass
    CUtensorMap mapBf;   // causal, when stash_S: the key features as [BH*N, m] bf16, for the backward pass
    int stash_S;
    const float *nK;     // [BH, N]      key norms in log2 units
    const float *cs;     // [BH, nslab]  key-side shift per slab (log2 units)
    float *pdr;          // [nslab, BH*N, 8]  partial normalisers of the four column groups (0..3), exponent the partial is scaled by (4)
    float *Sacc;         // [BH, m, DV]  fp32 state sums (non-causal key pass, atomics)
    float *zacc;         // [BH, m]
    // causal scan cut into nsplit segments of the sequence: the key pass stores one state per segment
    // (Sseg [BH, nsplit, m, DV], zseg [BH, nsplit, m]) instead of adding into Sacc; after an exclusive prefix over the
    // segments the causal kernel of segment s > 0 starts from Sseg[bh, s] (its bf16 copy comes through mapSb).
    float *Sseg, *zseg;
    float *zc;           // causal: z before chunk t for the backward pass, [BH, T, m] (row 0 not written)
    int *status;
    int N, H, Hkv, BH, m, nslab, T, nsplit;
};

enum { MODE_CAUSAL = 0, MODE_KEYS = 1, MODE_QUERIES = 2 };

// ------------------------------------------------------------------ forward scan kernels
// All three use 16 epilogue warps (warp w: TMEM lanes 32 (w % 4) .. +31, columns 32 (w / 4) .. +31) and one
// control warp whose first lane issues the TMA loads and the MMAs. phi(Q) and the masked kernel tile P are only
// ever the A operand of an MMA whose rows are tokens, so they are packed to bf16 in tensor memory and read
// by the MMA from there; phi(K) also serves transposed and as a B operand and goes to shared memory.

__device__ __forceinline__ void store_row_f32x32_bf16(const uint32_t (&v)[32], unsigned char *tile, int row, int col0)
{
#pragma unroll
    for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(tile_chunk(tile, row, col0 / 8 + q)) = pack8(v + 8 * q);
}

// phi(Q) of one row segment: row maximum over the slab's 128 features (exchanged with the three other warps
// of the lane quarter through red[4][128]), 2^(u - max) packed to bf16 into TMEM columns fq + col0/2.
// rmax receives the row maximum. WITH_Z: returns sum_l phi(Q)_l z_l over the segment (else 0).
template <bool WITH_Z>
__device__ __forceinline__ float query_features_to_tmem(uint32_t u_addr, uint32_t fq_addr, float *red, const float *z, int q4,
                                                        int g, int r, int col0, float &rmax)
{
    uint32_t v[32], pk[16];
    tmem_ld32(u_addr + col0, v);
    tmem_wait_ld();
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(v[j]));
    red[g * 128 + r] = mx;
    quarter_sync(q4);
    rmax = fmaxf(fmaxf(red[r], red[128 + r]), fmaxf(red[256 + r], red[384 + r]));
    float dz = 0.f;
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        const float f0 = ex2f(__uint_as_float(v[j]) - rmax), f1 = ex2f(__uint_as_float(v[j + 1]) - rmax);
        if constexpr (WITH_Z) {
            const float2 zz = *reinterpret_cast<const float2 *>(z + col0 + j);
            dz = fmaf(f0, zz.x, dz);
            dz = fmaf(f1, zz.y, dz);
        }
        pk[j / 2] = pack_bf16(f0, f1);
    }
    tmem_st16(fq_addr + col0 / 2, pk);
    tmem_wait_st();
    return dz;
}

template <int D, int DV>
struct FwdCausalSmem {
    static constexpr int kOm = 0;                          // folded projections of the slab, rounded    [128 l, D]
    static constexpr int kOml = kOm + 128 * D * 2;         // ... and what the rounding left out         [128 l, D]
    static constexpr int kQ = kOml + 128 * D * 2;
    static constexpr int kK = kQ + 128 * D * 2;
    static constexpr int kV = kK + 128 * D * 2;
    static constexpr int kFK = kV + 128 * DV * 2;          // phi(K)                              [128, 128]
    static constexpr int kSb = kFK + 32768;                // bf16 copy of the state              [128 l, DV]
    static constexpr int kRed = kSb + 128 * DV * 2;        // float[4][128]: row maxima exchanged between the warps of a row;
                                                           // mid-chunk the same 2 KB hold the ones operand of z += phi(K)^T 1
    static constexpr int kZ = kRed + 2048;                 // z_prev, float[128]
    static constexpr int kBars = kZ + 512;
    static constexpr int kTotal = kBars + 256;
};

// TMEM columns of the causal kernel: state S at 0 (DV), four partial sums of z at 128 (16 each: consecutive MMAs of
// z += phi(K)^T 1 go to different ones, so that none has to wait for the one before), packed phi(Q) at 192 (64),
// R1 at 256, R2 at 384.
constexpr uint32_t kColS = 0, kColZ = 128, kColFQ = 192, kColR1 = 256, kColR2 = 384;

enum CBars { CB_OM, CB_Q, CB_K, CB_V, CB_ST, CM1, CM2, CM3, CMS, CM4, CE0, CE1, CE2, CE3, CE4, CNBARS };

// Causal: one CTA per (b, h, slab) walks the chunks of the sequence.
//   R1: U_Q -> (phi(Q) read) -> P = phi(Q) phi(K)^T -> packed tril(P) (A operand of P V) -> U_Q of the next chunk
//   R2: U_K -> (phi(K) read) -> O = phi(Q) S_prev + P V -> (O read) -> U_K of the next chunk
// The epilogue warps work in this order: phi(K) of chunk t; the bf16 copy of the state through chunk t - 1 (while P
// runs); tril(P); the output tile and z; phi(Q) of chunk t + 1 (both projections of the next chunk are issued behind
// the output MMAs and run while the output is read). The state tile's buffer doubles as the staging tile of the
// output's TMA store: between the output MMAs of chunk t and the copy of the state through chunk t nobody reads it.
template <int D, int DV>
__global__ void __launch_bounds__(kThreads, 1) tc_fwd_causal_kernel(const __grid_constant__ MainParams p)
{
    using L = FwdCausalSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sOml = smem + L::kOml, *sQ = smem + L::kQ, *sK = smem + L::kK, *sV = smem + L::kV;
    unsigned char *sFK = smem + L::kFK, *sSb = smem + L::kSb;
    float *sZ = reinterpret_cast<float *>(smem + L::kZ), *sRed = reinterpret_cast<float *>(smem + L::kRed);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + CNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + CNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, seg = blockIdx.x % p.nsplit;
    const int bh = unit / p.nslab, slab = unit % p.nslab, h = bh % p.H;
    const int row0 = bh * p.N;
    const int tbeg = (int)((long long)p.T * seg / p.nsplit), tend = (int)((long long)p.T * (seg + 1) / p.nsplit);
    const bool fresh = (seg == 0);                 // the scan state starts at zero (else at the segment's prefix state)
    // the state through the segment's last chunk is also copied (and stored) when the backward pass will start the
    // next segment from it
    const bool copy_last = p.stash_S && tend < p.T;

    if (tid == 0) {
        for (int i = 0; i < CE0; ++i) mbar_init(bars + i, 1);
        for (int i = CE0; i < CNBARS; ++i) mbar_init(bars + i, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) sZ[tid] = fresh ? 0.f : p.zseg[((size_t)bh * p.nsplit + seg) * p.m + slab * 128 + tid];
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;
    if (!fresh && warp < kEpiWarps) {      // the segment's prefix state into the fp32 accumulators in TMEM
        const int lane = tid & 31, q4 = warp & 3, col0 = (warp >> 2) * 32, r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const size_t srow = ((size_t)bh * p.nsplit + seg) * p.m + slab * 128 + r;
        if (col0 < DV) {
            uint32_t v[32];
            const float4 *src = reinterpret_cast<const float4 *>(p.Sseg + srow * DV + col0);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float4 x = src[j];
                v[4 * j] = __float_as_uint(x.x); v[4 * j + 1] = __float_as_uint(x.y);
                v[4 * j + 2] = __float_as_uint(x.z); v[4 * j + 3] = __float_as_uint(x.w);
            }
            tmem_st32(lane_addr + kColS + col0, v);
        }
        {       // z: the prefix into the first partial sum, zero into the three others (one per column group's warp)
            uint32_t v[16];
            const uint32_t zv = (col0 == 0) ? __float_as_uint(sZ[r]) : 0u;
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = zv;
            tmem_st16(lane_addr + kColZ + (col0 / 32) * 16, v);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (tend <= tbeg) {
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            const int rowk0 = kv_row0(bh, p.H, p.Hkv, p.N);       // K and V may be shared by a group of query heads
            auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                const int base = (map == &p.mapQ) ? row0 : rowk0;
                mbar_expect_tx(bar, 128 * width * 2);
                for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, base + t * 128);
            };
            const int prow0 = (slab * p.BH + bh) * p.N;
            auto store_output = [&](int t) {       // this slab's part of the output rows of chunk t, staged in the state tile's buffer
                for (int a = 0; a < DV / 64; ++a) tma_store_2d(&p.mapPN, sSb + a * 16384, a * 64, prow0 + t * 128);
                tma_store_commit();
            };
            auto store_state = [&](int t) {        // the bf16 state before chunk t, for the backward pass
                for (int a = 0; a < DV / 64; ++a) tma_store_2d(&p.mapSst, sSb + a * 16384, a * 64, (bh * p.T + t) * p.m + slab * 128);
                tma_store_commit();
            };
            const TileDesc tOm(sOm), tOml(sOml), tQ(sQ), tK(sK), tV(sV), tFK(sFK), tSb(sSb);
            const uint64_t ones_desc = make_sdesc(smem_u32(sRed), 16384, 1024);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_o = make_idesc(128, DV, 0, 1);
            const uint32_t id_s = make_idesc(128, DV, 1, 1);
            const uint32_t id_z = make_idesc(128, 16, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2, FQ = tmem + kColFQ;

            mbar_expect_tx(bars + CB_OM, 2 * 128 * D * 2 + (fresh ? 0 : 128 * DV * 2));
            for (int a = 0; a < D / 64; ++a) {
                tma_load_2d(sOm + a * 16384, &p.mapOm, bars + CB_OM, a * 64, h * p.m + slab * 128);
                tma_load_2d(sOml + a * 16384, &p.mapOml, bars + CB_OM, a * 64, h * p.m + slab * 128);
            }
            if (!fresh)     // bf16 copy of the segment's prefix state
                for (int a = 0; a < DV / 64; ++a)
                    tma_load_2d(sSb + a * 16384, &p.mapSb, bars + CB_OM, a * 64, (bh * p.nsplit + seg) * p.m + slab * 128);
            load_tile(sQ, &p.mapQ, bars + CB_Q, D, tbeg);
            load_tile(sK, &p.mapK, bars + CB_K, D, tbeg);
            load_tile(sV, &p.mapV, bars + CB_V, DV, tbeg);

#define CWAIT(b, q) do { ok = wait_or_abort(bars + (b), (q), status, abort_flag); } while (0)
            bool ok = true;
            CWAIT(CB_OM, 0);
            if (ok) CWAIT(CB_Q, 0);
            if (ok) {
                tc_fence_after();
                issue_projection<D>(R1, tQ, tOm, tOml, id_kk);                                                    // U_Q of the first chunk
                mma_commit(bars + CM1);
                CWAIT(CB_K, 0);
            }
            if (ok) {
                tc_fence_after();
                issue_projection<D>(R2, tK, tOm, tOml, id_kk);                                                    // U_K of the first chunk
                mma_commit(bars + CM2);
                CWAIT(CE0, 0);                                                  // phi(Q) packed, Q tile consumed
            }
            if (ok && tbeg + 1 < tend) load_tile(sQ, &p.mapQ, bars + CB_Q, D, tbeg + 1);
            for (int t = tbeg; t < tend && ok; ++t) {
                const uint32_t ph = (t - tbeg) & 1;
                const bool first = (t == tbeg) && fresh, last = (t + 1 == tend);
                CWAIT(CE1, ph); if (!ok) break;                                 // phi(K) and the ones in smem, R2 read, K tile consumed
                if (!last) load_tile(sK, &p.mapK, bars + CB_K, D, t + 1);
                if (p.stash_S) {        // the backward kernels read the key features back instead of forming them again
                    tma_store_2d(&p.mapBf, sFK, slab * 128, row0 + t * 128);
                    tma_store_2d(&p.mapBf, sFK + 16384, slab * 128 + 64, row0 + t * 128);
                    tma_store_commit();
                }
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R1, FQ + k * 8, kdesc(tFK, k), id_kk, k > 0);                // P = phi(Q) phi(K)^T
                mma_commit(bars + CM3);
                if (!first) {
                    if (t > tbeg) {                                             // the bf16 state through chunk t - 1 is in smem
                        CWAIT(CE4, ph ^ 1); if (!ok) break;
                        if (p.stash_S) store_state(t);
                    }
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R2, FQ + k * 8, mndesc(tSb, k), id_o, k > 0);            // O = phi(Q) S_prev
                }
                _Pragma("unroll") for (int k = 0; k < 8; ++k)                                                                     // z += phi(K)^T 1
                    mma_ss(tmem + kColZ + 16 * (k & 3), mndesc(tFK, k), ones_desc, id_z, (!first) || k >= 4);
                CWAIT(CB_V, ph); if (!ok) break;
                CWAIT(CE2, ph); if (!ok) break;                                 // tril(P) packed in R1
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + k * 8, mndesc(tV, k), id_o, (!first) || k > 0);     // O += P V
                if (p.stash_S) tma_store_wait_read();       // the stash copies of the state before this chunk and of phi(K) have left their tiles: the output may be
                                                            // staged in the first, the next phi(K) written to the second
                mma_commit(bars + CM4);
                if (!last) {        // U_Q of the next chunk, while the epilogue warps read the output tile out
                    CWAIT(CB_Q, ph ^ 1); if (!ok) break;
                    tc_fence_after();
                    issue_projection<D>(R1, tQ, tOm, tOml, id_kk);
                    mma_commit(bars + CM1);
                }
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColS, mndesc(tFK, k), mndesc(tV, k), id_s, (!first) || k > 0);   // S += phi(K)^T V
                mma_commit(bars + CMS);
                CWAIT(CE3, ph); if (!ok) break;                                 // the output tile has been read out of R2 and staged
                store_output(t);
                if (!last) {
                    CWAIT(CB_K, ph ^ 1); if (!ok) break;
                    tc_fence_after();
                    issue_projection<D>(R2, tK, tOm, tOml, id_kk);                                                // U_K of the next chunk
                    mma_commit(bars + CM2);
                }
                if (!last || copy_last) { tma_store_wait_read(); mbar_arrive(bars + CB_ST); }     // the staged output has left the state tile's buffer
                CWAIT(CMS, ph); if (!ok) break;                                 // V tile consumed
                if (!last) {
                    load_tile(sV, &p.mapV, bars + CB_V, DV, t + 1);
                    CWAIT(CE0, ph ^ 1); if (!ok) break;                         // phi(Q) of the next chunk packed, its Q tile consumed
                    if (t + 2 < tend) load_tile(sQ, &p.mapQ, bars + CB_Q, D, t + 2);
                }
            }
            if (ok && copy_last) {      // the state through the segment's last chunk: what the backward pass starts the next segment from
                CWAIT(CE4, (tend - 1 - tbeg) & 1);
                if (ok) store_state(tend);
            }
#undef CWAIT
            tma_store_wait_all();
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, g = warp >> 2, col0 = g * 32;
        const int r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        const float cshift = load_key_shift(p.cs, bh * p.nslab + slab);
        const size_t prow0 = ((size_t)slab * p.BH + bh) * p.N;
        uint32_t *sOnes = reinterpret_cast<uint32_t *>(sRed);
        bool ok = true;
        float rmax = 0.f;                           // row maximum of the chunk whose phi(Q) was formed last
// A wait that gave up (here or, seen through the abort flag, in another warp) switches the warp to a dry run: it skips
// every later wait but keeps walking the same chunks, so that every named barrier below still gets all its arrivals and
// no warp is left waiting for one that has gone (what it reads and writes from then on is garbage; the status word says so).
#define EWAIT(b, q) do { ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + (b), (q), status, abort_flag)); } while (0)
        // phi(K): once the four warps of these rows are done with the exchanged maxima the array is filled with bf16 ones,
        // the B operand of z += phi(K)^T 1
        auto key_features = [&](float nk) {
            tc_fence_after();
            quarter_sync(q4);
            sOnes[g * 128 + r] = 0x3F803F80u;
            features_to_tile(R2 + col0, nk, sFK, r, col0);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + CE1);
        };
        float dz = 0.f;                             // phi(Q) z_prev over this thread's features, of the chunk whose phi(Q) was formed last
        auto query_features = [&]() {
            tc_fence_after();
            dz = query_features_to_tmem<true>(R1, lane_addr + kColFQ, sRed, sZ, q4, g, r, col0, rmax);
            tc_fence_before();
            mbar_arrive_warp(bars + CE0);
        };
        // the state through chunk t as the bf16 operand of phi(Q) S, once the staged output of chunk t has left the tile
        auto copy_state = [&](int t) {
            const uint32_t q = (t - tbeg) & 1;
            EWAIT(CB_ST, q);
            EWAIT(CMS, q);
            tc_fence_after();
            if (col0 < DV) tmem_row_to_tile(lane_addr + kColS + col0, sSb, r, col0);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + CE4);
        };
        EWAIT(CM1, 0);
        query_features();
        float nk_next = p.nK[(size_t)row0 + (size_t)tbeg * 128 + r] + cshift;
        for (int t = tbeg; t < tend; ++t) {
            const uint32_t ph = (t - tbeg) & 1;
            const bool last = (t + 1 == tend);
            const size_t prow = prow0 + (size_t)t * 128 + r;
            const float nk = nk_next;
            if (!last) nk_next = p.nK[(size_t)row0 + (size_t)(t + 1) * 128 + r] + cshift;     // needed a chunk from now

            EWAIT(CM2, ph);
            key_features(nk);
            if (t > tbeg) copy_state(t - 1);                // while P runs

            EWAIT(CM3, ph);
            tc_fence_after();
            float rowsum = 0.f;
            {
                uint32_t v[32], pk[16];
                tmem_ld32(R1 + col0, v);
                tmem_wait_ld();
                quarter_sync(q4);                   // every column group has read P before anyone overwrites it
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float x0 = (col0 + j <= r) ? __uint_as_float(v[j]) : 0.f;
                    const float x1 = (col0 + j + 1 <= r) ? __uint_as_float(v[j + 1]) : 0.f;
                    rowsum += x0 + x1;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + col0 / 2, pk);
                tmem_wait_st();
            }
            tc_fence_before();
            mbar_arrive_warp(bars + CE2);

            EWAIT(CM4, ph);         // the output tile; z through this chunk (its MMAs ran ahead of the output's)
            tc_fence_after();
            if (col0 < DV) {
                uint32_t v[32];
                tmem_ld32(R2 + col0, v);
                tmem_wait_ld();
                store_row_f32x32_bf16(v, sSb, r, col0);
            }
            if (g == 0 && t + 1 < p.T) {            // (also after a segment's last chunk: the next segment's backward needs it)
                const uint32_t z0 = tmem_ld1(lane_addr + kColZ), z1 = tmem_ld1(lane_addr + kColZ + 16);
                const uint32_t z2 = tmem_ld1(lane_addr + kColZ + 32), z3 = tmem_ld1(lane_addr + kColZ + 48);
                tmem_wait_ld();
                const float zv = (__uint_as_float(z0) + __uint_as_float(z1)) + (__uint_as_float(z2) + __uint_as_float(z3));
                sZ[r] = zv;
                p.zc[((size_t)bh * p.T + t + 1) * p.m + slab * 128 + r] = zv;
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + CE3);
            p.pdr[8 * prow + g] = rowsum + dz;
            if (g == 0) p.pdr[8 * prow + 4] = rmax + cshift;
            epi_sync();                             // every z is in place before anyone forms the next chunk's phi(Q)

            if (!last) {
                EWAIT(CM1, ph ^ 1);
                query_features();
            }
        }
        if (copy_last) copy_state(tend - 1);
#undef EWAIT
    }
    if (*abort_flag) __nanosleep(200000);   // error path only: let copies and MMAs in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ non-causal, key pass: S = phi(K)^T V, z = phi(K)^T 1
template <int D, int DV>
struct FwdKeysSmem {
    // K and V tiles sit in rings of kStages buffers (4 where they are small enough), so that a tile's load is issued
    // several tiles before its use; TMEM regions alternate between two, and so do the phi(K) tiles where two fit.
    static constexpr int kFixed = 2 * 128 * D * 2 + 2048 + 256;       // both halves of the folded projections, ones, barriers
    static constexpr int kStages = (kFixed + 4 * 128 * (D + DV) * 2 + 2 * 32768 <= 232448) ? 4 : 2;
    static constexpr int kFKs = (kFixed + kStages * 128 * (D + DV) * 2 + 2 * 32768 <= 232448) ? 2 : 1;
    static constexpr int kOm = 0;
    static constexpr int kOml = kOm + 128 * D * 2;
    static constexpr int kK = kOml + 128 * D * 2;
    static constexpr int kV = kK + kStages * 128 * D * 2;
    static constexpr int kFK = kV + kStages * 128 * DV * 2;   // phi(K) tiles
    static constexpr int kOnes = kFK + kFKs * 32768;
    static constexpr int kBars = kOnes + 2048;
    static constexpr int kTotal = kBars + 256;
};

// barriers of the key pass: Omega, K ring, V ring, then pairs (projection done, state update done, phi(K) written)
enum KyBars { YB_OM = 0, YB_K0 = 1, YB_V0 = 5, YM2_0 = 9, YM2_1, YMS_0, YMS_1, YE1_0, YE1_1, YNBARS };

// One CTA per (b, h, slab, token split); tiles alternate between two sets of buffers and two TMEM regions so that
// the projection of tile i+1 runs while the epilogue warps exponentiate tile i.
template <int D, int DV>
__global__ void __launch_bounds__(kThreads, 1) tc_fwd_keys_kernel(const __grid_constant__ MainParams p)
{
    using L = FwdKeysSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kXT = 128 * D * 2, kVT = 128 * DV * 2;
    unsigned char *sOm = smem + L::kOm, *sOml = smem + L::kOml, *sK = smem + L::kK, *sV = smem + L::kV, *sFK = smem + L::kFK, *sOnes = smem + L::kOnes;
    constexpr int kFKstride = (L::kFKs == 2) ? 32768 : 0;     // one phi(K) tile: tile i + 1 is written once the state update of tile i is done
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + YNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + YNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit;
    const int bh = unit / p.nslab, slab = unit % p.nslab, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    const int n = t1 - t0, row0 = bh * p.N, rowk0 = kv_row0(bh, p.H, p.Hkv, p.N);

    if (tid == 0) {
        for (int i = 0; i < YE1_0; ++i) mbar_init(bars + i, 1);
        mbar_init(bars + YE1_0, kEpiWarps); mbar_init(bars + YE1_1, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) {
        *reinterpret_cast<uint4 *>(sOnes + tid * 16) = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
        fence_async_smem();
    }
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (n <= 0) {
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            constexpr int NST = L::kStages;
            auto load_k = [&](int i) {
                const int b = i % NST;
                mbar_expect_tx(bars + YB_K0 + b, kXT);
                for (int a = 0; a < D / 64; ++a) tma_load_2d(sK + b * kXT + a * 16384, &p.mapK, bars + YB_K0 + b, a * 64, rowk0 + (t0 + i) * 128);
            };
            auto load_v = [&](int i) {
                const int b = i % NST;
                mbar_expect_tx(bars + YB_V0 + b, kVT);
                for (int a = 0; a < DV / 64; ++a) tma_load_2d(sV + b * kVT + a * 16384, &p.mapV, bars + YB_V0 + b, a * 64, rowk0 + (t0 + i) * 128);
            };
            const TileDesc tOm(sOm), tOml(sOml), tF0(sFK), tF1(sFK + kFKstride);
            const uint64_t ones_desc = make_sdesc(smem_u32(sOnes), 16384, 1024);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0), id_s = make_idesc(128, DV, 1, 1), id_z = make_idesc(128, 16, 1, 1);

            mbar_expect_tx(bars + YB_OM, 2 * 128 * D * 2);
            for (int a = 0; a < D / 64; ++a) {
                tma_load_2d(sOm + a * 16384, &p.mapOm, bars + YB_OM, a * 64, h * p.m + slab * 128);
                tma_load_2d(sOml + a * 16384, &p.mapOml, bars + YB_OM, a * 64, h * p.m + slab * 128);
            }
            for (int i = 0; i < NST && i < n; ++i) { load_k(i); load_v(i); }
            bool ok = wait_or_abort(bars + YB_OM, 0, status, abort_flag);
            if (ok) ok = wait_or_abort(bars + YB_K0, 0, status, abort_flag);
            if (ok) {
                tc_fence_after();
                const TileDesc tK0(sK);
                issue_projection<D>(tmem + kColR1, tK0, tOm, tOml, id_kk);
                mma_commit(bars + YM2_0);
            }
            for (int i = 0; i < n && ok; ++i) {
                const int b = i & 1;
                const uint32_t phb = (i >> 1) & 1;
                if (i + 1 < n) {       // projection of the next tile into the other region (read out two tiles ago)
                    const int sn = (i + 1) % NST;
                    ok = wait_or_abort(bars + YB_K0 + sn, ((i + 1) / NST) & 1, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const TileDesc tKn(sK + sn * kXT);
                    issue_projection<D>(tmem + (b ? kColR1 : kColR2), tKn, tOm, tOml, id_kk);
                    mma_commit(bars + YM2_0 + (b ^ 1));
                }
                ok = wait_or_abort(bars + YE1_0 + b, phb, status, abort_flag);      // phi(K) of tile i in smem; its K tile is consumed
                if (!ok) break;
                if (i + NST < n) load_k(i + NST);
                ok = wait_or_abort(bars + YB_V0 + i % NST, (i / NST) & 1, status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const TileDesc &tF = b ? tF1 : tF0;
                const TileDesc tVb(sV + (i % NST) * kVT);
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColS, mndesc(tF, k), mndesc(tVb, k), id_s, i > 0 || k > 0);
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColZ, mndesc(tF, k), ones_desc, id_z, i > 0 || k > 0);
                mma_commit(bars + YMS_0 + b);
                ok = wait_or_abort(bars + YMS_0 + b, phb, status, abort_flag);
                if (!ok) break;
                if (i + NST < n) load_v(i + NST);
            }
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, g = warp >> 2, col0 = g * 32;
        const int r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const float cshift = load_key_shift(p.cs, bh * p.nslab + slab);
        bool ok = true;
        for (int i = 0; i < n && ok; ++i) {
            const int b = i & 1;
            const uint32_t phb = (i >> 1) & 1;
            const float nk = p.nK[(size_t)row0 + (size_t)(t0 + i) * 128 + r] + cshift;
            ok = __all_sync(0xffffffffu, wait_or_abort(bars + YM2_0 + b, phb, status, abort_flag));
            if (!ok) break;
            if (L::kFKs == 1 && i > 0) {       // the one phi(K) tile is free once the state update of the tile before is done
                ok = __all_sync(0xffffffffu, wait_or_abort(bars + YMS_0 + (b ^ 1), ((i - 1) >> 1) & 1, status, abort_flag));
                if (!ok) break;
            }
            tc_fence_after();
            features_to_tile(lane_addr + (b ? kColR2 : kColR1) + col0, nk, sFK + b * kFKstride, r, col0);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + YE1_0 + b);
        }
        if (ok) ok = __all_sync(0xffffffffu, wait_or_abort(bars + YMS_0 + ((n - 1) & 1), ((n - 1) >> 1) & 1, status, abort_flag));
        if (ok) {        // add this CTA's state to the global sums, or store it as its segment's state
            tc_fence_after();
            const size_t srow = ((size_t)bh * p.nsplit + split) * p.m + slab * 128 + r;
            if (col0 < DV) {
                uint32_t v[32];
                tmem_ld32(lane_addr + kColS + col0, v);
                tmem_wait_ld();
                if (p.Sseg) {
                    float4 *dst = reinterpret_cast<float4 *>(p.Sseg + srow * DV + col0);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                } else {
                    float *dst = p.Sacc + ((size_t)bh * p.m + slab * 128 + r) * DV + col0;
#pragma unroll
                    for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(v[j]));
                }
            }
            if (g == 0) {
                uint32_t v[16];
                tmem_ld16(lane_addr + kColZ, v);
                tmem_wait_ld();
                if (p.Sseg) p.zseg[srow] = __uint_as_float(v[0]);
                else atomicAdd(p.zacc + (size_t)bh * p.m + slab * 128 + r, __uint_as_float(v[0]));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ non-causal, query pass: partial O = phi(Q) S, den = phi(Q) z
template <int D, int DV>
struct FwdQueriesSmem {
    // ring of Q tiles: 4 where they fit beside both halves of the folded projections, else 3
    static constexpr int kStages = (2 * 128 * D * 2 + 4 * 128 * D * 2 + 2 * 128 * DV * 2 + 512 + 2048 + 256 <= 232448) ? 4 : 3;
    static constexpr int kOm = 0;
    static constexpr int kOml = kOm + 128 * D * 2;
    static constexpr int kQ = kOml + 128 * D * 2;
    static constexpr int kSb = kQ + kStages * 128 * D * 2; // bf16 state of the slab [128 l, DV]
    static constexpr int kStg = kSb + 128 * DV * 2;
    static constexpr int kZ = kStg + 128 * DV * 2;
    static constexpr int kRed = kZ + 512;
    static constexpr int kBars = kRed + 2048;
    static constexpr int kTotal = kBars + 256;
};

enum QyBars { UB_OM = 0, UB_Q0 = 1, UM1_0 = 5, UM1_1, UM4_0, UM4_1, UE0_0, UE0_1, UE3_0, UE3_1, UNBARS };

// TMEM: packed phi(Q) of the two tiles in flight at 0 and 64; R1, R2 hold U_Q and then the output tile.
template <int D, int DV>
__global__ void __launch_bounds__(kThreads, 1) tc_fwd_queries_kernel(const __grid_constant__ MainParams p)
{
    using L = FwdQueriesSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kXT = 128 * D * 2;
    unsigned char *sOm = smem + L::kOm, *sOml = smem + L::kOml, *sQ = smem + L::kQ, *sSb = smem + L::kSb, *sStg = smem + L::kStg;
    float *sZ = reinterpret_cast<float *>(smem + L::kZ), *sRed = reinterpret_cast<float *>(smem + L::kRed);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + UNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + UNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit;
    const int bh = unit / p.nslab, slab = unit % p.nslab, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    const int n = t1 - t0, row0 = bh * p.N;

    if (tid == 0) {
        for (int i = 0; i < UE0_0; ++i) mbar_init(bars + i, 1);
        for (int i = UE0_0; i < UNBARS; ++i) mbar_init(bars + i, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) sZ[tid] = p.zacc[(size_t)bh * p.m + slab * 128 + tid];
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (n <= 0) {
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            constexpr int NST = L::kStages;
            auto load_q = [&](int i) {
                const int b = i % NST;
                mbar_expect_tx(bars + UB_Q0 + b, kXT);
                for (int a = 0; a < D / 64; ++a) tma_load_2d(sQ + b * kXT + a * 16384, &p.mapQ, bars + UB_Q0 + b, a * 64, row0 + (t0 + i) * 128);
            };
            const TileDesc tOm(sOm), tOml(sOml), tQ0(sQ), tSb(sSb);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0), id_o = make_idesc(128, DV, 0, 1);
            mbar_expect_tx(bars + UB_OM, 2 * 128 * D * 2 + 128 * DV * 2);
            for (int a = 0; a < D / 64; ++a) {
                tma_load_2d(sOm + a * 16384, &p.mapOm, bars + UB_OM, a * 64, h * p.m + slab * 128);
                tma_load_2d(sOml + a * 16384, &p.mapOml, bars + UB_OM, a * 64, h * p.m + slab * 128);
            }
            for (int a = 0; a < DV / 64; ++a) tma_load_2d(sSb + a * 16384, &p.mapSb, bars + UB_OM, a * 64, bh * p.m + slab * 128);
            for (int i = 0; i < NST && i < n; ++i) load_q(i);
            bool ok = wait_or_abort(bars + UB_OM, 0, status, abort_flag);
            if (ok) ok = wait_or_abort(bars + UB_Q0, 0, status, abort_flag);
            if (ok) {
                tc_fence_after();
                issue_projection<D>(tmem + kColR1, tQ0, tOm, tOml, id_kk);
                mma_commit(bars + UM1_0);
            }
            for (int i = 0; i < n && ok; ++i) {
                const int b = i & 1;
                const uint32_t phb = (i >> 1) & 1;
                if (i + 1 < n) {       // projection of the next tile into the other region, once its last output tile was read
                    ok = wait_or_abort(bars + UB_Q0 + (i + 1) % NST, ((i + 1) / NST) & 1, status, abort_flag);
                    if (ok && i >= 1) ok = wait_or_abort(bars + UE3_0 + (b ^ 1), ((i - 1) >> 1) & 1, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const TileDesc tQn(sQ + ((i + 1) % NST) * kXT);
                    issue_projection<D>(tmem + (b ? kColR1 : kColR2), tQn, tOm, tOml, id_kk);
                    mma_commit(bars + UM1_0 + (b ^ 1));
                }
                ok = wait_or_abort(bars + UE0_0 + b, phb, status, abort_flag);      // phi(Q) packed; U read; Q tile consumed
                if (!ok) break;
                if (i + NST < n) load_q(i + NST);
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(tmem + (b ? kColR2 : kColR1), tmem + b * 64 + k * 8, mndesc(tSb, k), id_o, k > 0);
                mma_commit(bars + UM4_0 + b);
            }
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, g = warp >> 2, col0 = g * 32;
        const int r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const float cshift = load_key_shift(p.cs, bh * p.nslab + slab);
        const size_t prow0 = ((size_t)slab * p.BH + bh) * p.N;
        bool ok = true;
        // (a wait that gave up switches the warp to a dry run over the remaining tiles: see the causal kernel)
        for (int i = 0; i < n; ++i) {
            const int b = i & 1;
            const uint32_t phb = (i >> 1) & 1;
            const uint32_t R = lane_addr + (b ? kColR2 : kColR1);
            float rmax;
            ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + UM1_0 + b, phb, status, abort_flag));
            tc_fence_after();
            const float dz = query_features_to_tmem<true>(R, lane_addr + b * 64, sRed, sZ, q4, g, r, col0, rmax);
            tc_fence_before();
            mbar_arrive_warp(bars + UE0_0 + b);

            ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + UM4_0 + b, phb, status, abort_flag));
            tc_fence_after();
            uint32_t v[32];
            if (col0 < DV) {
                tmem_ld32(R + col0, v);
                tmem_wait_ld();
            }
            tc_fence_before();
            mbar_arrive_warp(bars + UE3_0 + b);
            if (tid == 0) tma_store_wait_read();       // the previous tile's store has left the staging tile
            epi_sync();
            if (col0 < DV) store_row_f32x32_bf16(v, sStg, r, col0);
            sRed[g * 128 + r] = dz;
            fence_async_smem();
            epi_sync();
            if (tid == 0) {
                for (int a = 0; a < DV / 64; ++a) tma_store_2d(&p.mapPN, sStg + a * 16384, a * 64, (int)(prow0 + (size_t)(t0 + i) * 128));
                tma_store_commit();
            }
            if (g == 0) {
                const float den = sRed[r] + sRed[128 + r] + sRed[256 + r] + sRed[384 + r];
                float *dst = p.pdr + 8 * (prow0 + (size_t)(t0 + i) * 128 + r);
                *reinterpret_cast<float4 *>(dst) = make_float4(den, 0.f, 0.f, 0.f);
                dst[4] = rmax + cshift;
            }
            quarter_sync(q4);
        }
        if (tid == 0) tma_store_wait_all();
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// Sb[bh,l,:] = bf16(Sacc[bh,l,:])  (operand of the query pass); z is copied beside it where the backward pass
// will look for it (zout == z when that is the workspace itself)
__global__ void state_to_bf16_kernel(const float *S, __nv_bfloat16 *Sb, long long n, const float *z, float *zout, long long nz)
{
    const long long i0 = blockIdx.x * (long long)blockDim.x + threadIdx.x, step = (long long)gridDim.x * blockDim.x;
    for (long long i = i0; i < n; i += step) Sb[i] = __float2bfloat16_rn(S[i]);
    if (zout != z)
        for (long long i = i0; i < nz; i += step) zout[i] = z[i];
}

// In-place exclusive prefix over the segments of S[bh, seg, e] (e over m*dv) and z[bh, seg, l]; Sb receives the bf16
// copy of the prefixed S. One thread per (bh, e).
__global__ void segment_prefix_kernel(float *S, __nv_bfloat16 *Sb, float *z, int nseg, long long E, int m, long long total)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= total) return;
    const long long bh = i / E, e = i % E;
    float run = 0.f;
    for (int s = 0; s < nseg; ++s) {
        const long long at = (bh * nseg + s) * E + e;
        const float v = S[at];
        S[at] = run;
        Sb[at] = __float2bfloat16_rn(run);
        run += v;
    }
    if (e < m) {
        float zr = 0.f;
        for (int s = 0; s < nseg; ++s) {
            const long long at = (bh * nseg + s) * m + e;
            const float v = z[at];
            z[at] = zr;
            zr += v;
        }
    }
}

// O[row,:] = sum_s num_s[row,:] 2^(rho_s - rho) / sum_s den_s 2^(rho_s - rho), rho = max_s rho_s; den_s is the sum of
// the slab's four partial normalisers. One thread per 8 output columns. The combined normaliser and rho are also
// written to sv for the backward pass; a normaliser that is zero or not finite is reported through the status word.
// NS > 0: the number of slabs at compile time (all loads of a thread are issued before the first use).
template <int NS>
__global__ void combine_kernel(const __nv_bfloat16 *pnum, const float *pdr, __nv_bfloat16 *O, float2 *sv,
                               long long rows, int dv, int nslab_rt, int *status)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const int per_row = dv / 8;
    if (i >= rows * per_row) return;
    const long long row = i / per_row;
    const int c0 = (int)(i % per_row) * 8;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, den = 0.f, rho = -INFINITY;
    auto slab_den = [](const float4 &d4) { return (d4.x + d4.y) + (d4.z + d4.w); };
    if constexpr (NS > 0) {
        float4 d4[NS];
        float rh[NS];
        uint4 raw[NS];
#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const float *q = pdr + 8 * ((size_t)s * rows + row);
            d4[s] = *reinterpret_cast<const float4 *>(q);
            rh[s] = q[4];
            raw[s] = *reinterpret_cast<const uint4 *>(pnum + ((size_t)s * rows + row) * dv + c0);
        }
#pragma unroll
        for (int s = 0; s < NS; ++s) rho = fmaxf(rho, rh[s]);
#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const float w = exp2f(rh[s] - rho);
            den = fmaf(slab_den(d4[s]), w, den);
            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw[s]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __bfloat1622float2(h2[q]);
                acc[2 * q] = fmaf(f.x, w, acc[2 * q]);
                acc[2 * q + 1] = fmaf(f.y, w, acc[2 * q + 1]);
            }
        }
    } else {
        for (int s = 0; s < nslab_rt; ++s) rho = fmaxf(rho, pdr[8 * ((size_t)s * rows + row) + 4]);
        for (int s = 0; s < nslab_rt; ++s) {
            const float *q = pdr + 8 * ((size_t)s * rows + row);
            const float w = exp2f(q[4] - rho);
            den = fmaf(slab_den(*reinterpret_cast<const float4 *>(q)), w, den);
            const uint4 raw = *reinterpret_cast<const uint4 *>(pnum + ((size_t)s * rows + row) * dv + c0);
            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) {
                const float2 f = __bfloat1622float2(h2[q2]);
                acc[2 * q2] = fmaf(f.x, w, acc[2 * q2]);
                acc[2 * q2 + 1] = fmaf(f.y, w, acc[2 * q2 + 1]);
            }
        }
    }
    if (c0 == 0) {
        sv[row] = make_float2(den, rho);
        if (!(den > 0.f) || !isfinite(den)) atomicCAS(status, 0, (int)DARKATTN_ERR_NONFINITE);
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
    if constexpr (MODE == MODE_CAUSAL) {
        using L = FwdCausalSmem<D, DV>;
        static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
        cudaError_t e = cudaFuncSetAttribute(tc_fwd_causal_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e != cudaSuccess) return e;
        tc_fwd_causal_kernel<D, DV><<<grid, kThreads, L::kTotal, st>>>(P);
    } else if constexpr (MODE == MODE_KEYS) {
        using L = FwdKeysSmem<D, DV>;
        static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
        cudaError_t e = cudaFuncSetAttribute(tc_fwd_keys_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e != cudaSuccess) return e;
        tc_fwd_keys_kernel<D, DV><<<grid, kThreads, L::kTotal, st>>>(P);
    } else {
        using L = FwdQueriesSmem<D, DV>;
        static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
        cudaError_t e = cudaFuncSetAttribute(tc_fwd_queries_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e != cudaSuccess) return e;
        tc_fwd_queries_kernel<D, DV><<<grid, kThreads, L::kTotal, st>>>(P);
    }
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
    const long long units = (long long)BH * Y.nslab;
    if (!D.causal) {
        nsplit = pick_splits(units, Y.T, 1.4, 5.0, kMaxNsplit);
    } else if (units * 2 <= 148) {
        // few long sequences: cut each into segments (a key pass computes the segment states, the causal
        // kernels of all segments then run side by side), as many as fill the SMs, at least 4 chunks each
        nsplit = (int)(148 / units);
        if (nsplit > Y.T / 4) nsplit = Y.T / 4;
        if (nsplit > 16) nsplit = 16;
        if (nsplit < 1) nsplit = 1;
    }
    Y.nsplit = nsplit;
    const size_t nstate = D.causal ? (size_t)nsplit : 1;
    size_t off = 0;
    Y.status = take(off, 256);
    Y.Om = take(off, (size_t)D.H * m * d * 2);
    Y.Oml = take(off, (size_t)D.H * m * d * 2);
    Y.cs = take(off, BH * Y.nslab * 4);
    Y.nK = take(off, BH * N * 4);
    Y.pnum = take(off, (size_t)Y.nslab * BH * N * dv * 2);
    Y.pdr = take(off, (size_t)Y.nslab * BH * N * 32);
    Y.Sacc = take(off, BH * nstate * m * dv * 4);
    Y.zacc = take(off, BH * nstate * m * 4);
    Y.Sb = take(off, BH * nstate * m * dv * 2);
    Y.sv = take(off, BH * N * 8);
    Y.zc = take(off, D.causal ? BH * (size_t)Y.T * m * 4 : 0);
    plan->launches_fwd = D.causal ? (nsplit > 1 ? 7 : 5) : 7;
    {
        size_t so = 0;
        Y.sv_sv = take(so, BH * N * 8);
        Y.sv_nK = take(so, BH * N * 4);
        Y.sv_Om = take(so, (size_t)D.H * m * d * 2);
        Y.sv_Oml = take(so, (size_t)D.H * m * d * 2);
        Y.sv_cs = take(so, BH * Y.nslab * 4);
        Y.sv_zc = take(so, D.causal ? BH * (size_t)Y.T * m * 4 : 0);
        Y.sv_Sb = take(so, D.causal ? 0 : BH * m * dv * 2);
        Y.sv_zt = take(so, D.causal ? 0 : BH * m * 4);
        Y.sv_Sst = take(so, D.causal ? BH * (size_t)Y.T * m * dv * 2 : 0);
        Y.sv_Bphi = take(so, D.causal ? BH * N * m * 2 : 0);
        Y.sv_bytes = so;
        plan->saved_bytes = so;
    }
    // backward pass
    Y.Oscr = take(off, BH * N * dv * 2);
    Y.delta = take(off, BH * N * 4);
    Y.rhoc = take(off, D.causal ? BH * (size_t)Y.T * m * 4 : 0);
    Y.espart = take(off, (size_t)4 * Y.nslab * BH * N * 4);
    Y.Tacc = take(off, (size_t)D.H * m * d * 4);
    Y.dMn = take(off, (size_t)D.H * D.r * d * 4);
    Y.dKh = take(off, D.G > 1 ? BH * N * d * 2 : 0);
    Y.dVh = take(off, D.G > 1 ? BH * N * dv * 2 : 0);
    Y.Sst = take(off, D.causal ? BH * (size_t)Y.T * m * dv * 2 : 0);
    Y.Ahat = take(off, D.causal ? BH * N * m * 2 : 0);
    Y.Bphi = take(off, D.causal ? BH * N * m * 2 : 0);
    Y.Racc = take(off, D.causal ? 0 : BH * m * dv * 4);
    Y.rhot = take(off, D.causal ? 0 : BH * m * 4);
    Y.Rb = take(off, D.causal ? 0 : BH * m * dv * 2);
    // with `saved`; without it the forward launches come on top. Causal: delta, two scan kernels, dK finishing, the
    // dM product and the small kernel that adds the norm term's part; non-causal: one more for the rounding of R
    // between the two passes. (With per-kernel timing on, dM is one kernel.)
    plan->launches_bwd = (D.causal ? 6 : 7) + (D.G > 1 ? 2 : 0);      // (+ the two sums over the groups of query heads)
    Y.total_bytes = off;
    plan->workspace_bytes = Y.total_bytes;
}

cudaError_t tensor_prologue(const darkattn_plan_s *plan, const void *K, const void *M, const void *W, char *ws,
                            const Stash &out, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    PrepassParams PP;
    memset(&PP, 0, sizeof(PP));
    const size_t BHkv = (size_t)D.B * D.Hkv;
    if (!make_map(&PP.mapK, K, BHkv * N, D.d, 128) || !make_map(&PP.mapM, M, (size_t)D.H * D.r, D.d, 128) ||
        !make_map(&PP.mapOm, out.Om, (size_t)D.H * D.m, D.d, 128))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaSuccess;
    auto chk = [&]() { cudaError_t x = cudaGetLastError(); if (x != cudaSuccess && e == cudaSuccess) e = x; };

    // The two small kernels that read only M and W run on the plan's side stream (with per-kernel timing on,
    // everything stays on one stream).
    const bool beside = !plan->timer.on && ensure_aux(plan) == cudaSuccess;
    cudaStream_t sp = beside ? plan->aux_stream : st;
    if (beside) {
        e = cudaEventRecord(plan->aux_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sp, plan->aux_fork, 0);
    }
    timer_mark(plan, st, "fold_omega_kernel");
    if (D.d == 64)
        fold_omega_kernel<2><<<dim3(D.m / 16, D.H), 128, 0, sp>>>((const __nv_bfloat16 *)W, (const __nv_bfloat16 *)M, out.Om, out.Oml, D.m, D.r,
                                                               D.w_per_head, kLog2e * D.s);
    else
        fold_omega_kernel<4><<<dim3(D.m / 16, D.H), 128, 0, sp>>>((const __nv_bfloat16 *)W, (const __nv_bfloat16 *)M, out.Om, out.Oml, D.m, D.r,
                                                               D.w_per_head, kLog2e * D.s);
    chk();
    timer_mark(plan, st, "shift_init_kernel");
    shift_init_kernel<<<(unsigned)((BH * Y.nslab + 255) / 256), 256, 0, sp>>>(reinterpret_cast<int *>(out.cs), (int)(BH * Y.nslab));
    chk();
    if (beside && e == cudaSuccess) e = cudaEventRecord(plan->aux_join, sp);

    if (beside && e == cudaSuccess) e = cudaStreamWaitEvent(st, plan->aux_join, 0);

    // key norms and key-side shifts in one pass over K
    PP.nK = out.nK; PP.cs = reinterpret_cast<int *>(out.cs); PP.status = reinterpret_cast<int *>(ws + Y.status);
    PP.N = D.N; PP.H = D.H; PP.Hkv = D.Hkv; PP.T = Y.T; PP.m = D.m; PP.r = D.r; PP.nslab = Y.nslab; PP.npair = (Y.nslab + 1) / 2;
    PP.coef = kLog2e * 0.5f * D.s * D.s;
    const int per_sm = D.d == 64 ? 2 : 1;                           // CTAs of this kernel that fit one SM
    PP.nsplit = pick_splits((long long)BH * PP.npair, Y.T, 1.5, 3.0, 64, per_sm * 148);
    const int smem_bytes = 5 * 128 * D.d * 2 + 128;
    timer_mark(plan, st, "tc_key_prepass_kernel");
    if (D.d == 64) {
        cudaFuncSetAttribute(tc_key_prepass_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        tc_key_prepass_kernel<64><<<(unsigned)(BH * PP.npair * PP.nsplit), 160, smem_bytes, st>>>(PP);
    } else {
        cudaFuncSetAttribute(tc_key_prepass_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        tc_key_prepass_kernel<128><<<(unsigned)(BH * PP.npair * PP.nsplit), 160, smem_bytes, st>>>(PP);
    }
    chk();
    return e;
}

darkattn_status_t tensor_forward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                 const void *M, const void *W, void *O, void *saved, char *ws, cudaStream_t st, bool stash_states)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16 *>(ws + off); };
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    if (!encode_fn()) { set_cuda_error(cudaErrorNotSupported, "tensor_forward: cuTensorMapEncodeTiled unavailable"); return DARKATTN_ERR_CUDA; }

    const Stash stash = saved ? stash_in_saved(Y, saved) : stash_in_workspace(Y, ws);
    MainParams P;
    memset(&P, 0, sizeof(P));
    const size_t BHkv = (size_t)D.B * D.Hkv;
    bool ok = make_map(&P.mapQ, Q, BH * N, D.d, 128) && make_map(&P.mapK, K, BHkv * N, D.d, 128) &&
              make_map(&P.mapV, V, BHkv * N, D.dv, 128) && make_map(&P.mapOm, stash.Om, (size_t)D.H * D.m, D.d, 128) &&
              make_map(&P.mapOml, stash.Oml, (size_t)D.H * D.m, D.d, 128) &&
              make_map(&P.mapSb, D.causal ? bf(Y.Sb) : stash.Sb, BH * (D.causal ? Y.nsplit : 1) * D.m, D.dv, 128) &&
              make_map(&P.mapPN, bf(Y.pnum), (size_t)Y.nslab * BH * N, D.dv, 128);
    if (!ok) { set_cuda_error(cudaErrorInvalidValue, "tensor_forward: tensor map encode"); return DARKATTN_ERR_CUDA; }

    cudaError_t e = tensor_prologue(plan, K, M, W, ws, stash, st);
    auto chk = [&]() { cudaError_t x = cudaGetLastError(); if (x != cudaSuccess && e == cudaSuccess) e = x; };

    P.nK = stash.nK; P.cs = stash.cs; P.zc = stash.zc; P.pdr = fl(Y.pdr); P.Sacc = fl(Y.Sacc); P.zacc = fl(Y.zacc);
    P.status = reinterpret_cast<int *>(ws + Y.status);
    P.N = D.N; P.H = D.H; P.Hkv = D.Hkv; P.BH = D.BH; P.m = D.m; P.nslab = Y.nslab; P.T = Y.T; P.nsplit = Y.nsplit;
    P.stash_S = (D.causal && stash_states) ? 1 : 0;
    if (P.stash_S && !(make_map(&P.mapSst, stash.Sst, BH * Y.T * D.m, D.dv, 128) && make_map(&P.mapBf, stash.Bphi, BH * N, D.m, 128))) {
        set_cuda_error(cudaErrorInvalidValue, "tensor_forward: tensor map encode");
        return DARKATTN_ERR_CUDA;
    }
    const int units = (int)(BH * Y.nslab);
    if (D.causal) {
        if (Y.nsplit > 1) {      // segment states, then their exclusive prefix
            P.Sseg = fl(Y.Sacc); P.zseg = fl(Y.zacc);
            timer_mark(plan, st, "tc_fwd_keys_kernel");
            cudaError_t x = launch_main_shape<MODE_KEYS>(D.d, D.dv, P, units * Y.nsplit, st);
            if (x != cudaSuccess && e == cudaSuccess) e = x;
            const long long E = (long long)D.m * D.dv, total = (long long)BH * E;
            timer_mark(plan, st, "segment_prefix_kernel");
            segment_prefix_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(fl(Y.Sacc), bf(Y.Sb), fl(Y.zacc), Y.nsplit, E, D.m, total);
            chk();
        }
        timer_mark(plan, st, "tc_fwd_causal_kernel");
        cudaError_t x = launch_main_shape<MODE_CAUSAL>(D.d, D.dv, P, units * Y.nsplit, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
    } else {
        e = (e == cudaSuccess) ? cudaMemsetAsync(ws + Y.Sacc, 0, (Y.Sb - Y.Sacc), st) : e;   // S and z sums
        timer_mark(plan, st, "tc_fwd_keys_kernel");
        cudaError_t x = launch_main_shape<MODE_KEYS>(D.d, D.dv, P, units * Y.nsplit, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
        const long long n = (long long)BH * D.m * D.dv;
        timer_mark(plan, st, "state_to_bf16_kernel");
        state_to_bf16_kernel<<<(unsigned)((n + 1023) / 1024), 256, 0, st>>>(fl(Y.Sacc), stash.Sb, n, fl(Y.zacc), stash.zt, (long long)BH * D.m);
        chk();
        timer_mark(plan, st, "tc_fwd_queries_kernel");
        x = launch_main_shape<MODE_QUERIES>(D.d, D.dv, P, units * Y.nsplit, st);
        if (x != cudaSuccess && e == cudaSuccess) e = x;
    }
    {
        const long long rows = (long long)BH * N, threads = rows * (D.dv / 8);
        timer_mark(plan, st, "combine_kernel");
        const unsigned grid = (unsigned)((threads + 255) / 256);
        __nv_bfloat16 *Ob = (__nv_bfloat16 *)O;
        if (Y.nslab == 1) combine_kernel<1><<<grid, 256, 0, st>>>(bf(Y.pnum), fl(Y.pdr), Ob, stash.sv, rows, D.dv, 1, P.status);
        else if (Y.nslab == 2) combine_kernel<2><<<grid, 256, 0, st>>>(bf(Y.pnum), fl(Y.pdr), Ob, stash.sv, rows, D.dv, 2, P.status);
        else if (Y.nslab == 4) combine_kernel<4><<<grid, 256, 0, st>>>(bf(Y.pnum), fl(Y.pdr), Ob, stash.sv, rows, D.dv, 4, P.status);
        else combine_kernel<0><<<grid, 256, 0, st>>>(bf(Y.pnum), fl(Y.pdr), Ob, stash.sv, rows, D.dv, Y.nslab, P.status);
        chk();
    }
    if (e != cudaSuccess) { set_cuda_error(e, "tensor_forward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

}  // namespace darkattn
