// Tensor-core backward pass of causal DARK attention: gradients with respect to Q, K, V and M.
//
// Notation (per batch, head and slab of 128 features; log2 units as in the forward kernels):
//   A^_il   = 2^(U^Q_il - aq_i),  aq_i = rho_i - c + log2(den_i)     query features divided by the normaliser
//   Bf_jl   = 2^(U^K_jl - n_j - c)                                    key features
//   dP_ij   = dO_i . V_j - delta_i  (j <= i),  delta_i = dO_i . O_i   gradient of the unnormalised kernel value
//   E^Q_il  = A^_il ( sum_{j<=i} dP_ij Bf_jl )            = A^ .* ( dP Bf  +  dO S_prev^T - delta z_prev^T )
//   E^K_jl  = Bf_jl ( sum_{i>=j} dP_ij A^_il )            = Bf .* ( dP^T A^ +  V R_next^T + rho_next^T )
//   dV_j    = sum_{i>=j} (A^_i . Bf_j) dO_i               = P^^T dO + Bf R_next
//   S, z    : prefix sums of Bf^T V and Bf^T 1 over earlier chunks (forward direction)
//   R, rho  : suffix sums of A^^T dO and -A^^T delta over later chunks (reverse direction)
//   dQ = ln2 E^Q Omega,   dK = ln2 E^K Omega - rowsum(E^K) s^2 M^T M k,   T = E^Q^T Q + E^K^T K,
//   dM = s W^T T - s^2 sum_j rowsum(E^K)_j (M k_j) k_j^T
// (chain rule through the definitions of the feature map and of the attention; every stabilising
// shift is a constant because the output does not depend on it).
//
// Two scan kernels walk the chunks of a sequence, one CTA per (batch, head, slab): the query-side
// kernel forwards (state S in TMEM), the key-side kernel backwards (state R in TMEM). Features are
// recomputed from Q, K and the folded projections and never leave the SM. The 128 x 128 tiles dP
// (query side) and P^^T, dP^T (key side) are written back to tensor memory as bf16 and used as the
// A operand of the next MMA directly from there. Slab partials of dQ, dK, dV go to the workspace in
// bf16 and are summed by small kernels; the key-side one also applies the norm term with three MMAs.
#include "common.cuh"
#include "tc_common.cuh"

#include <math.h>
#include <string.h>

namespace darkattn {

using namespace tc;

namespace {

constexpr float kLn2 = 0.6931471805599453f;

struct BwdParams {
    CUtensorMap mapQ, mapK, mapV, mapG, mapOm;
    const float2 *sv;     // [BH*N]  (normaliser, exponent it is scaled by) from the forward pass
    const float *delta;   // [BH*N]  dO_i . O_i
    const float *nK;      // [BH*N]  key norms, log2 units
    const float *cs;      // [BH*nslab] key-side shift per slab
    float *rhoc;          // [BH, T, m] per-chunk -sum_i A^_il delta_i (written by the query-side kernel)
    __nv_bfloat16 *pdQ, *pdK, *pdV;   // slab partials
    float *espart;        // [nslab, BH*N] slab partials of rowsum(E^K)
    float *Tacc;          // [H, m, D]
    int *status;
    int N, H, BH, m, nslab, T;
};

template <int D, int DV>
struct BwdSmem {
    static constexpr int kDmax = D > DV ? D : DV;
    static constexpr int kOm = 0;                          // folded projections of the slab [128 l, D]
    static constexpr int kQA = kOm + 128 * D * 2;          // Q tile, then A^ (then E^Q)       [128, 128]
    static constexpr int kKB = kQA + 32768;                // K tile, then Bf (then E^K)        [128, 128]
    static constexpr int kV = kKB + 32768;                 // V tile                            [128, DV]
    static constexpr int kG = kV + 128 * DV * 2;           // dO tile; later the reloaded Q / K tile
    static constexpr int kSt = kG + 128 * kDmax * 2;       // bf16 copy of the scan state       [128 l, DV]
    static constexpr int kB1 = kSt + 128 * DV * 2;         // 16 x 128 operand: a row of ones
    static constexpr int kB2 = kB1 + 4096;                 // 16 x 128 operand: rows hi(-delta), lo(-delta)
    static constexpr int kVec = kB2 + 4096;                // two float[128]
    static constexpr int kBars = kVec + 1024;
    static constexpr int kTotal = kBars + 256;
};

// TMEM columns (512 allocated): scan state at 0, T at 128, scratch R1 at 256 and R2 at 384.
constexpr uint32_t kColState = 0, kColT = 128, kColR1 = 256, kColR2 = 384;

__device__ __forceinline__ unsigned char *tile_chunk(unsigned char *base, int row, int chunk16)
{
    return base + (chunk16 >> 3) * 16384 + swz128((uint32_t)row, (uint32_t)(chunk16 & 7));
}

__device__ __forceinline__ uint4 pack8(const uint32_t *v)
{
    return make_uint4(pack_bf16(__uint_as_float(v[0]), __uint_as_float(v[1])), pack_bf16(__uint_as_float(v[2]), __uint_as_float(v[3])),
                      pack_bf16(__uint_as_float(v[4]), __uint_as_float(v[5])), pack_bf16(__uint_as_float(v[6]), __uint_as_float(v[7])));
}

__device__ __forceinline__ void unpack8(const uint4 &raw, float *f)
{
    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 x = __bfloat1622float2(h2[q]);
        f[2 * q] = x.x;
        f[2 * q + 1] = x.y;
    }
}

// features 2^(U - offset) of one row: TMEM columns [col, col+128) -> bf16 tile row `row`
__device__ __forceinline__ void features_to_tile(uint32_t taddr, float offset, unsigned char *tile, int row)
{
    for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t v[32], pk[16];
        tmem_ld32(taddr + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; j += 2)
            pk[j / 2] = pack_bf16(ex2f(__uint_as_float(v[j]) - offset), ex2f(__uint_as_float(v[j + 1]) - offset));
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(tile_chunk(tile, row, c0 / 8 + q)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
    }
}

// fp32 TMEM columns [taddr, taddr + width) of one row -> bf16 tile row (swizzled smem)
template <int WIDTH>
__device__ __forceinline__ void tmem_row_to_tile(uint32_t taddr, unsigned char *tile, int row)
{
    for (int c0 = 0; c0 < WIDTH; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(taddr + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(tile_chunk(tile, row, c0 / 8 + q)) = pack8(v + 8 * q);
    }
}

// fp32 TMEM columns of one row -> bf16 row in global memory (dst points at the row)
template <int WIDTH>
__device__ __forceinline__ void tmem_row_to_global(uint32_t taddr, __nv_bfloat16 *dst)
{
    for (int c0 = 0; c0 < WIDTH; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(taddr + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(dst + c0 + 8 * q) = pack8(v + 8 * q);
    }
}

enum QBars { QB_OM, QB_Q, QB_K, QB_V, QB_G, QB_X2, QM1, QM2, QM3, QMS, QM4, QM5, QM6, QE1, QE2, QE3, QE4, QNBARS };

// ------------------------------------------------------------------ query side (forward direction)
template <int D, int DV>
__global__ void __launch_bounds__(160, 1) tc_bwd_q_kernel(const __grid_constant__ BwdParams p)
{
    using L = BwdSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sQA = smem + L::kQA, *sKB = smem + L::kKB, *sV = smem + L::kV;
    unsigned char *sG = smem + L::kG, *sSt = smem + L::kSt, *sB1 = smem + L::kB1, *sB2 = smem + L::kB2;
    float *sZ = reinterpret_cast<float *>(smem + L::kVec);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + QNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + QNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nslab, slab = blockIdx.x % p.nslab, h = bh % p.H;
    const int row0 = bh * p.N, T = p.T;

    if (tid == 0) {
        for (int i = 0; i < QE1; ++i) mbar_init(bars + i, 1);
        for (int i = QE1; i < QNBARS; ++i) mbar_init(bars + i, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) {
        for (int i = tid; i < 256; i += 128) {
            *reinterpret_cast<uint4 *>(sB1 + i * 16) = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
            *reinterpret_cast<uint4 *>(sB2 + i * 16) = make_uint4(0, 0, 0, 0);
        }
        sZ[tid] = 0.f;
    }
    if (warp == 4) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (warp == 4) {
        if ((tid & 31) == 0) {
            auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                mbar_expect_tx(bar, 128 * width * 2);
                for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, row0 + t * 128);
            };
            auto kdesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024); };
            auto mndesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + k * 2048, 16384, 1024); };
            auto bdesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + (k / 4) * 2048 + (k % 4) * 32, 16, 1024); };
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_vec = make_idesc(128, 16, 1, 0);
            const uint32_t id_state = make_idesc(128, DV, 1, 1);
            const uint32_t id_tm = make_idesc(128, 128, 0, 1);
            const uint32_t id_dx = make_idesc(128, D, 0, 1);
            const uint32_t id_t = make_idesc(128, D, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2;

            mbar_expect_tx(bars + QB_OM, 128 * D * 2);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sOm + a * 16384, &p.mapOm, bars + QB_OM, a * 64, h * p.m + slab * 128);
            load_tile(sQA, &p.mapQ, bars + QB_Q, D, 0);
            load_tile(sKB, &p.mapK, bars + QB_K, D, 0);
            load_tile(sV, &p.mapV, bars + QB_V, DV, 0);
            load_tile(sG, &p.mapG, bars + QB_G, DV, 0);

            bool ok = wait_or_abort(bars + QB_OM, 0, status, abort_flag);
            for (int t = 0; t < T && ok; ++t) {
                const uint32_t ph = t & 1;
                const bool first = (t == 0), last = (t + 1 == T);
#define QWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
                QWAIT(QB_Q); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k) mma_ss(R1, kdesc(sQA, k), kdesc(sOm, k), id_kk, k > 0);       // U_Q
                mma_commit(bars + QM1);
                QWAIT(QB_K); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k) mma_ss(R2, kdesc(sKB, k), kdesc(sOm, k), id_kk, k > 0);       // U_K
                mma_commit(bars + QM2);
                QWAIT(QE1); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ss(R2, mndesc(sKB, k), bdesc(sB1, k), id_vec, k > 0);           // z_c = Bf^T 1
                for (int k = 0; k < 8; ++k) mma_ss(R2 + 16, mndesc(sQA, k), bdesc(sB2, k), id_vec, k > 0);      // rho_c = -A^^T delta
                QWAIT(QB_V); if (!ok) break;
                QWAIT(QB_G); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < DV / 16; ++k) mma_ss(R1, kdesc(sG, k), kdesc(sV, k), id_kk, k > 0);         // dO V^T
                mma_commit(bars + QM3);
                for (int k = 0; k < 8; ++k) mma_ss(tmem + kColState, mndesc(sKB, k), mndesc(sV, k), id_state, (!first) || k > 0);   // S += Bf^T V
                mma_commit(bars + QMS);
                QWAIT(QE2); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + k * 8, mndesc(sKB, k), id_tm, k > 0);               // dP Bf
                if (!first)
                    for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(sG, k), kdesc(sSt, k), id_kk, 1);        // + dO S_prev^T
                mma_commit(bars + QM4);
                QWAIT(QM4); if (!ok) break;
                load_tile(sG, &p.mapQ, bars + QB_X2, D, t);                                                     // Q again, for T
                if (!last) { load_tile(sV, &p.mapV, bars + QB_V, DV, t + 1); load_tile(sKB, &p.mapK, bars + QB_K, D, t + 1); }
                QWAIT(QE3); if (!ok) break;
                QWAIT(QB_X2); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ss(R1, kdesc(sQA, k), mndesc(sOm, k), id_dx, k > 0);            // E Omega
                mma_commit(bars + QM5);
                for (int k = 0; k < 8; ++k) mma_ss(tmem + kColT, mndesc(sQA, k), mndesc(sG, k), id_t, (!first) || k > 0);   // T += E^T Q
                mma_commit(bars + QM6);
                QWAIT(QM6); if (!ok) break;
                if (!last) { load_tile(sQA, &p.mapQ, bars + QB_Q, D, t + 1); load_tile(sG, &p.mapG, bars + QB_G, DV, t + 1); }
                QWAIT(QE4); if (!ok) break;
#undef QWAIT
            }
        }
    } else {
        // ============================== epilogue threads: thread = TMEM lane = tile row
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        const float cshift = p.cs[bh * p.nslab + slab];
        float zrun = 0.f;
        bool ok = true;
        for (int t = 0; t < T && ok; ++t) {
            const uint32_t ph = t & 1;
            const bool last = (t + 1 == T);
            const size_t row = (size_t)row0 + (size_t)t * 128 + tid;
#define EWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
            const float2 svv = p.sv[row];
            const float del = p.delta[row];
            const float nk = p.nK[row] + cshift;
            const float aq = svv.y - cshift + log2f(svv.x);
            {   // rows 0 and 1 of the 16 x 128 operand: -delta split into two bf16 terms
                const __nv_bfloat16 hi = __float2bfloat16_rn(-del);
                const __nv_bfloat16 lo = __float2bfloat16_rn(-del - __bfloat162float(hi));
                const int atom = tid >> 6, kk = tid & 63, ch = kk >> 3;
                *reinterpret_cast<__nv_bfloat16 *>(sB2 + atom * 2048 + (ch << 4) + (kk & 7) * 2) = hi;
                *reinterpret_cast<__nv_bfloat16 *>(sB2 + atom * 2048 + 128 + ((ch ^ 1) << 4) + (kk & 7) * 2) = lo;
            }
            EWAIT(QM1); if (!ok) break;
            tc_fence_after();
            features_to_tile(R1, aq, sQA, tid);
            EWAIT(QM2); if (!ok) break;
            tc_fence_after();
            features_to_tile(R2, nk, sKB, tid);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bars + QE1);

            EWAIT(QM3); if (!ok) break;
            tc_fence_after();
            float znew;
            {
                uint32_t a[16], b[16];
                tmem_ld16(R2, a);
                tmem_ld16(R2 + 16, b);
                tmem_wait_ld();
                znew = zrun + __uint_as_float(a[0]);
                p.rhoc[((size_t)bh * T + t) * p.m + slab * 128 + tid] = __uint_as_float(b[0]) + __uint_as_float(b[1]);
            }
            for (int c0 = 0; c0 < 128; c0 += 32) {       // dP = tril(dO V^T - delta) as a bf16 operand in TMEM
                uint32_t v[32], pk[16];
                tmem_ld32(R1 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float x0 = (c0 + j <= tid) ? __uint_as_float(v[j]) - del : 0.f;
                    const float x1 = (c0 + j + 1 <= tid) ? __uint_as_float(v[j + 1]) - del : 0.f;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + c0 / 2, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bars + QE2);

            EWAIT(QM4); if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < 128; c0 += 32) {       // E = A^ .* (dP Bf + dO S^T - delta z^T), in place over A^
                uint32_t v[32];
                tmem_ld32(R2 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 *cell = reinterpret_cast<uint4 *>(tile_chunk(sQA, tid, c0 / 8 + q));
                    float a[8];
                    unpack8(*cell, a);
                    const float4 z0 = *reinterpret_cast<const float4 *>(sZ + c0 + 8 * q);
                    const float4 z1 = *reinterpret_cast<const float4 *>(sZ + c0 + 8 * q + 4);
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                    float e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) e[j] = a[j] * fmaf(-del, zz[j], __uint_as_float(v[8 * q + j]));
                    *cell = make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bars + QE3);

            EWAIT(QM5); if (!ok) break;
            tc_fence_after();
            tmem_row_to_global<D>(R1, p.pdQ + (((size_t)slab * p.BH + bh) * p.N + (size_t)t * 128 + tid) * D);
            EWAIT(QMS); if (!ok) break;
            zrun = znew;
            if (!last) {
                tmem_row_to_tile<DV>(lane_addr + kColState, sSt, tid);
                sZ[tid] = zrun;
                fence_async_smem();
            }
            tc_fence_before();
            mbar_arrive(bars + QE4);
#undef EWAIT
        }
        if (ok) ok = wait_or_abort(bars + QM6, (T - 1) & 1, status, abort_flag);
        if (ok) {
            tc_fence_after();
            float *dst = p.Tacc + ((size_t)h * p.m + slab * 128 + tid) * D;
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + kColT + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + c0 + j, __uint_as_float(v[j]));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);   // error path only: let copies and MMAs in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

enum KBars { KB_OM, KB_Q, KB_K, KB_V, KB_G, KB_X2, KM1, KM2, KM3, KM4, KM5, KM6, KM7, KM8, KM9, KE1, KE2, KE3, KE4, KE5, KNBARS };

// ------------------------------------------------------------------ key side (reverse direction)
template <int D, int DV>
__global__ void __launch_bounds__(160, 1) tc_bwd_k_kernel(const __grid_constant__ BwdParams p)
{
    using L = BwdSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sQA = smem + L::kQA, *sKB = smem + L::kKB, *sV = smem + L::kV;
    unsigned char *sG = smem + L::kG, *sSt = smem + L::kSt;
    float *sRho = reinterpret_cast<float *>(smem + L::kVec), *sDel = sRho + 128;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + KNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + KNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nslab, slab = blockIdx.x % p.nslab, h = bh % p.H;
    const int row0 = bh * p.N, T = p.T;

    if (tid == 0) {
        for (int i = 0; i < KE1; ++i) mbar_init(bars + i, 1);
        for (int i = KE1; i < KNBARS; ++i) mbar_init(bars + i, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) sRho[tid] = 0.f;
    if (warp == 4) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (warp == 4) {
        if ((tid & 31) == 0) {
            auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                mbar_expect_tx(bar, 128 * width * 2);
                for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, row0 + t * 128);
            };
            auto kdesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024); };
            auto mndesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + k * 2048, 16384, 1024); };
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_state = make_idesc(128, DV, 1, 1);
            const uint32_t id_dv_t = make_idesc(128, DV, 0, 1);
            const uint32_t id_tm = make_idesc(128, 128, 0, 1);
            const uint32_t id_dx = make_idesc(128, D, 0, 1);
            const uint32_t id_t = make_idesc(128, D, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2;

            mbar_expect_tx(bars + KB_OM, 128 * D * 2);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sOm + a * 16384, &p.mapOm, bars + KB_OM, a * 64, h * p.m + slab * 128);
            load_tile(sQA, &p.mapQ, bars + KB_Q, D, T - 1);
            load_tile(sKB, &p.mapK, bars + KB_K, D, T - 1);
            load_tile(sV, &p.mapV, bars + KB_V, DV, T - 1);
            load_tile(sG, &p.mapG, bars + KB_G, DV, T - 1);

            bool ok = wait_or_abort(bars + KB_OM, 0, status, abort_flag);
            for (int it = 0; it < T && ok; ++it) {
                const int t = T - 1 - it;
                const uint32_t ph = it & 1;
                const bool first = (it == 0), last = (it + 1 == T);
#define KWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
                KWAIT(KB_Q); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k) mma_ss(R1, kdesc(sQA, k), kdesc(sOm, k), id_kk, k > 0);       // U_Q
                mma_commit(bars + KM1);
                KWAIT(KB_K); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k) mma_ss(R2, kdesc(sKB, k), kdesc(sOm, k), id_kk, k > 0);       // U_K
                mma_commit(bars + KM2);
                KWAIT(KE1); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ss(R1, kdesc(sKB, k), kdesc(sQA, k), id_kk, k > 0);             // P^^T = Bf A^^T
                mma_commit(bars + KM3);
                KWAIT(KB_V); if (!ok) break;
                KWAIT(KB_G); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(sV, k), kdesc(sG, k), id_kk, k > 0);         // V dO^T
                mma_commit(bars + KM4);
                for (int k = 0; k < 8; ++k) mma_ss(tmem + kColState, mndesc(sQA, k), mndesc(sG, k), id_state, (!first) || k > 0);   // R += A^^T dO
                mma_commit(bars + KM5);
                KWAIT(KE2); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + k * 8, mndesc(sG, k), id_dv_t, k > 0);              // P^^T dO
                if (!first)
                    for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(sKB, k), mndesc(sSt, k), id_dv_t, 1);          // + Bf R_next
                mma_commit(bars + KM6);
                KWAIT(KE3); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + 64 + k * 8, mndesc(sQA, k), id_tm, k > 0);          // dP^T A^
                if (!first)
                    for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(sV, k), kdesc(sSt, k), id_kk, 1);        // + V R_next^T
                mma_commit(bars + KM7);
                KWAIT(KM7); if (!ok) break;
                load_tile(sG, &p.mapK, bars + KB_X2, D, t);                                                     // K again, for T
                if (!last) { load_tile(sQA, &p.mapQ, bars + KB_Q, D, t - 1); load_tile(sV, &p.mapV, bars + KB_V, DV, t - 1); }
                KWAIT(KE4); if (!ok) break;
                KWAIT(KB_X2); if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(sKB, k), mndesc(sOm, k), id_dx, k > 0);            // E Omega
                mma_commit(bars + KM8);
                for (int k = 0; k < 8; ++k) mma_ss(tmem + kColT, mndesc(sKB, k), mndesc(sG, k), id_t, (!first) || k > 0);   // T += E^T K
                mma_commit(bars + KM9);
                KWAIT(KM9); if (!ok) break;
                if (!last) { load_tile(sKB, &p.mapK, bars + KB_K, D, t - 1); load_tile(sG, &p.mapG, bars + KB_G, DV, t - 1); }
                KWAIT(KE5); if (!ok) break;
#undef KWAIT
            }
        }
    } else {
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        const float cshift = p.cs[bh * p.nslab + slab];
        bool ok = true;
        for (int it = 0; it < T && ok; ++it) {
            const int t = T - 1 - it;
            const uint32_t ph = it & 1;
            const bool last = (it + 1 == T);
            const size_t row = (size_t)row0 + (size_t)t * 128 + tid;
            const size_t prow = ((size_t)slab * p.BH + bh) * p.N + (size_t)t * 128 + tid;
#define EWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
            const float2 svv = p.sv[row];
            const float nk = p.nK[row] + cshift;
            const float aq = svv.y - cshift + log2f(svv.x);
            const float rho_c = p.rhoc[((size_t)bh * T + t) * p.m + slab * 128 + tid];
            sDel[tid] = p.delta[row];
            EWAIT(KM1); if (!ok) break;
            tc_fence_after();
            features_to_tile(R1, aq, sQA, tid);
            EWAIT(KM2); if (!ok) break;
            tc_fence_after();
            features_to_tile(R2, nk, sKB, tid);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bars + KE1);

            EWAIT(KM3); if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < 128; c0 += 32) {       // P^^T masked to queries i >= this key
                uint32_t v[32], pk[16];
                tmem_ld32(R1 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float x0 = (c0 + j >= tid) ? __uint_as_float(v[j]) : 0.f;
                    const float x1 = (c0 + j + 1 >= tid) ? __uint_as_float(v[j + 1]) : 0.f;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + c0 / 2, pk);
            }
            EWAIT(KM4); if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < 128; c0 += 32) {       // dP^T = (V dO^T - delta_i) masked
                uint32_t v[32], pk[16];
                tmem_ld32(R2 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float2 dl = *reinterpret_cast<const float2 *>(sDel + c0 + j);
                    const float x0 = (c0 + j >= tid) ? __uint_as_float(v[j]) - dl.x : 0.f;
                    const float x1 = (c0 + j + 1 >= tid) ? __uint_as_float(v[j + 1]) - dl.y : 0.f;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + 64 + c0 / 2, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bars + KE2);

            EWAIT(KM6); if (!ok) break;
            tc_fence_after();
            tmem_row_to_global<DV>(R2, p.pdV + prow * DV);
            tc_fence_before();
            mbar_arrive(bars + KE3);

            EWAIT(KM7); if (!ok) break;
            tc_fence_after();
            float es = 0.f;
            for (int c0 = 0; c0 < 128; c0 += 32) {       // E = Bf .* (dP^T A^ + V R^T + rho^T), in place over Bf
                uint32_t v[32];
                tmem_ld32(R2 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 *cell = reinterpret_cast<uint4 *>(tile_chunk(sKB, tid, c0 / 8 + q));
                    float b[8];
                    unpack8(*cell, b);
                    const float4 r0 = *reinterpret_cast<const float4 *>(sRho + c0 + 8 * q);
                    const float4 r1 = *reinterpret_cast<const float4 *>(sRho + c0 + 8 * q + 4);
                    const float rr[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
                    float e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) { e[j] = b[j] * (__uint_as_float(v[8 * q + j]) + rr[j]); es += e[j]; }
                    *cell = make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                }
            }
            p.espart[prow] = es;
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bars + KE4);

            EWAIT(KM8); if (!ok) break;
            tc_fence_after();
            tmem_row_to_global<D>(R2, p.pdK + prow * D);
            if (!last) {     // R (updated before KM6 completed) -> bf16 copy; rho_next for the chunk below
                tmem_row_to_tile<DV>(lane_addr + kColState, sSt, tid);
                sRho[tid] += rho_c;
                fence_async_smem();
            }
            tc_fence_before();
            mbar_arrive(bars + KE5);
#undef EWAIT
        }
        if (ok) ok = wait_or_abort(bars + KM9, (T - 1) & 1, status, abort_flag);
        if (ok) {
            tc_fence_after();
            float *dst = p.Tacc + ((size_t)h * p.m + slab * 128 + tid) * D;
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + kColT + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + c0 + j, __uint_as_float(v[j]));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ dK: slab sum + norm term (three MMAs per tile)
//   x~'  = K M^T                      (128 x r)
//   w_j  = -s^2 rowsum(E^K)_j x~'_j   (bf16 operand)
//   dK_j = ln2 sum_slabs part_j + w_j M          dMn += w^T K
struct FinishParams {
    CUtensorMap mapK, mapM;
    const __nv_bfloat16 *pdK;
    const float *espart;
    __nv_bfloat16 *dK;
    float *dMn;           // [H, r, D]
    int *status;
    int N, H, BH, T, nsplit, r, nslab;
    float s2;
};

template <int D>
__global__ void __launch_bounds__(160, 1) tc_bwd_finish_k_kernel(const __grid_constant__ FinishParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kTile = 128 * D * 2;
    unsigned char *sM = smem, *sK = smem + kTile, *sW = smem + 2 * kTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 2 * kTile + 32768);
    uint64_t *bar_m = bars, *bar_k = bars + 1, *m1 = bars + 2, *m2 = bars + 3, *m3 = bars + 4, *e1 = bars + 5, *e2 = bars + 6;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 7);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 8);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    if (tid == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(bars + i, 1);
        mbar_init(e1, 128); mbar_init(e2, 128);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128)      // columns >= r of the w tile stay zero
        for (int i = tid; i < 2048; i += 128) *reinterpret_cast<uint4 *>(sW + i * 16) = make_uint4(0, 0, 0, 0);
    if (warp == 4) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t C1 = 0, C2 = 128, C3 = 256;
    if (*abort_flag) { if (tid == 0) atomicExch(p.status, (int)DARKATTN_ERR_CUDA); }
    else if (t1 <= t0) {}
    else if (warp == 4) {
        if ((tid & 31) == 0) {
            auto kdesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + (k / 4) * 16384 + (k % 4) * 32, 16, 1024); };
            auto mndesc = [](unsigned char *base, int k) { return make_sdesc(smem_u32(base) + k * 2048, 16384, 1024); };
            mbar_expect_tx(bar_m, kTile);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sM + a * 16384, &p.mapM, bar_m, a * 64, h * p.r);
            mbar_expect_tx(bar_k, kTile);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sK + a * 16384, &p.mapK, bar_k, a * 64, bh * p.N + t0 * 128);
            const uint32_t id_x = make_idesc(128, p.r, 0, 0), id_d = make_idesc(128, D, 0, 1), id_t = make_idesc(128, D, 1, 1);
            bool ok = wait_or_abort(bar_m, 0, p.status, abort_flag);
            for (int t = t0; t < t1 && ok; ++t) {
                const uint32_t ph = (t - t0) & 1;
                ok = wait_or_abort(bar_k, ph, p.status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < D / 16; ++k) mma_ss(tmem + C1, kdesc(sK, k), kdesc(sM, k), id_x, k > 0);
                mma_commit(m1);
                ok = wait_or_abort(e1, ph, p.status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < p.r / 16; ++k) mma_ss(tmem + C2, kdesc(sW, k), mndesc(sM, k), id_d, k > 0);
                mma_commit(m2);
                for (int k = 0; k < 8; ++k) mma_ss(tmem + C3, mndesc(sW, k), mndesc(sK, k), id_t, (t > t0) || k > 0);
                mma_commit(m3);
                ok = wait_or_abort(m3, ph, p.status, abort_flag);
                if (!ok) break;
                if (t + 1 < t1) {
                    mbar_expect_tx(bar_k, kTile);
                    for (int a = 0; a < D / 64; ++a) tma_load_2d(sK + a * 16384, &p.mapK, bar_k, a * 64, bh * p.N + (t + 1) * 128);
                }
                ok = wait_or_abort(e2, ph, p.status, abort_flag);
            }
        }
    } else {
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const size_t rows = (size_t)p.BH * p.N;
        bool ok = true;
        for (int t = t0; t < t1 && ok; ++t) {
            const uint32_t ph = (t - t0) & 1;
            const size_t row = (size_t)bh * p.N + (size_t)t * 128 + tid;
            float es = 0.f;
            for (int s = 0; s < p.nslab; ++s) es += p.espart[(size_t)s * rows + row];
            const float coef = -p.s2 * es;
            ok = wait_or_abort(m1, ph, p.status, abort_flag);
            if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < p.r; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + C1 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(coef * __uint_as_float(v[j]));
                *reinterpret_cast<uint4 *>(tile_chunk(sW, tid, c0 / 8)) = pack8(v);
                *reinterpret_cast<uint4 *>(tile_chunk(sW, tid, c0 / 8 + 1)) = pack8(v + 8);
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(e1);
            ok = wait_or_abort(m2, ph, p.status, abort_flag);
            if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + C2 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    for (int s = 0; s < p.nslab; ++s) {
                        float f[8];
                        unpack8(*reinterpret_cast<const uint4 *>(p.pdK + ((size_t)s * rows + row) * D + c0 + 8 * q), f);
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[j] += f[j];
                    }
                    uint32_t o[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) o[j] = __float_as_uint(fmaf(kLn2, acc[j], __uint_as_float(v[8 * q + j])));
                    *reinterpret_cast<uint4 *>(p.dK + row * D + c0 + 8 * q) = pack8(o);
                }
            }
            tc_fence_before();
            mbar_arrive(e2);
        }
        if (ok) ok = wait_or_abort(m3, (t1 - 1 - t0) & 1, p.status, abort_flag);
        if (ok && tid < p.r) {
            tc_fence_after();
            float *dst = p.dMn + ((size_t)h * p.r + tid) * D;
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + C3 + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + c0 + j, __uint_as_float(v[j]));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ small SIMT kernels
// delta[row] = dO[row,:] . O[row,:]; one warp per row.
__global__ void delta_kernel(const __nv_bfloat16 *G, const __nv_bfloat16 *O, float *delta, long long rows, int dv)
{
    const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    float acc = 0.f;
    for (int c = lane * 2; c < dv; c += 64) {
        const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(G + row * dv + c));
        const float2 o = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(O + row * dv + c));
        acc = fmaf(g.x, o.x, fmaf(g.y, o.y, acc));
    }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) delta[row] = acc;
}

// out[row, c] = scale * sum_s part[s, row, c]; one thread per 8 columns.
__global__ void sum_slabs_kernel(const __nv_bfloat16 *part, __nv_bfloat16 *out, long long rows, int width, int nslab, float scale)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const int per_row = width / 8;
    if (i >= rows * per_row) return;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int s = 0; s < nslab; ++s) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4 *>(part + ((size_t)s * rows * per_row + i) * 8), f);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] += f[j];
    }
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) o[j] = __float_as_uint(scale * acc[j]);
    *reinterpret_cast<uint4 *>(out + i * 8) = pack8(o);
}

// dM[h,a,c] = s * sum_l W[l,a] T[h,l,c] + dMn[h,a,c]; one block per (a, h), one thread per c.
__global__ void dm_kernel(const __nv_bfloat16 *W, const float *Tacc, const float *dMn, float *dM, int m, int r, int d, int w_per_head, float s)
{
    const int a = blockIdx.x, h = blockIdx.y;
    const __nv_bfloat16 *w = W + (size_t)(w_per_head ? h : 0) * m * r;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float acc = 0.f;
        for (int l = 0; l < m; ++l) acc = fmaf(__bfloat162float(w[(size_t)l * r + a]), Tacc[((size_t)h * m + l) * d + c], acc);
        dM[((size_t)h * r + a) * d + c] = fmaf(s, acc, dMn[((size_t)h * r + a) * d + c]);
    }
}

template <int D, int DV>
cudaError_t launch_scan(const BwdParams &P, int grid, cudaStream_t st)
{
    using L = BwdSmem<D, DV>;
    static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_q_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tc_bwd_k_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    tc_bwd_q_kernel<D, DV><<<grid, 160, L::kTotal, st>>>(P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tc_bwd_k_kernel<D, DV><<<grid, 160, L::kTotal, st>>>(P);
    return cudaGetLastError();
}

template <int D>
cudaError_t launch_finish(const FinishParams &P, int grid, cudaStream_t st)
{
    constexpr int smem_bytes = 2 * 128 * D * 2 + 32768 + 128;
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_finish_k_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    tc_bwd_finish_k_kernel<D><<<grid, 160, smem_bytes, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

darkattn_status_t tensor_backward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                  const void *M, const void *W, const void *O, const void *dO, const void *saved,
                                  void *dQ, void *dK, void *dV, float *dM, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    if (!D.causal)   // the non-causal backward has no tensor-core kernels: FP32 path, same workspace
        return simt_backward(plan, Q, K, V, M, W, dO, dQ, dK, dV, dM, ws, st);
    const size_t BH = D.BH, N = D.N;
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16 *>(ws + off); };
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    if (!encode_fn()) { set_cuda_error(cudaErrorNotSupported, "tensor_backward: cuTensorMapEncodeTiled unavailable"); return DARKATTN_ERR_CUDA; }

    cudaError_t e = cudaSuccess;
    auto keep = [&](cudaError_t x) { if (x != cudaSuccess && e == cudaSuccess) e = x; };
    auto chk = [&]() { keep(cudaGetLastError()); };

    // The forward result and its per-row normalisers: taken from the caller when both are given,
    // otherwise recomputed into the workspace (that run also leaves the prologue's results there).
    const float2 *sv = reinterpret_cast<const float2 *>(saved);
    if (!O || !saved) {
        darkattn_status_t s = tensor_forward(plan, Q, K, V, M, W, bf(Y.Oscr), nullptr, ws, st);
        if (s != DARKATTN_OK) return s;
        O = bf(Y.Oscr);
        sv = reinterpret_cast<const float2 *>(ws + Y.sv);
    } else {
        keep(tensor_prologue(plan, K, M, W, ws, st));
    }

    const long long rows = (long long)BH * N;
    delta_kernel<<<(unsigned)((rows * 32 + 255) / 256), 256, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, fl(Y.delta), rows, D.dv);
    chk();
    keep(cudaMemsetAsync(ws + Y.Tacc, 0, (size_t)D.H * D.m * D.d * 4, st));
    keep(cudaMemsetAsync(ws + Y.dMn, 0, (size_t)D.H * D.r * D.d * 4, st));

    BwdParams P;
    memset(&P, 0, sizeof(P));
    bool ok = make_map(&P.mapQ, Q, BH * N, D.d, 128) && make_map(&P.mapK, K, BH * N, D.d, 128) &&
              make_map(&P.mapV, V, BH * N, D.dv, 128) && make_map(&P.mapG, dO, BH * N, D.dv, 128) &&
              make_map(&P.mapOm, bf(Y.Om), (size_t)D.H * D.m, D.d, 128);
    FinishParams F;
    memset(&F, 0, sizeof(F));
    ok = ok && make_map(&F.mapM, M, (size_t)D.H * D.r, D.d, 128);
    if (!ok) { set_cuda_error(cudaErrorInvalidValue, "tensor_backward: tensor map encode"); return DARKATTN_ERR_CUDA; }
    F.mapK = P.mapK;
    P.sv = sv; P.delta = fl(Y.delta); P.nK = fl(Y.nK); P.cs = fl(Y.cs); P.rhoc = fl(Y.rhoc);
    P.pdQ = bf(Y.pdQ); P.pdK = bf(Y.pdK); P.pdV = bf(Y.pdV); P.espart = fl(Y.espart); P.Tacc = fl(Y.Tacc);
    P.status = reinterpret_cast<int *>(ws + Y.status);
    P.N = D.N; P.H = D.H; P.BH = D.BH; P.m = D.m; P.nslab = Y.nslab; P.T = Y.T;
    const int units = (int)(BH * Y.nslab);
    if (D.d == 64 && D.dv == 64) keep(launch_scan<64, 64>(P, units, st));
    else if (D.d == 128 && D.dv == 128) keep(launch_scan<128, 128>(P, units, st));
    else if (D.d == 64 && D.dv == 128) keep(launch_scan<64, 128>(P, units, st));
    else keep(launch_scan<128, 64>(P, units, st));

    {
        const long long tq = rows * (D.d / 8), tv = rows * (D.dv / 8);
        sum_slabs_kernel<<<(unsigned)((tq + 255) / 256), 256, 0, st>>>(bf(Y.pdQ), (__nv_bfloat16 *)dQ, rows, D.d, Y.nslab, kLn2);
        chk();
        sum_slabs_kernel<<<(unsigned)((tv + 255) / 256), 256, 0, st>>>(bf(Y.pdV), (__nv_bfloat16 *)dV, rows, D.dv, Y.nslab, 1.f);
        chk();
    }
    F.pdK = bf(Y.pdK); F.espart = fl(Y.espart); F.dK = (__nv_bfloat16 *)dK; F.dMn = fl(Y.dMn);
    F.status = P.status;
    F.N = D.N; F.H = D.H; F.BH = D.BH; F.T = Y.T; F.r = D.r; F.nslab = Y.nslab; F.s2 = D.s * D.s;
    F.nsplit = (int)((148 * 2 + BH - 1) / BH);
    if (F.nsplit > Y.T) F.nsplit = Y.T;
    if (D.d == 64) keep(launch_finish<64>(F, (int)(BH * F.nsplit), st));
    else keep(launch_finish<128>(F, (int)(BH * F.nsplit), st));

    dm_kernel<<<dim3(D.r, D.H), 128, 0, st>>>((const __nv_bfloat16 *)W, fl(Y.Tacc), fl(Y.dMn), dM, D.m, D.r, D.d, D.w_per_head, D.s);
    chk();
    if (e != cudaSuccess) { set_cuda_error(e, "tensor_backward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

}  // namespace darkattn
