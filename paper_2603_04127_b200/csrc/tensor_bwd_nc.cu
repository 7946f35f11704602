// Tensor-core backward pass of non-causal DARK attention: the two passes over the sequence that
// produce dQ, dV, the projection part of dK, the row sums of E^K and T (Section 3, Eq. 3 differentiated).
//
// With no causal mask every query sees the same state, so (per batch, head and slab of 128
// features; log2 units and notation as in the causal backward kernels)
//   S = Bf^T V, z = Bf^T 1            key-side totals, kept by the forward pass
//   E^Q = A^ .* (dO S^T - delta z^T)   dQ = ln2 E^Q Omega
//   R = A^^T dO, rho = -A^^T delta     query-side totals, formed by the first pass
//   E^K = Bf .* (V R^T + rho^T)        dV = Bf R,   dK = ln2 E^K Omega - (norm term, applied later)
//   T = E^Q^T Q + E^K^T K
// The first kernel walks the query tiles of a slab (R in tensor memory, rho in registers), the
// second the key tiles. A sequence may be cut into pieces that run as separate CTAs: the pieces
// add their R, rho and T into fp32 buffers, and a small kernel rounds R to the bf16 operand of
// the second pass.
#include "common.cuh"
#include "tc_common.cuh"

#include <math.h>
#include <string.h>

namespace darkattn {

using namespace tc;

namespace {

constexpr float kLn2 = 0.6931471805599453f;

struct NcParams {
    CUtensorMap mapX, mapY, mapOm, mapOml, mapSt, mapOut, mapDV;   // X: Q or K; Y: dO or V; St: S or R (bf16); Out: dQ or dK
    const float2 *sv;     // [BH*N]  (normaliser, exponent it is scaled by) from the forward pass
    const float *delta;   // [BH*N]  dO_i . O_i
    const float *nK;      // [BH*N]  key norms, log2 units
    const float *cs;      // [BH*nslab] key-side shift per slab
    const float *zt;      // [BH, m] z of the whole sequence
    float *Racc;          // [BH, m, dv] sum of A^^T dO (query pass adds into it)
    float *rhot;          // [BH, m]     -sum of A^^T delta (query pass adds, key pass reads)
    float *espart;        // [4 nslab, BH*N] partials of rowsum(E^K): one per slab and 32-column group
    float *Tacc;          // [H, m, D]
    int *status;
    int N, H, Hkv, BH, m, nslab, T, nsplit;
    int add_kv;           // parts of dK and dV are added into the (zeroed) gradients: several slabs
    int out_per_head;     // grouped key/value heads: dK and dV rows are indexed by the query head (a later kernel sums each group)
};

template <int D, int DV>
struct NcSmem {
    static constexpr int kOm = 0;                          // folded projections of the slab [128 l, D]
    static constexpr int kOml = kOm + 128 * D * 2;         // what their rounding to bf16 left out [128 l, D]
    static constexpr int kX = kOml + 128 * D * 2;          // two buffers of the Q (K) tile     [128, D]; a tile's buffer also
                                                           // stages the tile's part of dQ (dK) once T += E^T X has read it
    static constexpr int kA = kX + 2 * 128 * D * 2;        // A^ (Bf), then E                   [128, 128]
    static constexpr int kY = kA + 32768;                  // dO (V) tile                       [128, DV]; key pass: then the staged dV tile
    static constexpr int kSt = kY + 128 * DV * 2;          // S (R) of the slab, bf16           [128 l, DV]
    // 3 KB of small things; query pass: the 16 x 128 K-major operand holding -delta (two swizzle atoms 1 KB apart of
    // which only rows 0 and 1, 256 bytes each, carry data; the MMA reads what lies behind them as rows 2..15, whose
    // products land in output columns nobody reads), barriers and z (rho) in between
    static constexpr int kSmall = kSt + 128 * DV * 2;
    static constexpr int kDel0 = kSmall;
    static constexpr int kBars = kSmall + 256;
    static constexpr int kVec = kSmall + 512;              // float[128]: z (rho) of the slab
    static constexpr int kTotal = kSmall + 3072;
};

constexpr uint32_t kColState = 0, kColT = 128, kColR1 = 256, kColR2 = 384;

__device__ __forceinline__ uint64_t vecdesc(const TileDesc &t, int k) { return t.kmaj + (uint64_t)(((k / 4) * 1024 + (k % 4) * 32) >> 4); }

enum NBars { NB_OM, NB_X0, NB_X1, NB_Y, NM1, NMA, NM2, NM3, NE1, NE2, NE3, NNBARS };

// Both passes share one schedule per tile t (R1, R2: scratch regions of tensor memory):
//   R1: U = X Omega^T (issued in the tail of the tile before) -> (features read) -> query pass: rho_c | key pass: dV = Bf R -> (read)
//   R2: dO S^T | V R^T (independent of the features, issued at once) -> (E formed) -> E Omega -> (read, stored)
// and the state updates R += A^^T dO, T += E^T X run behind them. KEYS selects the key pass.
template <int D, int DV, bool KEYS>
__global__ void __launch_bounds__(kThreads, 1) tc_bwd_nc_kernel(const __grid_constant__ NcParams p)
{
    using L = NcSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sOml = smem + L::kOml, *sX = smem + L::kX, *sA = smem + L::kA, *sY = smem + L::kY;
    unsigned char *sSt = smem + L::kSt, *sDelOp = smem + L::kDel0;
    float *sVec = reinterpret_cast<float *>(smem + L::kVec);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + NNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x / p.nsplit, piece = blockIdx.x % p.nsplit;
    const int bh = unit / p.nslab, slab = unit % p.nslab, h = bh % p.H;
    const int row0 = bh * p.N;
    // key pass: K, dK (X, Out) and V, dV (Y, DV) may be shared by a group of query heads; query pass: only V has no part in it
    const int rowx0 = KEYS ? kv_row0(bh, p.H, p.Hkv, p.N) : row0, rowy0 = rowx0;
    const int rowo0 = (KEYS && !p.out_per_head) ? rowx0 : row0;       // rows of the gradient tiles this pass writes
    const int tbeg = (int)((long long)p.T * piece / p.nsplit), tend = (int)((long long)p.T * (piece + 1) / p.nsplit);
    const int nt = tend - tbeg;

    if (tid == 0) {
        for (int i = 0; i < NE1; ++i) mbar_init(bars + i, 1);
        for (int i = NE1; i < NNBARS; ++i) mbar_init(bars + i, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) sVec[tid] = (KEYS ? p.rhot : p.zt)[(size_t)bh * p.m + slab * 128 + tid];
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (nt <= 0) {
        // nothing to do for this piece
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                mbar_expect_tx(bar, 128 * width * 2);
                const int base = (map == &p.mapX) ? rowx0 : rowy0;
                for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, base + t * 128);
            };
            const TileDesc tOm(sOm), tOml(sOml), tX0(sX), tX1(sX + 128 * D * 2), tA(sA), tY(sY), tSt(sSt), tDel(sDelOp);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_vec = make_idesc(128, 16, 1, 0);
            const uint32_t id_state = make_idesc(128, DV, 1, 1);
            const uint32_t id_dv = make_idesc(128, DV, 0, 1);
            const uint32_t id_dx = make_idesc(128, D, 0, 1);
            const uint32_t id_t = make_idesc(128, D, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2;

            mbar_expect_tx(bars + NB_OM, 2 * 128 * D * 2 + 128 * DV * 2);
            for (int a = 0; a < D / 64; ++a) {
                tma_load_2d(sOm + a * 16384, &p.mapOm, bars + NB_OM, a * 64, h * p.m + slab * 128);
                tma_load_2d(sOml + a * 16384, &p.mapOml, bars + NB_OM, a * 64, h * p.m + slab * 128);
            }
            for (int a = 0; a < DV / 64; ++a) tma_load_2d(sSt + a * 16384, &p.mapSt, bars + NB_OM, a * 64, bh * p.m + slab * 128);
            load_tile(sX, &p.mapX, bars + NB_X0, D, tbeg);
            load_tile(sY, &p.mapY, bars + NB_Y, DV, tbeg);

            bool ok = wait_or_abort(bars + NB_OM, 0, status, abort_flag);
            if (ok) ok = wait_or_abort(bars + NB_X0, 0, status, abort_flag);
            if (ok) {
                tc_fence_after();
                issue_projection<D>(R1, tX0, tOm, tOml, id_kk);                                                  // U of the first tile
                mma_commit(bars + NM1);
            }
            for (int it = 0; it < nt && ok; ++it) {
                const int t = tbeg + it;
                const uint32_t ph = it & 1;
                const bool first = (it == 0), last = (it + 1 == nt);
                const TileDesc &tX = (it & 1) ? tX1 : tX0;
#define NWAIT(b, q) do { ok = wait_or_abort(bars + (b), (q), status, abort_flag); } while (0)
                auto store_out = [&](const CUtensorMap *map, unsigned char *src, int width, int tt) {     // (adds into the gradient when the head has several slabs)
                    const bool add = KEYS ? (p.add_kv != 0) : (p.nslab > 1);
                    for (int a = 0; a < width / 64; ++a) {
                        if (add) tma_reduce_add_2d(map, src + a * 16384, a * 64, rowo0 + tt * 128);
                        else tma_store_2d(map, src + a * 16384, a * 64, rowo0 + tt * 128);
                    }
                    tma_store_commit();
                };
                NWAIT(NB_Y, ph); if (!ok) break;
                if (!first) {                                                       // the tile before: R2 read out, its part of dQ | dK staged in its X buffer
                    NWAIT(NE3, ph ^ 1); if (!ok) break;
                    store_out(&p.mapOut, sX + ((it + 1) & 1) * 128 * D * 2, D, t - 1);
                }
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(tY, k), kdesc(tSt, k), id_kk, k > 0);      // dO S^T | V R^T
                mma_commit(bars + NMA);
                if (!first) tma_store_wait_read();                                  // the staged tile has left the X buffer
                if (!last) load_tile(sX + ((it + 1) & 1) * 128 * D * 2, &p.mapX, bars + NB_X0 + ((it + 1) & 1), D, t + 1);
                NWAIT(NE1, ph); if (!ok) break;                                     // features in smem, R1 read
                tc_fence_after();
                if (KEYS) {
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R1, kdesc(tA, k), mndesc(tSt, k), id_dv, k > 0);        // dV = Bf R
                } else {
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R1, mndesc(tA, k), vecdesc(tDel, k), id_vec, k > 0);   // rho_c = -A^^T delta (columns 0, 1)
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColState, mndesc(tA, k), mndesc(tY, k), id_state, (!first) || k > 0);   // R += A^^T dO
                }
                mma_commit(bars + NM2);
                NWAIT(NE2, ph); if (!ok) break;                                     // E in smem; R1 and R2 read; key pass: dV staged over the V tile
                if (KEYS) store_out(&p.mapDV, sY, DV, t);
                else if (!last) load_tile(sY, &p.mapY, bars + NB_Y, DV, t + 1);
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(tA, k), mndesc(tOm, k), id_dx, k > 0);            // E Omega
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColT, mndesc(tA, k), mndesc(tX, k), id_t, (!first) || k > 0);   // T += E^T X
                mma_commit(bars + NM3);
                if (!last) {       // U of the next tile behind them (R1 has been read): its features can be formed at once
                    NWAIT(NB_X0 + ((it + 1) & 1), ((it + 1) >> 1) & 1); if (!ok) break;
                    tc_fence_after();
                    const TileDesc &tXn = ((it + 1) & 1) ? tX1 : tX0;
                    issue_projection<D>(R1, tXn, tOm, tOml, id_kk);
                    mma_commit(bars + NM1);
                }
                if (KEYS && !last) { tma_store_wait_read(); load_tile(sY, &p.mapY, bars + NB_Y, DV, t + 1); }     // the staged dV has left the V tile's buffer
                if (last) {        // the last tile's part of dQ | dK
                    NWAIT(NE3, ph); if (!ok) break;
                    store_out(&p.mapOut, sX + (it & 1) * 128 * D * 2, D, t);
                }
#undef NWAIT
            }
            tma_store_wait_all();
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, g = warp >> 2, col0 = g * 32;
        const int r = q4 * 32 + lane;                        // tile row = TMEM lane
        const bool g0 = (col0 == 0);                         // these 128 threads: row r also stands for feature r of the slab
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        const float cshift = load_key_shift(p.cs, bh * p.nslab + slab);
        const size_t rows = (size_t)p.BH * p.N;
        float rho_run = 0.f;
        bool ok = true;
        for (int it = 0; it < nt && ok; ++it) {
            const int t = tbeg + it;
            const uint32_t ph = it & 1;
            const size_t row = (size_t)row0 + (size_t)t * 128 + r;
#define EWAIT(b) do { ok = __all_sync(0xffffffffu, wait_or_abort(bars + (b), ph, status, abort_flag)); } while (0)
            float offset, del = 0.f;
            if (KEYS) {
                offset = p.nK[row] + cshift;
            } else {
                const float2 svv = p.sv[row];
                offset = svv.y - cshift + log2f(svv.x);
                del = p.delta[row];
            }
            float dtile[4] = {0.f, 0.f, 0.f, 0.f};       // query pass, warp 0: -delta of rows lane, lane + 32, ...
            if (!KEYS && warp == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) dtile[i] = -__ldg(p.delta + (size_t)row0 + (size_t)t * 128 + i * 32 + lane);
            }
            EWAIT(NM1); if (!ok) break;
            tc_fence_after();
            features_to_tile(R1 + col0, offset, sA, r, col0);                          // A^ | Bf
            if (warp == 0) {
                if (!KEYS) {
                    // 16 x 128 K-major operand of rho_c: row 0 = -delta rounded to bf16, row 1 = the rounding's remainder
                    // (its last reader, the MMAs of the tile before, completed before that tile's E was formed)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = i * 32 + lane;
                        const float dk = dtile[i];
                        const __nv_bfloat16 hi = __float2bfloat16_rn(dk);
                        const __nv_bfloat16 lo = __float2bfloat16_rn(dk - __bfloat162float(hi));
                        const int atom = k >> 6, kk = k & 63, ch = kk >> 3;
                        *reinterpret_cast<__nv_bfloat16 *>(sDelOp + atom * 1024 + (ch << 4) + (kk & 7) * 2) = hi;
                        *reinterpret_cast<__nv_bfloat16 *>(sDelOp + atom * 1024 + 128 + ((ch ^ 1) << 4) + (kk & 7) * 2) = lo;
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + NE1);

            EWAIT(NMA); if (!ok) break;
            EWAIT(NM2); if (!ok) break;
            tc_fence_after();
            if (KEYS) {
                if (col0 < DV) tmem_row_to_tile(R1 + col0, sY, r, col0);               // this slab's part of dV, staged over the V tile (V R^T is done)
            } else if (g0) {
                uint32_t v[16];
                tmem_ld16(R1, v);
                tmem_wait_ld();
                rho_run += __uint_as_float(v[0]) + __uint_as_float(v[1]);
            }
            {   // E = A^ .* (dO S^T - delta z^T)  |  Bf .* (V R^T + rho^T), in place over the features
                float es = 0.f;
                uint32_t v[32];
                tmem_ld32(R2 + col0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 *cell = reinterpret_cast<uint4 *>(tile_chunk(sA, r, col0 / 8 + q));
                    float a[8];
                    unpack8(*cell, a);
                    const float4 z0 = *reinterpret_cast<const float4 *>(sVec + col0 + 8 * q);
                    const float4 z1 = *reinterpret_cast<const float4 *>(sVec + col0 + 8 * q + 4);
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                    float e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float x = __uint_as_float(v[8 * q + j]);
                        e[j] = a[j] * (KEYS ? x + zz[j] : fmaf(-del, zz[j], x));
                        es += e[j];
                    }
                    *cell = make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                }
                if (KEYS) p.espart[((size_t)slab * 4 + g) * rows + row] = es;
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + NE2);

            EWAIT(NM3); if (!ok) break;     // E Omega in R2; T += E^T X has read this tile's X buffer: the control thread stores from there
            tc_fence_after();
            if (col0 < D) tmem_row_to_tile(R2 + col0, sX + (it & 1) * 128 * D * 2, r, col0, kLn2);  // this slab's part of dQ | dK (without the norm term)
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + NE3);
#undef EWAIT
        }
        // every MMA of this CTA completed before the last NM3 did: the accumulators can be read
        if (ok) {
            tc_fence_after();
            if (col0 < D) {
                float *dst = p.Tacc + ((size_t)h * p.m + slab * 128 + r) * D + col0;
                uint32_t v[32];
                tmem_ld32(lane_addr + kColT + col0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(v[j]));
            }
            if (!KEYS) {
                if (col0 < DV) {
                    float *dst = p.Racc + ((size_t)bh * p.m + slab * 128 + r) * DV + col0;
                    uint32_t v[32];
                    tmem_ld32(lane_addr + kColState + col0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(v[j]));
                }
                if (g0) atomicAdd(p.rhot + (size_t)bh * p.m + slab * 128 + r, rho_run);
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);   // error path only: let copies and MMAs in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// Rb = bf16(Racc): the operand of the key pass
__global__ void nc_round_state_kernel(const float *R, __nv_bfloat16 *Rb, long long n)
{
    for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * 4; i < n; i += (long long)gridDim.x * blockDim.x * 4) {
        const float4 x = *reinterpret_cast<const float4 *>(R + i);
        *reinterpret_cast<uint2 *>(Rb + i) = make_uint2(pack_bf16(x.x, x.y), pack_bf16(x.z, x.w));
    }
}

template <int D, int DV>
cudaError_t launch_nc(const darkattn_plan_s *plan, const NcParams &PQ, const NcParams &PK, const float *Racc, __nv_bfloat16 *Rb,
                      long long nstate, bool join, cudaStream_t st)
{
    using L = NcSmem<D, DV>;
    static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_nc_kernel<D, DV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tc_bwd_nc_kernel<D, DV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    const int grid = PQ.BH * PQ.nslab * PQ.nsplit;
    timer_mark(plan, st, "tc_bwd_nc_q_kernel");
    tc_bwd_nc_kernel<D, DV, false><<<grid, kThreads, L::kTotal, st>>>(PQ);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    timer_mark(plan, st, "nc_round_state_kernel");
    nc_round_state_kernel<<<(unsigned)((nstate / 4 + 255) / 256), 256, 0, st>>>(Racc, Rb, nstate);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (join) {
        e = cudaStreamWaitEvent(st, plan->aux_join, 0);      // dK and dV have been zeroed
        if (e != cudaSuccess) return e;
    }
    timer_mark(plan, st, "tc_bwd_nc_k_kernel");
    tc_bwd_nc_kernel<D, DV, true><<<grid, kThreads, L::kTotal, st>>>(PK);
    return cudaGetLastError();
}

}  // namespace

// The two passes of the non-causal backward. Expects delta computed, Tacc zeroed and (with several
// slabs) dQ zeroed on `st`, dK and dV zeroed behind plan->aux_join. With `per_head`, dK and dV are the per-query-head
// buffers of grouped key/value heads ([BH, N, *]).
cudaError_t tensor_backward_nc_passes(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V, const void *dO,
                                      const Stash &stash, void *dQ, void *dK, void *dV, bool per_head, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    __nv_bfloat16 *Rb = reinterpret_cast<__nv_bfloat16 *>(ws + Y.Rb);

    NcParams PQ;
    memset(&PQ, 0, sizeof(PQ));
    PQ.sv = stash.sv; PQ.delta = fl(Y.delta); PQ.nK = stash.nK; PQ.cs = stash.cs; PQ.zt = stash.zt;
    PQ.Racc = fl(Y.Racc); PQ.rhot = fl(Y.rhot); PQ.espart = fl(Y.espart); PQ.Tacc = fl(Y.Tacc);
    PQ.status = reinterpret_cast<int *>(ws + Y.status);
    const size_t BHkv = (size_t)D.B * D.Hkv;
    const bool add_kv = Y.nslab > 1;
    const size_t BHo = per_head ? BH : BHkv;          // rows of dK and dV (per query head with grouped key/value heads)
    PQ.out_per_head = per_head ? 1 : 0;
    PQ.N = D.N; PQ.H = D.H; PQ.Hkv = D.Hkv; PQ.BH = D.BH; PQ.m = D.m; PQ.nslab = Y.nslab; PQ.T = Y.T; PQ.add_kv = add_kv ? 1 : 0;
    PQ.nsplit = pick_splits((long long)BH * Y.nslab, Y.T, 3.0, 6.0, 64);
    NcParams PK = PQ;
    const bool ok = make_map(&PQ.mapX, Q, BH * N, D.d, 128) && make_map(&PQ.mapY, dO, BH * N, D.dv, 128) &&
                    make_map(&PQ.mapOm, stash.Om, (size_t)D.H * D.m, D.d, 128) && make_map(&PQ.mapOml, stash.Oml, (size_t)D.H * D.m, D.d, 128) &&
                    make_map(&PQ.mapSt, stash.Sb, BH * D.m, D.dv, 128) &&
                    make_map(&PQ.mapOut, dQ, BH * N, D.d, 128) && make_map(&PQ.mapDV, dV, BHo * N, D.dv, 128) &&
                    make_map(&PK.mapX, K, BHkv * N, D.d, 128) && make_map(&PK.mapY, V, BHkv * N, D.dv, 128) &&
                    make_map(&PK.mapSt, Rb, BH * D.m, D.dv, 128) && make_map(&PK.mapOut, dK, BHo * N, D.d, 128);
    if (!ok) return cudaErrorInvalidValue;
    PK.mapOm = PQ.mapOm;
    PK.mapOml = PQ.mapOml;
    PK.mapDV = PQ.mapDV;
    const long long nstate = (long long)BH * D.m * D.dv;
    cudaError_t e = cudaMemsetAsync(ws + Y.Racc, 0, (Y.rhot - Y.Racc) + BH * D.m * 4, st);      // R and rho sums (adjacent)
    if (e != cudaSuccess) return e;
    const bool join = add_kv;
    if (D.d == 64 && D.dv == 64) return launch_nc<64, 64>(plan, PQ, PK, fl(Y.Racc), Rb, nstate, join, st);
    if (D.d == 128 && D.dv == 128) return launch_nc<128, 128>(plan, PQ, PK, fl(Y.Racc), Rb, nstate, join, st);
    if (D.d == 64 && D.dv == 128) return launch_nc<64, 128>(plan, PQ, PK, fl(Y.Racc), Rb, nstate, join, st);
    return launch_nc<128, 64>(plan, PQ, PK, fl(Y.Racc), Rb, nstate, join, st);
}

}  // namespace darkattn
