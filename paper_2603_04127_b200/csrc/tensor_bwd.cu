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
// Two scan kernels. The query-side kernel takes the state S before every chunk and the key features Bf from the
// forward pass (bf16, through the stash), so its chunks are independent and spread evenly over the SMs; it forms
// A^ again from Q and both halves of the folded projections and leaves it in the workspace for the key-side kernel,
// which walks each (batch, head, slab) backwards with the state R in TMEM and reads A^ and Bf back. The 128 x 128
// tiles dP (query side) and P^^T, dP^T (key side) are written back to tensor memory as bf16 and used as the A operand
// of the next MMA directly from there. Each slab's parts of dQ, dK, dV are staged in a tile buffer that is free at
// that point and added into the (zeroed) gradients by TMA reduce-add stores; a finishing kernel applies the norm
// term of dK with three MMAs per tile.
#include "common.cuh"
#include "tc_common.cuh"

#include <math.h>
#include <string.h>

namespace darkattn {

using namespace tc;

namespace {

constexpr float kLn2 = 0.6931471805599453f;

struct BwdParams {
    CUtensorMap mapQ, mapK, mapV, mapG, mapOm, mapOml, mapDQ, mapDK, mapDV;   // the last three: the gradients, for the (adding) stores
    CUtensorMap mapAh, mapBf;   // A^ and Bf as [BH*N, m] bf16: A^ is written by the query-side kernel and read by the key-side one, Bf comes
                                // from the forward pass (through the stash) and is read by both
    CUtensorMap mapSst;         // S before every chunk as [BH*T*m, dv] bf16, from the forward pass
    const float2 *sv;     // [BH*N]  (normaliser, exponent it is scaled by) from the forward pass
    const float *delta;   // [BH*N]  dO_i . O_i
    const float *nK;      // [BH*N]  key norms, log2 units
    const float *cs;      // [BH*nslab] key-side shift per slab
    const float *zc;      // [BH, T, m] z before chunk t, from the forward pass (row 0 is not read)
    float *rhoc;          // [BH, T, m] per-chunk -sum_i A^_il delta_i (written by the query-side kernel)
    float *espart;        // [4 nslab, BH*N] partials of rowsum(E^K): one per slab and 32-column group
    float *Tacc;          // [H, m, D]
    int *status;
    int N, H, Hkv, BH, m, nslab, T;
    int add_kv;           // parts of dK and dV are added into the (zeroed) gradients: several slabs
    int out_per_head;     // grouped key/value heads: dK and dV rows are indexed by the query head (a later kernel sums each group)
};

template <int D, int DV>
struct BwdSmem {
    static constexpr int kDmax = D > DV ? D : DV;
    static constexpr int kOm = 0;                          // folded projections of the slab [128 l, D]
    static constexpr int kAux = kOm + 128 * D * 2;         // query side: what the rounding of the folded projections left out [128 l, D];
                                                           // key side: staging tile of the TMA stores of dV and dK
    static constexpr int kQA = kAux + 32768;               // Q tile, then A^ (then E^Q)       [128, 128]
    static constexpr int kKB = kQA + 32768;                // K tile, then Bf (then E^K)        [128, 128]
    static constexpr int kV = kKB + 32768;                 // V tile                            [128, DV]
    static constexpr int kG = kV + 128 * DV * 2;           // dO tile; later the reloaded Q / K tile
    static constexpr int kSt = kG + 128 * kDmax * 2;       // bf16 copy of the scan state       [128 l, DV]
                                                           // (32 KB: the query-side kernel also keeps a 128 x 128 feature tile there)
    // 3 KB of small things. Query side: the 16 x 128 K-major operand holding -delta (two swizzle atoms of which only the
    // rows 0 and 1, 256 bytes each, carry data: the MMA also reads the 768 bytes behind each and the kilobyte behind the
    // second atom as rows 2..15, whose products land in output columns nobody reads), barriers and z in between.
    static constexpr int kSmall = kSt + 32768;
    static constexpr int kDel0 = kSmall;                   // rows 0, 1 of the first atom (k = 0..63)
    static constexpr int kBars = kSmall + 256;
    static constexpr int kVec = kSmall + 512;              // query side: float[128] (z); key side: two float[128] (rho, delta)
    static constexpr int kDel1 = kSmall + 1024;            // rows 0, 1 of the second atom (k = 64..127)
    static constexpr int kTotal = kSmall + 3072;
    static_assert(kDel1 == kDel0 + 1024, "the two atoms of the -delta operand are 1 KB apart");
};

// TMEM columns (512 allocated): scan state at 0, T at 128, scratch R1 at 256 and R2 at 384.
constexpr uint32_t kColState = 0, kColT = 128, kColR1 = 256, kColR2 = 384;

// K-major 16 x 128 bf16 operand (two atoms 1 KB apart): step k covers 16 elements of K
__device__ __forceinline__ uint64_t vecdesc(const TileDesc &t, int k) { return t.kmaj + (uint64_t)(((k / 4) * 1024 + (k % 4) * 32) >> 4); }

enum QBars { QB_OM, QB_Q, QB_B, QB_V, QB_G, QB_S, QB_X2, QM1, QM3, QM4, QM5, QM6, QE1, QE2A, QE2, QE3, QE4, QET, QNBARS };

// ------------------------------------------------------------------ query side
// The state S before every chunk and the key features Bf come from the forward pass (bf16, through the stash), so the
// chunks are independent of one another here: the chunks of all (batch, head) pairs form one line that is cut evenly
// over groups of nslab CTAs, and a CTA walks its piece run by run (a run = consecutive chunks of one (batch, head) pair).
template <int D, int DV>
__global__ void __launch_bounds__(kThreads, 1) tc_bwd_q_kernel(const __grid_constant__ BwdParams p)
{
    using L = BwdSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sOml = smem + L::kAux, *sQA = smem + L::kQA, *sKB = smem + L::kKB, *sV = smem + L::kV;
    unsigned char *sG = smem + L::kG, *sSt = smem + L::kSt, *sDelOp = smem + L::kDel0;
    float *sZ = reinterpret_cast<float *>(smem + L::kVec);      // z before this chunk
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + QNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + QNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int T = p.T;
    // CTAs work in groups of nslab (one per slab of the head) on the same piece of the line of (batch, head, chunk)
    // items, so that the Q, V, dO tiles a group reads are fetched from HBM once
    const int slab = blockIdx.x % p.nslab, group = blockIdx.x / p.nslab, ngroups = gridDim.x / p.nslab;
    const long long total = (long long)p.BH * T;
    const long long lbeg = total * group / ngroups, lend = total * (group + 1) / ngroups;

    if (tid == 0) {
        for (int i = 0; i < QE1; ++i) mbar_init(bars + i, 1);
        for (int i = QE1; i < QNBARS; ++i) mbar_init(bars + i, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            const TileDesc tOm(sOm), tOml(sOml), tQA(sQA), tKB(sKB), tV(sV), tG(sG), tSt(sSt), tDel(sDelOp);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_vec = make_idesc(128, 16, 1, 0);
            const uint32_t id_tm = make_idesc(128, 128, 0, 1);
            const uint32_t id_dx = make_idesc(128, D, 0, 1);
            const uint32_t id_t = make_idesc(128, D, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2;
            // Schedule of one chunk (R1, R2, R3: scratch regions of TMEM). U_Q and dO V^T of the next chunk are issued in the
            // tail of the current one.
            //   R3: U_Q -> (A^ read) -> U_Q of the next chunk
            //   R2: dO V^T -> packed dP in [0,64) (A operand of dP Bf), rho_c in [64,80) -> dO V^T of the next chunk
            //   R1: dP Bf + dO S^T -> (E read) -> E Omega -> (dQ read)
            // Shared memory: X holds Q, then A^, then E, then the staged dQ tile, then the next chunk's state; S holds the
            // state, then the next chunk's Q (the two swap roles from chunk to chunk); the Bf tile's buffer takes the Q tile
            // again once dP Bf is done (T += E^T Q needs it) and the next chunk's Bf after that; V is free as soon as dO V^T
            // has been read out, so the next chunk's V tile, the first thing that chunk needs, loads earliest.
            const uint32_t R3 = tmem + kColState;
            bool ok = true;
            int it = 0, run = 0;        // chunks and runs done so far: the parities of the barriers
            for (long long l0 = lbeg; l0 < lend && ok; ++run) {
                const int bh = (int)(l0 / T), t0 = (int)(l0 % T);
                long long l1 = (long long)(bh + 1) * T;
                if (l1 > lend) l1 = lend;
                const int nrun = (int)(l1 - l0);
                l0 = l1;
                const int h = bh % p.H, row0 = bh * p.N, rowk0 = kv_row0(bh, p.H, p.Hkv, p.N);
                auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                    const int base = (map == &p.mapV) ? rowk0 : row0;      // V may be shared by a group of query heads
                    mbar_expect_tx(bar, 128 * width * 2);
                    for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, base + t * 128);
                };
                auto load_key_features = [&](int t) {                  // Bf of chunk t, as the forward pass formed it
                    mbar_expect_tx(bars + QB_B, 32768);
                    tma_load_2d(sKB, &p.mapBf, bars + QB_B, slab * 128, row0 + t * 128);
                    tma_load_2d(sKB + 16384, &p.mapBf, bars + QB_B, slab * 128 + 64, row0 + t * 128);
                };
                auto load_state = [&](unsigned char *dst, int t) {     // S before chunk t (for t = 0 the tile is loaded but not used)
                    mbar_expect_tx(bars + QB_S, 128 * DV * 2);
                    for (int a = 0; a < DV / 64; ++a) tma_load_2d(dst + a * 16384, &p.mapSst, bars + QB_S, a * 64, (bh * T + t) * p.m + slab * 128);
                };
                tma_store_wait_read();      // the last dQ tile of the run before has left its buffer
                mbar_expect_tx(bars + QB_OM, 2 * 128 * D * 2);
                for (int a = 0; a < D / 64; ++a) {
                    tma_load_2d(sOm + a * 16384, &p.mapOm, bars + QB_OM, a * 64, h * p.m + slab * 128);
                    tma_load_2d(sOml + a * 16384, &p.mapOml, bars + QB_OM, a * 64, h * p.m + slab * 128);
                }
                load_tile((it & 1) ? sSt : sQA, &p.mapQ, bars + QB_Q, D, t0);
                load_tile(sV, &p.mapV, bars + QB_V, DV, t0);
                load_tile(sG, &p.mapG, bars + QB_G, DV, t0);
                load_key_features(t0);
                load_state((it & 1) ? sQA : sSt, t0);
                ok = wait_or_abort(bars + QB_OM, run & 1, status, abort_flag);
                if (ok) ok = wait_or_abort(bars + QB_Q, it & 1, status, abort_flag);
                if (ok) {
                    tc_fence_after();
                    const TileDesc &tX0 = (it & 1) ? tSt : tQA;
                    issue_projection<D>(R3, tX0, tOm, tOml, id_kk);                                              // U_Q of the run's first chunk
                    mma_commit(bars + QM1);
                    ok = wait_or_abort(bars + QB_V, it & 1, status, abort_flag);
                    if (ok) ok = wait_or_abort(bars + QB_G, it & 1, status, abort_flag);
                }
                if (ok) {
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(tG, k), kdesc(tV, k), id_kk, k > 0);     // dO V^T of the run's first chunk
                    mma_commit(bars + QM3);
                }
                for (int c = 0; c < nrun && ok; ++c, ++it) {
                    const int t = t0 + c;
                    const uint32_t ph = it & 1;
                    const bool first = (t == 0), last = (c + 1 == nrun);
                    unsigned char *bX = ph ? sSt : sQA, *bS = ph ? sQA : sSt;
                    const TileDesc &tX = ph ? tSt : tQA, &tS = ph ? tQA : tSt;
#define QWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
                    QWAIT(QE1); if (!ok) break;                                                                  // A^ in X, R3 read, -delta operand written
                    tma_store_2d(&p.mapAh, bX, slab * 128, row0 + t * 128);                                      // A^ kept for the key-side kernel
                    tma_store_2d(&p.mapAh, bX + 16384, slab * 128 + 64, row0 + t * 128);
                    tma_store_commit();
                    QWAIT(QE2A); if (!ok) break;                                                                 // dO V^T read out of R2: V is done with
                    if (!last) load_tile(sV, &p.mapV, bars + QB_V, DV, t + 1);
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R2 + 64, mndesc(tX, k), vecdesc(tDel, k), id_vec, k > 0);  // rho_c = -A^^T delta (columns 0, 1)
                    QWAIT(QE2); if (!ok) break;                                                                  // dP packed in R2
                    QWAIT(QB_B); if (!ok) break;
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R1, R2 + k * 8, mndesc(tKB, k), id_tm, k > 0);           // dP Bf
                    QWAIT(QB_S); if (!ok) break;                                                                 // (for the first chunk the tile is loaded but not used)
                    if (!first) {
                        tc_fence_after();
                        _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R1, kdesc(tG, k), kdesc(tS, k), id_kk, 1);     // + dO S_prev^T
                    }
                    tma_store_wait_read();      // the A^ tile has left shared memory: E may overwrite it
                    mma_commit(bars + QM4);
                    QWAIT(QM4); if (!ok) break;                                                                  // Bf, dO and S of this chunk are done with
                    load_tile(sKB, &p.mapQ, bars + QB_X2, D, t);                                                // Q again, for T, where Bf was
                    if (!last) {
                        load_tile(sG, &p.mapG, bars + QB_G, DV, t + 1);
                        load_tile(bS, &p.mapQ, bars + QB_Q, D, t + 1);                                          // the state tile is done with: the next chunk's Q
                        for (int a = 0; a < DV / 64; ++a)                                                        // into L2 now: the next state's load can only be issued at the chunk's very end
                            tma_prefetch_l2_2d(&p.mapSst, a * 64, (bh * T + t + 1) * p.m + slab * 128);
                    }
                    QWAIT(QE3); if (!ok) break;
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R1, kdesc(tX, k), mndesc(tOm, k), id_dx, k > 0);         // E Omega
                    mma_commit(bars + QM5);
                    QWAIT(QB_X2); if (!ok) break;
                    if (c == 0 && run > 0) {                                                                     // T of the previous run has been read out
                        ok = wait_or_abort(bars + QET, (run - 1) & 1, status, abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColT, mndesc(tX, k), mndesc(tKB, k), id_t, (c > 0) || k > 0);   // T += E^T Q
                    mma_commit(bars + QM6);
                    if (!last) {
                        ok = wait_or_abort(bars + QB_Q, ph ^ 1, status, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_projection<D>(R3, tS, tOm, tOml, id_kk);                                           // U_Q of the next chunk (its Q sits in S)
                        mma_commit(bars + QM1);
                        ok = wait_or_abort(bars + QB_V, ph ^ 1, status, abort_flag);
                        if (ok) ok = wait_or_abort(bars + QB_G, ph ^ 1, status, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(tG, k), kdesc(tV, k), id_kk, k > 0); // dO V^T of the next chunk
                        mma_commit(bars + QM3);
                    }
                    QWAIT(QM6); if (!ok) break;                                                                  // the Q tile is done with:
                    if (!last) load_key_features(t + 1);                                                         // the next chunk's Bf
                    QWAIT(QE4); if (!ok) break;                                                                  // this slab's part of dQ is staged where E was
                    for (int a = 0; a < D / 64; ++a) {
                        if (p.nslab > 1) tma_reduce_add_2d(&p.mapDQ, bX + a * 16384, a * 64, row0 + t * 128);
                        else tma_store_2d(&p.mapDQ, bX + a * 16384, a * 64, row0 + t * 128);
                    }
                    tma_store_commit();
                    if (!last) {
                        tma_store_wait_read();
                        load_state(bX, t + 1);                                                                   // the next chunk's state
                    }
#undef QWAIT
                }
            }
            tma_store_wait_all();
        }
    } else {
        // ============================== epilogue threads (see kEpiWarps)
        const int lane = tid & 31, q4 = warp & 3, col0 = (warp >> 2) * 32;
        const int r = q4 * 32 + lane;                        // tile row = TMEM lane
        const bool g0 = (col0 == 0);                         // these 128 threads: row r also stands for feature r of the slab
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        // A wait that gave up (here or, seen through the abort flag, in another warp) switches the warp to a dry run: it skips
        // every later wait but keeps walking the same chunks, so that every named barrier still gets all its arrivals.
        bool ok = true;
        int it = 0, run = 0;
        for (long long l0 = lbeg; l0 < lend; ++run) {
            const int bh = (int)(l0 / T), t0 = (int)(l0 % T);
            long long l1 = (long long)(bh + 1) * T;
            if (l1 > lend) l1 = lend;
            const int nrun = (int)(l1 - l0);
            l0 = l1;
            const int h = bh % p.H, row0 = bh * p.N;
            const float cshift = load_key_shift(p.cs, bh * p.nslab + slab);
            if (g0) sZ[r] = (t0 > 0) ? __ldg(p.zc + ((size_t)bh * T + t0) * p.m + slab * 128 + r) : 0.f;
            float2 svv_next = p.sv[(size_t)row0 + (size_t)t0 * 128 + r];
            float del_next = p.delta[(size_t)row0 + (size_t)t0 * 128 + r];
            epi_sync();
            for (int c = 0; c < nrun; ++c, ++it) {
                const int t = t0 + c;
                const uint32_t ph = it & 1;
                const bool last = (c + 1 == nrun);
                const size_t row = (size_t)row0 + (size_t)t * 128 + r;
#define EWAIT(b) do { ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + (b), ph, status, abort_flag)); } while (0)
                const float2 svv = svv_next;                 // (loaded a chunk ahead: their latency is off the chunk's critical path)
                const float del = del_next;
                if (!last) { svv_next = p.sv[row + 128]; del_next = p.delta[row + 128]; }
                const float aq = svv.y - cshift + log2f(svv.x);
                // z before the next chunk, from the forward pass (loaded early, used at the end of the chunk)
                const float znext = (g0 && !last) ? __ldg(p.zc + ((size_t)bh * T + t + 1) * p.m + slab * 128 + r) : 0.f;
                float dtile[4] = {0.f, 0.f, 0.f, 0.f};       // warp 0: -delta of rows lane, lane + 32, ... for the operand of rho_c
                if (warp == 0) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) dtile[i] = -__ldg(p.delta + (size_t)row0 + (size_t)t * 128 + i * 32 + lane);
                }
                unsigned char *bX = ph ? sSt : sQA;          // this chunk's Q / A^ / E tile
                EWAIT(QM1);
                tc_fence_after();
                features_to_tile(lane_addr + kColState + col0, aq, bX, r, col0);           // A^
                if (warp == 0) {
                    // 16 x 128 K-major operand of rho_c = -A^^T delta: row 0 = -delta rounded to bf16, row 1 = the rounding's
                    // remainder (its last reader, the chunk before's MMAs, completed before that chunk's E was formed)
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
                fence_async_smem();
                tc_fence_before();
                mbar_arrive_warp(bars + QE1);

                EWAIT(QM3);
                tc_fence_after();
                {   // dP = tril(dO V^T - delta) as a bf16 operand in TMEM (packed over the fp32 tile)
                    uint32_t v[32], pk[16];
                    tmem_ld32(R2 + col0, v);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive_warp(bars + QE2A);
                    quarter_sync(q4);                         // every column group has read before anyone overwrites
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float x0 = (col0 + j <= r) ? __uint_as_float(v[j]) - del : 0.f;
                        const float x1 = (col0 + j + 1 <= r) ? __uint_as_float(v[j + 1]) - del : 0.f;
                        pk[j / 2] = pack_bf16(x0, x1);
                    }
                    tmem_st16(R2 + col0 / 2, pk);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive_warp(bars + QE2);

                EWAIT(QM4);
                tc_fence_after();
                if (g0) {       // rho_c of feature r (TMEM lane r; its MMAs ran ahead of dP Bf), for the key-side kernel
                    uint32_t v[16];
                    tmem_ld16(R2 + 64, v);
                    tmem_wait_ld();
                    p.rhoc[((size_t)bh * T + t) * p.m + slab * 128 + r] = __uint_as_float(v[0]) + __uint_as_float(v[1]);
                }
                {   // E = A^ .* (dP Bf + dO S^T - delta z^T), in place over A^
                    uint32_t v[32];
                    tmem_ld32(R1 + col0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 *cell = reinterpret_cast<uint4 *>(tile_chunk(bX, r, col0 / 8 + q));
                        float a[8];
                        unpack8(*cell, a);
                        const float4 z0 = *reinterpret_cast<const float4 *>(sZ + col0 + 8 * q);
                        const float4 z1 = *reinterpret_cast<const float4 *>(sZ + col0 + 8 * q + 4);
                        const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                        float e[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) e[j] = a[j] * fmaf(-del, zz[j], __uint_as_float(v[8 * q + j]));
                        *cell = make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                    }
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive_warp(bars + QE3);

                EWAIT(QM5);
                tc_fence_after();
                {   // this slab's part of dQ: out of tensor memory, then (once T += E^T Q has read E) staged over E; the control
                    // thread adds the tile into dQ
                    uint32_t v[32];
                    if (col0 < D) {
                        tmem_ld32(R1 + col0, v);
                        tmem_wait_ld();
                    }
                    EWAIT(QM6);
                    if (col0 < D) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(kLn2 * __uint_as_float(v[j]));
#pragma unroll
                        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(tile_chunk(bX, r, col0 / 8 + q)) = pack8(v + 8 * q);
                    }
                }
                fence_async_smem();
                if (g0 && !last) sZ[r] = znext;       // every reader of z is past its E step (E Omega was issued behind all of them)
                tc_fence_before();
                mbar_arrive_warp(bars + QE4);
#undef EWAIT
            }
            // the run's T: every MMA of the run completed before its last T += E^T Q did
            ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + QM6, (it - 1) & 1, status, abort_flag));
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
                tc_fence_before();
                mbar_arrive_warp(bars + QET);
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);   // error path only: let copies and MMAs in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

enum KBars { KB_OM, KB_A, KB_B, KB_V, KB_G, KB_X2, KM3, KM4, KM5, KM6, KM7, KM8, KE2, KE3, KE4, KE5, KNBARS };

// ------------------------------------------------------------------ key side (reverse direction)
template <int D, int DV>
__global__ void __launch_bounds__(kThreads, 1) tc_bwd_k_kernel(const __grid_constant__ BwdParams p)
{
    using L = BwdSmem<D, DV>;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *sOm = smem + L::kOm, *sQA = smem + L::kQA, *sKB = smem + L::kKB, *sV = smem + L::kV;
    unsigned char *sG = smem + L::kG, *sSt = smem + L::kSt, *sStg = smem + L::kAux;
    float *sRho = reinterpret_cast<float *>(smem + L::kVec), *sDel = sRho + 128;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + KNBARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + KNBARS + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nslab, slab = blockIdx.x % p.nslab, h = bh % p.H;
    const int row0 = bh * p.N, rowk0 = kv_row0(bh, p.H, p.Hkv, p.N), T = p.T;      // rowk0: K and V may be shared by a group of query heads
    const int rowo0 = p.out_per_head ? row0 : rowk0;                                 // rows of dK and dV

    if (tid == 0) {
        for (int i = 0; i < KE2; ++i) mbar_init(bars + i, 1);
        for (int i = KE2; i < KNBARS; ++i) mbar_init(bars + i, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128) sRho[tid] = 0.f;
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    int *status = p.status;

    if (*abort_flag) {
        if (tid == 0) atomicExch(status, (int)DARKATTN_ERR_CUDA);
    } else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            auto load_tile = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int width, int t) {
                mbar_expect_tx(bar, 128 * width * 2);
                const int base = (map == &p.mapG) ? row0 : rowk0;
                for (int a = 0; a < width / 64; ++a) tma_load_2d(dst + a * 16384, map, bar, a * 64, base + t * 128);
            };
            auto load_features = [&](unsigned char *dst, const CUtensorMap *map, uint64_t *bar, int t) {
                mbar_expect_tx(bar, 32768);
                tma_load_2d(dst, map, bar, slab * 128, row0 + t * 128);
                tma_load_2d(dst + 16384, map, bar, slab * 128 + 64, row0 + t * 128);
            };
            auto prefetch_features = [&](const CUtensorMap *map, int t) {
                tma_prefetch_l2_2d(map, slab * 128, row0 + t * 128);
                tma_prefetch_l2_2d(map, slab * 128 + 64, row0 + t * 128);
            };
            const TileDesc tOm(sOm), tQA(sQA), tKB(sKB), tV(sV), tG(sG), tSt(sSt), tStg(sStg);
            const uint32_t id_kk = make_idesc(128, 128, 0, 0);
            const uint32_t id_state = make_idesc(128, DV, 1, 1);
            const uint32_t id_dv_t = make_idesc(128, DV, 0, 1);
            const uint32_t id_tm = make_idesc(128, 128, 0, 1);
            const uint32_t id_dx = make_idesc(128, D, 0, 1);
            const uint32_t id_t = make_idesc(128, D, 1, 1);
            const uint32_t R1 = tmem + kColR1, R2 = tmem + kColR2;

            mbar_expect_tx(bars + KB_OM, 128 * D * 2);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sOm + a * 16384, &p.mapOm, bars + KB_OM, a * 64, h * p.m + slab * 128);
            load_tile(sV, &p.mapV, bars + KB_V, DV, T - 1);
            load_tile(sG, &p.mapG, bars + KB_G, DV, T - 1);
            load_features(sQA, &p.mapAh, bars + KB_A, T - 1);
            load_features(sKB, &p.mapBf, bars + KB_B, T - 1);

            // Schedule of one chunk. A^ comes from the query-side kernel through the workspace, Bf from the forward pass
            // through the stash; V dO^T of the next chunk is issued in the tail of the current one.
            //   R1: V dO^T -> packed dP^T [0,64) and P^^T [64,128) (A operands) -> V dO^T of the next chunk
            //   R2: Bf A^^T -> (read) -> dV -> (read) -> dBf -> (E formed) -> dK partial -> (read)
            // Shared memory: the spare tile stages dV, then holds the K tile that T += E^T K needs, then stages dK; so
            // A^ of the next chunk can be fetched as soon as dP^T A^ is done, V and dO with it, Bf once E Omega is done.
            auto store_out = [&](const CUtensorMap *map, int width, int t) {     // the staged tile into (or, with several slabs, added into) the gradient
                for (int a = 0; a < width / 64; ++a) {
                    if (p.add_kv) tma_reduce_add_2d(map, sStg + a * 16384, a * 64, rowo0 + t * 128);
                    else tma_store_2d(map, sStg + a * 16384, a * 64, rowo0 + t * 128);
                }
                tma_store_commit();
            };
            bool ok = wait_or_abort(bars + KB_OM, 0, status, abort_flag);
            if (ok) ok = wait_or_abort(bars + KB_V, 0, status, abort_flag);
            if (ok) ok = wait_or_abort(bars + KB_G, 0, status, abort_flag);
            if (ok) {
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R1, kdesc(tV, k), kdesc(tG, k), id_kk, k > 0);         // V dO^T of the last chunk
                mma_commit(bars + KM3);
            }
            for (int it = 0; it < T && ok; ++it) {
                const int t = T - 1 - it;
                const uint32_t ph = it & 1;
                const bool first = (it == 0), last = (it + 1 == T);
#define KWAIT(b) do { ok = wait_or_abort(bars + (b), ph, status, abort_flag); } while (0)
                KWAIT(KB_A); if (!ok) break;
                KWAIT(KB_B); if (!ok) break;
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(tKB, k), kdesc(tQA, k), id_kk, k > 0);             // P^^T = Bf A^^T
                mma_commit(bars + KM4);
                if (!last) prefetch_features(&p.mapBf, t - 1);      // into L2 now: its load can only be issued late in the chunk
                KWAIT(KE2); if (!ok) break;                                                                      // dP^T and P^^T packed in R1
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + 64 + k * 8, mndesc(tG, k), id_dv_t, k > 0);         // P^^T dO
                if (!first)
                    _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(tKB, k), mndesc(tSt, k), id_dv_t, 1);          // + Bf R_next
                tma_store_wait_read();      // the dK tile of the chunk before has left the spare tile: dV may be staged there
                mma_commit(bars + KM6);
                // the state update is not on the chunk's critical path: it runs while dV is read out
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColState, mndesc(tQA, k), mndesc(tG, k), id_state, (!first) || k > 0);   // R += A^^T dO
                mma_commit(bars + KM5);
                KWAIT(KE3); if (!ok) break;                                                                      // dV read out of R2 and staged
                store_out(&p.mapDV, DV, t);
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ts(R2, R1 + k * 8, mndesc(tQA, k), id_tm, k > 0);               // dP^T A^
                if (!first)
                    _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R2, kdesc(tV, k), kdesc(tSt, k), id_kk, 1);        // + V R_next^T
                mma_commit(bars + KM7);
                KWAIT(KM7); if (!ok) break;                                                                      // A^, V and dO of this chunk are done with
                tma_store_wait_read();                                                                           // the staged dV has left the spare tile:
                load_tile(sStg, &p.mapK, bars + KB_X2, D, t);                                                   // the K tile, for T
                if (!last) {
                    load_features(sQA, &p.mapAh, bars + KB_A, t - 1);
                    load_tile(sV, &p.mapV, bars + KB_V, DV, t - 1);
                    load_tile(sG, &p.mapG, bars + KB_G, DV, t - 1);
                }
                KWAIT(KE4); if (!ok) break;                                                                      // E in smem, R2 read
                KWAIT(KB_X2); if (!ok) break;
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + kColT, mndesc(tKB, k), mndesc(tStg, k), id_t, (!first) || k > 0);   // T += E^T K
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(R2, kdesc(tKB, k), mndesc(tOm, k), id_dx, k > 0);            // E Omega
                mma_commit(bars + KM8);
                if (!last) {
                    ok = wait_or_abort(bars + KB_V, ph ^ 1, status, abort_flag);
                    if (ok) ok = wait_or_abort(bars + KB_G, ph ^ 1, status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    _Pragma("unroll") for (int k = 0; k < DV / 16; ++k) mma_ss(R1, kdesc(tV, k), kdesc(tG, k), id_kk, k > 0);     // V dO^T of the next chunk
                    mma_commit(bars + KM3);
                }
                KWAIT(KM8); if (!ok) break;                                                                      // E and the K tile are done with
                if (!last) load_features(sKB, &p.mapBf, bars + KB_B, t - 1);
                KWAIT(KE5); if (!ok) break;                                                                      // dK read out of R2 and staged; bf16 copy of R in place
                store_out(&p.mapDK, D, t);
#undef KWAIT
            }
            tma_store_wait_all();
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, g = warp >> 2, col0 = g * 32;
        const int r = q4 * 32 + lane;
        const bool g0 = (col0 == 0);
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t R1 = lane_addr + kColR1, R2 = lane_addr + kColR2;
        const size_t rows = (size_t)p.BH * p.N;
        bool ok = true;     // (a wait that gave up switches the warp to a dry run over the remaining chunks: see the query-side kernel)
        for (int it = 0; it < T; ++it) {
            const int t = T - 1 - it;
            const uint32_t ph = it & 1;
            const bool last = (it + 1 == T);
            const size_t row = (size_t)row0 + (size_t)t * 128 + r;
#define EWAIT(b) do { ok = ok && __all_sync(0xffffffffu, wait_or_abort(bars + (b), ph, status, abort_flag)); } while (0)
            float rho_c = 0.f;
            if (g0) {
                rho_c = p.rhoc[((size_t)bh * T + t) * p.m + slab * 128 + r];
                sDel[r] = p.delta[row];
            }
            EWAIT(KM3);
            tc_fence_after();
            {   // dP^T = (V dO^T - delta_i) masked to queries i >= this key, packed over the fp32 tile
                uint32_t v[32], pk[16];
                tmem_ld32(R1 + col0, v);
                tmem_wait_ld();
                epi_sync();          // every column group has read before anyone overwrites; delta of every row is in place
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float2 dl = *reinterpret_cast<const float2 *>(sDel + col0 + j);
                    const float x0 = (col0 + j >= r) ? __uint_as_float(v[j]) - dl.x : 0.f;
                    const float x1 = (col0 + j + 1 >= r) ? __uint_as_float(v[j + 1]) - dl.y : 0.f;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + col0 / 2, pk);
            }
            EWAIT(KM4);
            tc_fence_after();
            {   // P^^T masked the same way, packed behind dP^T
                uint32_t v[32], pk[16];
                tmem_ld32(R2 + col0, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float x0 = (col0 + j >= r) ? __uint_as_float(v[j]) : 0.f;
                    const float x1 = (col0 + j + 1 >= r) ? __uint_as_float(v[j + 1]) : 0.f;
                    pk[j / 2] = pack_bf16(x0, x1);
                }
                tmem_st16(R1 + 64 + col0 / 2, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive_warp(bars + KE2);

            EWAIT(KM6);
            tc_fence_after();
            if (col0 < DV) tmem_row_to_tile(R2 + col0, sStg, r, col0);      // this slab's part of dV, staged: the control thread adds it into dV
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + KE3);

            EWAIT(KM7);
            tc_fence_after();
            {   // E = Bf .* (dP^T A^ + V R^T + rho^T), in place over Bf
                float es = 0.f;
                uint32_t v[32];
                tmem_ld32(R2 + col0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 *cell = reinterpret_cast<uint4 *>(tile_chunk(sKB, r, col0 / 8 + q));
                    float b[8];
                    unpack8(*cell, b);
                    const float4 r0 = *reinterpret_cast<const float4 *>(sRho + col0 + 8 * q);
                    const float4 r1 = *reinterpret_cast<const float4 *>(sRho + col0 + 8 * q + 4);
                    const float rr[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
                    float e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) { e[j] = b[j] * (__uint_as_float(v[8 * q + j]) + rr[j]); es += e[j]; }
                    *cell = make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                }
                p.espart[((size_t)slab * 4 + g) * rows + row] = es;
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + KE4);
            // while T += E^T K and E Omega run: R (updated behind the dV MMAs, its last reader V R^T done before E was formed) -> bf16 copy
            if (!last && col0 < DV) tmem_row_to_tile(lane_addr + kColState + col0, sSt, r, col0);

            EWAIT(KM8);     // (T += E^T K, issued ahead of E Omega, has read the K tile in the spare tile)
            tc_fence_after();
            if (col0 < D) tmem_row_to_tile(R2 + col0, sStg, r, col0, kLn2); // this slab's part of dK (without the norm term), staged: the control thread adds it into dK
            if (g0 && !last) sRho[r] += rho_c;      // rho_next for the chunk below (every reader of rho is past its E step)
            fence_async_smem();
            tc_fence_before();
            mbar_arrive_warp(bars + KE5);
#undef EWAIT
        }
        ok = ok && wait_or_abort(bars + KM8, (T - 1) & 1, status, abort_flag);
        if (ok && col0 < D) {
            tc_fence_after();
            float *dst = p.Tacc + ((size_t)h * p.m + slab * 128 + r) * D + col0;
            uint32_t v[32];
            tmem_ld32(lane_addr + kColT + col0, v);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(v[j]));
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ dK: slab sum + norm term (three MMAs per tile)
//   x~'  = K M^T                      (128 x r)
//   w_j  = -s^2 rowsum(E^K)_j x~'_j   (bf16 operand)
//   dK_j = (dK_j as the scan kernel left it) + w_j M          dMn += w^T K
struct FinishParams {
    CUtensorMap mapK, mapM, mapOut;   // K, M, dK (the norm term's part is added into it)
    const float *espart;  // [nes, BH*N]
    float *dMn;           // [H, r, D]
    int *status;
    int N, H, Hkv, BH, T, nsplit, r, nes;
    int out_per_head;     // dK rows are indexed by the query head (grouped key/value heads)
    float s2;
};

// Shared memory: M tile, two K tiles, the w tile (32 KB), the output staging tile, barriers. The norm term's part of
// dK is added into dK (which holds what the key-side pass added up) by TMA reduce-add stores.
template <int D>
__global__ void __launch_bounds__(kThreads, 1) tc_bwd_finish_k_kernel(const __grid_constant__ FinishParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int kTile = 128 * D * 2;
    unsigned char *sM = smem, *sK0 = smem + kTile, *sW = smem + 3 * kTile, *sOut = sW + 32768;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sOut + kTile);
    uint64_t *bar_m = bars, *bar_k = bars + 1 /* two */, *m1 = bars + 4, *m2 = bars + 5, *m3 = bars + 6;
    uint64_t *e1 = bars + 7, *e2 = bars + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 10);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 11);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.nsplit, split = blockIdx.x % p.nsplit, h = bh % p.H;
    const int t0 = (int)((long long)p.T * split / p.nsplit), t1 = (int)((long long)p.T * (split + 1) / p.nsplit);
    const size_t rows = (size_t)p.BH * p.N;
    if (tid == 0) {
        for (int i = 0; i < 7; ++i) mbar_init(bars + i, 1);
        mbar_init(e1, kEpiWarps); mbar_init(e2, kEpiWarps);
        *abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        fence_mbar_init();
    }
    if (tid < 128)      // columns >= r of the w tile stay zero
        for (int i = tid; i < 2048; i += 128) *reinterpret_cast<uint4 *>(sW + i * 16) = make_uint4(0, 0, 0, 0);
    if (warp == kEpiWarps) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t C1 = 0, C2 = 128, C3 = 256;
    if (*abort_flag) { if (tid == 0) atomicExch(p.status, (int)DARKATTN_ERR_CUDA); }
    else if (t1 <= t0) {}
    else if (warp == kEpiWarps) {
        if ((tid & 31) == 0) {
            const TileDesc tM(sM), tW(sW), tK0(sK0), tK1(sK0 + kTile);
            auto load_k = [&](int t) {
                const int b = (t - t0) & 1;
                mbar_expect_tx(bar_k + b, kTile);
                for (int a = 0; a < D / 64; ++a) tma_load_2d(sK0 + b * kTile + a * 16384, &p.mapK, bar_k + b, a * 64, kv_row0(bh, p.H, p.Hkv, p.N) + t * 128);
            };
            mbar_expect_tx(bar_m, kTile);
            for (int a = 0; a < D / 64; ++a) tma_load_2d(sM + a * 16384, &p.mapM, bar_m, a * 64, h * p.r);
            load_k(t0);
            const uint32_t id_x = make_idesc(128, p.r, 0, 0), id_d = make_idesc(128, D, 0, 1), id_t = make_idesc(128, D, 1, 1);
            // K M^T of tile i+1 is issued right behind the two products of tile i, so that it runs while the epilogue
            // warps still write tile i out.
            bool ok = wait_or_abort(bar_m, 0, p.status, abort_flag);
            if (t0 + 1 < t1) load_k(t0 + 1);
            if (ok) ok = wait_or_abort(bar_k, 0, p.status, abort_flag);
            if (ok) {
                tc_fence_after();
                _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(tmem + C1, kdesc(tK0, k), kdesc(tM, k), id_x, k > 0);
                mma_commit(m1);
            }
            for (int t = t0; t < t1 && ok; ++t) {
                const int i = t - t0, b = i & 1;
                const uint32_t ph = i & 1;
                const TileDesc &tK = b ? tK1 : tK0;
                ok = wait_or_abort(e1, ph, p.status, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < p.r / 16; ++k) mma_ss(tmem + C2, kdesc(tW, k), mndesc(tM, k), id_d, k > 0);
                mma_commit(m2);
                _Pragma("unroll") for (int k = 0; k < 8; ++k) mma_ss(tmem + C3, mndesc(tW, k), mndesc(tK, k), id_t, (t > t0) || k > 0);
                mma_commit(m3);
                if (t + 1 < t1) {
                    ok = wait_or_abort(bar_k + (b ^ 1), ((i + 1) >> 1) & 1, p.status, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const TileDesc &tKn = b ? tK0 : tK1;
                    _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(tmem + C1, kdesc(tKn, k), kdesc(tM, k), id_x, k > 0);
                    mma_commit(m1);
                }
                ok = wait_or_abort(m3, ph, p.status, abort_flag);
                if (!ok) break;
                if (t + 2 < t1) load_k(t + 2);          // this tile's K buffer has been read by both of its products
                ok = wait_or_abort(e2, ph, p.status, abort_flag);
            }
        }
    } else {
        const int lane = tid & 31, q4 = warp & 3, col0 = (warp >> 2) * 32;
        const int r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        bool ok = true;
        // rowsum(E) of a tile's row: its partials are loaded one tile ahead (their latency is hidden behind a tile's work)
        auto row_sum = [&](int t) {
            const size_t rw = (size_t)bh * p.N + (size_t)t * 128 + r;
            float e = 0.f;
            for (int s = 0; s < p.nes; ++s) e += __ldg(p.espart + (size_t)s * rows + rw);
            return e;
        };
        float es_next = row_sum(t0);
        // (a wait that gave up switches the warp to a dry run over the remaining tiles, so that epi_sync still gets every arrival)
        for (int t = t0; t < t1; ++t) {
            const uint32_t ph = (t - t0) & 1;
            const float coef = -p.s2 * es_next;
            ok = ok && __all_sync(0xffffffffu, wait_or_abort(m1, ph, p.status, abort_flag));
            tc_fence_after();
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int c = col0 + 16 * hh;
                if (c < p.r) {
                    uint32_t v[16];
                    tmem_ld16(lane_addr + C1 + c, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(coef * __uint_as_float(v[j]));
                    *reinterpret_cast<uint4 *>(tile_chunk(sW, r, c / 8)) = pack8(v);
                    *reinterpret_cast<uint4 *>(tile_chunk(sW, r, c / 8 + 1)) = pack8(v + 8);
                }
            }
            fence_async_smem();
            if (tid == 0) tma_store_wait_read();          // the staging tile of the previous store is free again
            tc_fence_before();
            mbar_arrive_warp(e1);
            if (t + 1 < t1) es_next = row_sum(t + 1);

            ok = ok && __all_sync(0xffffffffu, wait_or_abort(m2, ph, p.status, abort_flag));
            tc_fence_after();
            if (col0 < D) {
                uint32_t v[32];
                tmem_ld32(lane_addr + C2 + col0, v);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(tile_chunk(sOut, r, col0 / 8 + q)) = pack8(v + 8 * q);
            }
            fence_async_smem();
            epi_sync();
            if (tid == 0) {
                for (int a = 0; a < D / 64; ++a)
                    tma_reduce_add_2d(&p.mapOut, sOut + a * 16384, a * 64, (p.out_per_head ? bh * p.N : kv_row0(bh, p.H, p.Hkv, p.N)) + t * 128);
                tma_store_commit();
            }
            tc_fence_before();
            mbar_arrive_warp(e2);
        }
        if (tid == 0) tma_store_wait_all();
        if (ok) ok = wait_or_abort(m3, (t1 - 1 - t0) & 1, p.status, abort_flag);
        if (ok && q4 * 32 < p.r && col0 < D) {      // whole warps: the tensor-memory load is a warp-wide instruction
            tc_fence_after();
            float *dst = p.dMn + ((size_t)h * p.r + r) * D + col0;
            uint32_t v[32];
            tmem_ld32(lane_addr + C3 + col0, v);
            tmem_wait_ld();
            if (r < p.r) {                           // r may end inside the warp's 32 rows (r = 16, 48, ...)
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(v[j]));
            }
        }
    }
    if (*abort_flag) __nanosleep(200000);
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ small SIMT kernels
// Grouped key/value heads: out[(b,hk),i,:] = sum_g src[(b, hk G + g),i,:], added up in fp32 and rounded once; eight
// elements per thread.
__global__ void group_sum_kernel(const __nv_bfloat16 *src, __nv_bfloat16 *out, int N, int w, int H, int Hkv, long long total8)
{
    const long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (t >= total8) return;
    const int per_row = w / 8, G = H / Hkv;
    const int c8 = (int)(t % per_row);
    const long long row = t / per_row;
    const int i = (int)(row % N);
    const long long bhk = row / N, b = bhk / Hkv, hk = bhk % Hkv;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int g = 0; g < G; ++g) {
        float x[8];
        unpack8(*reinterpret_cast<const uint4 *>(src + (((b * H + hk * G + g) * N + i) * (long long)w + c8 * 8)), x);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] += x[j];
    }
    uint32_t pk[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) pk[j] = __float_as_uint(acc[j]);
    *reinterpret_cast<uint4 *>(out + t * 8) = pack8(pk);
}

// delta[row] = dO[row,:] . O[row,:]; dv/8 threads per row, 16 bytes of each tensor per thread.
__global__ void delta_kernel(const __nv_bfloat16 *G, const __nv_bfloat16 *O, float *delta, long long rows, int dv)
{
    const int per_row = dv / 8;                       // 8 or 16: a power of two that divides the warp
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long row = i / per_row;
    float acc = 0.f;
    if (row < rows) {
        float g[8], o[8];
        unpack8(*reinterpret_cast<const uint4 *>(G + i * 8), g);
        unpack8(*reinterpret_cast<const uint4 *>(O + i * 8), o);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc = fmaf(g[j], o[j], acc);
    }
    for (int o = per_row / 2; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (row < rows && (i % per_row) == 0) delta[row] = acc;
}

// dM[h,a,c] += s * sum_{l in this block's 64 rows} W[l,a] T[h,l,c]  (+ dMn[h,a,c] from the first block of rows);
// dM is zeroed before the launch. One block per (8 rows a, head, 64 rows l), one thread per column c: many small
// blocks, because the kernel is bound by the latency of its loads.
__global__ void dm_kernel(const __nv_bfloat16 *W, const float *Tacc, const float *dMn, float *dM, int m, int r, int d, int w_per_head, float s)
{
    __shared__ float sw[64 * 8];
    const int a0 = blockIdx.x * 8, h = blockIdx.y, lb = blockIdx.z * 64, c = threadIdx.x;
    const __nv_bfloat16 *w = W + (size_t)(w_per_head ? h : 0) * m * r;
    for (int i = threadIdx.x; i < 64 * 8; i += blockDim.x) {
        const int l = i / 8, j = i % 8;
        sw[i] = (a0 + j < r) ? __bfloat162float(w[(size_t)(lb + l) * r + a0 + j]) : 0.f;
    }
    __syncthreads();
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const float *Th = Tacc + ((size_t)h * m + lb) * d + c;
    for (int l0 = 0; l0 < 64; l0 += 16) {
        float tv[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) tv[i] = Th[(size_t)(l0 + i) * d];
#pragma unroll
        for (int i = 0; i < 16; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = fmaf(sw[(l0 + i) * 8 + j], tv[i], acc[j]);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
        if (a0 + j < r) {
            float v = s * acc[j];
            if (lb == 0 && dMn) v += dMn[((size_t)h * r + a0 + j) * d + c];
            atomicAdd(dM + ((size_t)h * r + a0 + j) * d + c, v);
        }
}

// dM += dMn (the norm term's part, when dm_kernel ran beside the kernel that produces it)
__global__ void dm_add_kernel(float *dM, const float *dMn, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dM[i] += dMn[i];
}

// dW[(h,) l, a] = s * sum_c T[h,l,c] M[h,a,c], summed over the heads when W is shared: through the folded projection
// u_l = s w_l . (M x) the gradient of w_l is s M (sum_i E_il x_i). One block per row l (and head), one thread per a.
__global__ void dw_kernel(const float *Tacc, const __nv_bfloat16 *M, float *dW, int H, int m, int r, int d, int w_per_head, float s)
{
    const int l = blockIdx.x, a = threadIdx.x;
    const int h0 = w_per_head ? blockIdx.y : 0, h1 = w_per_head ? blockIdx.y + 1 : H;
    float acc = 0.f;
    for (int h = h0; h < h1; ++h) {
        const float *T = Tacc + ((size_t)h * m + l) * d;
        const __nv_bfloat16 *Ma = M + ((size_t)h * r + a) * d;
        for (int c = 0; c < d; c += 8) {
            float f[8];
            unpack8(*reinterpret_cast<const uint4 *>(Ma + c), f);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc = fmaf(T[c + j], f[j], acc);
        }
    }
    dW[((size_t)(w_per_head ? blockIdx.y : 0) * m + l) * r + a] = s * acc;
}

int sm_count()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) n = v;
        else n = 148;
    }
    return n;
}

template <int D, int DV>
cudaError_t launch_scan(const darkattn_plan_s *plan, const BwdParams &P, int grid, cudaStream_t st)
{
    using L = BwdSmem<D, DV>;
    static_assert(L::kTotal <= 232448, "shared memory budget of one CTA exceeded");
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_q_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tc_bwd_k_kernel<D, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    // the query-side kernel divides all chunks evenly over the SMs: groups of nslab CTAs, one group per piece
    long long groups = sm_count() / P.nslab;
    if (groups < 1) groups = 1;
    if (groups > (long long)P.BH * P.T) groups = (long long)P.BH * P.T;
    const int qgrid = (int)groups * P.nslab;
    timer_mark(plan, st, "tc_bwd_q_kernel");
    tc_bwd_q_kernel<D, DV><<<qgrid, kThreads, L::kTotal, st>>>(P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (P.add_kv) {
        e = cudaStreamWaitEvent(st, plan->aux_join, 0);      // dK and dV have been zeroed
        if (e != cudaSuccess) return e;
    }
    timer_mark(plan, st, "tc_bwd_k_kernel");
    tc_bwd_k_kernel<D, DV><<<grid, kThreads, L::kTotal, st>>>(P);
    return cudaGetLastError();
}

template <int D>
cudaError_t launch_finish(FinishParams &P, int grid, cudaStream_t st)
{
    constexpr int kTile = 128 * D * 2, smem_bytes = 4 * kTile + 32768 + 128;    // M, two K tiles, staging; w; barriers
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_finish_k_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    tc_bwd_finish_k_kernel<D><<<grid, kThreads, smem_bytes, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

darkattn_status_t tensor_backward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                  const void *M, const void *W, const void *O, const void *dO, const void *saved,
                                  void *dQ, void *dK, void *dV, float *dM, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    const size_t BH = D.BH, N = D.N;
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16 *>(ws + off); };
    auto fl = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    if (!encode_fn()) { set_cuda_error(cudaErrorNotSupported, "tensor_backward: cuTensorMapEncodeTiled unavailable"); return DARKATTN_ERR_CUDA; }

    cudaError_t e = cudaSuccess;
    auto keep = [&](cudaError_t x) { if (x != cudaSuccess && e == cudaSuccess) e = x; };
    auto chk = [&]() { keep(cudaGetLastError()); };

    // The forward result and what the forward pass stashed (per-row normalisers, key norms, folded
    // projections, key shifts): taken from the caller when both are given, otherwise recomputed into the
    // workspace by running the forward kernels again.
    Stash stash;
    if (!O || !saved) {
        darkattn_status_t s = tensor_forward(plan, Q, K, V, M, W, bf(Y.Oscr), nullptr, ws, st, true);
        if (s != DARKATTN_OK) return s;
        O = bf(Y.Oscr);
        stash = stash_in_workspace(Y, ws);
    } else {
        stash = stash_in_saved(Y, const_cast<void *>(saved));
    }

    const long long rows = (long long)BH * N;
    timer_mark(plan, st, "delta_kernel");
    delta_kernel<<<(unsigned)((rows * (D.dv / 8) + 255) / 256), 256, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, fl(Y.delta), rows, D.dv);
    chk();
    keep(cudaMemsetAsync(ws + Y.Tacc, 0, (size_t)D.H * D.m * D.d * 4, st));
    keep(cudaMemsetAsync(ws + Y.dMn, 0, (size_t)D.H * D.r * D.d * 4, st));
    const size_t BHkv = (size_t)D.B * D.Hkv;
    // Grouped key/value heads: every query head's part of dK and dV goes to rows of its own in the workspace (so that an
    // element is rounded to bf16 as often as without groups), and a last kernel adds each group up in fp32.
    const bool per_head = D.G > 1;
    void *dKo = per_head ? (void *)bf(Y.dKh) : dK, *dVo = per_head ? (void *)bf(Y.dVh) : dV;
    const size_t BHo = per_head ? BH : BHkv;
    const bool add_kv = Y.nslab > 1;
    if (add_kv) {
        // The slabs of a head add their parts into the gradients, which therefore start at zero. dQ is needed first; dK and
        // dV are zeroed on a side stream while the query-side scan runs (it leaves SMs and bandwidth free).
        keep(ensure_aux(plan));
        if (e != cudaSuccess) { set_cuda_error(e, "tensor_backward: side stream"); return DARKATTN_ERR_CUDA; }
        keep(cudaEventRecord(plan->aux_fork, st));
        keep(cudaStreamWaitEvent(plan->aux_stream, plan->aux_fork, 0));
        keep(cudaMemsetAsync(dKo, 0, BHo * N * D.d * 2, plan->aux_stream));
        keep(cudaMemsetAsync(dVo, 0, BHo * N * D.dv * 2, plan->aux_stream));
        keep(cudaEventRecord(plan->aux_join, plan->aux_stream));
    }
    if (Y.nslab > 1) keep(cudaMemsetAsync(dQ, 0, BH * N * D.d * 2, st));

    FinishParams F;
    memset(&F, 0, sizeof(F));
    if (!make_map(&F.mapM, M, (size_t)D.H * D.r, D.d, 128) || !make_map(&F.mapK, K, BHkv * N, D.d, 128)) {
        set_cuda_error(cudaErrorInvalidValue, "tensor_backward: tensor map encode");
        return DARKATTN_ERR_CUDA;
    }
    if (D.causal) {
        BwdParams P;
        memset(&P, 0, sizeof(P));
        const bool ok = make_map(&P.mapQ, Q, BH * N, D.d, 128) && make_map(&P.mapK, K, BHkv * N, D.d, 128) &&
                        make_map(&P.mapV, V, BHkv * N, D.dv, 128) && make_map(&P.mapG, dO, BH * N, D.dv, 128) &&
                        make_map(&P.mapOm, stash.Om, (size_t)D.H * D.m, D.d, 128) &&
                        make_map(&P.mapOml, stash.Oml, (size_t)D.H * D.m, D.d, 128) &&
                        make_map(&P.mapDQ, dQ, BH * N, D.d, 128) && make_map(&P.mapDK, dKo, BHo * N, D.d, 128) &&
                        make_map(&P.mapDV, dVo, BHo * N, D.dv, 128) &&
                        make_map(&P.mapAh, bf(Y.Ahat), BH * N, D.m, 128) && make_map(&P.mapBf, stash.Bphi, BH * N, D.m, 128) &&
                        make_map(&P.mapSst, stash.Sst, BH * Y.T * D.m, D.dv, 128);
        if (!ok) { set_cuda_error(cudaErrorInvalidValue, "tensor_backward: tensor map encode"); return DARKATTN_ERR_CUDA; }
        P.sv = stash.sv; P.delta = fl(Y.delta); P.nK = stash.nK; P.cs = stash.cs; P.zc = stash.zc; P.rhoc = fl(Y.rhoc);
        P.espart = fl(Y.espart); P.Tacc = fl(Y.Tacc);
        P.status = reinterpret_cast<int *>(ws + Y.status);
        P.N = D.N; P.H = D.H; P.Hkv = D.Hkv; P.BH = D.BH; P.m = D.m; P.nslab = Y.nslab; P.T = Y.T; P.add_kv = add_kv ? 1 : 0;
        P.out_per_head = per_head ? 1 : 0;
        const int units = (int)(BH * Y.nslab);
        if (D.d == 64 && D.dv == 64) keep(launch_scan<64, 64>(plan, P, units, st));
        else if (D.d == 128 && D.dv == 128) keep(launch_scan<128, 128>(plan, P, units, st));
        else if (D.d == 64 && D.dv == 128) keep(launch_scan<64, 128>(plan, P, units, st));
        else keep(launch_scan<128, 64>(plan, P, units, st));
    } else {
        keep(tensor_backward_nc_passes(plan, Q, K, V, dO, stash, dQ, dKo, dVo, per_head, ws, st));
    }

    if (!make_map(&F.mapOut, dKo, BHo * N, D.d, 128)) { set_cuda_error(cudaErrorInvalidValue, "tensor_backward: tensor map encode"); return DARKATTN_ERR_CUDA; }
    F.espart = fl(Y.espart); F.dMn = fl(Y.dMn);
    F.status = reinterpret_cast<int *>(ws + Y.status);
    F.N = D.N; F.H = D.H; F.Hkv = D.Hkv; F.BH = D.BH; F.T = Y.T; F.r = D.r; F.nes = 4 * Y.nslab; F.s2 = D.s * D.s; F.out_per_head = per_head ? 1 : 0;
    F.nsplit = pick_splits((long long)BH, Y.T, 3.5, 5.0, 64);
    // dM = s W^T T + (norm term). T is complete once the key-side pass is done, so its product runs on the side
    // stream next to the kernel that produces the norm term, and a small kernel adds the two. (With per-kernel
    // timing on, everything stays on one stream.)
    const dim3 dm_grid((D.r + 7) / 8, D.H, D.m / 64);
    const bool beside = !plan->timer.on && ensure_aux(plan) == cudaSuccess;
    if (beside) {
        keep(cudaEventRecord(plan->aux_fork, st));
        keep(cudaStreamWaitEvent(plan->aux_stream, plan->aux_fork, 0));
        keep(cudaMemsetAsync(dM, 0, (size_t)D.H * D.r * D.d * 4, plan->aux_stream));
        dm_kernel<<<dm_grid, D.d, 0, plan->aux_stream>>>((const __nv_bfloat16 *)W, fl(Y.Tacc), nullptr, dM, D.m, D.r, D.d, D.w_per_head, D.s);
        chk();
        keep(cudaEventRecord(plan->aux_join, plan->aux_stream));
    }
    timer_mark(plan, st, "tc_bwd_finish_k_kernel");
    if (D.d == 64) keep(launch_finish<64>(F, (int)(BH * F.nsplit), st));
    else keep(launch_finish<128>(F, (int)(BH * F.nsplit), st));

    if (beside) {
        keep(cudaStreamWaitEvent(st, plan->aux_join, 0));
        const int n = D.H * D.r * D.d;
        dm_add_kernel<<<(n + 255) / 256, 256, 0, st>>>(dM, fl(Y.dMn), n);
        chk();
    } else {
        timer_mark(plan, st, "dm_kernel");
        keep(cudaMemsetAsync(dM, 0, (size_t)D.H * D.r * D.d * 4, st));
        dm_kernel<<<dm_grid, D.d, 0, st>>>((const __nv_bfloat16 *)W, fl(Y.Tacc), fl(Y.dMn), dM, D.m, D.r, D.d, D.w_per_head, D.s);
        chk();
    }
    if (per_head) {
        const long long nk = (long long)BHkv * N * D.d / 8, nv = (long long)BHkv * N * D.dv / 8;
        timer_mark(plan, st, "group_sum_kernel (dK)");
        group_sum_kernel<<<(unsigned)((nk + 255) / 256), 256, 0, st>>>(bf(Y.dKh), (__nv_bfloat16 *)dK, D.N, D.d, D.H, D.Hkv, nk);
        chk();
        timer_mark(plan, st, "group_sum_kernel (dV)");
        group_sum_kernel<<<(unsigned)((nv + 255) / 256), 256, 0, st>>>(bf(Y.dVh), (__nv_bfloat16 *)dV, D.N, D.dv, D.H, D.Hkv, nv);
        chk();
    }
    if (e != cudaSuccess) { set_cuda_error(e, "tensor_backward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

darkattn_status_t tensor_backward_dw(const darkattn_plan_s *plan, const void *M, float *dW, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const TensorLayout &Y = plan->tensor;
    timer_mark(plan, st, "dw_kernel");
    dw_kernel<<<dim3(D.m, D.w_per_head ? D.H : 1), D.r, 0, st>>>(reinterpret_cast<const float *>(ws + Y.Tacc), (const __nv_bfloat16 *)M, dW,
                                                                D.H, D.m, D.r, D.d, D.w_per_head, D.s);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, "tensor_backward_dw"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

}  // namespace darkattn
