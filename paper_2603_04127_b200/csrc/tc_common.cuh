// Blackwell (sm_100a) building blocks used by the tensor-core kernels: mbarriers with bounded waits,
// TMA tile loads/stores, TMEM allocation, tcgen05.mma issue/commit, TMEM loads, and the shared-memory
// matrix descriptors of the 128-byte-swizzled operand layouts.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>

namespace darkattn {
namespace tc {

// Upper bound on one mbarrier wait, in nanoseconds of the global timer. A healthy wait finishes in
// microseconds; when the bound runs out the kernel records DARKATTN_ERR_TIMEOUT in the status word
// and unwinds instead of spinning forever.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One arrival for the whole warp: every lane's earlier writes are ordered before it by the warp barrier.
__device__ __forceinline__ void mbar_arrive_warp(uint64_t *bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}
// Returns false (after setting *status) if the phase did not complete within kWaitLimitNs.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int *status)
{
    for (int i = 0; i < 64; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kWaitLimitNs) break;
    }
    atomicExch(status, 5 /* DARKATTN_ERR_TIMEOUT */);
    return false;
}

// ---------------------------------------------------------------- proxies and fences
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---------------------------------------------------------------- TMA (tiled, 2-D, no multicast)
// The innermost coordinate x times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
// Brings a tile into L2 only (no shared-memory destination, nothing to wait for): issued a chunk ahead of the tile's
// load, which then finds its lines in L2 instead of paying the latency of HBM.
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap *map, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, const void *smem_src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}
// Element-wise add of a shared-memory tile into global memory (the additions are done in the tensor's type, bf16
// here, by the memory system): several CTAs may add into the same tile.
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, const void *smem_src, int x, int y)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... of all but the most recently committed group (groups complete in the order they were committed)
__device__ __forceinline__ void tma_store_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---------------------------------------------------------------- TMEM
// Warp-collective. ncols: power of two in [32, 512]. The base address is written to *smem_slot.
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_slot, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base lane + t).
// A warp may only touch the TMEM lane quarter 32*(warp_id % 4) .. +31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// one 32-bit column: thread t of the warp receives lane (base lane + t)
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr)
{
    uint32_t v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(taddr) : "memory");
    return v;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- tcgen05.mma (bf16 x bf16 -> fp32)
// Instruction descriptor, kind::f16: D fp32, A and B bf16, dense, no negation.
// a_mn / b_mn: 1 when that operand is stored MN-major (the M or N index contiguous), 0 for K-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn, int b_mn)
{
    return (1u << 4)        // D format: F32
         | (1u << 7)        // A format: BF16
         | (1u << 10)       // B format: BF16
         | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
         | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Shared-memory matrix descriptor for a 128-byte-swizzled operand (the layout TMA writes with
// CU_TENSOR_MAP_SWIZZLE_128B into a 1024-byte aligned tile whose rows are 128 bytes).
//   K-major operand : rows = M/N index, 128-byte row = 64 bf16 along K. sbo = bytes between groups of
//                     8 rows (1024 when rows are dense); lbo is not used by the hardware (set to 16).
//                     One MMA (K = 16) reads 32 bytes of each row: advance the start address by 32.
//   MN-major operand: rows = K index, 128-byte row = 64 bf16 along M/N. sbo = bytes between groups of
//                     8 K-rows (1024), lbo = bytes between 64-element blocks along M/N.
//                     One MMA (K = 16) reads 16 rows: advance the start address by 2048.
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;      // descriptor version of sm_100
    d |= (uint64_t)2 << 61;      // layout type: 128-byte swizzle
    return d;
}

// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread. accumulate = 0 overwrites D.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]. A is a 128-row bf16 operand held in tensor memory: lane = row,
// each 32-bit column holds two consecutive K elements (even K in the low half), K-major only.
// One MMA (K = 16) reads 8 columns: advance the A address by 8 per step.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Make the mbarrier observe completion of all MMAs this thread issued so far (implies the
// tcgen05 before_thread_sync fence).
__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Byte offset of element (row, 16-byte chunk) inside a 128-byte-swizzled tile with 128-byte rows.
__device__ __forceinline__ uint32_t swz128(uint32_t row, uint32_t chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Floats as integers whose order is the floats' order (for atomicMax on signed integers), and back.
__device__ __forceinline__ int float_order_key(float x) { const int b = __float_as_int(x); return b >= 0 ? b : b ^ 0x7fffffff; }
__device__ __forceinline__ float float_from_order_key(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }
// The key-side shift of a (batch, head, slab): kept as such an integer by the kernel that takes the maximum over the keys.
__device__ __forceinline__ float load_key_shift(const float *cs, int i) { return float_from_order_key(reinterpret_cast<const int *>(cs)[i]); }

// mbarrier wait that also gives up when another thread of the CTA already did.
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, int *status, volatile int *abort_flag)
{
    for (int i = 0; i < 128; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > kWaitLimitNs) break;
    }
    *abort_flag = 1;
    atomicExch(status, 5 /* DARKATTN_ERR_TIMEOUT */);
    return false;
}

// ---------------------------------------------------------------- tiles, epilogue layout, descriptors
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

// Epilogue thread layout: 16 warps. Warp w works on TMEM lanes (tile rows) 32 (w % 4) .. +31, the only
// ones it may touch, and on the 32 columns starting at 32 (w / 4); four warps share each row.
constexpr int kEpiWarps = 16, kEpiThreads = 512, kThreads = 544;

// the four warps that share a lane quarter
__device__ __forceinline__ void quarter_sync(int q) { asm volatile("bar.sync %0, 128;" ::"r"(q + 1) : "memory"); }
// all epilogue threads
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 5, 512;" ::: "memory"); }

// features 2^(U - offset): 32 TMEM columns at taddr -> bf16 tile row `row`, columns [col0, col0 + 32)
__device__ __forceinline__ void features_to_tile(uint32_t taddr, float offset, unsigned char *tile, int row, int col0)
{
    uint32_t v[32], pk[16];
    tmem_ld32(taddr, v);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; j += 2)
        pk[j / 2] = pack_bf16(ex2f(__uint_as_float(v[j]) - offset), ex2f(__uint_as_float(v[j + 1]) - offset));
#pragma unroll
    for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4 *>(tile_chunk(tile, row, col0 / 8 + q)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
}

// 32 fp32 TMEM columns at taddr, times scale -> bf16 tile row (swizzled smem), columns [col0, col0 + 32)
__device__ __forceinline__ void tmem_row_to_tile(uint32_t taddr, unsigned char *tile, int row, int col0, float scale = 1.f)
{
    uint32_t v[32];
    tmem_ld32(taddr, v);
    tmem_wait_ld();
    if (scale != 1.f) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(scale * __uint_as_float(v[j]));
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(tile_chunk(tile, row, col0 / 8 + q)) = pack8(v + 8 * q);
}

// Matrix descriptors are built once per tile buffer; step k of an MMA loop only adds a constant to the
// start-address field (units of 16 bytes), so that the issuing thread spends one add per instruction.
struct TileDesc {
    uint64_t kmaj, mnmaj;
    __device__ __forceinline__ explicit TileDesc(const unsigned char *base)
        : kmaj(make_sdesc(smem_u32(base), 16, 1024)), mnmaj(make_sdesc(smem_u32(base), 16384, 1024)) {}
};
// K-major operand, 64-element atoms 16 KB apart: step k covers 16 elements (32 bytes) of K
__device__ __forceinline__ uint64_t kdesc(const TileDesc &t, int k) { return t.kmaj + (uint64_t)(((k / 4) * 16384 + (k % 4) * 32) >> 4); }
// MN-major operand: step k covers 16 K-rows of 128 bytes
__device__ __forceinline__ uint64_t mndesc(const TileDesc &t, int k) { return t.mnmaj + (uint64_t)((k * 2048) >> 4); }

// X (Om + Oml)^T into a TMEM region: the projection against both halves of the folded matrix (its bf16 rounding and
// the bf16 rounding of what that left out), accumulated in fp32
template <int D>
__device__ __forceinline__ void issue_projection(uint32_t dst, const TileDesc &tX, const TileDesc &tOm, const TileDesc &tOml, uint32_t idesc)
{
    _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(dst, kdesc(tX, k), kdesc(tOm, k), idesc, k > 0);
    _Pragma("unroll") for (int k = 0; k < D / 16; ++k) mma_ss(dst, kdesc(tX, k), kdesc(tOml, k), idesc, 1);
}

// First row, in the [B * H_kv * N, width] view of K, V, dK, dV, of the key/value head that query head bh = b H + h reads
// (grouped key/value heads: G = H / H_kv consecutive query heads share one).
__device__ __forceinline__ int kv_row0(int bh, int H, int Hkv, int N) { return ((bh / H) * Hkv + (bh % H) / (H / Hkv)) * N; }

// ---------------------------------------------------------------- host side: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor [rows, cols] (cols contiguous), box = 64 columns x box_rows rows, 128-byte swizzle.
inline bool make_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace darkattn
