// Single-token decode step of causal DARK attention: the recurrent form of the causal scan. Per (batch, head) the
// caller keeps the running state S = sum_j phi(k_j) v_j^T (m x dv) and z = sum_j phi(k_j) (m), both float32; one step
// adds the new token's key and value and reads the new token's query out:
//     S += phi(k) v^T,   z += phi(k),   o = phi(q)^T S / phi(q)^T z          (Section 2's ordering phi(Q) (phi(K)^T V), one row at a time)
// Stabiliser (cancels in o, and is the same at every step, so the state of one step is valid for the next): keys use
// the per-feature shift c_l = |w_l|^2 / 2, i.e. phi(k)_l = exp(u_l - |x~|^2/2 - c_l) = exp(-|x~ - w_l|^2 / 2) <= 1;
// queries use exp(u_l + c_l - max_l(u_l + c_l)).
// The step is bound by the traffic of the state (read and written once): plain SIMT, FP32, coalesced over dv.
#include "common.cuh"

#include <math.h>

namespace darkattn {

namespace {

template <typename T>
__device__ __forceinline__ float ldf(const T *p, size_t i)
{
    if constexpr (sizeof(T) == 2) return __bfloat162float(p[i]);
    else return p[i];
}

// Features of one (batch, head)'s new token, by a block of 256 threads: fk[l] = phi(k)_l and, when WITH_Q, fq[l] = phi(q)_l
// (shared memory: xq[r], xk[r], fq[m], fk[m], red[...]).
template <typename T, bool WITH_Q>
__device__ __forceinline__ void token_features(const T *qv, const T *kv, const T *Mh, const T *Wh, float *xq, float *xk, float *fq,
                                               float *fk, float *red, int d, int r, int m, float s)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // x~ = s M x for the query and the key: one warp per row of M, its lanes along the row (coalesced), shuffle sum
    for (int a = warp; a < r; a += 8) {
        float aq = 0.f, ak = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float mv = ldf(Mh, (size_t)a * d + c);
            if constexpr (WITH_Q) aq = fmaf(mv, ldf(qv, c), aq);
            ak = fmaf(mv, ldf(kv, c), ak);
        }
        for (int off = 16; off; off >>= 1) {
            if constexpr (WITH_Q) aq += __shfl_xor_sync(0xffffffffu, aq, off);
            ak += __shfl_xor_sync(0xffffffffu, ak, off);
        }
        if (lane == 0) { xq[a] = s * aq; xk[a] = s * ak; }
    }
    __syncthreads();
    float nk = 0.f;
    for (int a = lane; a < r; a += 32) nk = fmaf(xk[a], xk[a], nk);
    for (int off = 16; off; off >>= 1) nk += __shfl_xor_sync(0xffffffffu, nk, off);
    nk *= 0.5f;
    float mx = -INFINITY;
    for (int l = warp; l < m; l += 8) {             // exponents of the features: one warp per row of W
        float uq = 0.f, uk = 0.f, c = 0.f;
        for (int a = lane; a < r; a += 32) {
            const float w = ldf(Wh, (size_t)l * r + a);
            if constexpr (WITH_Q) uq = fmaf(w, xq[a], uq);
            uk = fmaf(w, xk[a], uk);
            c = fmaf(w, w, c);
        }
        for (int off = 16; off; off >>= 1) {
            if constexpr (WITH_Q) uq += __shfl_xor_sync(0xffffffffu, uq, off);
            uk += __shfl_xor_sync(0xffffffffu, uk, off);
            c += __shfl_xor_sync(0xffffffffu, c, off);
        }
        c *= 0.5f;
        if (lane == 0) { fk[l] = __expf(uk - nk - c); fq[l] = uq + c; }
        mx = fmaxf(mx, uq + c);
    }
    if constexpr (WITH_Q) {
        for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        if ((tid & 31) == 0) red[tid >> 5] = mx;
        __syncthreads();
        mx = red[0];
        for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
        __syncthreads();
        for (int l = tid; l < m; l += 256) fq[l] = __expf(fq[l] - mx);
    }
    __syncthreads();
}

// grid = (dv / 32 column blocks, B*H); block = 256 threads = 32 columns x 8 groups of features. Every column block of a
// (batch, head) needs z + phi(k) for the normaliser; none of them stores it (the blocks are not ordered among themselves):
// decode_z_kernel, launched behind this one on the same stream, applies z += phi(k).
template <typename T>
__global__ void __launch_bounds__(256) decode_step_kernel(const T *q, const T *k, const T *v, const T *M, const T *W, float *S,
                                                           const float *z, T *o, int H, int Hkv, int d, int r, int m, int dv, int w_per_head,
                                                           float s)
{
    extern __shared__ float sm[];
    float *xq = sm, *xk = xq + r, *fq = xk + r, *fk = fq + m, *red = fk + m;   // red: 8 x 32 partial numerators + 8 partial normalisers + scratch
    const int bh = blockIdx.y, h = bh % H, tid = threadIdx.x;
    const int kvh = (bh / H) * Hkv + h / (H / Hkv);     // the key/value head this query head reads (grouped key/value heads)
    token_features<T, true>(q + (size_t)bh * d, k + (size_t)kvh * d, M + (size_t)h * r * d, W + (size_t)(w_per_head ? h : 0) * m * r,
                            xq, xk, fq, fk, red, d, r, m, s);

    // state update and read-out: thread = (column, feature group)
    const int col = blockIdx.x * 32 + (tid & 31), grp = tid >> 5;
    const float vv = ldf(v, (size_t)kvh * dv + col);
    float *Sb = S + (size_t)bh * m * dv;
    const float *zb = z + (size_t)bh * m;
    float num = 0.f, den = 0.f;
    for (int l = grp; l < m; l += 8) {
        const float snew = fmaf(fk[l], vv, Sb[(size_t)l * dv + col]);
        Sb[(size_t)l * dv + col] = snew;
        num = fmaf(fq[l], snew, num);
        if ((tid & 31) == 0) {                       // one lane per group carries the normaliser
            den = fmaf(fq[l], zb[l] + fk[l], den);
        }
    }
    red[grp * 32 + (tid & 31)] = num;
    if ((tid & 31) == 0) red[256 + grp] = den;
    __syncthreads();
    if (tid < 32) {
        float n = 0.f, dn = 0.f;
        for (int g = 0; g < 8; ++g) { n += red[g * 32 + tid]; dn += red[256 + g]; }
        const float out = n / dn;
        if constexpr (sizeof(T) == 2) o[(size_t)bh * dv + blockIdx.x * 32 + tid] = __float2bfloat16_rn(out);
        else o[(size_t)bh * dv + blockIdx.x * 32 + tid] = out;
    }
}

// z += phi(k) of the new token; one block per (batch, head).
template <typename T>
__global__ void __launch_bounds__(256) decode_z_kernel(const T *k, const T *M, const T *W, float *z, int H, int Hkv, int d, int r, int m,
                                                        int w_per_head, float s)
{
    extern __shared__ float sm[];
    float *xq = sm, *xk = xq + r, *fq = xk + r, *fk = fq + m, *red = fk + m;
    const int bh = blockIdx.x, h = bh % H;
    token_features<T, false>(nullptr, k + (size_t)((bh / H) * Hkv + h / (H / Hkv)) * d, M + (size_t)h * r * d, W + (size_t)(w_per_head ? h : 0) * m * r, xq, xk, fq,
                             fk, red, d, r, m, s);
    for (int l = threadIdx.x; l < m; l += 256) z[(size_t)bh * m + l] += fk[l];
}

}  // namespace

}  // namespace darkattn

using namespace darkattn;

extern "C" darkattn_status_t darkattn_decode_step(darkattn_plan_t plan, const void *q, const void *k, const void *v, const void *M,
                                                  const void *W, float *S, float *z, void *o, void *cuda_stream)
{
    if (!plan || !q || !k || !v || !M || !W || !S || !z || !o) return DARKATTN_ERR_INVALID_ARG;
    const Dims &D = plan->dims;
    if (!D.causal) return DARKATTN_ERR_UNSUPPORTED;          // the recurrent form is the causal one
    if (D.dv % 32) return DARKATTN_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = (size_t)(2 * D.r + 2 * D.m + 256 + 16) * sizeof(float);
    if (smem > 48 * 1024) return DARKATTN_ERR_UNSUPPORTED;
    const dim3 grid(D.dv / 32, D.BH);
    if (D.bf16)
        decode_step_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v,
                                                                  (const __nv_bfloat16 *)M, (const __nv_bfloat16 *)W, S, z, (__nv_bfloat16 *)o,
                                                                  D.H, D.Hkv, D.d, D.r, D.m, D.dv, D.w_per_head, D.s);
    else
        decode_step_kernel<float><<<grid, 256, smem, st>>>((const float *)q, (const float *)k, (const float *)v, (const float *)M,
                                                           (const float *)W, S, z, (float *)o, D.H, D.Hkv, D.d, D.r, D.m, D.dv, D.w_per_head, D.s);
    if (D.bf16)
        decode_z_kernel<__nv_bfloat16><<<D.BH, 256, smem, st>>>((const __nv_bfloat16 *)k, (const __nv_bfloat16 *)M, (const __nv_bfloat16 *)W, z,
                                                              D.H, D.Hkv, D.d, D.r, D.m, D.w_per_head, D.s);
    else
        decode_z_kernel<float><<<D.BH, 256, smem, st>>>((const float *)k, (const float *)M, (const float *)W, z, D.H, D.Hkv, D.d, D.r, D.m,
                                                        D.w_per_head, D.s);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, "decode_step"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}
