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

// Dot products of one row of a matrix with up to two vectors held in shared memory, and the row's squared norm. Eight lanes
// share a row: lane `sub` of the eight takes every eighth 16-byte piece of it, so a warp's load covers four rows in pieces
// of 128 contiguous bytes (every sector it fetches is used), and three shuffle steps add the eight parts up (all eight
// lanes end with the sums). Rows whose length is not a multiple of 16 bytes are read element by element, eight apart.
// Every lane of the warp must call this (the shuffles name the full warp).
template <typename T, bool TWO>
__device__ __forceinline__ void row_dots(const T *row, const float *x0, const float *x1, int n, int sub, bool vec, float &d0, float &d1,
                                         float &nn)
{
    d0 = d1 = nn = 0.f;
    constexpr int V = 16 / (int)sizeof(T);          // elements per 16-byte load
    if (vec) {
#pragma unroll 4
        for (int c = sub * V; c < n; c += 8 * V) {
            float w[V];
            if constexpr (sizeof(T) == 2) {         // eight bf16: the upper half of an fp32 each
                const uint4 raw = *reinterpret_cast<const uint4 *>(row + c);
                const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) { w[2 * j] = __uint_as_float(u[j] << 16); w[2 * j + 1] = __uint_as_float(u[j] & 0xffff0000u); }
            }
            else { const float4 f = *reinterpret_cast<const float4 *>(row + c); w[0] = f.x; w[1] = f.y; w[2] = f.z; w[3] = f.w; }
#pragma unroll
            for (int j = 0; j < V; ++j) {
                d0 = fmaf(w[j], x0[c + j], d0);
                if constexpr (TWO) d1 = fmaf(w[j], x1[c + j], d1);
                nn = fmaf(w[j], w[j], nn);
            }
        }
    } else {
        for (int c = sub; c < n; c += 8) {
            const float w = ldf(row, c);
            d0 = fmaf(w, x0[c], d0);
            if constexpr (TWO) d1 = fmaf(w, x1[c], d1);
            nn = fmaf(w, w, nn);
        }
    }
#pragma unroll
    for (int off = 1; off < 8; off <<= 1) {
        d0 += __shfl_xor_sync(0xffffffffu, d0, off);
        if constexpr (TWO) d1 += __shfl_xor_sync(0xffffffffu, d1, off);
        nn += __shfl_xor_sync(0xffffffffu, nn, off);
    }
}

// Features of one (batch, head)'s new token, by the whole block (a multiple of 32 threads, at most 1024): fk[l] = phi(k)_l and, when WITH_Q, fq[l] = phi(q)_l
// (shared memory: vq[d], vk[d], xq[r], xk[r], fq[m], fk[m], red[...]).
template <typename T, bool WITH_Q>
__device__ __forceinline__ void token_features(const T *qv, const T *kv, const T *Mh, const T *Wh, float *vq, float *vk, float *xq,
                                               float *xk, float *fq, float *fk, float *red, int d, int r, int m, float s)
{
    const int tid = threadIdx.x, lane = tid & 31;
    const int nt = blockDim.x, sub = tid & 7, grp = tid >> 3, ngrp = nt >> 3;
    constexpr int V = 16 / (int)sizeof(T);
    for (int c = tid; c < d; c += nt) {
        vk[c] = ldf(kv, c);
        if constexpr (WITH_Q) vq[c] = ldf(qv, c);
    }
    __syncthreads();
    // x~ = s M x for the query and the key: eight lanes per row of M (whole warps walk the loop: rows past the end are read
    // from the last row and not stored)
    const bool vec_m = (d % V == 0) && (reinterpret_cast<uintptr_t>(Mh) & 15) == 0;
    for (int a0 = 0; a0 < r; a0 += ngrp) {
        const int a = a0 + grp, ac = a < r ? a : r - 1;
        float aq, ak, nn;
        row_dots<T, WITH_Q>(Mh + (size_t)ac * d, WITH_Q ? vq : vk, vk, d, sub, vec_m, aq, ak, nn);
        if (a < r && sub == 0) {
            if constexpr (WITH_Q) { xq[a] = s * aq; xk[a] = s * ak; }
            else xk[a] = s * aq;
        }
    }
    __syncthreads();
    float nk = 0.f;
    for (int a = lane; a < r; a += 32) nk = fmaf(xk[a], xk[a], nk);
    for (int off = 16; off; off >>= 1) nk += __shfl_xor_sync(0xffffffffu, nk, off);
    nk *= 0.5f;
    float mx = -INFINITY;
    const bool vec_w = (r % V == 0) && (reinterpret_cast<uintptr_t>(Wh) & 15) == 0;
    for (int l0 = 0; l0 < m; l0 += ngrp) {          // exponents of the features: eight lanes per row of W
        const int l = l0 + grp, lc = l < m ? l : m - 1;
        float uq, uk, c;
        row_dots<T, WITH_Q>(Wh + (size_t)lc * r, WITH_Q ? xq : xk, xk, r, sub, vec_w, uq, uk, c);
        if constexpr (!WITH_Q) uk = uq;
        c *= 0.5f;
        if (l < m) {
            if (sub == 0) {
                fk[l] = __expf(uk - nk - c);
                if constexpr (WITH_Q) fq[l] = uq + c;
            }
            if constexpr (WITH_Q) mx = fmaxf(mx, uq + c);
        }
    }
    if constexpr (WITH_Q) {
        for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        if (lane == 0) red[tid >> 5] = mx;
        __syncthreads();
        mx = red[0];
        for (int w = 1; w < nt / 32; ++w) mx = fmaxf(mx, red[w]);
        __syncthreads();
        for (int l = tid; l < m; l += nt) fq[l] = __expf(fq[l] - mx);
    }
    __syncthreads();
}

// One block of NT threads per (batch, head): thread = (four columns of the state, group of rows). The block owns
// the head's z, so it reads z for the normaliser and stores z + phi(k) itself. NT = 512 when the blocks are few (each is
// a chain of load latencies: more threads shorten it); NT = 256 when there are several per SM, so that two share an SM
// and one's feature phase, which moves no state, runs under the other's state traffic.
template <typename T, int NT>
__global__ void __launch_bounds__(NT, 512 / NT) decode_step_kernel(const T *q, const T *k, const T *v, const T *M, const T *W, float *S,
                                                           float *z, T *o, int H, int Hkv, int d, int r, int m, int dv, int w_per_head,
                                                           float s)
{
    extern __shared__ float sm[];
    float *vq = sm, *vk = vq + d, *xq = vk + d, *xk = xq + r, *fq = xk + r, *fk = fq + m, *red = fk + m;   // red: up to 2048 partial numerators + 16 partial normalisers
    const int bh = blockIdx.x, h = bh % H, tid = threadIdx.x, lane = tid & 31;
    const int kvh = (bh / H) * Hkv + h / (H / Hkv);     // the key/value head this query head reads (grouped key/value heads)
    token_features<T, true>(q + (size_t)bh * d, k + (size_t)kvh * d, M + (size_t)h * r * d, W + (size_t)(w_per_head ? h : 0) * m * r,
                            vq, vk, xq, xk, fq, fk, red, d, r, m, s);

    // normaliser phi(q) . (z + phi(k)) and the new z: one feature per thread
    float *zb = z + (size_t)bh * m;
    float den = 0.f;
    for (int l = tid; l < m; l += NT) {
        const float zn = zb[l] + fk[l];
        zb[l] = zn;
        den = fmaf(fq[l], zn, den);
    }
    for (int off = 16; off; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);

    // state update and read-out: a thread owns four neighbouring columns of every (NT / (dv / 4))-th row and keeps 16 of
    // its rows (256 bytes) in flight
    const int tpr = dv / 4, nrg = NT / tpr, c4 = (tid % tpr) * 4, rg = tid / tpr;
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rg < nrg) {
        const float4 vv = make_float4(ldf(v, (size_t)kvh * dv + c4), ldf(v, (size_t)kvh * dv + c4 + 1), ldf(v, (size_t)kvh * dv + c4 + 2),
                                      ldf(v, (size_t)kvh * dv + c4 + 3));
        float4 *Sb = reinterpret_cast<float4 *>(S + (size_t)bh * m * dv + c4);
        for (int l0 = rg; l0 < m; l0 += 16 * nrg) {
            float4 sv[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) { const int l = l0 + nrg * j; sv[j] = (l < m) ? Sb[(size_t)l * tpr] : make_float4(0.f, 0.f, 0.f, 0.f); }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int l = l0 + nrg * j;
                if (l < m) {
                    const float f = fk[l], g = fq[l];
                    const float4 sn = make_float4(fmaf(f, vv.x, sv[j].x), fmaf(f, vv.y, sv[j].y), fmaf(f, vv.z, sv[j].z), fmaf(f, vv.w, sv[j].w));
                    Sb[(size_t)l * tpr] = sn;
                    num.x = fmaf(g, sn.x, num.x); num.y = fmaf(g, sn.y, num.y); num.z = fmaf(g, sn.z, num.z); num.w = fmaf(g, sn.w, num.w);
                }
            }
        }
        float *rd = red + rg * dv + c4;
        rd[0] = num.x; rd[1] = num.y; rd[2] = num.z; rd[3] = num.w;
    }
    if (lane == 0) red[2048 + (tid >> 5)] = den;
    __syncthreads();
    if (tid < dv) {
        float n = 0.f, dn = 0.f;
        for (int g = 0; g < nrg; ++g) n += red[g * dv + tid];
        for (int w = 0; w < NT / 32; ++w) dn += red[2048 + w];
        const float out = n / dn;
        if constexpr (sizeof(T) == 2) o[(size_t)bh * dv + tid] = __float2bfloat16_rn(out);
        else o[(size_t)bh * dv + tid] = out;
    }
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
    if (D.dv > 512) return DARKATTN_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(2 * D.d + 2 * D.r + 2 * D.m + 2048 + 16) * sizeof(float);
    if (smem > 48 * 1024) return DARKATTN_ERR_UNSUPPORTED;
    const bool many = D.BH >= 2 * 148 && D.dv <= 256;      // several blocks per SM: two smaller blocks share one
#define DARKATTN_DECODE_LAUNCH(T, NT)                                                                                              \
    decode_step_kernel<T, NT><<<(unsigned)D.BH, NT, smem, st>>>((const T *)q, (const T *)k, (const T *)v, (const T *)M, (const T *)W, S, z, \
                                                                (T *)o, D.H, D.Hkv, D.d, D.r, D.m, D.dv, D.w_per_head, D.s)
    if (D.bf16) { if (many) DARKATTN_DECODE_LAUNCH(__nv_bfloat16, 256); else DARKATTN_DECODE_LAUNCH(__nv_bfloat16, 512); }
    else { if (many) DARKATTN_DECODE_LAUNCH(float, 256); else DARKATTN_DECODE_LAUNCH(float, 512); }
#undef DARKATTN_DECODE_LAUNCH
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e, "decode_step"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}
