// FP32 path of libdarkattn: every step of DARK attention as FP32 FFMA kernels with FP32 accumulation.
//
// This is the path that meets the 1e-4 tolerance (tensor-core operand types round the argument of
// the exponential too coarsely), and the path that accepts any shape. It is built from one strided
// batched GEMM kernel plus small row-wise kernels, and keeps its intermediates in the workspace.
//
// Stabiliser (cancels in O): keys use one shift per (batch, head, feature), c_l = max_j (u_jl - n_j),
// queries use e_il = u_il + c_l - max_l(u_il + c_l); the query's own norm term is a per-row constant
// and is dropped. The product phi(q_i)_l phi(k_j)_l is then the unshifted one times a per-row factor.
#include "common.cuh"

#include <math.h>

namespace darkattn {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

struct GemmP {
    const float *A, *B;
    float *C;
    int M, N, K;
    long long sAm, sAk, sBk, sBn, sCm, sCn;   // element strides
    int nb1;                                  // batch index z = z0 * nb1 + z1
    long long A0, A1, B0, B1, C0, C1;         // batch strides for z0, z1
    float alpha;
    int accumulate;                           // C += instead of C =
    int mask;                                 // 0 none; 1 keep col <= row (others written as 0)
    int tilesM, tilesN;
};

// C[z] (+)= alpha * A[z] * B[z], A is M x K, B is K x N, all with arbitrary element strides.
__global__ void __launch_bounds__(256) gemm_kernel(GemmP p)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tiles = p.tilesM * p.tilesN;
    const long long z = blockIdx.x / tiles;
    const int t = blockIdx.x % tiles;
    const int m0 = (t / p.tilesN) * BM, n0 = (t % p.tilesN) * BN;
    const long long z0 = z / p.nb1, z1 = z % p.nb1;
    const float *A = p.A + z0 * p.A0 + z1 * p.A1;
    const float *B = p.B + z0 * p.B0 + z1 * p.B1;
    float *C = p.C + z0 * p.C0 + z1 * p.C1;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const bool dead = (p.mask == 1 && n0 > m0 + BM - 1);   // tile entirely above the diagonal
    if (!dead) {
        for (int k0 = 0; k0 < p.K; k0 += BK) {
            if (p.sAk == 1) {
                const int row = tid / 4, kk = (tid % 4) * 4;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int k = k0 + kk + i;
                    As[kk + i][row] = (m0 + row < p.M && k < p.K) ? A[(long long)(m0 + row) * p.sAm + k] : 0.f;
                }
            } else {
                const int kk = tid / 16, mm = (tid % 16) * 4;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    As[kk][mm + i] = (m0 + mm + i < p.M && k0 + kk < p.K)
                                         ? A[(long long)(m0 + mm + i) * p.sAm + (long long)(k0 + kk) * p.sAk] : 0.f;
            }
            if (p.sBk == 1) {
                const int col = tid / 4, kk = (tid % 4) * 4;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int k = k0 + kk + i;
                    Bs[kk + i][col] = (n0 + col < p.N && k < p.K) ? B[(long long)(n0 + col) * p.sBn + k] : 0.f;
                }
            } else {
                const int kk = tid / 16, nn = (tid % 16) * 4;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    Bs[kk][nn + i] = (n0 + nn + i < p.N && k0 + kk < p.K)
                                         ? B[(long long)(k0 + kk) * p.sBk + (long long)(n0 + nn + i) * p.sBn] : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < BK; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
                for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
        if (row >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = n0 + tx * 4 + j;
            if (col >= p.N) continue;
            float v = p.alpha * acc[i][j];
            if (p.mask == 1 && col > row) v = 0.f;
            float *dst = C + (long long)row * p.sCm + (long long)col * p.sCn;
            *dst = p.accumulate ? (*dst + v) : v;
        }
    }
}

__global__ void cast_bf16_f32_kernel(const __nv_bfloat16 *in, float *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        out[i] = __bfloat162float(in[i]);
}

__global__ void fill_kernel(float *p, float v, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) p[i] = v;
}

// n[row] = 0.5 * |xt[row,:]|^2, one warp per row.
__global__ void half_sqnorm_kernel(const float *xt, float *n, long long rows, int r)
{
    const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    float acc = 0.f;
    for (int a = lane; a < r; a += 32) { const float v = xt[row * r + a]; acc = fmaf(v, v, acc); }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) n[row] = 0.5f * acc;
}

__device__ __forceinline__ void atomic_max_float(float *addr, float v)
{
    if (v >= 0.f) atomicMax(reinterpret_cast<int *>(addr), __float_as_int(v));
    else atomicMin(reinterpret_cast<unsigned int *>(addr), __float_as_uint(v));
}

// cK[bh,l] = max_j (u[bh,j,l] - n[bh,j]); block = (rows block of 128, bh); thread per column.
__global__ void key_colmax_kernel(const float *u, const float *n, float *cK, int N, int Npad, int m)
{
    const int bh = blockIdx.y;
    const int j0 = blockIdx.x * 128, j1 = min(N, j0 + 128);
    for (int l = threadIdx.x; l < m; l += blockDim.x) {
        float mx = -INFINITY;
        for (int j = j0; j < j1; ++j) mx = fmaxf(mx, u[((long long)bh * Npad + j) * m + l] - n[(long long)bh * N + j]);
        if (j1 > j0) atomic_max_float(&cK[(long long)bh * m + l], mx);
    }
}

// f[bh,j,l] = exp(u - n_j - cK_l) for j < N, 0 for padding rows.
__global__ void key_features_kernel(float *f, const float *n, const float *cK, int N, int Npad, int m, long long total)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int l = (int)(i % m);
        const long long row = i / m;
        const int j = (int)(row % Npad);
        const long long bh = row / Npad;
        f[i] = (j < N) ? expf(f[i] - n[bh * N + j] - cK[bh * m + l]) : 0.f;
    }
}

// f[bh,i,l] = exp(u + cK_l - max_l(u + cK_l)) for i < N, 0 for padding rows; one warp per row.
__global__ void query_features_kernel(float *f, const float *cK, int N, int Npad, int m, long long rows)
{
    const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    const int i = (int)(row % Npad);
    const long long bh = row / Npad;
    float *fr = f + row * m;
    if (i >= N) { for (int l = lane; l < m; l += 32) fr[l] = 0.f; return; }
    const float *c = cK + bh * m;
    float mx = -INFINITY;
    for (int l = lane; l < m; l += 32) mx = fmaxf(mx, fr[l] + c[l]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    for (int l = lane; l < m; l += 32) fr[l] = expf(fr[l] + c[l] - mx);
}

// Va[bh,j,:] = [V_j | 1] for j < N, 0 for padding rows.
__global__ void augment_values_kernel(const float *V, float *Va, int N, int Npad, int dv, long long total)
{
    const int dva = dv + 1;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % dva);
        const long long row = i / dva;
        const int j = (int)(row % Npad);
        const long long bh = row / Npad;
        Va[i] = (j >= N) ? 0.f : (c < dv ? V[(bh * N + j) * dv + c] : 1.f);
    }
}

// In-place exclusive scan over the chunk index of S[bh, c, e] (forward or reverse order).
__global__ void chunk_scan_kernel(float *S, int nc, long long E, long long total, int reverse)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= total) return;
    const long long bh = i / E, e = i % E;
    float *base = S + bh * nc * E + e;
    float run = 0.f;
    for (int k = 0; k < nc; ++k) {
        const int c = reverse ? nc - 1 - k : k;
        const float v = base[(long long)c * E];
        base[(long long)c * E] = run;
        run += v;
    }
}

// out[bh,i,c] = src[bh,i,c] (/ src[bh,i,div_col]) for i < N, c < w, cast to the storage type.
template <typename T>
__global__ void emit_rows_kernel(T *out, const float *src, int N, int w, long long src_batch, int src_row,
                                 int div_col, long long total)
{
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(t % w);
        const long long row = t / w;
        const int i = (int)(row % N);
        const long long bh = row / N;
        const float *s = src + bh * src_batch + (long long)i * src_row;
        float v = s[c];
        if (div_col >= 0) v = v / s[div_col];
        if constexpr (sizeof(T) == 2) out[t] = __float2bfloat16_rn(v);
        else out[t] = v;
    }
}

// Grouped key/value heads. out[(b,hk),i,c] = sum_g src[(b, hk G + g),i,c]: the gradient of a shared key or value row
// collects the parts of the G query heads that read it.
template <typename T>
__global__ void emit_grouped_kernel(T *out, const float *src, int N, int w, long long src_batch, int src_row, int H, int Hkv,
                                    long long total)
{
    const int G = H / Hkv;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(t % w);
        const long long row = t / w;
        const int i = (int)(row % N);
        const long long bhk = row / N, b = bhk / Hkv, hk = bhk % Hkv;
        float v = 0.f;
        for (int g = 0; g < G; ++g) v += src[(b * H + hk * G + g) * src_batch + (long long)i * src_row + c];
        if constexpr (sizeof(T) == 2) out[t] = __float2bfloat16_rn(v);
        else out[t] = v;
    }
}

// out[(b,h),i,c] = in[(b, h / G),i,c] as fp32: every query head gets its own copy of the key/value head it reads.
template <typename T>
__global__ void expand_kv_kernel(const T *in, float *out, long long per_head, int H, int Hkv, long long total)
{
    const int G = H / Hkv;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        const long long bh = t / per_head, e = t % per_head, b = bh / H, h = bh % H;
        const T x = in[(b * Hkv + h / G) * per_head + e];
        if constexpr (sizeof(T) == 2) out[t] = __bfloat162float(x);
        else out[t] = x;
    }
}

// Ga[bh,i,:] = [G_i / den_i | -(G_i . O_i) / den_i], O_i = num_i / den_i; one warp per row.
__global__ void grad_aug_kernel(const float *G, const float *num, float *Ga, int N, int Npad, int dv, long long rows)
{
    const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    const int dva = dv + 1;
    const int i = (int)(row % Npad);
    const long long bh = row / Npad;
    float *g = Ga + row * dva;
    if (i >= N) { for (int c = lane; c < dva; c += 32) g[c] = 0.f; return; }
    const float *nr = num + row * dva;
    const float *Gr = G + (bh * N + i) * dv;
    const float inv = 1.f / nr[dv];
    float delta = 0.f;
    for (int c = lane; c < dv; c += 32) { const float gv = Gr[c]; g[c] = gv * inv; delta = fmaf(gv, nr[c] * inv, delta); }
    for (int o = 16; o; o >>= 1) delta += __shfl_xor_sync(0xffffffffu, delta, o);
    if (lane == 0) g[dv] = -delta * inv;
}

// E = dphi .* phi in place (into dphi); es[bh,i] = sum_l E_il for i < N; one warp per row.
__global__ void feature_grad_kernel(float *dphi, const float *phi, float *es, int N, int Npad, int m, long long rows)
{
    const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / 32;
    const int lane = threadIdx.x % 32;
    if (row >= rows) return;
    const int i = (int)(row % Npad);
    const long long bh = row / Npad;
    float acc = 0.f;
    for (int l = lane; l < m; l += 32) { const float e = dphi[row * m + l] * phi[row * m + l]; dphi[row * m + l] = e; acc += e; }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0 && i < N) es[bh * N + i] = acc;
}

// dxt[row,a] -= es[row] * xt[row,a]
__global__ void norm_term_kernel(float *dxt, const float *xt, const float *es, int r, long long total)
{
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x)
        dxt[t] = fmaf(-es[t / r], xt[t], dxt[t]);
}

// dM[h,:] = sum_b dMp[b,h,:]
__global__ void reduce_batch_kernel(const float *dMp, float *dM, int B, long long per_b, long long total)
{
    const long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (t >= total) return;
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc += dMp[b * per_b + t];
    dM[t] = acc;
}

struct Launcher {
    cudaStream_t st;
    int count = 0;
    cudaError_t err = cudaSuccess;
    void check() { cudaError_t e = cudaGetLastError(); if (e != cudaSuccess && err == cudaSuccess) err = e; ++count; }
    static int blocks(long long n, int per) { long long b = (n + per - 1) / per; return (int)(b < 1 ? 1 : (b > 148LL * 64 ? 148LL * 64 : b)); }

    void gemm(const float *A, const float *B, float *C, int M, int N, int K, long long sAm, long long sAk,
              long long sBk, long long sBn, long long sCm, long long sCn, long long nbatch, int nb1,
              long long A0, long long A1, long long B0, long long B1, long long C0, long long C1, float alpha,
              int accumulate, int mask)
    {
        GemmP p{A, B, C, M, N, K, sAm, sAk, sBk, sBn, sCm, sCn, nb1, A0, A1, B0, B1, C0, C1, alpha, accumulate, mask,
                (M + BM - 1) / BM, (N + BN - 1) / BN};
        const long long grid = nbatch * p.tilesM * p.tilesN;
        gemm_kernel<<<(unsigned)grid, 256, 0, st>>>(p);
        check();
    }
    void cast(const void *in, float *out, long long n)
    {
        cast_bf16_f32_kernel<<<blocks(n, 1024), 256, 0, st>>>((const __nv_bfloat16 *)in, out, n);
        check();
    }
    void fill(float *p, float v, long long n) { fill_kernel<<<blocks(n, 1024), 256, 0, st>>>(p, v, n); check(); }
    void expand_kv(const void *in, int bf16, float *out, long long per_head, int B, int H, int Hkv)
    {
        const long long total = (long long)B * H * per_head;
        if (bf16) expand_kv_kernel<__nv_bfloat16><<<blocks(total, 1024), 256, 0, st>>>((const __nv_bfloat16 *)in, out, per_head, H, Hkv, total);
        else expand_kv_kernel<float><<<blocks(total, 1024), 256, 0, st>>>((const float *)in, out, per_head, H, Hkv, total);
        check();
    }
    void emit_grouped(void *out, int bf16, const float *src, int B, int H, int Hkv, int N, int w, long long src_batch, int src_row)
    {
        const long long total = (long long)B * Hkv * N * w;
        if (bf16) emit_grouped_kernel<__nv_bfloat16><<<blocks(total, 1024), 256, 0, st>>>((__nv_bfloat16 *)out, src, N, w, src_batch, src_row, H, Hkv, total);
        else emit_grouped_kernel<float><<<blocks(total, 1024), 256, 0, st>>>((float *)out, src, N, w, src_batch, src_row, H, Hkv, total);
        check();
    }
    void emit(void *out, int bf16, const float *src, long long BH, int N, int w, long long src_batch, int src_row, int div_col)
    {
        const long long total = BH * N * w;
        if (bf16) emit_rows_kernel<__nv_bfloat16><<<blocks(total, 1024), 256, 0, st>>>((__nv_bfloat16 *)out, src, N, w, src_batch, src_row, div_col, total);
        else emit_rows_kernel<float><<<blocks(total, 1024), 256, 0, st>>>((float *)out, src, N, w, src_batch, src_row, div_col, total);
        check();
    }
};

inline int warp_rows_grid(long long rows) { return (int)((rows * 32 + 255) / 256); }

struct Bufs {
    const float *Q, *K, *V, *M, *W;
    float *xtQ, *xtK, *nQ, *nK, *fQ, *fK, *cK, *Va, *Sloc, *P, *num;
};

// Steps shared by forward and backward: features, states, numerators (all left in the workspace).
void run_forward_stages(const darkattn_plan_s *plan, Launcher &L, const void *Q, const void *K, const void *V,
                        const void *M, const void *W, char *ws, Bufs &b)
{
    const Dims &D = plan->dims;
    const SimtLayout &Y = plan->simt;
    const long long BH = D.BH, N = D.N, Np = D.Npad, d = D.d, r = D.r, m = D.m, dv = D.dv, dva = D.dva, C = D.C, nc = D.nc;
    auto F = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    if (D.bf16) {
        L.cast(Q, F(Y.Qf), BH * N * d);
        L.cast(M, F(Y.Mf), (long long)D.H * r * d); L.cast(W, F(Y.Wf), (long long)(D.w_per_head ? D.H : 1) * m * r);
        b.Q = F(Y.Qf); b.M = F(Y.Mf); b.W = F(Y.Wf);
    } else {
        b.Q = (const float *)Q; b.M = (const float *)M; b.W = (const float *)W;
    }
    if (D.G > 1) {          // grouped key/value heads: every query head works on its own fp32 copy of the head it reads
        L.expand_kv(K, D.bf16, F(Y.Kf), N * d, D.B, D.H, D.Hkv); L.expand_kv(V, D.bf16, F(Y.Vf), N * dv, D.B, D.H, D.Hkv);
        b.K = F(Y.Kf); b.V = F(Y.Vf);
    } else if (D.bf16) {
        L.cast(K, F(Y.Kf), BH * N * d); L.cast(V, F(Y.Vf), BH * N * dv);
        b.K = F(Y.Kf); b.V = F(Y.Vf);
    } else {
        b.K = (const float *)K; b.V = (const float *)V;
    }
    b.xtQ = F(Y.xtQ); b.xtK = F(Y.xtK); b.nQ = F(Y.nQ); b.nK = F(Y.nK); b.fQ = F(Y.fQ); b.fK = F(Y.fK);
    b.cK = F(Y.cK); b.Va = F(Y.Va); b.Sloc = F(Y.Sloc); b.P = F(Y.P); b.num = F(Y.num);
    const long long wb1 = D.w_per_head ? m * r : 0;

    for (int side = 0; side < 2; ++side) {
        const float *X = side ? b.K : b.Q;
        float *xt = side ? b.xtK : b.xtQ, *f = side ? b.fK : b.fQ;
        // x~ = s X M^T
        L.gemm(X, b.M, xt, (int)N, (int)r, (int)d, d, 1, 1, d, r, 1, BH, D.H, D.H * N * d, N * d, 0, r * d, D.H * N * r, N * r, D.s, 0, 0);
        // u = x~ W^T
        L.gemm(xt, b.W, f, (int)N, (int)m, (int)r, r, 1, 1, r, m, 1, BH, D.H, D.H * N * r, N * r, 0, wb1, D.H * Np * m, Np * m, 1.f, 0, 0);
    }
    half_sqnorm_kernel<<<warp_rows_grid(BH * N), 256, 0, L.st>>>(b.xtK, b.nK, BH * N, (int)r); L.check();
    L.fill(b.cK, -INFINITY, BH * m);
    key_colmax_kernel<<<dim3((unsigned)((N + 127) / 128), (unsigned)BH), 256, 0, L.st>>>(b.fK, b.nK, b.cK, (int)N, (int)Np, (int)m); L.check();
    key_features_kernel<<<Launcher::blocks(BH * Np * m, 1024), 256, 0, L.st>>>(b.fK, b.nK, b.cK, (int)N, (int)Np, (int)m, BH * Np * m); L.check();
    query_features_kernel<<<warp_rows_grid(BH * Np), 256, 0, L.st>>>(b.fQ, b.cK, (int)N, (int)Np, (int)m, BH * Np); L.check();
    augment_values_kernel<<<Launcher::blocks(BH * Np * dva, 1024), 256, 0, L.st>>>(b.V, b.Va, (int)N, (int)Np, (int)dv, BH * Np * dva); L.check();

    if (!D.causal) {
        // S = phi(K)^T [V|1]; num = phi(Q) S
        L.gemm(b.fK, b.Va, b.Sloc, (int)m, (int)dva, (int)Np, 1, m, dva, 1, dva, 1, BH, 1, Np * m, 0, Np * dva, 0, m * dva, 0, 1.f, 0, 0);
        L.gemm(b.fQ, b.Sloc, b.num, (int)Np, (int)dva, (int)m, m, 1, dva, 1, dva, 1, BH, 1, Np * m, 0, m * dva, 0, Np * dva, 0, 1.f, 0, 0);
    } else {
        const long long Z = BH * nc;
        // chunk-local states, then exclusive prefix over chunks
        L.gemm(b.fK, b.Va, b.Sloc, (int)m, (int)dva, (int)C, 1, m, dva, 1, dva, 1, Z, (int)nc, Np * m, C * m, Np * dva, C * dva, nc * m * dva, m * dva, 1.f, 0, 0);
        chunk_scan_kernel<<<(unsigned)((BH * m * dva + 255) / 256), 256, 0, L.st>>>(b.Sloc, (int)nc, m * dva, BH * m * dva, 0); L.check();
        // P = tril(phi(Q_c) phi(K_c)^T); num = P [V|1] + phi(Q_c) S_prev
        L.gemm(b.fQ, b.fK, b.P, (int)C, (int)C, (int)m, m, 1, 1, m, C, 1, Z, (int)nc, Np * m, C * m, Np * m, C * m, nc * C * C, C * C, 1.f, 0, 1);
        L.gemm(b.P, b.Va, b.num, (int)C, (int)dva, (int)C, C, 1, dva, 1, dva, 1, Z, (int)nc, nc * C * C, C * C, Np * dva, C * dva, Np * dva, C * dva, 1.f, 0, 0);
        L.gemm(b.fQ, b.Sloc, b.num, (int)C, (int)dva, (int)m, m, 1, dva, 1, dva, 1, Z, (int)nc, Np * m, C * m, nc * m * dva, m * dva, Np * dva, C * dva, 1.f, 1, 0);
    }
}

size_t take(size_t &off, long long floats)
{
    const size_t at = off;
    off += (((size_t)floats * sizeof(float)) + 255) / 256 * 256;
    return at;
}

}  // namespace

void simt_make_layout(darkattn_plan_s *plan)
{
    const Dims &D = plan->dims;
    SimtLayout &Y = plan->simt;
    const long long BH = D.BH, N = D.N, Np = D.Npad, d = D.d, r = D.r, m = D.m, dv = D.dv, dva = D.dva, C = D.C, nc = D.nc;
    size_t off = 0;
    Y.status = take(off, 64);
    Y.Qf = Y.Kf = Y.Vf = Y.Mf = Y.Wf = 0;
    if (D.bf16) {
        Y.Qf = take(off, BH * N * d);
        Y.Mf = take(off, (long long)D.H * r * d); Y.Wf = take(off, (long long)(D.w_per_head ? D.H : 1) * m * r);
    }
    if (D.bf16 || D.G > 1) { Y.Kf = take(off, BH * N * d); Y.Vf = take(off, BH * N * dv); }
    Y.xtQ = take(off, BH * N * r); Y.xtK = take(off, BH * N * r);
    Y.nQ = take(off, BH * N); Y.nK = take(off, BH * N);
    Y.fQ = take(off, BH * Np * m); Y.fK = take(off, BH * Np * m);
    Y.cK = take(off, BH * m);
    Y.Va = take(off, BH * Np * dva);
    Y.Sloc = take(off, BH * nc * m * dva);
    Y.P = D.causal ? take(off, BH * nc * C * C) : 0;
    Y.num = take(off, BH * Np * dva);
    Y.fwd_bytes = off;
    Y.Gf = D.bf16 ? take(off, BH * N * dv) : 0;
    Y.Ga = take(off, BH * Np * dva);
    Y.dP = D.causal ? take(off, BH * nc * C * C) : 0;
    Y.Rloc = take(off, BH * nc * m * dva);
    Y.dA = take(off, BH * Np * m); Y.dBf = take(off, BH * Np * m);
    Y.dVa = take(off, BH * Np * dva);
    Y.esQ = take(off, BH * N); Y.esK = take(off, BH * N);
    Y.dxtQ = take(off, BH * N * r); Y.dxtK = take(off, BH * N * r);
    Y.dXf = take(off, BH * N * d);
    Y.dMp = take(off, BH * r * d);
    Y.dWp = take(off, BH * m * r);
    Y.total_bytes = off;
}

darkattn_status_t simt_forward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                               const void *M, const void *W, void *O, char *ws, cudaStream_t st, bool)
{
    const Dims &D = plan->dims;
    Launcher L{st};
    Bufs b;
    run_forward_stages(plan, L, Q, K, V, M, W, ws, b);
    L.emit(O, D.bf16, b.num, D.BH, D.N, D.dv, (long long)D.Npad * D.dva, D.dva, D.dv);
    if (L.err != cudaSuccess) { set_cuda_error(L.err, "simt_forward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

darkattn_status_t simt_backward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                const void *M, const void *W, const void *dO, void *dQ, void *dK, void *dV,
                                float *dM, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const SimtLayout &Y = plan->simt;
    const long long BH = D.BH, N = D.N, Np = D.Npad, d = D.d, r = D.r, m = D.m, dv = D.dv, dva = D.dva, C = D.C, nc = D.nc;
    auto F = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    Launcher L{st};
    Bufs b;
    run_forward_stages(plan, L, Q, K, V, M, W, ws, b);

    const float *G;
    if (D.bf16) { L.cast(dO, F(Y.Gf), BH * N * dv); G = F(Y.Gf); } else G = (const float *)dO;
    float *Ga = F(Y.Ga), *dP = F(Y.dP), *Rl = F(Y.Rloc), *dA = F(Y.dA), *dBf = F(Y.dBf), *dVa = F(Y.dVa);
    grad_aug_kernel<<<warp_rows_grid(BH * Np), 256, 0, st>>>(G, b.num, Ga, (int)N, (int)Np, (int)dv, BH * Np); L.check();

    if (!D.causal) {
        // dA = Ga S^T ; R = phi(Q)^T Ga ; dBf = [V|1] R^T ; d[V|1] = phi(K) R
        L.gemm(Ga, b.Sloc, dA, (int)Np, (int)m, (int)dva, dva, 1, 1, dva, m, 1, BH, 1, Np * dva, 0, m * dva, 0, Np * m, 0, 1.f, 0, 0);
        L.gemm(b.fQ, Ga, Rl, (int)m, (int)dva, (int)Np, 1, m, dva, 1, dva, 1, BH, 1, Np * m, 0, Np * dva, 0, m * dva, 0, 1.f, 0, 0);
        L.gemm(b.Va, Rl, dBf, (int)Np, (int)m, (int)dva, dva, 1, 1, dva, m, 1, BH, 1, Np * dva, 0, m * dva, 0, Np * m, 0, 1.f, 0, 0);
        L.gemm(b.fK, Rl, dVa, (int)Np, (int)dva, (int)m, m, 1, dva, 1, dva, 1, BH, 1, Np * m, 0, m * dva, 0, Np * dva, 0, 1.f, 0, 0);
    } else {
        const long long Z = BH * nc;
        const long long sP0 = nc * C * C, sP1 = C * C, sF0 = Np * m, sF1 = C * m, sV0 = Np * dva, sV1 = C * dva, sS0 = nc * m * dva, sS1 = m * dva;
        // dP = tril(Ga_c [V|1]_c^T)
        L.gemm(Ga, b.Va, dP, (int)C, (int)C, (int)dva, dva, 1, 1, dva, C, 1, Z, (int)nc, sV0, sV1, sV0, sV1, sP0, sP1, 1.f, 0, 1);
        // dA_c = dP_c phi(K_c) + Ga_c S_prev^T
        L.gemm(dP, b.fK, dA, (int)C, (int)m, (int)C, C, 1, m, 1, m, 1, Z, (int)nc, sP0, sP1, sF0, sF1, sF0, sF1, 1.f, 0, 0);
        L.gemm(Ga, b.Sloc, dA, (int)C, (int)m, (int)dva, dva, 1, 1, dva, m, 1, Z, (int)nc, sV0, sV1, sS0, sS1, sF0, sF1, 1.f, 1, 0);
        // reverse states R_c = phi(Q_c)^T Ga_c, exclusive suffix over chunks
        L.gemm(b.fQ, Ga, Rl, (int)m, (int)dva, (int)C, 1, m, dva, 1, dva, 1, Z, (int)nc, sF0, sF1, sV0, sV1, sS0, sS1, 1.f, 0, 0);
        chunk_scan_kernel<<<(unsigned)((BH * m * dva + 255) / 256), 256, 0, st>>>(Rl, (int)nc, m * dva, BH * m * dva, 1); L.check();
        // dBf_c = dP_c^T phi(Q_c) + [V|1]_c R_next^T
        L.gemm(dP, b.fQ, dBf, (int)C, (int)m, (int)C, 1, C, m, 1, m, 1, Z, (int)nc, sP0, sP1, sF0, sF1, sF0, sF1, 1.f, 0, 0);
        L.gemm(b.Va, Rl, dBf, (int)C, (int)m, (int)dva, dva, 1, 1, dva, m, 1, Z, (int)nc, sV0, sV1, sS0, sS1, sF0, sF1, 1.f, 1, 0);
        // d[V|1]_c = P_c^T Ga_c + phi(K_c) R_next
        L.gemm(b.P, Ga, dVa, (int)C, (int)dva, (int)C, 1, C, dva, 1, dva, 1, Z, (int)nc, sP0, sP1, sV0, sV1, sV0, sV1, 1.f, 0, 0);
        L.gemm(b.fK, Rl, dVa, (int)C, (int)dva, (int)m, m, 1, dva, 1, dva, 1, Z, (int)nc, sF0, sF1, sS0, sS1, sV0, sV1, 1.f, 1, 0);
    }
    if (D.G > 1) L.emit_grouped(dV, D.bf16, dVa, D.B, D.H, D.Hkv, (int)N, (int)dv, Np * dva, (int)dva);
    else L.emit(dV, D.bf16, dVa, BH, (int)N, (int)dv, Np * dva, (int)dva, -1);

    const long long wb1 = D.w_per_head ? m * r : 0;
    for (int side = 0; side < 2; ++side) {
        float *dphi = side ? dBf : dA;
        const float *phi = side ? b.fK : b.fQ, *xt = side ? b.xtK : b.xtQ, *X = side ? b.K : b.Q;
        float *es = F(side ? Y.esK : Y.esQ), *dxt = F(side ? Y.dxtK : Y.dxtQ), *dXf = F(Y.dXf);
        feature_grad_kernel<<<warp_rows_grid(BH * Np), 256, 0, st>>>(dphi, phi, es, (int)N, (int)Np, (int)m, BH * Np); L.check();
        // dx~ = E W - rowsum(E) x~
        L.gemm(dphi, b.W, dxt, (int)N, (int)r, (int)m, m, 1, r, 1, r, 1, BH, D.H, D.H * Np * m, Np * m, 0, wb1, D.H * N * r, N * r, 1.f, 0, 0);
        norm_term_kernel<<<Launcher::blocks(BH * N * r, 1024), 256, 0, st>>>(dxt, xt, es, (int)r, BH * N * r); L.check();
        // dX = s dx~ M
        L.gemm(dxt, b.M, dXf, (int)N, (int)d, (int)r, r, 1, d, 1, d, 1, BH, D.H, D.H * N * r, N * r, 0, r * d, D.H * N * d, N * d, D.s, 0, 0);
        if (side && D.G > 1) L.emit_grouped(dK, D.bf16, dXf, D.B, D.H, D.Hkv, (int)N, (int)d, N * d, (int)d);
        else L.emit(side ? dK : dQ, D.bf16, dXf, BH, (int)N, (int)d, N * d, (int)d, -1);
        // dM_(b,h) (+)= s dx~^T X
        L.gemm(dxt, X, F(Y.dMp), (int)r, (int)d, (int)N, 1, r, d, 1, d, 1, BH, 1, N * r, 0, N * d, 0, r * d, 0, D.s, side, 0);
    }
    reduce_batch_kernel<<<(unsigned)(((long long)D.H * r * d + 255) / 256), 256, 0, st>>>(F(Y.dMp), dM, D.B, (long long)D.H * r * d, (long long)D.H * r * d); L.check();
    if (L.err != cudaSuccess) { set_cuda_error(L.err, "simt_backward"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

// dW_l = sum_i E_il x~_i over queries and keys: E (in the buffers dA, dBf) and x~ are still in the workspace after
// simt_backward. Per (b,h) products, then the sum over the batch (and over the heads when W is shared).
__global__ void reduce_dw_kernel(const float *dWp, float *dW, int B, int H, long long per_head, int w_per_head, long long total)
{
    const long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (t >= total) return;
    float acc = 0.f;
    if (w_per_head) {
        const long long h = t / per_head, e = t % per_head;
        for (int b = 0; b < B; ++b) acc += dWp[((long long)b * H + h) * per_head + e];
    } else {
        for (int bh = 0; bh < B * H; ++bh) acc += dWp[(long long)bh * per_head + t];
    }
    dW[t] = acc;
}

darkattn_status_t simt_backward_dw(const darkattn_plan_s *plan, float *dW, char *ws, cudaStream_t st)
{
    const Dims &D = plan->dims;
    const SimtLayout &Y = plan->simt;
    const long long BH = D.BH, N = D.N, Np = D.Npad, r = D.r, m = D.m;
    auto F = [&](size_t off) { return reinterpret_cast<float *>(ws + off); };
    Launcher L{st};
    for (int side = 0; side < 2; ++side) {
        const float *E = F(side ? Y.dBf : Y.dA), *xt = F(side ? Y.xtK : Y.xtQ);
        // dWp_(b,h) (+)= E^T x~   [m x r], contraction over the N tokens (padding rows of E are zero, but x~ has only N rows)
        L.gemm(E, xt, F(Y.dWp), (int)m, (int)r, (int)N, 1, m, r, 1, r, 1, BH, 1, Np * m, 0, N * r, 0, m * r, 0, 1.f, side, 0);
    }
    const long long per_head = m * r, total = (D.w_per_head ? D.H : 1) * per_head;
    reduce_dw_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(F(Y.dWp), dW, D.B, D.H, per_head, D.w_per_head, total);
    L.check();
    if (L.err != cudaSuccess) { set_cuda_error(L.err, "simt_backward_dw"); return DARKATTN_ERR_CUDA; }
    return DARKATTN_OK;
}

}  // namespace darkattn
