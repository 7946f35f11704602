// Internal declarations shared by the translation units of libdarkattn.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "darkattn.h"

namespace darkattn {

// Resolved problem description (defaults filled in).
struct Dims {
    int B, H, N, d, r, m, dv;
    int BH;          // B * H
    int Hkv, G;      // key/value heads and query heads per key/value head (H = Hkv * G)
    int C;           // causal chunk length
    int nc;          // number of chunks = ceil(N / C)   (1 when not causal)
    int Npad;        // nc * C when causal, else N
    int dva;         // dv + 1: values with a ones column appended (its sums are the normaliser)
    int causal;
    int bf16;        // storage type of the tensors is bf16
    int w_per_head;
    float s;         // sqrt(scale), applied to Mq and to Mk
};

// Offsets (bytes) into the caller's workspace of the SIMT path's intermediates.
struct SimtLayout {
    size_t status;                 // device status word (first 256 bytes)
    size_t Qf, Kf, Vf, Mf, Wf, Gf; // fp32 copies of bf16 inputs (unused for f32 storage)
    size_t xtQ, xtK;               // x~            [BH, N, r]
    size_t nQ, nK;                 // |x~|^2 / 2    [BH, N]
    size_t fQ, fK;                 // exponents, then features  [BH, Npad, m]
    size_t cK;                     // per-feature key shift     [BH, m]
    size_t Va;                     // [V | 1]       [BH, Npad, dva]
    size_t Sloc;                   // chunk states, then exclusive prefixes [BH, nc, m, dva]
    size_t P;                      // masked intra-chunk kernel  [BH, nc, C, C]   (causal)
    size_t num;                    // numerators and normaliser  [BH, Npad, dva]
    // backward only
    size_t Ga;                     // [dO/den | -delta/den]      [BH, Npad, dva]
    size_t dP;                     // [BH, nc, C, C]             (causal)
    size_t Rloc;                   // reverse states             [BH, nc, m, dva]
    size_t dA, dBf;                // feature gradients, then E  [BH, Npad, m]
    size_t dVa;                    // [BH, Npad, dva]
    size_t esQ, esK;               // rowsum(E)                  [BH, N]
    size_t dxtQ, dxtK;             // dx~                        [BH, N, r]
    size_t dXf;                    // fp32 dX before the cast    [BH, N, d]
    size_t dMp;                    // per-(b,h) dM               [BH, r, d]
    size_t dWp;                    // per-(b,h) dW               [BH, m, r]
    size_t fwd_bytes, total_bytes;
};

// Offsets (bytes) into the workspace of the tensor-core forward path.
struct TensorLayout {
    size_t status;
    size_t Om;      // folded projections log2(e) s W M, bf16 [H, m, d]
    size_t Oml;     // what the rounding of Om to bf16 left out, bf16 [H, m, d]: the projections are taken against Om + Oml
    size_t cs;      // key-side shift per (bh, slab), fp32
    size_t nK;      // key norms, fp32 [BH, N]
    size_t pnum;    // partial numerators, bf16 [nslab, BH, N, dv]
    size_t pdr;     // per slab and row: the partial normalisers of the four 32-column groups and the exponent the partial is
                    // scaled by, fp32 [nslab, BH, N, 8] (entries 0..3 and 4; 5..7 unused)
    size_t Sacc;    // non-causal state sums, fp32 [BH, m, dv]
    size_t zacc;    // fp32 [BH, m]
    size_t Sb;      // bf16 copy of the state, [BH, m, dv]
    size_t sv;      // per-row normaliser and the exponent it is scaled by, float2 [BH, N] (forward -> backward)
    // backward only
    size_t Oscr;    // forward output when backward has to recompute it, bf16 [BH, N, dv]
    size_t delta;   // dO_i . O_i, fp32 [BH, N]
    size_t rhoc;    // per-chunk sums -sum_i A^_il delta_i, fp32 [BH, T, m]
    size_t espart;  // partials of rowsum(E_K) per slab and 32-column group, fp32 [4 nslab, BH, N]
    size_t Tacc;    // sum_i E_i^T x_i over both sides and the batch, fp32 [H, m, d]
    size_t dMn;     // gradient of M through the key norm term, fp32 [H, r, d]
    size_t dKh, dVh; // grouped key/value heads: dK and dV per query head, bf16 [BH, N, d] and [BH, N, dv], summed over each group in fp32 at the end
    size_t Sst;     // workspace copy of the stash's per-chunk S (causal): bf16 [BH, T, m, dv], S before chunk t (t = 0 not written)
    size_t Ahat;    // causal backward: A^ of every (token, feature), bf16 [BH, N, m] (query-side kernel -> key-side kernel)
    size_t Bphi;    // workspace copy of the stash's key features Bf (causal), bf16 [BH, N, m]: forward scan -> both backward kernels
    size_t Racc;    // non-causal backward: sum of A^^T dO, fp32 [BH, m, dv]; rhot directly behind it
    size_t rhot;    // non-causal backward: -sum of A^^T delta, fp32 [BH, m]
    size_t Rb;      // bf16 copy of Racc
    size_t total_bytes;
    // the forward -> backward stash (`saved`): per-row normalisers, key norms, folded projections, key shifts
    size_t sv_sv, sv_nK, sv_Om, sv_Oml, sv_cs, sv_zc, sv_Sb, sv_zt, sv_Sst, sv_Bphi, sv_bytes;
    size_t zc;      // workspace copy of the stash's per-chunk z (causal): sum_j phi(K)_jl over the chunks before t, fp32 [BH, T, m]
    int nslab, T, nsplit;
};

// Where one call keeps what the prologue and the forward pass leave for the backward pass: in the
// caller's `saved` buffer when there is one, else in the workspace.
struct Stash {
    float2 *sv;
    float *nK;
    __nv_bfloat16 *Om, *Oml;
    float *cs;
    float *zc;      // causal: z before chunk t, [BH, T, m] (row t = 0 is not written: it is zero)
    __nv_bfloat16 *Sb;   // non-causal: S of the whole sequence, bf16 [BH, m, dv]
    float *zt;      // non-causal: z of the whole sequence, [BH, m]
    __nv_bfloat16 *Sst;  // causal: S before chunk t, bf16 [BH, T, m, dv] (t = 0 is not written: it is zero)
    __nv_bfloat16 *Bphi; // causal: the key features Bf of every (token, feature), bf16 [BH, N, m], as the forward scan formed them
};
inline Stash stash_in_workspace(const TensorLayout &Y, char *ws)
{
    return Stash{reinterpret_cast<float2 *>(ws + Y.sv), reinterpret_cast<float *>(ws + Y.nK),
                 reinterpret_cast<__nv_bfloat16 *>(ws + Y.Om), reinterpret_cast<__nv_bfloat16 *>(ws + Y.Oml),
                 reinterpret_cast<float *>(ws + Y.cs),
                 reinterpret_cast<float *>(ws + Y.zc), reinterpret_cast<__nv_bfloat16 *>(ws + Y.Sb),
                 reinterpret_cast<float *>(ws + Y.zacc), reinterpret_cast<__nv_bfloat16 *>(ws + Y.Sst),
                 reinterpret_cast<__nv_bfloat16 *>(ws + Y.Bphi)};
}
inline Stash stash_in_saved(const TensorLayout &Y, void *saved)
{
    char *b = static_cast<char *>(saved);
    return Stash{reinterpret_cast<float2 *>(b + Y.sv_sv), reinterpret_cast<float *>(b + Y.sv_nK),
                 reinterpret_cast<__nv_bfloat16 *>(b + Y.sv_Om), reinterpret_cast<__nv_bfloat16 *>(b + Y.sv_Oml),
                 reinterpret_cast<float *>(b + Y.sv_cs),
                 reinterpret_cast<float *>(b + Y.sv_zc), reinterpret_cast<__nv_bfloat16 *>(b + Y.sv_Sb),
                 reinterpret_cast<float *>(b + Y.sv_zt), reinterpret_cast<__nv_bfloat16 *>(b + Y.sv_Sst),
                 reinterpret_cast<__nv_bfloat16 *>(b + Y.sv_Bphi)};
}

}  // namespace darkattn

namespace darkattn {
// Optional per-kernel timing: an event before every kernel of a call and one after the last.
struct KernelTimer {
    static constexpr int kMaxMarks = 96, kMaxKernels = 32;
    bool on = false, created = false;
    int n = 0;                               // marks since the last harvest
    cudaEvent_t ev[kMaxMarks];
    const char *name[kMaxMarks];             // nullptr: closing mark of a call
    int nk = 0;                              // accumulated per kernel name
    const char *kname[kMaxKernels];
    double kms[kMaxKernels];
    int kcount[kMaxKernels];
};
}  // namespace darkattn

struct darkattn_plan_s {
    darkattn_desc_t desc;
    darkattn::Dims dims;
    int path;                      // resolved DARKATTN_PATH_*
    darkattn::SimtLayout simt;
    darkattn::TensorLayout tensor;
    size_t workspace_bytes;
    size_t saved_bytes;
    int launches_fwd, launches_bwd;
    mutable darkattn::KernelTimer timer;
    // side stream of the tensor-core backward (created by its first call on the device current then) and the two
    // events that fork it from and join it back into the caller's stream
    mutable cudaStream_t aux_stream = nullptr;
    mutable cudaEvent_t aux_fork = nullptr, aux_join = nullptr;
};

namespace darkattn {

void set_cuda_error(cudaError_t e, const char *where);
// The plan's side stream and the two events that fork work onto it and join it back (created on first use).
inline cudaError_t ensure_aux(const darkattn_plan_s *plan)
{
    if (plan->aux_stream) return cudaSuccess;
    cudaError_t e = cudaStreamCreateWithFlags(&plan->aux_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->aux_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->aux_join, cudaEventDisableTiming);
    return e;
}

// Records an event in front of the kernel `name` (nullptr: after the last kernel of a call) when timing is on.
void timer_mark(const darkattn_plan_s *plan, cudaStream_t st, const char *name);

// SIMT (FP32 FFMA) path
void simt_make_layout(darkattn_plan_s *plan);
darkattn_status_t simt_forward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                               const void *M, const void *W, void *O, char *ws, cudaStream_t st,
                               bool keep_for_backward);
darkattn_status_t simt_backward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                const void *M, const void *W, const void *dO, void *dQ, void *dK,
                                void *dV, float *dM, char *ws, cudaStream_t st);

// Tensor-core (tcgen05 / TMEM / TMA) path, bf16 operands with fp32 accumulation
bool tensor_supported(const darkattn_plan_s *plan);
void tensor_make_layout(darkattn_plan_s *plan);
darkattn_status_t tensor_forward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                 const void *M, const void *W, void *O, void *saved, char *ws, cudaStream_t st, bool stash_states);
// Folded projections, key-side shifts and key norms (written to `out`).
cudaError_t tensor_prologue(const darkattn_plan_s *plan, const void *K, const void *M, const void *W, char *ws,
                            const Stash &out, cudaStream_t st);
// dW from what the last backward call left in the workspace
darkattn_status_t simt_backward_dw(const darkattn_plan_s *plan, float *dW, char *ws, cudaStream_t st);
cudaError_t tensor_backward_nc_passes(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V, const void *dO,
                                      const Stash &stash, void *dQ, void *dK, void *dV, bool per_head, char *ws, cudaStream_t st);
darkattn_status_t tensor_backward_dw(const darkattn_plan_s *plan, const void *M, float *dW, char *ws, cudaStream_t st);
darkattn_status_t tensor_backward(const darkattn_plan_s *plan, const void *Q, const void *K, const void *V,
                                  const void *M, const void *W, const void *O, const void *dO, const void *saved,
                                  void *dQ, void *dK, void *dV, float *dM, char *ws, cudaStream_t st);

// Number of pieces (1..max_splits, at most T) to cut each of `units` sequences of T tiles into, for kernels that run one CTA
// per piece and SM: the count that minimises (waves of CTAs over the 148 SMs) x (time of one CTA), one CTA costing
// us_per_tile per tile plus us_fixed to start and to flush its accumulators.
inline int pick_splits(long long units, int T, double us_per_tile, double us_fixed, int max_splits, int slots = 148)
{
    int best_c = 1;
    double best = 1e30;
    for (int c = 1; c <= max_splits && c <= T; ++c) {
        const long long waves = (units * c + slots - 1) / slots;
        const double cost = (double)waves * (us_per_tile * ((T + c - 1) / c) + us_fixed);
        if (cost < best) { best = cost; best_c = c; }
    }
    return best_c;
}

#define DARKATTN_CUDA_TRY(expr, where)                                   \
    do {                                                                 \
        cudaError_t e__ = (expr);                                        \
        if (e__ != cudaSuccess) {                                        \
            ::darkattn::set_cuda_error(e__, where);                      \
            return DARKATTN_ERR_CUDA;                                    \
        }                                                                \
    } while (0)

}  // namespace darkattn
