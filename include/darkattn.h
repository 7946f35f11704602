/*
 * darkattn.h -- C ABI of libdarkattn: random-feature attention for the data-aligned softmax kernel
 * exp(q^T Sigma k), Sigma = M^T M (DARKFormer, Section 4.1), on NVIDIA B200 (sm_100a).
 *
 * What the library computes, per batch b and head h (Q,K in R^{N x d}, V in R^{N x dv},
 * M_h in R^{r x d}, W in R^{m x r} with Gaussian rows w_l, s = sqrt(scale)):
 *
 *   x~      = s * M_h x                      re-embedding x -> Mx (Section 4.1; Appendix C)
 *   phi(x)_l = exp(w_l . x~ - |x~|^2 / 2)    positive random feature for omega~_l = M^T w_l ~ N(0,Sigma)
 *                                            (Section 4.1 feature map; Appendix B reparametrisation)
 *   O_i     = sum_j phi(q_i).phi(k_j) v_j / sum_j phi(q_i).phi(k_j)
 *                                            evaluated as phi(Q) (phi(K)^T V), never forming N x N
 *                                            (Section 2, "Efficient Attention via Random Feature Kernels")
 *   causal: the sums run over j <= i; they are evaluated as a chunked prefix scan.
 *
 * The common factor 1/sqrt(m) of the feature map and every stabilising shift of the exponent cancel
 * in O and are not observable through this interface.
 *
 * All tensor arguments are DEVICE pointers to contiguous arrays, last index fastest, base address
 * aligned to 16 bytes. The caller owns every buffer, including `workspace` and `saved`; the library
 * allocates no device memory and keeps no pointer after a call returns. Calls are asynchronous on the
 * given CUDA stream and never synchronise it (except darkattn_last_device_status). Argument errors are
 * reported on the host before anything is launched. There is no CPU fallback.
 *
 *   Q, dQ          [B, H, N, d]      desc.dtype
 *   K, dK          [B, H_kv, N, d]   desc.dtype   (H_kv = H unless desc.H_kv says otherwise: grouped key/value heads)
 *   V, dV          [B, H_kv, N, dv]  desc.dtype
 *   O, dO          [B, H, N, dv]     desc.dtype
 *   M              [H, r, d]         desc.dtype   (row a of M_h produces coordinate a of M_h x)
 *   W              [m, r]            desc.dtype   (or [H, m, r] when desc.w_per_head != 0)
 *   dM             [H, r, d]         float32, OVERWRITTEN (summed over the batch inside the call)
 */
#ifndef DARKATTN_H_
#define DARKATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DARKATTN_OK = 0,
    DARKATTN_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, misaligned pointer            */
    DARKATTN_ERR_UNSUPPORTED = 2,  /* shape / dtype / path combination that no kernel here covers     */
    DARKATTN_ERR_WORKSPACE = 3,    /* workspace missing, or too small a built-in one (forward_static) */
    DARKATTN_ERR_CUDA = 4,         /* a CUDA runtime or driver call failed (see darkattn_last_cuda_error) */
    DARKATTN_ERR_TIMEOUT = 5,      /* a bounded device-side wait gave up (device status word)         */
    DARKATTN_ERR_NONFINITE = 6     /* a normaliser was zero or not finite (device status word)        */
} darkattn_status_t;

typedef enum { DARKATTN_F32 = 0, DARKATTN_BF16 = 1 } darkattn_dtype_t;

/* Which kernels carry the work.
 *   AUTO   : F32 -> SIMT; BF16 -> TENSOR where the shape is covered, else SIMT.
 *   SIMT   : FP32 FFMA kernels with FP32 accumulation (any shape; the only path that meets the
 *            1e-4 tolerance, because TF32/BF16 operands round the exponent's argument).
 *   TENSOR : tcgen05 / TMEM / TMA kernels, BF16 operands, FP32 accumulation (BF16 dtype only;
 *            DARKATTN_ERR_UNSUPPORTED at plan time if the shape is not covered).               */
typedef enum { DARKATTN_PATH_AUTO = 0, DARKATTN_PATH_SIMT = 1, DARKATTN_PATH_TENSOR = 2 } darkattn_path_t;

typedef struct {
    int32_t B, H, N;      /* batch, heads, sequence length (all >= 1)                              */
    int32_t d;            /* query/key width                                                       */
    int32_t r;            /* rows of M (r <= d in the paper; any r >= 1 accepted); 0 means r = d   */
    int32_t m;            /* number of random features                                             */
    int32_t dv;           /* value width; 0 means dv = d                                           */
    int32_t dtype;        /* darkattn_dtype_t of Q,K,V,M,W,O,dO,dQ,dK,dV                            */
    int32_t causal;       /* 0: every key; 1: keys j <= i                                          */
    int32_t chunk;        /* causal chunk length of the prefix scan; 0 means 128                   */
    float   scale;        /* multiplies q^T Sigma k; 0 means 1/sqrt(d) (Section 2 footnote: the
                             scaling is absorbed symmetrically, sqrt(scale) into Mq and into Mk)   */
    int32_t w_per_head;   /* 0: W [m,r] shared by all heads; 1: W [H,m,r]                          */
    int32_t path;         /* darkattn_path_t                                                       */
    int32_t H_kv;         /* key/value heads; 0 means H. Must divide H: query heads h*G .. h*G+G-1 (G = H / H_kv)
                             attend to key/value head h. The paper's feature map applies one M to queries and keys
                             alike (Appendix B: q~ = Mq, k~ = Mk), and M is per query head: a shared key is mapped
                             with the M of the query head that reads it, so its features differ from head to head of
                             the group and only the storage of K and V is shared. dK and dV sum over the group.     */
} darkattn_desc_t;

typedef struct darkattn_plan_s *darkattn_plan_t;

/* Validate a descriptor and fix the kernel selection and the workspace layout. Host only: touches
 * no GPU state. On success *out owns a small host object; release it with darkattn_destroy.     */
darkattn_status_t darkattn_plan(const darkattn_desc_t *desc, darkattn_plan_t *out);

/* Bytes of device scratch the caller must pass as `workspace` to forward / backward (the larger of
 * the two needs). Contents need not be preserved between calls.                                  */
size_t darkattn_workspace_bytes(darkattn_plan_t plan);

/* Bytes of the forward->backward stash (`saved`): what the forward pass computed and the backward
 * pass needs again (on the tensor-core path the per-row normalisers, the key norms, the folded
 * projections, the key-side shifts and the key-side sums: z before every chunk when causal, S and
 * z of the whole sequence otherwise). 0 means there is none. `saved` may always be NULL in both
 * calls: backward then recomputes what it needs, at the cost of running the forward kernels again. */
size_t darkattn_saved_bytes(darkattn_plan_t plan);

/* The path (DARKATTN_PATH_SIMT or DARKATTN_PATH_TENSOR) the plan resolved to.                   */
int32_t darkattn_plan_path(darkattn_plan_t plan);

/* O = normalised random-feature attention (formulas at the top of this file).                   */
darkattn_status_t darkattn_forward(darkattn_plan_t plan, const void *Q, const void *K, const void *V,
                                   const void *M, const void *W, void *O, void *saved /* nullable */,
                                   void *workspace, void *cuda_stream);

/* Gradients of L = sum(dO .* O) with respect to Q, K, V and M (the paper learns M by
 * back-propagation, Section 4; the formulas follow from the chain rule through the definitions at
 * the top of this file, with every stabilising shift held constant, which is exact because O does
 * not depend on them). `O` is the forward result for the same inputs (may be NULL: recomputed).
 * On the tensor-core path part of the zeroing of dK and dV runs on a stream of the plan's own (created by the
 * first such call, non-blocking), forked from `cuda_stream` and joined back into it with events before the
 * call's later kernels: to the caller everything still happens in stream order on `cuda_stream`.           */
darkattn_status_t darkattn_backward(darkattn_plan_t plan, const void *Q, const void *K, const void *V,
                                    const void *M, const void *W, const void *O, const void *dO,
                                    const void *saved /* nullable */, void *dQ, void *dK, void *dV,
                                    float *dM, void *workspace, void *cuda_stream);

/* Gradient of L with respect to the projection rows W, for the variant of the model that trains them (the
 * learned-feature kernel the paper compares against, Section 5: the random projections are replaced by
 * trainable vectors). Chain rule through u_l = w_l . x~: dW_l = sum_i (dphi .* phi)_il x~_i over queries and keys,
 * batches (and heads, when W is shared by the heads).
 * Call it after darkattn_backward, with the same plan, M and `workspace` and nothing else run on that workspace in
 * between: it is computed from accumulators that call left there. dW is float32, laid out like W ([m, r], or
 * [H, m, r] when desc.w_per_head != 0), OVERWRITTEN. Asynchronous on `cuda_stream`.                           */
darkattn_status_t darkattn_backward_dw(darkattn_plan_t plan, const void *M, float *dW, void *workspace,
                                       void *cuda_stream);

/* One decode step of causal attention in its recurrent form. Section 2 ("Efficient Attention via Random Feature
 * Kernels") evaluates the attention as phi(Q) (phi(K)^T V) without forming the L x L matrix; with the causal mask the
 * same ordering, taken one token at a time, needs only the running sums S = sum_{j<=i} phi(k_j) v_j^T and
 * z = sum_{j<=i} phi(k_j) (the Discussion names long-context use as a direction). For every (batch, head) this call
 * adds the new token's key and value to the caller's running state and returns the new token's output,
 *     S += phi(k) v^T,   z += phi(k),   o = phi(q)^T S / phi(q)^T z.
 * q, k [B, H, d] and v, o [B, H, dv] in desc.dtype; S [B, H, m, dv] and z [B, H, m] float32, owned by the caller and
 * updated in place: zero them before the first token. The features are scaled by exp(-|w_l|^2/2) (keys) and its
 * inverse (queries), which cancels in o, is the same at every step and keeps every key feature <= 1; the state is
 * therefore only meaningful to this call. Needs a causal plan (B, H, d, r, m, dv, dtype, scale, w_per_head are taken
 * from it; N is not used) with dv a multiple of 32, at most 512 (else DARKATTN_ERR_UNSUPPORTED). No workspace. One
 * kernel launch, asynchronous on `cuda_stream`.                                                                   */
darkattn_status_t darkattn_decode_step(darkattn_plan_t plan, const void *q, const void *k, const void *v, const void *M,
                                       const void *W, float *S, float *z, void *o, void *cuda_stream);

/* Synchronise `cuda_stream`, then read the device status word kept at the start of `workspace`
 * (written by kernels whose bounded waits gave up, or that met a normaliser that is zero or not
 * finite). Returns DARKATTN_OK, DARKATTN_ERR_TIMEOUT, DARKATTN_ERR_NONFINITE or DARKATTN_ERR_CUDA.  */
darkattn_status_t darkattn_last_device_status(darkattn_plan_t plan, const void *workspace,
                                              void *cuda_stream);

void darkattn_destroy(darkattn_plan_t plan);
const char *darkattn_status_string(darkattn_status_t status);
/* Text of the last CUDA error this thread's calls into the library ran into ("" if none).       */
const char *darkattn_last_cuda_error(void);

/* Measure this GPU's throughput of the two ALU resources the feature map leans on, so that the
 * exponent leg of the roofline has a measured denominator: which = 0 -> ex2.approx.f32 (MUFU),
 * which = 1 -> FP32 FMA. Launches a register-only kernel on every SM `iters` times on `cuda_stream`,
 * times it with CUDA events and writes operations per second to *ops_per_second (host pointer).
 * Synchronises the stream.                                                                        */
darkattn_status_t darkattn_measure_alu_peak(int32_t which, int32_t iters, double *ops_per_second,
                                            void *cuda_stream);

/* Self-test of the bounded device-side wait the scan kernels rely on: launches one small kernel whose
 * only thread waits on a barrier nobody arrives on. The wait must give up after its limit (2 s),
 * record DARKATTN_ERR_TIMEOUT in a device status word and let the kernel end normally. Writes that
 * status word and the kernel's device time in seconds to the two host pointers; synchronises the
 * stream. Nothing faults, the context stays usable. Returns DARKATTN_OK when the launch itself ran. */
darkattn_status_t darkattn_selftest_wait_limit(int32_t *device_status, double *seconds, void *cuda_stream);

/* Forward pass that needs no workspace from the caller and allocates nothing.
 *
 * (The paper has no counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Some hosts of this library cannot hand it scratch memory: an inference server that gave the whole
 * GPU to its own pool at start-up and forbids cudaMalloc afterwards because it stalls every stream,
 * a plug-in that is passed input and output buffers but has no access to its host's allocator, a
 * latency-critical loop that must not allocate once it is running. For them this call runs the same
 * FP32 forward as darkattn_forward on the SIMT path (any dtype, any shape, causal or not), with its
 * intermediates in an array of DARKATTN_STATIC_SCRATCH_BYTES that is part of the library's device
 * image: every GPU that loads the library holds that much memory until the process exits.
 *
 *  - The caller still passes Q, K, V, M, W (inputs) and O (output), laid out as for darkattn_forward.
 *  - darkattn_static_scratch_needed(plan) tells how much of the array a plan would use. A plan that
 *    needs more than DARKATTN_STATIC_SCRATCH_BYTES is refused with DARKATTN_ERR_WORKSPACE before
 *    anything touches the GPU; use darkattn_forward with a workspace of your own for it.
 *  - The first call on each device looks up the array's device address (with that device current).
 *    Make that first call at start-up, before any stream capture begins and before the host's own pool
 *    takes the rest of the GPU: under CUDA's default lazy module loading the driver only places the
 *    array in device memory when its address is first asked for (or set CUDA_MODULE_LOADING=EAGER), so
 *    this first call is the one that can still fail for lack of memory. The address is kept per
 *    device; cudaDeviceReset invalidates it (the library is not meant to outlive a reset).
 *  - No cudaMalloc, cudaFree or other allocating routine is called by the library, now or later.
 *  - The status word of this call lives in the library's own array, out of reach of
 *    darkattn_last_device_status: the FP32 kernels it runs never write one.
 *  - All calls on a device share the one array, and it keeps the previous call's contents; the call
 *    clears the words that must start at zero itself. Two calls whose GPU work overlaps (different
 *    streams, or different host threads) race on the array: serialise them on one stream.         */
#define DARKATTN_STATIC_SCRATCH_BYTES (16u << 20)
size_t darkattn_static_scratch_needed(darkattn_plan_t plan);
darkattn_status_t darkattn_forward_static(darkattn_plan_t plan, const void *Q, const void *K, const void *V,
                                          const void *M, const void *W, void *O, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DARKATTN_H_ */
