/*
 * darkattn_ref.c -- float64 CPU oracle for DARK random-feature attention.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the method computes,
 * written from the paper; it shares no code with the CUDA library and must never be called from
 * the product path. Only the test-suite, the smoke check and the benchmark's CPU-baseline leg
 * may link or load it.
 *
 * Every function takes host pointers to contiguous row-major double arrays (last index fastest).
 * Loops are written in the order of the definitions; the only parallelism is OpenMP over the
 * independent (batch, head) pairs.
 *
 * Notation (per batch b and head h):  Q,K in R^{N x d}, V in R^{N x dv}, M in R^{r x d},
 * W in R^{m x r} with rows w_l.  s = sqrt(scale) is applied to both Mq and Mk, so that the kernel
 * being estimated is exp(scale * q^T M^T M k)  (Section 2 footnote: q and k absorb the 1/sqrt(d)).
 *
 *   x~_i     = s * M x_i                                   (Section 4.1, x~ := M x)
 *   u_il     = w_l^T x~_i                                  (Appendix B: w^T(Mq) = (M^T w)^T q)
 *   phi(x_i)_l = exp(u_il - ||x~_i||^2/2 - shift) / sqrt(m)   (Section 4.1 feature map, h(x~))
 *   O_i      = sum_j phi(q_i)^T phi(k_j) v_j / sum_j phi(q_i)^T phi(k_j)    (Section 2, normalised;
 *              evaluated as phi(Q)(phi(K)^T V), the linear ordering of Section 2)
 *   causal:  the sums run over j <= i (diagonal included).
 *
 * `shift` is an optional constant subtracted in the exponent (one per query row, one per
 * (batch, head) for the keys). It cancels in O; it exists so that tests can check exactly that.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REF_OK 0
#define REF_ERR_ARG 1
#define REF_ERR_MEM 2

int darkattn_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Feature map of Section 4.1 for N rows.
 * X [N,d], M [r,d], W [m,r]; shift [N] or NULL; phi [N,m] out; xt [N,r] out or NULL.        */
int darkattn_ref_features(int N, int d, int r, int m, double s,
                          const double *X, const double *M, const double *W,
                          const double *shift, double *phi, double *xt_out)
{
    if (N < 0 || d <= 0 || r <= 0 || m <= 0 || !X || !M || !W || !phi) return REF_ERR_ARG;
    double *xt = (double *)malloc(sizeof(double) * (size_t)r);
    if (!xt) return REF_ERR_MEM;
    const double inv_sqrt_m = 1.0 / sqrt((double)m);
    for (int i = 0; i < N; ++i) {
        const double *x = X + (size_t)i * d;
        double nrm2 = 0.0;
        for (int a = 0; a < r; ++a) {                 /* x~ = s * M x */
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += M[(size_t)a * d + c] * x[c];
            xt[a] = s * acc;
            nrm2 += xt[a] * xt[a];
        }
        const double h = 0.5 * nrm2 + (shift ? shift[i] : 0.0);
        for (int l = 0; l < m; ++l) {                 /* u_l = w_l . x~ ; phi_l = exp(u_l - h)/sqrt(m) */
            double u = 0.0;
            for (int a = 0; a < r; ++a) u += W[(size_t)l * r + a] * xt[a];
            phi[(size_t)i * m + l] = exp(u - h) * inv_sqrt_m;
        }
        if (xt_out) memcpy(xt_out + (size_t)i * r, xt, sizeof(double) * (size_t)r);
    }
    free(xt);
    return REF_OK;
}

/* One (batch, head): normalised random-feature attention, Section 2 ordering.
 * phiQ, phiK [N,m]; V [N,dv]; O [N,dv]. Scratch S [m,dv], z [m].                               */
static void attend_one(int N, int m, int dv, int causal,
                       const double *phiQ, const double *phiK, const double *V,
                       double *S, double *z, double *O)
{
    memset(S, 0, sizeof(double) * (size_t)m * dv);
    memset(z, 0, sizeof(double) * (size_t)m);
    if (!causal) {
        for (int j = 0; j < N; ++j)                    /* S = phi(K)^T V, z = phi(K)^T 1 */
            for (int l = 0; l < m; ++l) {
                const double f = phiK[(size_t)j * m + l];
                z[l] += f;
                for (int c = 0; c < dv; ++c) S[(size_t)l * dv + c] += f * V[(size_t)j * dv + c];
            }
    }
    for (int i = 0; i < N; ++i) {
        if (causal) {                                  /* prefix sums include the diagonal j = i */
            for (int l = 0; l < m; ++l) {
                const double f = phiK[(size_t)i * m + l];
                z[l] += f;
                for (int c = 0; c < dv; ++c) S[(size_t)l * dv + c] += f * V[(size_t)i * dv + c];
            }
        }
        double den = 0.0;
        for (int l = 0; l < m; ++l) den += phiQ[(size_t)i * m + l] * z[l];
        for (int c = 0; c < dv; ++c) {
            double num = 0.0;
            for (int l = 0; l < m; ++l) num += phiQ[(size_t)i * m + l] * S[(size_t)l * dv + c];
            O[(size_t)i * dv + c] = num / den;
        }
    }
}

/* Forward for all (b,h).
 * Q,K [B,H,N,d]; V,O [B,H,N,dv]; M [H,r,d]; W [m,r] (or [H,m,r] when w_per_head);
 * shift_q [B,H,N] or NULL; shift_k [B,H] or NULL.                                              */
int darkattn_ref_forward(int B, int H, int N, int d, int r, int m, int dv, int causal,
                         double scale, int w_per_head,
                         const double *Q, const double *K, const double *V,
                         const double *M, const double *W,
                         const double *shift_q, const double *shift_k, double *O)
{
    if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || r <= 0 || m <= 0 || dv <= 0 || !(scale > 0.0) ||
        !Q || !K || !V || !M || !W || !O)
        return REF_ERR_ARG;
    const double s = sqrt(scale);
    int status = REF_OK;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        const int h = bh % H;
        const double *Mh = M + (size_t)h * r * d;
        const double *Wh = W + (w_per_head ? (size_t)h * m * r : 0);
        double *phiQ = (double *)malloc(sizeof(double) * (size_t)N * m);
        double *phiK = (double *)malloc(sizeof(double) * (size_t)N * m);
        double *S = (double *)malloc(sizeof(double) * (size_t)m * dv);
        double *z = (double *)malloc(sizeof(double) * (size_t)m);
        double *sk = (double *)malloc(sizeof(double) * (size_t)N);
        if (!phiQ || !phiK || !S || !z || !sk) {
#pragma omp critical
            status = REF_ERR_MEM;
        } else {
            for (int j = 0; j < N; ++j) sk[j] = shift_k ? shift_k[bh] : 0.0;
            darkattn_ref_features(N, d, r, m, s, Q + (size_t)bh * N * d, Mh, Wh,
                                  shift_q ? shift_q + (size_t)bh * N : NULL, phiQ, NULL);
            darkattn_ref_features(N, d, r, m, s, K + (size_t)bh * N * d, Mh, Wh, sk, phiK, NULL);
            attend_one(N, m, dv, causal, phiQ, phiK, V + (size_t)bh * N * dv, S, z,
                       O + (size_t)bh * N * dv);
        }
        free(phiQ); free(phiK); free(S); free(z); free(sk);
    }
    return status;
}

/* Chain rule through the feature map for one side (queries or keys) of one (b,h).
 *   E = dphi (.) phi                     (derivative of exp; the shift is a constant)
 *   dx~_i = W^T E_i - (sum_l E_il) x~_i  (u = W x~ and the -||x~||^2/2 term)
 *   dx_i  = s * M^T dx~_i
 *   dM   += s * dx~_i x_i^T,   dW += E_i x~_i^T
 */
static void features_backward(int N, int d, int r, int m, double s,
                              const double *X, const double *Mh, const double *Wh,
                              const double *phi, const double *xt, const double *dphi,
                              double *dX, double *dM, double *dW, double *dxt /* scratch [r] */)
{
    for (int i = 0; i < N; ++i) {
        double esum = 0.0;
        for (int a = 0; a < r; ++a) dxt[a] = 0.0;
        for (int l = 0; l < m; ++l) {
            const double e = dphi[(size_t)i * m + l] * phi[(size_t)i * m + l];
            esum += e;
            for (int a = 0; a < r; ++a) {
                dxt[a] += Wh[(size_t)l * r + a] * e;
                dW[(size_t)l * r + a] += e * xt[(size_t)i * r + a];
            }
        }
        for (int a = 0; a < r; ++a) dxt[a] -= esum * xt[(size_t)i * r + a];
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int a = 0; a < r; ++a) acc += Mh[(size_t)a * d + c] * dxt[a];
            dX[(size_t)i * d + c] = s * acc;
        }
        for (int a = 0; a < r; ++a)
            for (int c = 0; c < d; ++c) dM[(size_t)a * d + c] += s * dxt[a] * X[(size_t)i * d + c];
    }
}

/* Backward for all (b,h): gradients of L = sum(dO (.) O) with respect to Q, K, V, M (and W).
 *
 * With A = phi(Q), Bf = phi(K), S_i = sum_{j in J(i)} Bf_j v_j^T, z_i = sum_{j in J(i)} Bf_j,
 * den_i = A_i . z_i, O_i = A_i^T S_i / den_i, G = dO, delta_i = G_i . O_i
 * (J(i) = all j, or j <= i when causal):
 *   dA_i  = (S_i G_i - delta_i z_i) / den_i
 *   R_j   = sum_{i in I(j)} A_i (G_i/den_i)^T,  rho_j = - sum_{i in I(j)} A_i delta_i/den_i
 *   dBf_j = R_j v_j + rho_j,   dV_j = R_j^T Bf_j          (I(j) = all i, or i >= j when causal)
 * followed by features_backward for both sides.
 *
 * dQ,dK [B,H,N,d]; dV [B,H,N,dv]; dM [H,r,d] (summed over the batch); dW [m,r] or [H,m,r]
 * (summed over the batch, and over heads when W is shared); dW may be NULL.                    */
int darkattn_ref_backward(int B, int H, int N, int d, int r, int m, int dv, int causal,
                          double scale, int w_per_head,
                          const double *Q, const double *K, const double *V,
                          const double *M, const double *W, const double *dO,
                          const double *shift_q, const double *shift_k,
                          double *dQ, double *dK, double *dV, double *dM, double *dW)
{
    if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || r <= 0 || m <= 0 || dv <= 0 || !(scale > 0.0) ||
        !Q || !K || !V || !M || !W || !dO || !dQ || !dK || !dV || !dM)
        return REF_ERR_ARG;
    const double s = sqrt(scale);
    const int BH = B * H;
    double *dM_part = (double *)calloc((size_t)BH * r * d, sizeof(double));
    double *dW_part = (double *)calloc((size_t)BH * m * r, sizeof(double));
    if (!dM_part || !dW_part) { free(dM_part); free(dW_part); return REF_ERR_MEM; }
    int status = REF_OK;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < BH; ++bh) {
        const int h = bh % H;
        const double *Mh = M + (size_t)h * r * d;
        const double *Wh = W + (w_per_head ? (size_t)h * m * r : 0);
        const double *Qb = Q + (size_t)bh * N * d, *Kb = K + (size_t)bh * N * d;
        const double *Vb = V + (size_t)bh * N * dv, *Gb = dO + (size_t)bh * N * dv;
        const size_t nm = (size_t)N * m;
        double *buf = (double *)malloc(sizeof(double) *
                                       (4 * nm + 2 * (size_t)N * r + 2 * (size_t)N + (size_t)N * dv +
                                        2 * (size_t)m * dv + 2 * (size_t)m + (size_t)N + r));
        if (!buf) {
#pragma omp critical
            status = REF_ERR_MEM;
            continue;
        }
        double *phiQ = buf, *phiK = phiQ + nm, *dA = phiK + nm, *dBf = dA + nm;
        double *xtQ = dBf + nm, *xtK = xtQ + (size_t)N * r;
        double *den = xtK + (size_t)N * r, *delta = den + N;
        double *Oi = delta + N;                          /* [N,dv] recomputed outputs */
        double *S = Oi + (size_t)N * dv, *R = S + (size_t)m * dv;
        double *z = R + (size_t)m * dv, *rho = z + m;
        double *sk = rho + m, *dxt = sk + N;

        for (int j = 0; j < N; ++j) sk[j] = shift_k ? shift_k[bh] : 0.0;
        darkattn_ref_features(N, d, r, m, s, Qb, Mh, Wh, shift_q ? shift_q + (size_t)bh * N : NULL,
                              phiQ, xtQ);
        darkattn_ref_features(N, d, r, m, s, Kb, Mh, Wh, sk, phiK, xtK);

        /* forward-direction pass: S_i, z_i, den_i, O_i, delta_i, dA_i */
        memset(S, 0, sizeof(double) * (size_t)m * dv);
        memset(z, 0, sizeof(double) * (size_t)m);
        if (!causal)
            for (int j = 0; j < N; ++j)
                for (int l = 0; l < m; ++l) {
                    const double f = phiK[(size_t)j * m + l];
                    z[l] += f;
                    for (int c = 0; c < dv; ++c) S[(size_t)l * dv + c] += f * Vb[(size_t)j * dv + c];
                }
        for (int i = 0; i < N; ++i) {
            if (causal)
                for (int l = 0; l < m; ++l) {
                    const double f = phiK[(size_t)i * m + l];
                    z[l] += f;
                    for (int c = 0; c < dv; ++c) S[(size_t)l * dv + c] += f * Vb[(size_t)i * dv + c];
                }
            double dn = 0.0;
            for (int l = 0; l < m; ++l) dn += phiQ[(size_t)i * m + l] * z[l];
            den[i] = dn;
            double dl = 0.0;
            for (int c = 0; c < dv; ++c) {
                double num = 0.0;
                for (int l = 0; l < m; ++l) num += phiQ[(size_t)i * m + l] * S[(size_t)l * dv + c];
                Oi[(size_t)i * dv + c] = num / dn;
                dl += Gb[(size_t)i * dv + c] * Oi[(size_t)i * dv + c];
            }
            delta[i] = dl;
            for (int l = 0; l < m; ++l) {
                double acc = 0.0;
                for (int c = 0; c < dv; ++c) acc += S[(size_t)l * dv + c] * Gb[(size_t)i * dv + c];
                dA[(size_t)i * m + l] = (acc - dl * z[l]) / dn;
            }
        }

        /* reverse-direction pass: R_j, rho_j, dBf_j, dV_j */
        memset(R, 0, sizeof(double) * (size_t)m * dv);
        memset(rho, 0, sizeof(double) * (size_t)m);
        if (!causal)
            for (int i = 0; i < N; ++i)
                for (int l = 0; l < m; ++l) {
                    const double a = phiQ[(size_t)i * m + l];
                    rho[l] -= a * delta[i] / den[i];
                    for (int c = 0; c < dv; ++c)
                        R[(size_t)l * dv + c] += a * Gb[(size_t)i * dv + c] / den[i];
                }
        for (int j = N - 1; j >= 0; --j) {
            if (causal)
                for (int l = 0; l < m; ++l) {
                    const double a = phiQ[(size_t)j * m + l];
                    rho[l] -= a * delta[j] / den[j];
                    for (int c = 0; c < dv; ++c)
                        R[(size_t)l * dv + c] += a * Gb[(size_t)j * dv + c] / den[j];
                }
            for (int l = 0; l < m; ++l) {
                double acc = rho[l];
                for (int c = 0; c < dv; ++c) acc += R[(size_t)l * dv + c] * Vb[(size_t)j * dv + c];
                dBf[(size_t)j * m + l] = acc;
            }
            for (int c = 0; c < dv; ++c) {
                double acc = 0.0;
                for (int l = 0; l < m; ++l) acc += R[(size_t)l * dv + c] * phiK[(size_t)j * m + l];
                dV[(size_t)bh * N * dv + (size_t)j * dv + c] = acc;
            }
        }

        double *dMp = dM_part + (size_t)bh * r * d, *dWp = dW_part + (size_t)bh * m * r;
        features_backward(N, d, r, m, s, Qb, Mh, Wh, phiQ, xtQ, dA, dQ + (size_t)bh * N * d, dMp, dWp, dxt);
        features_backward(N, d, r, m, s, Kb, Mh, Wh, phiK, xtK, dBf, dK + (size_t)bh * N * d, dMp, dWp, dxt);
        free(buf);
    }
    /* reduce the per-(b,h) parameter gradients in a fixed order */
    memset(dM, 0, sizeof(double) * (size_t)H * r * d);
    if (dW) memset(dW, 0, sizeof(double) * (size_t)(w_per_head ? H : 1) * m * r);
    for (int bh = 0; bh < BH; ++bh) {
        const int h = bh % H;
        for (size_t t = 0; t < (size_t)r * d; ++t) dM[(size_t)h * r * d + t] += dM_part[(size_t)bh * r * d + t];
        if (dW) {
            double *dst = dW + (w_per_head ? (size_t)h * m * r : 0);
            for (size_t t = 0; t < (size_t)m * r; ++t) dst[t] += dW_part[(size_t)bh * m * r + t];
        }
    }
    free(dM_part); free(dW_part);
    return status;
}
