/*
 * la_oracle.c -- fp64 CPU oracle for linear attention ("Transformers are RNNs").
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * CUDA library must compute.  It shares no code, header, table or helper with
 * the CUDA path, and only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may call it.  Nothing in the product path may link it.
 *
 * Everything is double precision, scalar loops, one (batch, head) pair at a
 * time; the only parallelism is an OpenMP "parallel for" over the independent
 * (batch, head) pairs.  No blocking, chunking or reordering beyond what the
 * cited equation or algorithm states.
 *
 * Layout of every array: row-major contiguous
 *     Q, K, dQ, dK : [B, H, N, D]      V, O, G, dV : [B, H, N, M]
 *     den          : [B, H, N]         S : [B, H, D, M]     Z : [B, H, D]
 *
 * Two independent statements of the same function are provided:
 *   (1) "quadratic": the definition, Eq. 3 (non-causal) / Eq. 8 (causal) with
 *       sim(q, k) = phi(q)^T phi(k) (Eq. 4), on the explicit N x N matrix, and
 *       its gradient by the explicit chain rule on that matrix;
 *   (2) "linear": Eq. 5-6 (non-causal) / Eq. 9-12 and Algorithm 1 (causal),
 *       with the gradients of Eq. 13-15 (Algorithm 1, backward) applied to the
 *       value matrix extended by a column of ones, which carries the
 *       normaliser Z (Eq. 11) and its gradient; the recurrent step is
 *       Eq. 16-20 restricted to the attention part, and the causal form
 *       continued from a given state is that recurrence started from it.
 * The tests pin (1) to closed forms, a hand-worked rational example, library
 * one-liners and finite differences, and (2) to (1).  No function here is
 * "parity unpinned".
 *
 * phi selector: 0 = elu(x)+1 (Eq. 7, alpha = 1), 1 = identity (inputs are
 * already feature-mapped, the convention of Algorithm 1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define LA_ORACLE_PHI_ELU1 0
#define LA_ORACLE_PHI_IDENTITY 1

/* Eq. 7: phi(x) = elu(x) + 1 = x + 1 for x > 0, exp(x) otherwise. */
static double phi_value(double x, int phi)
{
    if (phi == LA_ORACLE_PHI_IDENTITY) return x;
    return x > 0.0 ? x + 1.0 : exp(x);
}

/* d phi / dx: 1 for x > 0, exp(x) otherwise (both branches give 1 at 0). */
static double phi_slope(double x, int phi)
{
    if (phi == LA_ORACLE_PHI_IDENTITY) return 1.0;
    return x > 0.0 ? 1.0 : exp(x);
}

int la_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void la_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Eq. 7 elementwise; deriv != 0 returns the slope instead of the value. */
void la_oracle_feature_map(const double *x, double *y, int64_t n, int deriv)
{
    for (int64_t i = 0; i < n; ++i)
        y[i] = deriv ? phi_slope(x[i], LA_ORACLE_PHI_ELU1)
                     : phi_value(x[i], LA_ORACLE_PHI_ELU1);
}

static double *mapped(const double *x, int64_t n, int phi)
{
    double *y = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
    for (int64_t i = 0; i < n; ++i) y[i] = phi_value(x[i], phi);
    return y;
}

/* ------------------------------------------------------------------------- */
/* (1) The definition: Eq. 3 / Eq. 8 with the kernel of Eq. 4.                */
/* ------------------------------------------------------------------------- */

/*
 * O_i = sum_j A_ij V_j / (sum_j A_ij + eps),  A_ij = phi(Q_i) . phi(K_j),
 * j <= i when causal (Eq. 8), all j otherwise (Eq. 3).
 * W, if not NULL, receives the normalised weights A_ij / (den_i + eps) as
 * [B, H, N, N] with zeros where masked.
 */
void la_oracle_attention_quadratic(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                                   int causal, int phi, double eps,
                                   const double *Q, const double *K, const double *V,
                                   double *O, double *W)
{
    int64_t BH = B * H;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Vh = V + bh * N * M;
        double *Oh = O + bh * N * M;
        double *q = mapped(Q + bh * N * D, N * D, phi);
        double *k = mapped(K + bh * N * D, N * D, phi);
        double *a = (double *)malloc((size_t)(N > 0 ? N : 1) * sizeof(double));
        for (int64_t i = 0; i < N; ++i) {
            int64_t last = causal ? i : N - 1;
            double den = 0.0;
            for (int64_t j = 0; j <= last; ++j) {
                double s = 0.0;
                for (int64_t d = 0; d < D; ++d) s += q[i * D + d] * k[j * D + d];
                a[j] = s;
                den += s;
            }
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t j = 0; j <= last; ++j) num += a[j] * Vh[j * M + e];
                Oh[i * M + e] = num / (den + eps);
            }
            if (W) {
                double *Wr = W + (bh * N + i) * N;
                for (int64_t j = 0; j < N; ++j) Wr[j] = j <= last ? a[j] / (den + eps) : 0.0;
            }
        }
        free(a); free(k); free(q);
    }
}

/*
 * Gradient of L = sum_{i,e} G_ie O_ie by the chain rule on the N x N matrix:
 *   dL/dA_ij = G_i . (V_j - O_i) / (den_i + eps)      (allowed j only)
 *   grad phi(Q_i) = sum_j dL/dA_ij phi(K_j),  grad phi(K_j) = sum_i dL/dA_ij phi(Q_i),
 *   grad V_j = sum_i A_ij G_i / (den_i + eps),
 * then the slope of Eq. 7 is chained in for the raw Q, K.
 */
void la_oracle_attention_quadratic_backward(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                                            int causal, int phi, double eps,
                                            const double *Q, const double *K, const double *V,
                                            const double *G,
                                            double *dQ, double *dK, double *dV)
{
    int64_t BH = B * H;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Qh = Q + bh * N * D, *Kh = K + bh * N * D;
        const double *Vh = V + bh * N * M, *Gh = G + bh * N * M;
        double *dQh = dQ + bh * N * D, *dKh = dK + bh * N * D, *dVh = dV + bh * N * M;
        double *q = mapped(Qh, N * D, phi);
        double *k = mapped(Kh, N * D, phi);
        double *a = (double *)malloc((size_t)(N > 0 ? N : 1) * sizeof(double));
        double *o = (double *)malloc((size_t)(M > 0 ? M : 1) * sizeof(double));
        for (int64_t i = 0; i < N * D; ++i) { dQh[i] = 0.0; dKh[i] = 0.0; }
        for (int64_t i = 0; i < N * M; ++i) dVh[i] = 0.0;
        for (int64_t i = 0; i < N; ++i) {
            int64_t last = causal ? i : N - 1;
            double den = 0.0;
            for (int64_t j = 0; j <= last; ++j) {
                double s = 0.0;
                for (int64_t d = 0; d < D; ++d) s += q[i * D + d] * k[j * D + d];
                a[j] = s;
                den += s;
            }
            double dn = den + eps;
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t j = 0; j <= last; ++j) num += a[j] * Vh[j * M + e];
                o[e] = num / dn;
            }
            for (int64_t j = 0; j <= last; ++j) {
                double da = 0.0;
                for (int64_t e = 0; e < M; ++e) da += Gh[i * M + e] * (Vh[j * M + e] - o[e]);
                da /= dn;
                for (int64_t d = 0; d < D; ++d) {
                    dQh[i * D + d] += da * k[j * D + d];
                    dKh[j * D + d] += da * q[i * D + d];
                }
                for (int64_t e = 0; e < M; ++e) dVh[j * M + e] += a[j] * Gh[i * M + e] / dn;
            }
        }
        for (int64_t i = 0; i < N * D; ++i) {
            dQh[i] *= phi_slope(Qh[i], phi);
            dKh[i] *= phi_slope(Kh[i], phi);
        }
        free(o); free(a); free(k); free(q);
    }
}

/* ------------------------------------------------------------------------- */
/* (2) The linear-time forms.                                                 */
/* ------------------------------------------------------------------------- */

/*
 * Causal: Algorithm 1 "forward" with S of Eq. 10 and Z of Eq. 11 kept side by
 * side, then Eq. 12:   for i = 1..N:  S += phi(K_i) V_i^T ; Z += phi(K_i) ;
 *                      O_i = phi(Q_i)^T S / (phi(Q_i)^T Z + eps).
 * Non-causal: Eq. 5 -- S and Z are the sums over all j, formed once and used
 * for every query.
 * den (may be NULL) receives phi(Q_i)^T Z (without eps).  S_out / Z_out (may
 * be NULL) receive the final state S_N, Z_N.
 */
void la_oracle_linear(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                      int causal, int phi, double eps,
                      const double *Q, const double *K, const double *V,
                      double *O, double *den, double *S_out, double *Z_out)
{
    int64_t BH = B * H;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Vh = V + bh * N * M;
        double *Oh = O + bh * N * M;
        double *q = mapped(Q + bh * N * D, N * D, phi);
        double *k = mapped(K + bh * N * D, N * D, phi);
        double *S = (double *)calloc((size_t)(D * M > 0 ? D * M : 1), sizeof(double));
        double *Z = (double *)calloc((size_t)(D > 0 ? D : 1), sizeof(double));
        if (!causal) {
            for (int64_t j = 0; j < N; ++j)
                for (int64_t d = 0; d < D; ++d) {
                    for (int64_t e = 0; e < M; ++e) S[d * M + e] += k[j * D + d] * Vh[j * M + e];
                    Z[d] += k[j * D + d];
                }
        }
        for (int64_t i = 0; i < N; ++i) {
            if (causal) {
                for (int64_t d = 0; d < D; ++d) {
                    for (int64_t e = 0; e < M; ++e) S[d * M + e] += k[i * D + d] * Vh[i * M + e];
                    Z[d] += k[i * D + d];
                }
            }
            double dn = 0.0;
            for (int64_t d = 0; d < D; ++d) dn += q[i * D + d] * Z[d];
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t d = 0; d < D; ++d) num += q[i * D + d] * S[d * M + e];
                Oh[i * M + e] = num / (dn + eps);
            }
            if (den) den[bh * N + i] = dn;
        }
        if (S_out) memcpy(S_out + bh * D * M, S, (size_t)(D * M) * sizeof(double));
        if (Z_out) memcpy(Z_out + bh * D, Z, (size_t)D * sizeof(double));
        free(Z); free(S); free(k); free(q);
    }
}

/*
 * Causal form continued from a given state: the recurrence of Eq. 16-20 (attention part) started
 * from s_0 = S0, z_0 = Z0 instead of zero, which is what the state carried over from the tokens
 * before this call amounts to (a long sequence processed in several calls):
 *     for i = 1..N:  s_i = s_{i-1} + phi(K_i) V_i^T ;  z_i = z_{i-1} + phi(K_i) ;
 *                    O_i = phi(Q_i)^T s_i / (phi(Q_i)^T z_i + eps).
 * S0 / Z0: [B, H, D, M] / [B, H, D].  den, S_out, Z_out as in la_oracle_linear.
 */
void la_oracle_causal_from_state(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                                 int phi, double eps,
                                 const double *Q, const double *K, const double *V,
                                 const double *S0, const double *Z0,
                                 double *O, double *den, double *S_out, double *Z_out)
{
    int64_t BH = B * H;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Vh = V + bh * N * M;
        double *Oh = O + bh * N * M;
        double *q = mapped(Q + bh * N * D, N * D, phi);
        double *k = mapped(K + bh * N * D, N * D, phi);
        double *s = (double *)malloc((size_t)(D * M > 0 ? D * M : 1) * sizeof(double));
        double *z = (double *)malloc((size_t)(D > 0 ? D : 1) * sizeof(double));
        memcpy(s, S0 + bh * D * M, (size_t)(D * M) * sizeof(double));
        memcpy(z, Z0 + bh * D, (size_t)D * sizeof(double));
        for (int64_t i = 0; i < N; ++i) {
            for (int64_t d = 0; d < D; ++d) {
                for (int64_t e = 0; e < M; ++e) s[d * M + e] += k[i * D + d] * Vh[i * M + e];
                z[d] += k[i * D + d];
            }
            double dn = 0.0;
            for (int64_t d = 0; d < D; ++d) dn += q[i * D + d] * z[d];
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t d = 0; d < D; ++d) num += q[i * D + d] * s[d * M + e];
                Oh[i * M + e] = num / (dn + eps);
            }
            if (den) den[bh * N + i] = dn;
        }
        if (S_out) memcpy(S_out + bh * D * M, s, (size_t)(D * M) * sizeof(double));
        if (Z_out) memcpy(Z_out + bh * D, z, (size_t)D * sizeof(double));
        free(z); free(s); free(k); free(q);
    }
}

/*
 * Gradients in linear time and constant memory.  The paper derives the
 * gradient of the numerator only (Eq. 13-15) and leaves the division to
 * automatic differentiation.  Reading used here: extend V_j by a constant 1,
 * so that the extended numerator is [num_i | den_i]; the gradient of
 * L = sum G.O with respect to that extended numerator is
 *     Gt_i = [ G_i / den_i ,  -(G_i . O_i) / den_i ]      (den_i includes eps)
 * and Eq. 13-15 / Algorithm 1 "backward" apply unchanged:
 *     St = 0; for i = 1..N: St += phi(K_i) [V_i,1]^T ; grad phi(Q_i) = St Gt_i
 *     Rt = 0; for i = N..1: Rt += phi(Q_i) Gt_i^T ;
 *                           grad V_i = (Rt^T phi(K_i))[0:M] ; grad phi(K_i) = Rt [V_i,1]
 * (the constant 1 receives no gradient).  Non-causal: St and Rt are the full
 * sums, used for every i.  Finally the slope of Eq. 7 is chained in.
 */
void la_oracle_linear_backward(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                               int causal, int phi, double eps,
                               const double *Q, const double *K, const double *V,
                               const double *G,
                               double *dQ, double *dK, double *dV)
{
    int64_t BH = B * H;
    int64_t M1 = M + 1;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Qh = Q + bh * N * D, *Kh = K + bh * N * D;
        const double *Vh = V + bh * N * M, *Gh = G + bh * N * M;
        double *dQh = dQ + bh * N * D, *dKh = dK + bh * N * D, *dVh = dV + bh * N * M;
        double *q = mapped(Qh, N * D, phi);
        double *k = mapped(Kh, N * D, phi);
        double *St = (double *)calloc((size_t)(D * M1), sizeof(double));
        double *Rt = (double *)calloc((size_t)(D * M1), sizeof(double));
        double *Gt = (double *)malloc((size_t)(N > 0 ? N * M1 : 1) * sizeof(double));

        /* forward sweep: state, outputs, extended upstream gradient, grad phi(Q) */
        if (!causal) {
            for (int64_t j = 0; j < N; ++j)
                for (int64_t d = 0; d < D; ++d) {
                    for (int64_t e = 0; e < M; ++e) St[d * M1 + e] += k[j * D + d] * Vh[j * M + e];
                    St[d * M1 + M] += k[j * D + d];
                }
        }
        for (int64_t i = 0; i < N; ++i) {
            if (causal) {
                for (int64_t d = 0; d < D; ++d) {
                    for (int64_t e = 0; e < M; ++e) St[d * M1 + e] += k[i * D + d] * Vh[i * M + e];
                    St[d * M1 + M] += k[i * D + d];
                }
            }
            double dn = eps;
            for (int64_t d = 0; d < D; ++d) dn += q[i * D + d] * St[d * M1 + M];
            double go = 0.0;
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t d = 0; d < D; ++d) num += q[i * D + d] * St[d * M1 + e];
                go += Gh[i * M + e] * (num / dn);
                Gt[i * M1 + e] = Gh[i * M + e] / dn;
            }
            Gt[i * M1 + M] = -go / dn;
            if (causal) {
                for (int64_t d = 0; d < D; ++d) {          /* Eq. 13 */
                    double s = 0.0;
                    for (int64_t e = 0; e < M1; ++e) s += St[d * M1 + e] * Gt[i * M1 + e];
                    dQh[i * D + d] = s;
                }
            }
        }
        if (!causal) {
            for (int64_t i = 0; i < N; ++i)
                for (int64_t d = 0; d < D; ++d) {
                    double s = 0.0;
                    for (int64_t e = 0; e < M1; ++e) s += St[d * M1 + e] * Gt[i * M1 + e];
                    dQh[i * D + d] = s;
                }
            for (int64_t j = 0; j < N; ++j)
                for (int64_t d = 0; d < D; ++d)
                    for (int64_t e = 0; e < M1; ++e) Rt[d * M1 + e] += q[j * D + d] * Gt[j * M1 + e];
        }
        /* reverse sweep: Eq. 14 and Eq. 15 */
        for (int64_t i = N - 1; i >= 0; --i) {
            if (causal) {
                for (int64_t d = 0; d < D; ++d)
                    for (int64_t e = 0; e < M1; ++e) Rt[d * M1 + e] += q[i * D + d] * Gt[i * M1 + e];
            }
            for (int64_t e = 0; e < M; ++e) {              /* Eq. 15 */
                double s = 0.0;
                for (int64_t d = 0; d < D; ++d) s += Rt[d * M1 + e] * k[i * D + d];
                dVh[i * M + e] = s;
            }
            for (int64_t d = 0; d < D; ++d) {              /* Eq. 14 */
                double s = Rt[d * M1 + M];
                for (int64_t e = 0; e < M; ++e) s += Rt[d * M1 + e] * Vh[i * M + e];
                dKh[i * D + d] = s;
            }
        }
        for (int64_t i = 0; i < N * D; ++i) {
            dQh[i] *= phi_slope(Qh[i], phi);
            dKh[i] *= phi_slope(Kh[i], phi);
        }
        free(Gt); free(Rt); free(St); free(k); free(q);
    }
}

/*
 * Gradient of the causal form continued from a state (la_oracle_causal_from_state), for
 *     L = sum_{i,e} G_ie O_ie + <dS_N, S_N> + <dZ_N, Z_N>,
 * i.e. an upstream gradient on the outputs and (optionally, NULL = zero) on the final state, as
 * needed when a sequence is processed, and differentiated, in several calls.  With the values
 * extended by a constant 1 (see la_oracle_linear_backward) the state is st_i = [s_i | z_i],
 * st_0 = [S0 | Z0], and Algorithm 1 "backward" applies with two changes only: the forward
 * running sum starts from st_0, and the reverse running sum starts from the upstream gradient
 * of the final state instead of zero:
 *     St = [S0|Z0]; for i = 1..N: St += phi(K_i) [V_i,1]^T ; grad phi(Q_i) = St Gt_i       (Eq. 13)
 *     Rt = [dS_N|dZ_N]; for i = N..1: Rt += phi(Q_i) Gt_i^T ;
 *                       grad V_i = (Rt^T phi(K_i))[0:M] ; grad phi(K_i) = Rt [V_i,1]      (Eq. 14-15)
 * and the state the call started from receives what is left in the reverse sum:
 *     [dS0 | dZ0] = Rt after the sweep      (st_0 enters every st_i with coefficient one).
 */
void la_oracle_causal_backward_from_state(int64_t B, int64_t H, int64_t N, int64_t D, int64_t M,
                                          int phi, double eps,
                                          const double *Q, const double *K, const double *V,
                                          const double *S0, const double *Z0,
                                          const double *G, const double *dSN, const double *dZN,
                                          double *dQ, double *dK, double *dV, double *dS0, double *dZ0)
{
    int64_t BH = B * H;
    int64_t M1 = M + 1;
#pragma omp parallel for schedule(dynamic)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *Qh = Q + bh * N * D, *Kh = K + bh * N * D;
        const double *Vh = V + bh * N * M, *Gh = G + bh * N * M;
        double *dQh = dQ + bh * N * D, *dKh = dK + bh * N * D, *dVh = dV + bh * N * M;
        double *q = mapped(Qh, N * D, phi);
        double *k = mapped(Kh, N * D, phi);
        double *St = (double *)calloc((size_t)(D * M1), sizeof(double));
        double *Rt = (double *)calloc((size_t)(D * M1), sizeof(double));
        double *Gt = (double *)malloc((size_t)(N > 0 ? N * M1 : 1) * sizeof(double));
        for (int64_t d = 0; d < D; ++d) {
            for (int64_t e = 0; e < M; ++e) {
                St[d * M1 + e] = S0[bh * D * M + d * M + e];
                if (dSN) Rt[d * M1 + e] = dSN[bh * D * M + d * M + e];
            }
            St[d * M1 + M] = Z0[bh * D + d];
            if (dZN) Rt[d * M1 + M] = dZN[bh * D + d];
        }
        for (int64_t i = 0; i < N; ++i) {
            for (int64_t d = 0; d < D; ++d) {
                for (int64_t e = 0; e < M; ++e) St[d * M1 + e] += k[i * D + d] * Vh[i * M + e];
                St[d * M1 + M] += k[i * D + d];
            }
            double dn = eps;
            for (int64_t d = 0; d < D; ++d) dn += q[i * D + d] * St[d * M1 + M];
            double go = 0.0;
            for (int64_t e = 0; e < M; ++e) {
                double num = 0.0;
                for (int64_t d = 0; d < D; ++d) num += q[i * D + d] * St[d * M1 + e];
                go += Gh[i * M + e] * (num / dn);
                Gt[i * M1 + e] = Gh[i * M + e] / dn;
            }
            Gt[i * M1 + M] = -go / dn;
            for (int64_t d = 0; d < D; ++d) {
                double s = 0.0;
                for (int64_t e = 0; e < M1; ++e) s += St[d * M1 + e] * Gt[i * M1 + e];
                dQh[i * D + d] = s;
            }
        }
        for (int64_t i = N - 1; i >= 0; --i) {
            for (int64_t d = 0; d < D; ++d)
                for (int64_t e = 0; e < M1; ++e) Rt[d * M1 + e] += q[i * D + d] * Gt[i * M1 + e];
            for (int64_t e = 0; e < M; ++e) {
                double s = 0.0;
                for (int64_t d = 0; d < D; ++d) s += Rt[d * M1 + e] * k[i * D + d];
                dVh[i * M + e] = s;
            }
            for (int64_t d = 0; d < D; ++d) {
                double s = Rt[d * M1 + M];
                for (int64_t e = 0; e < M; ++e) s += Rt[d * M1 + e] * Vh[i * M + e];
                dKh[i * D + d] = s;
            }
        }
        for (int64_t i = 0; i < N * D; ++i) {
            dQh[i] *= phi_slope(Qh[i], phi);
            dKh[i] *= phi_slope(Kh[i], phi);
        }
        for (int64_t d = 0; d < D; ++d) {
            for (int64_t e = 0; e < M; ++e) dS0[bh * D * M + d * M + e] = Rt[d * M1 + e];
            dZ0[bh * D + d] = Rt[d * M1 + M];
        }
        free(Gt); free(Rt); free(St); free(k); free(q);
    }
}

/*
 * One recurrent step, Eq. 18-20 (attention part): the state is updated first
 * and read afterwards.   S += phi(k) v^T ; Z += phi(k) ;
 *                        out = phi(q)^T S / (phi(q)^T Z + eps).
 * q, k: [B, H, D]; v, out: [B, H, M]; S: [B, H, D, M] and Z: [B, H, D] are
 * updated in place (zero for a new sequence, Eq. 16-17).
 */
void la_oracle_recurrent_step(int64_t B, int64_t H, int64_t D, int64_t M,
                              int phi, double eps,
                              const double *q, const double *k, const double *v,
                              double *S, double *Z, double *out)
{
    int64_t BH = B * H;
#pragma omp parallel for schedule(static)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const double *qh = q + bh * D, *kh = k + bh * D, *vh = v + bh * M;
        double *Sh = S + bh * D * M, *Zh = Z + bh * D, *oh = out + bh * M;
        for (int64_t d = 0; d < D; ++d) {
            double kd = phi_value(kh[d], phi);
            for (int64_t e = 0; e < M; ++e) Sh[d * M + e] += kd * vh[e];
            Zh[d] += kd;
        }
        double dn = eps;
        for (int64_t d = 0; d < D; ++d) dn += phi_value(qh[d], phi) * Zh[d];
        for (int64_t e = 0; e < M; ++e) {
            double num = 0.0;
            for (int64_t d = 0; d < D; ++d) num += phi_value(qh[d], phi) * Sh[d * M + e];
            oh[e] = num / dn;
        }
    }
}
