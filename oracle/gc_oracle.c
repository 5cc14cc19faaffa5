/*
 * CPU oracle for the Gradient Cache "Step 2" computation (arXiv 2101.06983, Section 3.3):
 * the in-batch-negative contrastive loss over all B query and N passage representations and
 * its exact gradients with respect to every representation.
 *
 * THIS IS TEST INFRASTRUCTURE, not the product.  It is deliberately plain and slow: double
 * precision, the whole B x N logit matrix S stored explicitly, an explicit softmax, ordinary
 * loops, no blocking, no BLAS.  It shares no code with the CUDA library and is only executed
 * by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Parity pins (see tests/test_oracle_pins.py): central finite differences of the loss, row
 * sums of softmax-minus-onehot, closed forms for identical representations and for the 1x2
 * logistic case, scale and permutation symmetries, and the paper's exactness claim on a linear
 * encoder; gco_query_rows and gco_passage_rows by the same hand-worked example, finite
 * differences and closed form, row for row; gco_cache_apply (Step 3 for a linear encoder) by the
 * finite-difference gradient with respect to the encoder matrix and a hand-worked example;
 * gco_build_variant (cosine similarity, several positives, two-direction loss, dL/dtau) in
 * tests/test_oracle_variants.py; gco_dist_loss / gco_dist_w (Distance Gradient Cache, Section 5)
 * in tests/test_oracle_distance.py.  No function here is "parity unpinned".
 *
 * Notation (paper, Section 3.1-3.2): Q row i is f(s_i), P row j is g(t_j), pos_idx[i] is r_i,
 * tau the temperature, S_ij = <f(s_i), g(t_j)> / tau.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define GCO_MASK_NONE 0
#define GCO_MASK_SELF 1

/* Mask reading (not in the paper, which has no mask): with GCO_MASK_SELF the pair (i, i) is
 * removed from the denominator of Eq. 1 altogether, so p_ii = 0 exactly. */
static int allowed(int mask_mode, int64_t i, int64_t j) {
    return !(mask_mode == GCO_MASK_SELF && i == j);
}

int gco_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int check_args(const int32_t* pos_idx, int64_t B, int64_t N, int64_t d, double tau,
                      int mask_mode) {
    if (B <= 0 || N <= 0 || d <= 0) return 1;
    if (!(tau > 0.0) || !isfinite(tau)) return 2;
    if (mask_mode != GCO_MASK_NONE && mask_mode != GCO_MASK_SELF) return 3;
    for (int64_t i = 0; i < B; ++i) {
        if (pos_idx[i] < 0 || pos_idx[i] >= N) return 4;
        if (!allowed(mask_mode, i, pos_idx[i])) return 5;
    }
    return 0;
}

/* Logits of one query row: S_ij = (sum_k Q_ik P_jk) / tau  (exponent of Eq. 1). */
static void logits_row(const double* Q, const double* P, int64_t i, int64_t N, int64_t d,
                       double tau, double* S_row) {
    const double* q = Q + i * d;
    for (int64_t j = 0; j < N; ++j) {
        const double* p = P + j * d;
        double acc = 0.0;
        for (int64_t k = 0; k < d; ++k) acc += q[k] * p[k];
        S_row[j] = acc / tau;
    }
}

/* Natural-log logsumexp of one row over the allowed columns (denominator of Eq. 1 / Eq. 4). */
static double lse_row(const double* S_row, int64_t i, int64_t N, int mask_mode) {
    double m = -INFINITY;
    for (int64_t j = 0; j < N; ++j)
        if (allowed(mask_mode, i, j) && S_row[j] > m) m = S_row[j];
    double sum = 0.0;
    for (int64_t j = 0; j < N; ++j)
        if (allowed(mask_mode, i, j)) sum += exp(S_row[j] - m);
    return m + log(sum);
}

/*
 * Full computation with S and G stored explicitly.
 *   loss      : Eq. 1, mean over the B queries of (lse_i - S_{i, r_i})
 *   row_lse   : [B]  lse_i
 *   pos_logit : [B]  S_{i, r_i}
 *   dQ        : [B x d]  Eq. 5 (generalised to any tau: the exact derivative of Eq. 1)
 *   dP        : [N x d]  Eq. 6-7, with eps_j read as the SUM of f(s_k) over all k with r_k = j
 * Any output pointer may be NULL except that gradients need nothing else.
 * Returns 0 on success, a positive code for bad arguments, -1 when out of memory.
 */
int gco_build_cache(const double* Q, const double* P, const int32_t* pos_idx, int64_t B,
                    int64_t N, int64_t d, double tau, int mask_mode, double* loss,
                    double* row_lse, double* pos_logit, double* dQ, double* dP) {
    int rc = check_args(pos_idx, B, N, d, tau, mask_mode);
    if (rc) return rc;
    double* S = (double*)malloc(sizeof(double) * (size_t)B * (size_t)N);
    double* lse = (double*)malloc(sizeof(double) * (size_t)B);
    if (!S || !lse) { free(S); free(lse); return -1; }

    /* S = Q P^T / tau */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < B; ++i) logits_row(Q, P, i, N, d, tau, S + i * N);

    /* lse_i, and the loss of Eq. 1 */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < B; ++i) lse[i] = lse_row(S + i * N, i, N, mask_mode);
    double total = 0.0;
    for (int64_t i = 0; i < B; ++i) total += lse[i] - S[i * N + pos_idx[i]];
    if (loss) *loss = total / (double)B;
    if (row_lse) memcpy(row_lse, lse, sizeof(double) * (size_t)B);
    if (pos_logit)
        for (int64_t i = 0; i < B; ++i) pos_logit[i] = S[i * N + pos_idx[i]];

    if (dQ || dP) {
        /* G_ij = (p_ij - [j == r_i]) / B, with p_ij of Eq. 4 (0 where masked); in place of S */
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < B; ++i) {
            double* row = S + i * N;
            for (int64_t j = 0; j < N; ++j) {
                double p = allowed(mask_mode, i, j) ? exp(row[j] - lse[i]) : 0.0;
                double onehot = (j == pos_idx[i]) ? 1.0 : 0.0;
                row[j] = (p - onehot) / (double)B;
            }
        }
        const double* G = S;
        if (dQ) {
            /* Eq. 5: dL/df(s_i) = (1/tau) sum_j G_ij g(t_j) */
#pragma omp parallel for schedule(static)
            for (int64_t i = 0; i < B; ++i) {
                double* out = dQ + i * d;
                for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
                for (int64_t j = 0; j < N; ++j) {
                    double g = G[i * N + j];
                    const double* p = P + j * d;
                    for (int64_t k = 0; k < d; ++k) out[k] += g * p[k];
                }
                for (int64_t k = 0; k < d; ++k) out[k] /= tau;
            }
        }
        if (dP) {
            /* Eq. 6-7: dL/dg(t_j) = (1/tau) sum_i G_ij f(s_i) */
#pragma omp parallel for schedule(static)
            for (int64_t j = 0; j < N; ++j) {
                double* out = dP + j * d;
                for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
                for (int64_t i = 0; i < B; ++i) {
                    double g = G[i * N + j];
                    const double* q = Q + i * d;
                    for (int64_t k = 0; k < d; ++k) out[k] += g * q[k];
                }
                for (int64_t k = 0; k < d; ++k) out[k] /= tau;
            }
        }
    }
    free(S);
    free(lse);
    return 0;
}

/*
 * Row-sampled variant for sizes where B x N doubles do not fit: for each listed query row i
 * (n_rows of them) compute lse_i, S_{i,r_i} and (optionally) row i of dQ.  Each row needs only
 * its own row of S, held in a per-thread buffer; the arithmetic is the same as above.
 * dQ_rows is [n_rows x d].
 */
int gco_query_rows(const double* Q, const double* P, const int32_t* pos_idx, int64_t B, int64_t N,
                   int64_t d, double tau, int mask_mode, const int64_t* rows, int64_t n_rows,
                   double* row_lse, double* pos_logit, double* dQ_rows) {
    int rc = check_args(pos_idx, B, N, d, tau, mask_mode);
    if (rc) return rc;
    for (int64_t r = 0; r < n_rows; ++r)
        if (rows[r] < 0 || rows[r] >= B) return 6;
    int failed = 0;
#pragma omp parallel
    {
        double* S_row = (double*)malloc(sizeof(double) * (size_t)N);
        if (!S_row) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!S_row) continue;
            int64_t i = rows[r];
            logits_row(Q, P, i, N, d, tau, S_row);
            double lse = lse_row(S_row, i, N, mask_mode);
            if (row_lse) row_lse[r] = lse;
            if (pos_logit) pos_logit[r] = S_row[pos_idx[i]];
            if (dQ_rows) {
                double* out = dQ_rows + r * d;
                for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
                for (int64_t j = 0; j < N; ++j) {
                    double p = allowed(mask_mode, i, j) ? exp(S_row[j] - lse) : 0.0;
                    double g = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / (double)B;
                    const double* pj = P + j * d;
                    for (int64_t k = 0; k < d; ++k) out[k] += g * pj[k];
                }
                for (int64_t k = 0; k < d; ++k) out[k] /= tau;
            }
        }
        free(S_row);
    }
    return failed ? -1 : 0;
}

/*
 * Row-sampled dP: for each listed passage row j compute row j of dP (Eq. 6-7) given lse_i for
 * ALL queries (row_lse, length B, from gco_build_cache or gco_query_rows over every row).
 * dP_rows is [n_rows x d].
 */
int gco_passage_rows(const double* Q, const double* P, const int32_t* pos_idx, int64_t B,
                     int64_t N, int64_t d, double tau, int mask_mode, const double* row_lse,
                     const int64_t* rows, int64_t n_rows, double* dP_rows) {
    int rc = check_args(pos_idx, B, N, d, tau, mask_mode);
    if (rc) return rc;
    for (int64_t r = 0; r < n_rows; ++r)
        if (rows[r] < 0 || rows[r] >= N) return 6;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t j = rows[r];
        const double* pj = P + j * d;
        double* out = dP_rows + r * d;
        for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
        for (int64_t i = 0; i < B; ++i) {
            const double* q = Q + i * d;
            double s = 0.0;
            for (int64_t k = 0; k < d; ++k) s += q[k] * pj[k];
            s /= tau;
            double p = allowed(mask_mode, i, j) ? exp(s - row_lse[i]) : 0.0;
            double g = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / (double)B;
            for (int64_t k = 0; k < d; ++k) out[k] += g * q[k];
        }
        for (int64_t k = 0; k < d; ++k) out[k] /= tau;
    }
    return 0;
}

/*
 * Step 3 for a linear encoder f(s) = W s (Section 3.3, Eq. 8; Eq. 9 for g): the representation
 * gradients u_i of one sub-batch, taken from the cache, are pushed through the encoder's
 * parameters.  For the linear map, d f(s_i) / d W applied to u_i is the outer product u_i s_i^T,
 * so the sub-batch's term of Eq. 8 is
 *
 *     dW[a][b] (+)= sum_i U[i][a] * X[i][b]        U: rows x d (cache slice), X: rows x d_in
 *
 * With accumulate == 0 dW is overwritten (first sub-batch), otherwise the sum is added to it
 * (the outer summation of Eq. 8 over sub-batches).  Pinned by the finite-difference gradient of
 * the full-batch loss with respect to W and by a hand-worked integer example.
 */
int gco_cache_apply(const double* U, const double* X, int64_t rows, int64_t d, int64_t d_in,
                    int accumulate, double* dW) {
    if (!U || !X || !dW || rows <= 0 || d <= 0 || d_in <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < d; ++a) {
        for (int64_t b = 0; b < d_in; ++b) {
            double s = 0.0;
            for (int64_t i = 0; i < rows; ++i) s += U[i * d + a] * X[i * d_in + b];
            if (accumulate) dW[a * d_in + b] += s;
            else dW[a * d_in + b] = s;
        }
    }
    return 0;
}

/*
 * Variants of the loss that the paper leaves to automatic differentiation (Section 3.3, Step 2:
 * any loss on the stored representations works).  Still Step 2: the loss over all B x N pairs
 * and its gradient with respect to every representation, plus the derivative with respect to the
 * temperature.  Everything explicit, in double; S and G stored whole.
 *
 *   cosine != 0      similarity is the cosine: S_ij = <q_i/|q_i|, p_j/|p_j|> / tau.  dQ, dP are
 *                    the gradients with respect to the UN-normalised rows (the Jacobian of the
 *                    normalisation, (I - n n^T)/|x| with n = x/|x|, applied to the gradient with
 *                    respect to the unit rows).
 *   positives        CSR: query i has the positives pos_list[pos_ptr[i] .. pos_ptr[i+1]) (at least
 *                    one, distinct, none on the masked diagonal).  Loss of query i = mean over its
 *                    positives of -log p_ir, so G_ij = (p_ij - [j in R_i]/|R_i|)/B.  One positive
 *                    per query is Eq. 1.
 *   two_direction    (needs exactly one positive per query) L = (L_row + L_col)/2 with L_row =
 *                    Eq. 1 and L_col its mirror image over the same B positive pairs: passage r_i
 *                    is the anchor, the B queries are its candidates,
 *                        L_col = (1/B) sum_i (log sum_{i'} exp(S_{i' r_i}) - S_{i r_i}),
 *                    the sum over i' running over the allowed pairs.  N may exceed B: passages
 *                    that are nobody's positive only appear in the row softmax.
 *   dtau             dL/dtau = -(1/tau) sum_ij G_ij S_ij  (S = <.,.>/tau).
 * Outputs may be NULL.  Returns 0, a positive code for bad arguments, -1 when out of memory.
 * Pinned in tests/test_oracle_variants.py by finite differences with respect to every input and
 * tau, Euler's identity for the joint scaling of Q and tau, orthogonality of the cosine
 * gradients to their rows, the role-swap symmetry of the two-direction loss and reduction to
 * gco_build_cache.
 */
int gco_build_variant(const double* Q, const double* P, const int64_t* pos_ptr,
                      const int32_t* pos_list, int64_t B, int64_t N, int64_t d, double tau,
                      int mask_mode, int cosine, int two_direction, double* loss, double* dQ,
                      double* dP, double* dtau) {
    if (B <= 0 || N <= 0 || d <= 0) return 1;
    if (!(tau > 0.0) || !isfinite(tau)) return 2;
    if (mask_mode != GCO_MASK_NONE && mask_mode != GCO_MASK_SELF) return 3;
    if (pos_ptr[0] != 0) return 4;
    for (int64_t i = 0; i < B; ++i) {
        int64_t n = pos_ptr[i + 1] - pos_ptr[i];
        if (n < 1) return 4;
        if (two_direction && n != 1) return 7;
        for (int64_t a = pos_ptr[i]; a < pos_ptr[i + 1]; ++a) {
            if (pos_list[a] < 0 || pos_list[a] >= N) return 4;
            if (!allowed(mask_mode, i, pos_list[a])) return 5;
            for (int64_t b = pos_ptr[i]; b < a; ++b)
                if (pos_list[b] == pos_list[a]) return 6;
        }
    }
    double* Qn = (double*)malloc(sizeof(double) * (size_t)B * (size_t)d);
    double* Pn = (double*)malloc(sizeof(double) * (size_t)N * (size_t)d);
    double* qnorm = (double*)malloc(sizeof(double) * (size_t)B);
    double* pnorm = (double*)malloc(sizeof(double) * (size_t)N);
    double* S = (double*)malloc(sizeof(double) * (size_t)B * (size_t)N);
    double* G = (double*)malloc(sizeof(double) * (size_t)B * (size_t)N);
    double* gQ = (double*)malloc(sizeof(double) * (size_t)B * (size_t)d);
    double* gP = (double*)malloc(sizeof(double) * (size_t)N * (size_t)d);
    if (!Qn || !Pn || !qnorm || !pnorm || !S || !G || !gQ || !gP) {
        free(Qn); free(Pn); free(qnorm); free(pnorm); free(S); free(G); free(gQ); free(gP);
        return -1;
    }
    /* the rows the similarity is taken of: the inputs, or their unit vectors */
    for (int64_t i = 0; i < B; ++i) {
        double s = 0.0;
        for (int64_t k = 0; k < d; ++k) s += Q[i * d + k] * Q[i * d + k];
        qnorm[i] = cosine ? sqrt(s) : 1.0;
        for (int64_t k = 0; k < d; ++k) Qn[i * d + k] = Q[i * d + k] / qnorm[i];
    }
    for (int64_t j = 0; j < N; ++j) {
        double s = 0.0;
        for (int64_t k = 0; k < d; ++k) s += P[j * d + k] * P[j * d + k];
        pnorm[j] = cosine ? sqrt(s) : 1.0;
        for (int64_t k = 0; k < d; ++k) Pn[j * d + k] = P[j * d + k] / pnorm[j];
    }
    for (int64_t i = 0; i < B; ++i) logits_row(Qn, Pn, i, N, d, tau, S + i * N);

    /* row direction: every query against all passages */
    double total = 0.0;
    for (int64_t i = 0; i < B; ++i) {
        const double lse = lse_row(S + i * N, i, N, mask_mode);
        const int64_t np = pos_ptr[i + 1] - pos_ptr[i];
        for (int64_t j = 0; j < N; ++j)
            G[i * N + j] = (allowed(mask_mode, i, j) ? exp(S[i * N + j] - lse) : 0.0) / (double)B;
        for (int64_t a = pos_ptr[i]; a < pos_ptr[i + 1]; ++a) {
            total += (lse - S[i * N + pos_list[a]]) / (double)np;
            G[i * N + pos_list[a]] -= 1.0 / ((double)np * (double)B);
        }
    }
    double L = total / (double)B;

    if (two_direction) {
        /* column direction: the positive passage of query i against all queries */
        double total_c = 0.0;
        for (int64_t i = 0; i < B; ++i) {
            const int64_t j = pos_list[pos_ptr[i]];
            double m = -INFINITY;
            for (int64_t k = 0; k < B; ++k)
                if (allowed(mask_mode, k, j) && S[k * N + j] > m) m = S[k * N + j];
            double sum = 0.0;
            for (int64_t k = 0; k < B; ++k)
                if (allowed(mask_mode, k, j)) sum += exp(S[k * N + j] - m);
            const double lse_c = m + log(sum);
            total_c += lse_c - S[i * N + j];
            /* d/dS of this term: softmax over the column, minus one at (i, j); both halves
             * of the loss weigh 1/2 */
            for (int64_t k = 0; k < B; ++k) {
                double pc = allowed(mask_mode, k, j) ? exp(S[k * N + j] - lse_c) : 0.0;
                G[k * N + j] += pc / (double)B;
            }
            G[i * N + j] -= 1.0 / (double)B;
        }
        L = 0.5 * (L + total_c / (double)B);
        for (int64_t e = 0; e < B * N; ++e) G[e] *= 0.5;
    }
    if (loss) *loss = L;

    /* gradients with respect to the rows the similarity saw, and with respect to tau */
    for (int64_t i = 0; i < B; ++i)
        for (int64_t k = 0; k < d; ++k) {
            double s = 0.0;
            for (int64_t j = 0; j < N; ++j) s += G[i * N + j] * Pn[j * d + k];
            gQ[i * d + k] = s / tau;
        }
    for (int64_t j = 0; j < N; ++j)
        for (int64_t k = 0; k < d; ++k) {
            double s = 0.0;
            for (int64_t i = 0; i < B; ++i) s += G[i * N + j] * Qn[i * d + k];
            gP[j * d + k] = s / tau;
        }
    if (dtau) {
        double s = 0.0;
        for (int64_t e = 0; e < B * N; ++e) s += G[e] * S[e];
        *dtau = -s / tau;
    }
    /* back through the normalisation: dx = (g - n <n, g>) / |x| */
    if (dQ)
        for (int64_t i = 0; i < B; ++i) {
            double dot = 0.0;
            for (int64_t k = 0; k < d; ++k) dot += Qn[i * d + k] * gQ[i * d + k];
            for (int64_t k = 0; k < d; ++k)
                dQ[i * d + k] = cosine ? (gQ[i * d + k] - Qn[i * d + k] * dot) / qnorm[i]
                                       : gQ[i * d + k];
        }
    if (dP)
        for (int64_t j = 0; j < N; ++j) {
            double dot = 0.0;
            for (int64_t k = 0; k < d; ++k) dot += Pn[j * d + k] * gP[j * d + k];
            for (int64_t k = 0; k < d; ++k)
                dP[j * d + k] = cosine ? (gP[j * d + k] - Pn[j * d + k] * dot) / pnorm[j]
                                       : gP[j * d + k];
        }
    free(Qn); free(Pn); free(qnorm); free(pnorm); free(S); free(G); free(gQ); free(gP);
    return 0;
}

/*
 * Distance Gradient Cache (Section 5, Eq. 10-13).  The similarity is a general distance
 * d_ij = Phi(f(s_i), g(t_j)); the loss is Eq. 1 with d_ij / tau as the logit of pair (i, j).
 *
 *   gco_dist_loss   the loss as a function of the B x N matrix of distances D, and lse_i.
 *   gco_dist_w      the Distance Gradient Cache w_ij = dL/dd_ij = (p_ij - [j == r_i]) / (B tau),
 *                   p the row softmax of D / tau over the allowed pairs (0 where masked).
 * With these, Eq. 11 is dL/dOmega = sum_ij w_ij dPhi_ij/dOmega and Eq. 12-13 are u_i = sum_j w_ij
 * dd_ij/df(s_i), v_j = sum_i w_ij dd_ij/dg(t_j); for the dot product d_ij = <f_i, g_j> they reduce
 * to Eq. 5-7.  Pinned in tests/test_oracle_distance.py.
 */
int gco_dist_loss(const double* D, const int32_t* pos_idx, int64_t B, int64_t N, double tau,
                  int mask_mode, double* loss, double* row_lse) {
    int rc = check_args(pos_idx, B, N, 1, tau, mask_mode);
    if (rc) return rc;
    double total = 0.0;
    for (int64_t i = 0; i < B; ++i) {
        double m = -INFINITY;
        for (int64_t j = 0; j < N; ++j)
            if (allowed(mask_mode, i, j) && D[i * N + j] / tau > m) m = D[i * N + j] / tau;
        double sum = 0.0;
        for (int64_t j = 0; j < N; ++j)
            if (allowed(mask_mode, i, j)) sum += exp(D[i * N + j] / tau - m);
        const double lse = m + log(sum);
        if (row_lse) row_lse[i] = lse;
        total += lse - D[i * N + pos_idx[i]] / tau;
    }
    if (loss) *loss = total / (double)B;
    return 0;
}

int gco_dist_w(const double* D, const int32_t* pos_idx, int64_t B, int64_t N, double tau,
               int mask_mode, double* W) {
    int rc = check_args(pos_idx, B, N, 1, tau, mask_mode);
    if (rc) return rc;
    double* lse = (double*)malloc(sizeof(double) * (size_t)B);
    if (!lse) return -1;
    rc = gco_dist_loss(D, pos_idx, B, N, tau, mask_mode, NULL, lse);
    for (int64_t i = 0; i < B && !rc; ++i)
        for (int64_t j = 0; j < N; ++j) {
            double p = allowed(mask_mode, i, j) ? exp(D[i * N + j] / tau - lse[i]) : 0.0;
            W[i * N + j] = (p - ((j == pos_idx[i]) ? 1.0 : 0.0)) / ((double)B * tau);
        }
    free(lse);
    return rc;
}
