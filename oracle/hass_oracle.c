/*
 * fp64 CPU oracle for the fused LM-head + Top-K distillation loss of HASS
 * (Harmonized Objective Distillation, Section 3.1, Eq. 1) and its gradient with
 * respect to the draft features.
 *
 * THIS IS TEST INFRASTRUCTURE. It is slow on purpose, shares no code with the
 * CUDA library and must never be called from the product path. Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Per row i (rows are independent), in the paper's notation (q: target LLM's
 * next-token distribution, p: draft model's, Omega: vocabulary, Omega_hat: the K
 * tokens with the highest target probability):
 *
 *   step 1  z_t[v] = sum_k H_t[i,k] W[v,k],  z_d[v] = sum_k H_d[i,k] W[v,k]
 *           (the shared LM head applied to target and draft features; training listing of the
 *            appendix "Implementation of Harmonized Context Alignment":
 *            lm_head(hidden_states_target), lm_head(predict))
 *   step 2  q = softmax(z_t), p = softmax(z_d) over the whole vocabulary (Eq. 1: q and p
 *           are next-token probability distributions; they are NOT renormalised over
 *           Omega_hat - that is the separate "Normed Top-K" variant of Section 4.3)
 *   step 3  Omega_hat = K largest q (Section 3.1), by a full sort on (-z_t, index):
 *           ties go to the lower index
 *   step 4  L = - sum_{x in Omega_hat} q(x) log p(x)                        (Eq. 1)
 *   step 5  dL/dz_d[v] = g (S_q p[v] - q[v] [v in Omega_hat]),  S_q = sum_{x in Omega_hat} q(x)
 *           dH_d[i,:] = sum_v dL/dz_d[v] W[v,:]
 *           (derivative of Eq. 1 with q and Omega_hat constant: the target side needs no
 *            gradient, Appendix "Training Overhead"; g is the upstream weight of row i)
 *
 * Combined objective (Section 3.2: the training objective of one aligning step is the cross-entropy
 * between the target's and the draft's next-token distributions plus auxiliary terms, one of which is the
 * Top-K loss with weight w, Section 4.1): the *_objective entries also return
 *   L_CE = - sum_{x in Omega} q(x) log p(x)
 * and differentiate  w_ce L_CE + w_topk L_TopK:
 *   dL/dz_d[v] = g ( w_ce (p[v] - q[v]) + w_topk (S_q p[v] - q[v] [v in Omega_hat]) ).
 * The plain entries are the case w_ce = 0, w_topk = 1.
 *
 * Loss variants of Section 4.3 (the paper describes them in one sentence each; the readings are this
 * file's), selected by `variant` in the *_variant entries, all with q and Omega_hat constant:
 *   1  Top-P:        Omega_hat = the shortest prefix of the tokens sorted by descending q whose cumulative
 *                    probability is larger than P, at most K tokens; loss and gradient as Eq. 1 on that set.
 *   2  Normed Top-K: q and p are both renormalised over Omega_hat (linear normalisation of the
 *                    probabilities, which equals a softmax over the logits restricted to Omega_hat):
 *                    L = - sum_{x in Omega_hat} qn(x) log pn(x), qn = q / S_q, pn = p / S_p;
 *                    dL/dz_d[x] = g (pn(x) - qn(x)) on Omega_hat and 0 elsewhere.
 *   3  Bi-directional Top-K: Omega_hat = (K most probable tokens under q) united with (K most probable
 *                    under p); loss and gradient as Eq. 1 on that set, the set being a constant:
 *                    L = - sum_{x in U} q(x) log p(x), dL/dz_d[v] = g (S_U p[v] - q[v] [v in U]).
 *                    idx / q_k then hold up to 2K entries: the target's K in descending q, followed by the
 *                    draft's tokens that are not among them in descending p.
 *
 * Inputs of the feature-level entry are bf16 bit patterns widened exactly to fp64.
 * The only liberty taken with summation order is SIMD reassociation of the inner
 * dot-product loop (omp simd reduction), i.e. rounding order.
 *
 * Pins (tests/test_oracle_pins.py): K = V reduces to soft-target cross-entropy
 * (library log_softmax), one-hot target gives NLL, shift invariances, brute-force
 * subset enumeration with a literal unshifted Eq. 1, finite differences, and an
 * autograd restatement. Every function here is pinned by at least one of them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#if defined(__x86_64__) && defined(__GNUC__) && !defined(__clang__)
#define HASS_CLONES __attribute__((target_clones("avx512f", "avx2,fma", "default")))
#else
#define HASS_CLONES
#endif

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int hass_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- step 1 helpers ------------------------------------------------------- */

HASS_CLONES
static void dot2(const double* a, const double* b, const double* w, int64_t d, double* out_a,
                 double* out_b) {
    double sa = 0.0, sb = 0.0;
#pragma omp simd reduction(+ : sa, sb)
    for (int64_t k = 0; k < d; ++k) {
        sa += a[k] * w[k];
        sb += b[k] * w[k];
    }
    *out_a = sa;
    *out_b = sb;
}

HASS_CLONES
static void axpy(double alpha, const double* w, double* y, int64_t d) {
    for (int64_t k = 0; k < d; ++k) y[k] += alpha * w[k];
}

HASS_CLONES
static void widen_bf16(const uint16_t* src, double* dst, int64_t d) {
    for (int64_t k = 0; k < d; ++k) dst[k] = bf16_to_f64(src[k]);
}

/* ---- steps 2-5 on given logits ------------------------------------------------ */

typedef struct {
    double z;
    int32_t v;
} zi_t;

static int cmp_desc(const void* pa, const void* pb) {
    const zi_t* a = (const zi_t*)pa;
    const zi_t* b = (const zi_t*)pb;
    if (a->z > b->z) return -1;
    if (a->z < b->z) return 1;
    return (a->v > b->v) - (a->v < b->v);
}

static double log_sum_exp(const double* z, int64_t V) {
    double m = z[0];
    for (int64_t v = 1; v < V; ++v)
        if (z[v] > m) m = z[v];
    double s = 0.0;
    for (int64_t v = 0; v < V; ++v) s += exp(z[v] - m);
    return m + log(s);
}

/*
 * Steps 2-5 for one row from its logits.
 *   forced_idx  NULL: Omega_hat is the top-K of z_t (step 3). Otherwise K indices that are
 *               taken as Omega_hat as given (used to score a row whose K-th and (K+1)-th
 *               target logits are a near-tie on a set the caller supplies).
 *   idx, q_k    [K] out: Omega_hat in descending q (ties: lower index first) and q there.
 *   dz_d        [V] out or NULL.
 * Returns 0, or -1 on bad arguments.
 */
int hass_oracle_row_objective(const double* z_t, const double* z_d, int64_t V, int32_t K, double g, double w_ce,
                              double w_topk, const int32_t* forced_idx, double* loss_ce, double* loss, int32_t* idx,
                              double* q_k, double* lse_t_out, double* lse_d_out, double* dz_d) {
    if (V < 1 || K < 1 || K > V) return -1;
    const double lse_t = log_sum_exp(z_t, V);
    const double lse_d = log_sum_exp(z_d, V);

    zi_t* order = NULL;
    if (forced_idx) {
        order = (zi_t*)malloc(sizeof(zi_t) * (size_t)K);
        for (int32_t j = 0; j < K; ++j) {
            if (forced_idx[j] < 0 || forced_idx[j] >= V) {
                free(order);
                return -1;
            }
            order[j].z = z_t[forced_idx[j]];
            order[j].v = forced_idx[j];
        }
        qsort(order, (size_t)K, sizeof(zi_t), cmp_desc);
    } else {
        order = (zi_t*)malloc(sizeof(zi_t) * (size_t)V);
        for (int64_t v = 0; v < V; ++v) {
            order[v].z = z_t[v];
            order[v].v = (int32_t)v;
        }
        qsort(order, (size_t)V, sizeof(zi_t), cmp_desc);
    }

    double S_q = 0.0, L = 0.0;
    for (int32_t j = 0; j < K; ++j) {
        const int32_t x = order[j].v;
        const double q = exp(z_t[x] - lse_t);
        const double logp = z_d[x] - lse_d;
        idx[j] = x;
        q_k[j] = q;
        S_q += q;
        L -= q * logp;
    }
    *loss = L;
    if (lse_t_out) *lse_t_out = lse_t;
    if (lse_d_out) *lse_d_out = lse_d;
    if (loss_ce) {
        /* full-vocabulary cross-entropy between q and p */
        double ce = 0.0;
        for (int64_t v = 0; v < V; ++v) ce -= exp(z_t[v] - lse_t) * (z_d[v] - lse_d);
        *loss_ce = ce;
    }

    if (dz_d) {
        for (int64_t v = 0; v < V; ++v) {
            const double p = exp(z_d[v] - lse_d);
            const double q = exp(z_t[v] - lse_t);
            dz_d[v] = g * (w_ce * (p - q) + w_topk * S_q * p);
        }
        for (int32_t j = 0; j < K; ++j) dz_d[idx[j]] -= g * w_topk * q_k[j];
    }
    free(order);
    return 0;
}

/*
 * Loss variants (see the header). variant 0 = Eq. 1, 1 = Top-P (param = P, K = cap), 2 = Normed Top-K.
 * n_out receives |Omega_hat|; idx / q_k beyond it are -1 / 0.
 */
int hass_oracle_row_variant(const double* z_t, const double* z_d, int64_t V, int32_t K, double g, int variant,
                            double param, double* loss, int32_t* idx, double* q_k, int32_t* n_out,
                            double* lse_t_out, double* lse_d_out, double* dz_d) {
    if (variant < 0 || variant > 3) return -1;
    if (variant == 3) {
        /* union of the two Top-K sets; idx and q_k have room for 2K entries */
        double l0, lt, ld;
        int32_t* it = (int32_t*)malloc(sizeof(int32_t) * (size_t)K * 2);
        double* qt = (double*)malloc(sizeof(double) * (size_t)K * 2);
        int rc3 = hass_oracle_row_objective(z_t, z_d, V, K, g, 0.0, 1.0, NULL, NULL, &l0, it, qt, &lt, &ld, NULL);
        if (rc3 == 0) /* the draft's own Top-K: the same selection with the roles of the logits exchanged */
            rc3 = hass_oracle_row_objective(z_d, z_d, V, K, g, 0.0, 1.0, NULL, NULL, &l0, it + K, qt + K, NULL, NULL, NULL);
        if (rc3 != 0) {
            free(it);
            free(qt);
            return rc3;
        }
        int32_t n = 0;
        double S_U = 0.0, L = 0.0;
        for (int32_t j = 0; j < 2 * K; ++j) {
            int dup = 0;
            for (int32_t i = 0; i < n; ++i) dup |= (idx[i] == it[j]);
            if (dup) continue;
            idx[n] = it[j];
            q_k[n] = exp(z_t[it[j]] - lt);
            S_U += q_k[n];
            L -= q_k[n] * (z_d[it[j]] - ld);
            ++n;
        }
        for (int32_t j = n; j < 2 * K; ++j) {
            idx[j] = -1;
            q_k[j] = 0.0;
        }
        *loss = L;
        if (lse_t_out) *lse_t_out = lt;
        if (lse_d_out) *lse_d_out = ld;
        if (dz_d) {
            for (int64_t v = 0; v < V; ++v) dz_d[v] = g * S_U * exp(z_d[v] - ld);
            for (int32_t j = 0; j < n; ++j) dz_d[idx[j]] -= g * q_k[j];
        }
        if (n_out) *n_out = n;
        free(it);
        free(qt);
        return 0;
    }
    int rc = hass_oracle_row_objective(z_t, z_d, V, K, g, 0.0, 1.0, NULL, NULL, loss, idx, q_k, lse_t_out, lse_d_out,
                                       variant == 0 ? dz_d : NULL);
    if (rc != 0) return rc;
    int32_t n = K;
    if (variant == 0) {
        if (n_out) *n_out = n;
        return 0;
    }
    const double lse_d = log_sum_exp(z_d, V);
    if (variant == 1) {
        /* shortest sorted prefix whose cumulative target probability is larger than P */
        double cum = 0.0;
        n = 0;
        while (n < K) {
            cum += q_k[n];
            ++n;
            if (cum > param) break;
        }
        double S_q = 0.0, L = 0.0;
        for (int32_t j = 0; j < n; ++j) {
            S_q += q_k[j];
            L -= q_k[j] * (z_d[idx[j]] - lse_d);
        }
        *loss = L;
        if (dz_d) {
            for (int64_t v = 0; v < V; ++v) dz_d[v] = g * S_q * exp(z_d[v] - lse_d);
            for (int32_t j = 0; j < n; ++j) dz_d[idx[j]] -= g * q_k[j];
        }
        for (int32_t j = n; j < K; ++j) {
            idx[j] = -1;
            q_k[j] = 0.0;
        }
    } else {
        /* both distributions renormalised over Omega_hat */
        double S_q = 0.0, m = z_d[idx[0]];
        for (int32_t j = 0; j < K; ++j) {
            S_q += q_k[j];
            if (z_d[idx[j]] > m) m = z_d[idx[j]];
        }
        double se = 0.0;
        for (int32_t j = 0; j < K; ++j) se += exp(z_d[idx[j]] - m);
        const double lse_k = m + log(se);
        double L = 0.0;
        for (int32_t j = 0; j < K; ++j) L -= (q_k[j] / S_q) * (z_d[idx[j]] - lse_k);
        *loss = L;
        if (dz_d) {
            for (int64_t v = 0; v < V; ++v) dz_d[v] = 0.0;
            for (int32_t j = 0; j < K; ++j) dz_d[idx[j]] = g * (exp(z_d[idx[j]] - lse_k) - q_k[j] / S_q);
        }
    }
    if (n_out) *n_out = n;
    return 0;
}

/*
 * Eq. 1 (normed = 0) or the Normed Top-K loss (normed = 1) of one row on a GIVEN token set: the sum of Eq. 1
 * runs over `set` (n distinct token ids) instead of over a selection made here. Used to score a row on a set
 * that a caller found by other means, when two selections are equally valid (a near-tie at the K-th place).
 *   q_set  [n] out: q at the set's tokens, in the given order.
 * Returns 0, or -1 on bad arguments (empty set, id out of range, repeated id).
 */
int hass_oracle_row_on_set(const double* z_t, const double* z_d, int64_t V, const int32_t* set, int32_t n, double g,
                           int normed, double* loss, double* q_set, double* lse_t_out, double* lse_d_out,
                           double* dz_d) {
    if (V < 1 || n < 1 || n > V) return -1;
    for (int32_t j = 0; j < n; ++j) {
        if (set[j] < 0 || set[j] >= V) return -1;
        for (int32_t i = 0; i < j; ++i)
            if (set[i] == set[j]) return -1;
    }
    const double lse_t = log_sum_exp(z_t, V);
    const double lse_d = log_sum_exp(z_d, V);
    if (lse_t_out) *lse_t_out = lse_t;
    if (lse_d_out) *lse_d_out = lse_d;
    double S = 0.0;
    for (int32_t j = 0; j < n; ++j) {
        q_set[j] = exp(z_t[set[j]] - lse_t);
        S += q_set[j];
    }
    double L = 0.0;
    if (!normed) {
        for (int32_t j = 0; j < n; ++j) L -= q_set[j] * (z_d[set[j]] - lse_d);
        if (dz_d) {
            for (int64_t v = 0; v < V; ++v) dz_d[v] = g * S * exp(z_d[v] - lse_d);
            for (int32_t j = 0; j < n; ++j) dz_d[set[j]] -= g * q_set[j];
        }
    } else {
        double m = z_d[set[0]];
        for (int32_t j = 1; j < n; ++j)
            if (z_d[set[j]] > m) m = z_d[set[j]];
        double se = 0.0;
        for (int32_t j = 0; j < n; ++j) se += exp(z_d[set[j]] - m);
        const double lse_k = m + log(se);
        for (int32_t j = 0; j < n; ++j) L -= (q_set[j] / S) * (z_d[set[j]] - lse_k);
        if (dz_d) {
            for (int64_t v = 0; v < V; ++v) dz_d[v] = 0.0;
            for (int32_t j = 0; j < n; ++j) dz_d[set[j]] = g * (exp(z_d[set[j]] - lse_k) - q_set[j] / S);
        }
    }
    *loss = L;
    return 0;
}

/* Feature-level loss variants for a set of rows (bf16 bit patterns); outputs as hass_oracle_features plus n.
 * forced_idx: NULL, or [n_rows, kk] (kk = 2K for variant 3, else K) token sets to score instead of the
 * oracle's own selection: a row's entries >= 0 are its Omega_hat (hass_oracle_row_on_set); idx repeats them. */
int hass_oracle_features_variant(const uint16_t* H_t, const uint16_t* H_d, const uint16_t* W, int64_t N, int64_t d,
                                 int64_t V, int32_t K, int variant, double param, const double* grad_loss,
                                 const int64_t* rows, int64_t n_rows, const int32_t* forced_idx, double* loss,
                                 int32_t* idx, double* q_k, int32_t* n_out, double* lse_t, double* lse_d,
                                 double* dH_d) {
    if (N < 1 || d < 1 || V < 1 || K < 1 || K > V || n_rows < 0 || !rows) return -1;
    int status = 0;
#pragma omp parallel
    {
        double* ht = (double*)malloc(sizeof(double) * (size_t)d);
        double* hd = (double*)malloc(sizeof(double) * (size_t)d);
        double* wr = (double*)malloc(sizeof(double) * (size_t)d);
        double* zt = (double*)malloc(sizeof(double) * (size_t)V);
        double* zd = (double*)malloc(sizeof(double) * (size_t)V);
        double* dz = (double*)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t i = rows[r];
            if (i < 0 || i >= N) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            const double g = grad_loss ? grad_loss[i] : 1.0;
            widen_bf16(H_t + i * d, ht, d);
            widen_bf16(H_d + i * d, hd, d);
            for (int64_t v = 0; v < V; ++v) {
                widen_bf16(W + v * d, wr, d);
                dot2(ht, hd, wr, d, &zt[v], &zd[v]);
            }
            const int64_t kk = variant == 3 ? 2 * (int64_t)K : K;   /* entries per row of idx / q_k */
            int rc;
            if (forced_idx) {
                int32_t n = 0;
                for (int64_t j = 0; j < kk; ++j) {
                    idx[r * kk + j] = -1;
                    q_k[r * kk + j] = 0.0;
                }
                for (int64_t j = 0; j < kk; ++j)
                    if (forced_idx[r * kk + j] >= 0) idx[r * kk + n++] = forced_idx[r * kk + j];
                n_out[r] = n;
                rc = hass_oracle_row_on_set(zt, zd, V, idx + r * kk, n, g, variant == 2, &loss[r], q_k + r * kk,
                                            &lse_t[r], &lse_d[r], dz);
            } else {
                rc = hass_oracle_row_variant(zt, zd, V, K, g, variant, param, &loss[r], idx + r * kk, q_k + r * kk,
                                             &n_out[r], &lse_t[r], &lse_d[r], dz);
            }
            if (rc != 0) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            double* out = dH_d + r * d;
            for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
            for (int64_t v = 0; v < V; ++v) {
                if (dz[v] == 0.0) continue;
                widen_bf16(W + v * d, wr, d);
                axpy(dz[v], wr, out, d);
            }
        }
        free(ht);
        free(hd);
        free(wr);
        free(zt);
        free(zd);
        free(dz);
    }
    return status;
}

int hass_oracle_row_from_logits(const double* z_t, const double* z_d, int64_t V, int32_t K, double g,
                                const int32_t* forced_idx, double* loss, int32_t* idx, double* q_k,
                                double* lse_t_out, double* lse_d_out, double* dz_d) {
    return hass_oracle_row_objective(z_t, z_d, V, K, g, 0.0, 1.0, forced_idx, NULL, loss, idx, q_k, lse_t_out,
                                     lse_d_out, dz_d);
}

/* ---- feature-level entries -------------------------------------------------------- */

/*
 * Steps 1-5 for a set of rows.
 *   elem_bytes  2: H_t, H_d, W hold bf16 bit patterns; 8: they hold doubles.
 *   rows        NULL (all N rows, n_rows == N) or n_rows row numbers into H_t / H_d.
 *   grad_loss   NULL (g = 1) or [N] upstream weights, indexed by the original row number.
 *   forced_idx  NULL or [n_rows, K].
 * Outputs are indexed by position in `rows`: loss, lse_t, lse_d [n_rows]; idx, q_k [n_rows, K];
 * dH_d [n_rows, d] (may be NULL to skip step 5's back-projection).
 */
int hass_oracle_features_objective(const void* H_t, const void* H_d, const void* W, int elem_bytes, int64_t N,
                                   int64_t d, int64_t V, int32_t K, double w_ce, double w_topk,
                                   const double* grad_loss, const int64_t* rows, int64_t n_rows,
                                   const int32_t* forced_idx, double* loss_ce, double* loss, int32_t* idx,
                                   double* q_k, double* lse_t, double* lse_d, double* dH_d) {
    if (N < 1 || d < 1 || V < 1 || K < 1 || K > V || n_rows < 0) return -1;
    if (elem_bytes != 2 && elem_bytes != 8) return -1;
    if (!rows && n_rows != N) return -1;
    for (int64_t r = 0; r < n_rows; ++r)
        if (rows && (rows[r] < 0 || rows[r] >= N)) return -1;
    int status = 0;

#pragma omp parallel
    {
        double* ht = (double*)malloc(sizeof(double) * (size_t)d);
        double* hd = (double*)malloc(sizeof(double) * (size_t)d);
        double* wr = (double*)malloc(sizeof(double) * (size_t)d);
        double* zt = (double*)malloc(sizeof(double) * (size_t)V);
        double* zd = (double*)malloc(sizeof(double) * (size_t)V);
        double* dz = (double*)malloc(sizeof(double) * (size_t)V);

#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t i = rows ? rows[r] : r;
            const double g = grad_loss ? grad_loss[i] : 1.0;
            if (elem_bytes == 2) {
                widen_bf16((const uint16_t*)H_t + i * d, ht, d);
                widen_bf16((const uint16_t*)H_d + i * d, hd, d);
            } else {
                memcpy(ht, (const double*)H_t + i * d, sizeof(double) * (size_t)d);
                memcpy(hd, (const double*)H_d + i * d, sizeof(double) * (size_t)d);
            }
            /* step 1 */
            for (int64_t v = 0; v < V; ++v) {
                const double* w;
                if (elem_bytes == 2) {
                    widen_bf16((const uint16_t*)W + v * d, wr, d);
                    w = wr;
                } else {
                    w = (const double*)W + v * d;
                }
                dot2(ht, hd, w, d, &zt[v], &zd[v]);
            }
            /* steps 2-5 on the logits */
            int rc = hass_oracle_row_objective(zt, zd, V, K, g, w_ce, w_topk, forced_idx ? forced_idx + r * K : NULL,
                                               loss_ce ? &loss_ce[r] : NULL, &loss[r], idx + r * K, q_k + r * K,
                                               &lse_t[r], &lse_d[r], dH_d ? dz : NULL);
            if (rc != 0) {
#pragma omp atomic write
                status = -1;
                continue;
            }
            /* step 5: back-projection through the LM head */
            if (dH_d) {
                double* out = dH_d + r * d;
                for (int64_t k = 0; k < d; ++k) out[k] = 0.0;
                for (int64_t v = 0; v < V; ++v) {
                    const double* w;
                    if (elem_bytes == 2) {
                        widen_bf16((const uint16_t*)W + v * d, wr, d);
                        w = wr;
                    } else {
                        w = (const double*)W + v * d;
                    }
                    axpy(dz[v], w, out, d);
                }
            }
        }
        free(ht);
        free(hd);
        free(wr);
        free(zt);
        free(zd);
        free(dz);
    }
    return status;
}

int hass_oracle_features(const void* H_t, const void* H_d, const void* W, int elem_bytes, int64_t N,
                         int64_t d, int64_t V, int32_t K, const double* grad_loss, const int64_t* rows,
                         int64_t n_rows, const int32_t* forced_idx, double* loss, int32_t* idx,
                         double* q_k, double* lse_t, double* lse_d, double* dH_d) {
    return hass_oracle_features_objective(H_t, H_d, W, elem_bytes, N, d, V, K, 0.0, 1.0, grad_loss, rows, n_rows,
                                          forced_idx, NULL, loss, idx, q_k, lse_t, lse_d, dH_d);
}

/* Step 1 for selected (row, token) pairs: z[j] = sum_k H[row_j, k] W[tok_j, k], bf16 inputs.
 * The parity comparator uses it to look up target logits of tokens the GPU selected. */
int hass_oracle_logits_at(const uint16_t* H, const uint16_t* W, int64_t N, int64_t d, int64_t V,
                          const int64_t* row, const int32_t* tok, int64_t n, double* z) {
    for (int64_t j = 0; j < n; ++j) {
        if (row[j] < 0 || row[j] >= N || tok[j] < 0 || tok[j] >= V) return -1;
        double s = 0.0;
        for (int64_t k = 0; k < d; ++k)
            s += bf16_to_f64(H[row[j] * d + k]) * bf16_to_f64(W[(int64_t)tok[j] * d + k]);
        z[j] = s;
    }
    return 0;
}
