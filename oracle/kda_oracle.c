/*
 * KDA oracle: the token-by-token recurrence in fp64.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked against.  Only the
 * tests, the smoke check and the CPU-baseline leg of the benchmark may build, load or call it; it
 * shares no code, header, table or helper with the CUDA path and the product never routes through
 * it.
 *
 * What it computes (Kimi Linear paper, Section 3, Eq. 1), per sequence n and head h independently,
 * with S a dk x dv matrix:
 *
 *     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T ,   o_t = S_t^T q_t
 *
 * written out as: decay the rows of S by alpha_t = exp(log_alpha_t); form the residual
 * r = v_t - S^T k_t against the *decayed* state; add the rank-one term beta_t k_t r^T; read the
 * output from the *updated* state.  The chunkwise algorithm of Section 3.1 is an exact regrouping
 * of this recurrence (Appendix B proves it), so this definition is the expected result of the
 * chunk kernel as well as of the decode kernel.
 *
 * Inputs are float arrays holding the exact stored values (bf16 values widen exactly to float);
 * every operation below is carried out in double.
 *
 * Layouts (d contiguous):  q,k,log_alpha [T_total,H,dk]  v,o [T_total,H,dv]  beta [T_total,H]
 *                          S0,S_T [n_seqs,H,dk,dv]        cu_seqlens [n_seqs+1] (token offsets)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* One token of Eq. 1 on one head's state S (dk x dv, row-major).  o may be NULL. */
static void kda_token_step(double *S, const float *q, const float *k, const float *v,
                           const float *log_alpha, double beta, double scale, int dk, int dv,
                           double *r, double *o)
{
    /* Diag(alpha_t) S_{t-1}: row i of S is scaled by alpha_{t,i}. */
    for (int i = 0; i < dk; ++i) {
        double a = exp((double)log_alpha[i]);
        double *Si = S + (size_t)i * dv;
        for (int j = 0; j < dv; ++j) Si[j] *= a;
    }
    /* r = v_t - (decayed S)^T k_t */
    for (int j = 0; j < dv; ++j) r[j] = (double)v[j];
    for (int i = 0; i < dk; ++i) {
        double ki = (double)k[i];
        const double *Si = S + (size_t)i * dv;
        for (int j = 0; j < dv; ++j) r[j] -= ki * Si[j];
    }
    /* S_t = decayed S + beta_t k_t r^T   ( = (I - beta k k^T) Diag(alpha) S + beta k v^T ) */
    for (int i = 0; i < dk; ++i) {
        double bk = beta * (double)k[i];
        double *Si = S + (size_t)i * dv;
        for (int j = 0; j < dv; ++j) Si[j] += bk * r[j];
    }
    /* o_t = scale * S_t^T q_t */
    if (o) {
        for (int j = 0; j < dv; ++j) o[j] = 0.0;
        for (int i = 0; i < dk; ++i) {
            double qi = (double)q[i];
            const double *Si = S + (size_t)i * dv;
            for (int j = 0; j < dv; ++j) o[j] += qi * Si[j];
        }
        for (int j = 0; j < dv; ++j) o[j] *= scale;
    }
}

/*
 * Whole sequences (Eq. 1 applied to every token in order).
 *   S0   : initial states or NULL (= zeros)
 *   o    : [T_total,H,dv] or NULL
 *   S_T  : final states or NULL
 *   cu_seqlens : n_seqs+1 token offsets, cu[0] = 0, non-decreasing
 * Returns 0, or -1 on a bad argument / failed allocation.
 */
int kda_oracle_recurrence(const float *q, const float *k, const float *v, const float *log_alpha,
                          const float *beta, const double *S0, double *o, double *S_T,
                          const int64_t *cu_seqlens, int n_seqs, int H, int dk, int dv,
                          double scale, int n_threads)
{
    if (!k || !v || !log_alpha || !beta || !cu_seqlens || n_seqs < 0 || H <= 0 || dk <= 0 || dv <= 0)
        return -1;
    if (o && !q) return -1;
    int failed = 0;
    long n_items = (long)n_seqs * H;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (long item = 0; item < n_items; ++item) {
        int n = (int)(item / H), h = (int)(item % H);
        double *S = (double *)malloc(sizeof(double) * dk * dv);
        double *r = (double *)malloc(sizeof(double) * dv);
        if (!S || !r) {
            failed = 1;
            free(S);
            free(r);
            continue;
        }
        size_t sofs = ((size_t)n * H + h) * dk * dv;
        if (S0) memcpy(S, S0 + sofs, sizeof(double) * dk * dv);
        else memset(S, 0, sizeof(double) * dk * dv);
        for (int64_t t = cu_seqlens[n]; t < cu_seqlens[n + 1]; ++t) {
            size_t th = (size_t)t * H + h;
            kda_token_step(S, q ? q + th * dk : NULL, k + th * dk, v + th * dv,
                           log_alpha + th * dk, (double)beta[th], scale, dk, dv, r,
                           o ? o + th * dv : NULL);
        }
        if (S_T) memcpy(S_T + sofs, S, sizeof(double) * dk * dv);
        free(S);
        free(r);
    }
    return failed ? -1 : 0;
}

/*
 * One decode step (the body of the recurrence once per sequence and head), state updated in place.
 *   q,k,log_alpha [n_seqs,H,dk]   v,o [n_seqs,H,dv]   beta [n_seqs,H]
 *   S [n_slots,H,dk,dv]; sequence n uses slot state_slot[n] (or n when state_slot is NULL)
 */
int kda_oracle_decode_step(const float *q, const float *k, const float *v, const float *log_alpha,
                           const float *beta, double *S, const int32_t *state_slot, double *o,
                           int n_seqs, int H, int dk, int dv, double scale, int n_threads)
{
    if (!q || !k || !v || !log_alpha || !beta || !S || !o || n_seqs < 0 || H <= 0) return -1;
    int failed = 0;
    long n_items = (long)n_seqs * H;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(static)
    for (long item = 0; item < n_items; ++item) {
        int n = (int)(item / H), h = (int)(item % H);
        double *r = (double *)malloc(sizeof(double) * dv);
        if (!r) {
            failed = 1;
            continue;
        }
        size_t th = (size_t)n * H + h;
        size_t slot = state_slot ? (size_t)state_slot[n] : (size_t)n;
        kda_token_step(S + (slot * H + h) * dk * dv, q + th * dk, k + th * dk, v + th * dv,
                       log_alpha + th * dk, (double)beta[th], scale, dk, dv, r, o + th * dv);
        free(r);
    }
    return failed ? -1 : 0;
}

/*
 * General diagonal-plus-low-rank recurrence (Section 3.2 and Section 6.1, "Relation to DPLR"), the
 * comparison workload of the paper's kernel-time figure.  Per sequence and head, with S a dk x dv
 * matrix, g the per-channel log-decay and a, b the two low-rank vectors:
 *
 *     S_t = (Diag(exp(g_t)) + b_t a_t^T) S_{t-1} + k_t v_t^T ,      o_t = scale * S_t^T q_t
 *
 * i.e. a_t is contracted with the state as the previous token left it (x = S_{t-1}^T a_t), and the
 * state then receives the decay, the rank-one term b_t x^T and the new key/value pair.  This is the
 * reading of the paper's chunkwise DPLR pseudo-code taken here: its decay factor between the row of
 * a and the column of b or k stops one token before the row, and its state update adds b-weighted
 * and k-weighted terms.  With a = alpha . k, b = -beta k and the key replaced by beta k it is Eq. 1
 * (the correspondence the paper states, up to the sign convention of the low-rank term).
 *
 * Layouts as above; a, b, g are [T_total,H,dk].
 */
int kda_oracle_dplr_recurrence(const float *q, const float *k, const float *v, const float *a,
                               const float *b, const float *g, const double *S0, double *o,
                               double *S_T, const int64_t *cu_seqlens, int n_seqs, int H, int dk,
                               int dv, double scale, int n_threads)
{
    if (!k || !v || !a || !b || !g || !cu_seqlens || n_seqs < 0 || H <= 0 || dk <= 0 || dv <= 0)
        return -1;
    if (o && !q) return -1;
    int failed = 0;
    long n_items = (long)n_seqs * H;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (long item = 0; item < n_items; ++item) {
        int n = (int)(item / H), h = (int)(item % H);
        double *S = (double *)malloc(sizeof(double) * dk * dv);
        double *x = (double *)malloc(sizeof(double) * dv);
        if (!S || !x) {
            failed = 1;
            free(S);
            free(x);
            continue;
        }
        size_t sofs = ((size_t)n * H + h) * dk * dv;
        if (S0) memcpy(S, S0 + sofs, sizeof(double) * dk * dv);
        else memset(S, 0, sizeof(double) * dk * dv);
        for (int64_t t = cu_seqlens[n]; t < cu_seqlens[n + 1]; ++t) {
            size_t th = (size_t)t * H + h;
            const float *at = a + th * dk, *bt = b + th * dk, *gt = g + th * dk, *kt = k + th * dk;
            const float *vt = v + th * dv;
            /* x = S_{t-1}^T a_t */
            for (int j = 0; j < dv; ++j) x[j] = 0.0;
            for (int i = 0; i < dk; ++i) {
                double ai = (double)at[i];
                const double *Si = S + (size_t)i * dv;
                for (int j = 0; j < dv; ++j) x[j] += ai * Si[j];
            }
            /* S_t = Diag(exp(g_t)) S_{t-1} + b_t x^T + k_t v_t^T */
            for (int i = 0; i < dk; ++i) {
                double d = exp((double)gt[i]), bi = (double)bt[i], ki = (double)kt[i];
                double *Si = S + (size_t)i * dv;
                for (int j = 0; j < dv; ++j) Si[j] = d * Si[j] + bi * x[j] + ki * (double)vt[j];
            }
            if (o) {
                const float *qt = q + th * dk;
                double *ot = o + th * dv;
                for (int j = 0; j < dv; ++j) ot[j] = 0.0;
                for (int i = 0; i < dk; ++i) {
                    double qi = (double)qt[i];
                    const double *Si = S + (size_t)i * dv;
                    for (int j = 0; j < dv; ++j) ot[j] += qi * Si[j];
                }
                for (int j = 0; j < dv; ++j) ot[j] *= scale;
            }
        }
        if (S_T) memcpy(S_T + sofs, S, sizeof(double) * dk * dv);
        free(S);
        free(x);
    }
    return failed ? -1 : 0;
}

/*
 * Gradients of Eq. 1 (backward pass; the paper trains with the recurrence, Section 5, but prints no
 * backward algorithm, so this is Eq. 1 differentiated by hand).  For the scalar
 *
 *     L = sum_t <d_o_t, o_t> + <dS_T, S_T>
 *
 * it returns dL/dq, dL/dk, dL/dv, dL/dlog_alpha, dL/dbeta and dL/dS0.  With the forward step
 * written as  S' = Diag(alpha_t) S_{t-1},  r = v_t - S'^T k_t,  S_t = S' + beta_t k_t r^T,
 * o_t = scale S_t^T q_t,  and Lam the adjoint of the state, the steps are taken in reverse order:
 *
 *     Lam  += scale q_t d_o_t^T                 dq_t = scale S_t d_o_t
 *     dbeta_t = k_t^T Lam r                     dk_t  = beta_t Lam r
 *     dr = beta_t Lam^T k_t                     dv_t  = dr
 *     Lam' = Lam - k_t dr^T                     dk_t -= S' dr
 *     dlog_alpha_t = rowsum(Lam' . S')          Lam  <- Diag(alpha_t) Lam'          (for t-1)
 *
 * (dlog_alpha uses alpha_t dS'/dalpha_t = S', so nothing is divided by alpha.)  The forward states
 * of one sequence and head are all kept in memory: sizes are for tests (T * dk * dv doubles).
 *
 * Layouts as above; d_o [T_total,H,dv] may be NULL (= zeros), dS_T [n_seqs,H,dk,dv] may be NULL
 * (= zeros); every output pointer may be NULL.
 */
int kda_oracle_backward(const float *q, const float *k, const float *v, const float *log_alpha,
                        const float *beta, const double *S0, const double *d_o, const double *dS_T,
                        double *dq, double *dk_out, double *dv_out, double *dg, double *dbeta,
                        double *dS0, const int64_t *cu_seqlens, int n_seqs, int H, int dk, int dv,
                        double scale, int n_threads)
{
    if (!q || !k || !v || !log_alpha || !beta || !cu_seqlens || n_seqs < 0 || H <= 0 || dk <= 0 || dv <= 0)
        return -1;
    int failed = 0;
    long n_items = (long)n_seqs * H;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (long item = 0; item < n_items; ++item) {
        int n = (int)(item / H), h = (int)(item % H);
        int64_t t0 = cu_seqlens[n], t1 = cu_seqlens[n + 1];
        size_t len = (size_t)(t1 - t0), sz = (size_t)dk * dv;
        /* Sd[t] = decayed state S' of token t, Sp[t] = state S_t after token t, R[t] = residual r */
        double *Sd = (double *)malloc(sizeof(double) * sz * (len ? len : 1));
        double *Sp = (double *)malloc(sizeof(double) * sz * (len ? len : 1));
        double *R = (double *)malloc(sizeof(double) * dv * (len ? len : 1));
        double *Lam = (double *)malloc(sizeof(double) * sz);
        double *S = (double *)malloc(sizeof(double) * sz);
        double *dr = (double *)malloc(sizeof(double) * dv);
        double *lr = (double *)malloc(sizeof(double) * dk);
        if (!Sd || !Sp || !R || !Lam || !S || !dr || !lr) {
            failed = 1;
            free(Sd); free(Sp); free(R); free(Lam); free(S); free(dr); free(lr);
            continue;
        }
        size_t sofs = ((size_t)n * H + h) * sz;
        if (S0) memcpy(S, S0 + sofs, sizeof(double) * sz);
        else memset(S, 0, sizeof(double) * sz);
        /* forward, keeping every intermediate */
        for (size_t s = 0; s < len; ++s) {
            size_t th = (size_t)(t0 + (int64_t)s) * H + h;
            const float *kt = k + th * dk, *vt = v + th * dv, *gt = log_alpha + th * dk;
            double b = (double)beta[th];
            double *Sds = Sd + s * sz, *Sps = Sp + s * sz, *r = R + s * dv;
            for (int i = 0; i < dk; ++i) {
                double al = exp((double)gt[i]);
                for (int j = 0; j < dv; ++j) Sds[(size_t)i * dv + j] = al * S[(size_t)i * dv + j];
            }
            for (int j = 0; j < dv; ++j) r[j] = (double)vt[j];
            for (int i = 0; i < dk; ++i)
                for (int j = 0; j < dv; ++j) r[j] -= (double)kt[i] * Sds[(size_t)i * dv + j];
            for (int i = 0; i < dk; ++i)
                for (int j = 0; j < dv; ++j)
                    Sps[(size_t)i * dv + j] = Sds[(size_t)i * dv + j] + b * (double)kt[i] * r[j];
            memcpy(S, Sps, sizeof(double) * sz);
        }
        /* reverse */
        if (dS_T) memcpy(Lam, dS_T + sofs, sizeof(double) * sz);
        else memset(Lam, 0, sizeof(double) * sz);
        for (size_t s = len; s-- > 0;) {
            size_t th = (size_t)(t0 + (int64_t)s) * H + h;
            const float *qt = q + th * dk, *kt = k + th * dk, *gt = log_alpha + th * dk;
            double b = (double)beta[th];
            const double *Sds = Sd + s * sz, *Sps = Sp + s * sz, *r = R + s * dv;
            const double *dot = d_o ? d_o + th * dv : NULL;
            /* o_t = scale S_t^T q_t */
            for (int i = 0; i < dk; ++i) {
                double acc = 0.0;
                for (int j = 0; j < dv; ++j) {
                    double g_o = dot ? dot[j] : 0.0;
                    Lam[(size_t)i * dv + j] += scale * (double)qt[i] * g_o;
                    acc += Sps[(size_t)i * dv + j] * g_o;
                }
                if (dq) dq[th * dk + i] = scale * acc;
            }
            /* S_t = S' + beta k r^T */
            double db = 0.0;
            for (int i = 0; i < dk; ++i) {
                double acc = 0.0;
                for (int j = 0; j < dv; ++j) acc += Lam[(size_t)i * dv + j] * r[j];
                lr[i] = acc;                       /* (Lam r)_i */
                db += (double)kt[i] * acc;
            }
            if (dbeta) dbeta[th] = db;
            for (int j = 0; j < dv; ++j) {
                double acc = 0.0;
                for (int i = 0; i < dk; ++i) acc += Lam[(size_t)i * dv + j] * (double)kt[i];
                dr[j] = b * acc;
                if (dv_out) dv_out[th * dv + j] = dr[j];   /* r = v - S'^T k */
            }
            for (int i = 0; i < dk; ++i) {
                double sdr = 0.0, gsum = 0.0, al = exp((double)gt[i]);
                for (int j = 0; j < dv; ++j) {
                    double lp = Lam[(size_t)i * dv + j] - (double)kt[i] * dr[j];   /* Lam' */
                    sdr += Sds[(size_t)i * dv + j] * dr[j];
                    gsum += lp * Sds[(size_t)i * dv + j];
                    Lam[(size_t)i * dv + j] = al * lp;                             /* adjoint of S_{t-1} */
                }
                if (dk_out) dk_out[th * dk + i] = b * lr[i] - sdr;
                if (dg) dg[th * dk + i] = gsum;
            }
        }
        if (dS0) memcpy(dS0 + sofs, Lam, sizeof(double) * sz);
        free(Sd); free(Sp); free(R); free(Lam); free(S); free(dr); free(lr);
    }
    return failed ? -1 : 0;
}

int kda_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
