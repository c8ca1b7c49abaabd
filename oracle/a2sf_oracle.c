/*
 * A2SF oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, fp64 CPU statement of what the A2SF hot path computes, written
 * from the paper's definitions.  Only tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it.  It shares no code with the CUDA library.
 *
 * Every function works on ONE (batch, head) unit unless its name ends in
 * "_batch"; the batch drivers only spread independent units over threads.
 *
 * Notation (0-based positions): n prompt length, d head dimension, M cache
 * budget, R recent window.  The paper's Eq. 5 weight alpha^(n-q) (1-based q)
 * is alpha^(n-1-i) for 0-based row i.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py
 * (closed forms, invariants, brute force, library cross-checks).  The absolute
 * accuracy figures of the paper's Tables 1-2 are "parity unpinned": they need
 * trained weights and datasets.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * Masked softmax row (paper Sec. 1 causal mask; Eq. 3: S_{q,k} = 0 for q < k).
 * Row i attends to keys 0..i.  Writes P[0..i]; returns the log-sum-exp of the
 * scaled logits.  P[j] for j > i is not touched (it is zero by Eq. 3).
 * ---------------------------------------------------------------------- */
double a2sf_oracle_softmax_row(const double *Q, const double *K, int d, double scale,
                               int i, double *P)
{
    const double *q = Q + (size_t)i * d;
    double m = -INFINITY;
    for (int j = 0; j <= i; ++j) {
        const double *k = K + (size_t)j * d;
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += q[c] * k[c];
        s *= scale;
        P[j] = s;
        if (s > m) m = s;
    }
    double l = 0.0;
    for (int j = 0; j <= i; ++j) {
        P[j] = exp(P[j] - m);
        l += P[j];
    }
    for (int j = 0; j <= i; ++j) P[j] /= l;
    return m + log(l);
}

/* ------------------------------------------------------------------------
 * Prefill over rows [i0, i1) of one unit.
 *   out  [(i1-i0)][d]   out_i = sum_j P_ij v_j                (masked attention)
 *   lse  [i1-i0]        log sum_j exp(s_ij)
 *   S    [n_alpha][n]   S_j += alpha^(n-1-i) P_ij for i in [i0,i1), i >= j
 *                       (Eq. 5; Eq. 6 ends at the diagonal term S_{k,k}).
 * With i0 = 0, i1 = n this is the whole definition.  S is zeroed here.
 * The weight is built by repeated multiplication from w_{n-1} = 1, so that
 * 0^0 = 1 (alpha = 0 keeps only the last row).
 * ---------------------------------------------------------------------- */
void a2sf_oracle_prefill_rows(const double *Q, const double *K, const double *V,
                              int n, int d, double scale,
                              const double *alphas, int n_alpha,
                              int i0, int i1,
                              double *out, double *lse, double *S)
{
    double *P = (double *)malloc(sizeof(double) * (size_t)n);
    double *w = (double *)malloc(sizeof(double) * (size_t)n * (size_t)(n_alpha > 0 ? n_alpha : 1));
    for (int a = 0; a < n_alpha; ++a) {
        double *wa = w + (size_t)a * n;
        wa[n - 1] = 1.0;
        for (int i = n - 2; i >= 0; --i) wa[i] = wa[i + 1] * alphas[a];
        memset(S + (size_t)a * n, 0, sizeof(double) * (size_t)n);
    }
    for (int i = i0; i < i1; ++i) {
        double l = a2sf_oracle_softmax_row(Q, K, d, scale, i, P);
        if (lse) lse[i - i0] = l;
        if (out) {
            double *o = out + (size_t)(i - i0) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int j = 0; j <= i; ++j) {
                const double *v = V + (size_t)j * d;
                for (int c = 0; c < d; ++c) o[c] += P[j] * v[c];
            }
        }
        for (int a = 0; a < n_alpha; ++a) {
            double wi = w[(size_t)a * n + i];
            double *Sa = S + (size_t)a * n;
            for (int j = 0; j <= i; ++j) Sa[j] += wi * P[j];
        }
    }
    free(w);
    free(P);
}

/* ------------------------------------------------------------------------
 * Selection (paper Sec. 3.1: tokens with small score are removed; Sec. 4.1:
 * budget = local window + selective part).  Keep every position >= n-R and,
 * of the others, all but the n-M smallest under the total order (S_j, j)
 * ascending -- among equal scores the lowest position is removed first.
 * n <= M keeps everything.  kept[] is ascending; returns its length.
 * ---------------------------------------------------------------------- */
typedef struct { double s; int32_t j; } a2sf_cand;

static int cand_cmp(const void *a, const void *b)
{
    const a2sf_cand *x = (const a2sf_cand *)a, *y = (const a2sf_cand *)b;
    if (x->s < y->s) return -1;
    if (x->s > y->s) return 1;
    return (x->j > y->j) - (x->j < y->j);
}

static int i32_cmp(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int a2sf_oracle_select(const double *S, int n, int M, int R, int32_t *kept)
{
    if (n <= M) {
        for (int j = 0; j < n; ++j) kept[j] = j;
        return n;
    }
    int ncand = n - R;
    int drop = n - M;
    a2sf_cand *c = (a2sf_cand *)malloc(sizeof(a2sf_cand) * (size_t)(ncand > 0 ? ncand : 1));
    for (int j = 0; j < ncand; ++j) { c[j].s = S[j]; c[j].j = j; }
    qsort(c, (size_t)ncand, sizeof(a2sf_cand), cand_cmp);
    int m = 0;
    for (int r = drop; r < ncand; ++r) kept[m++] = c[r].j;
    for (int j = ncand; j < n; ++j) kept[m++] = j;
    qsort(kept, (size_t)m, sizeof(int32_t), i32_cmp);
    free(c);
    return m;
}

/* ------------------------------------------------------------------------
 * Pruned cache of one unit, slot-indexed.
 *   Kc, Vc [M][d]; Sc [M]; pos [M]; *count resident slots; *len tokens seen.
 * Initial cache: slot s holds token kept[s].
 * ---------------------------------------------------------------------- */
void a2sf_oracle_cache_load(const double *K, const double *V, const double *S,
                            const int32_t *kept, int m, int n, int d,
                            double *Kc, double *Vc, double *Sc, int32_t *pos,
                            int32_t *count, int32_t *len)
{
    for (int s = 0; s < m; ++s) {
        int j = kept[s];
        memcpy(Kc + (size_t)s * d, K + (size_t)j * d, sizeof(double) * (size_t)d);
        memcpy(Vc + (size_t)s * d, V + (size_t)j * d, sizeof(double) * (size_t)d);
        Sc[s] = S[j];
        pos[s] = j;
    }
    *count = m;
    *len = n;
}

/* ------------------------------------------------------------------------
 * One generation step on one unit.
 *  (i)   logits of the new query against every cached key and against the new
 *        key itself (the diagonal term of Eq. 6)
 *  (ii)  softmax over cached + self (the pruned denominator, Sec. 2.2)
 *  (iii) out = sum a_slot V[slot] + a_self v_new
 *  (iv)  S[slot] <- alpha S[slot] + a_slot ;  S_new = a_self     (Eq. 5 as a recurrence)
 *  (v)   cache not full: append.  Full: the candidates are the slots whose
 *        position is <= p - R (p = position of the new token), plus the new
 *        token itself iff R == 0; the (S, pos)-smallest candidate is evicted and
 *        the new token takes its slot in place.
 *  (vi)  len++.
 * info[0] = slot actually vacated (-1 appended, -2 the new token itself was dropped)
 * info[1] = the rule's own choice (equals info[0] unless forced)
 * info[2] = the rule's runner-up among the candidates (-1 none, -2 the new token)
 * scores3[0..2] = post-update scores of those three.
 * force_evict >= 0 (or -2) overrides the choice when the cache is full (used to
 * re-synchronise a comparison after an excused near-tie); -3 = the normal rule.
 * ---------------------------------------------------------------------- */
void a2sf_oracle_decode_step(double *Kc, double *Vc, double *Sc, int32_t *pos,
                             int32_t *count, int32_t *len,
                             const double *q, const double *k_new, const double *v_new,
                             int d, double scale, double alpha, int M, int R,
                             int force_evict,
                             double *out, int32_t *info, double *scores3)
{
    int cnt = *count;
    int p = *len;
    double *a = (double *)malloc(sizeof(double) * (size_t)(cnt + 1));
    double m = -INFINITY;
    for (int s = 0; s <= cnt; ++s) {
        const double *k = (s < cnt) ? Kc + (size_t)s * d : k_new;
        double t = 0.0;
        for (int c = 0; c < d; ++c) t += q[c] * k[c];
        t *= scale;
        a[s] = t;
        if (t > m) m = t;
    }
    double l = 0.0;
    for (int s = 0; s <= cnt; ++s) { a[s] = exp(a[s] - m); l += a[s]; }
    for (int s = 0; s <= cnt; ++s) a[s] /= l;

    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int s = 0; s <= cnt; ++s) {
        const double *v = (s < cnt) ? Vc + (size_t)s * d : v_new;
        for (int c = 0; c < d; ++c) out[c] += a[s] * v[c];
    }

    for (int s = 0; s < cnt; ++s) Sc[s] = alpha * Sc[s] + a[s];
    double s_new = a[cnt];

    info[0] = -1; info[1] = -1; info[2] = -1;
    scores3[0] = 0.0; scores3[1] = 0.0; scores3[2] = 0.0;
    int target;
    if (cnt < M) {
        target = cnt;
        *count = cnt + 1;
    } else {
        /* best and second best candidate under (S, pos) ascending */
        int best = -1, second = -1;            /* -2 stands for the new token */
        double bs = 0.0, ss = 0.0; int bp = 0, sp = 0;
        int ncand = cnt + (R == 0 ? 1 : 0);
        for (int t = 0; t < ncand; ++t) {
            int slot = (t < cnt) ? t : -2;
            double sc = (t < cnt) ? Sc[t] : s_new;
            int ps = (t < cnt) ? pos[t] : p;
            if (t < cnt && !(ps <= p - R)) continue;
            int lt_best = (best == -1) || sc < bs || (sc == bs && ps < bp);
            if (lt_best) {
                second = best; ss = bs; sp = bp;
                best = slot; bs = sc; bp = ps;
            } else {
                int lt_second = (second == -1) || sc < ss || (sc == ss && ps < sp);
                if (lt_second) { second = slot; ss = sc; sp = ps; }
            }
        }
        info[1] = best; info[2] = second; scores3[1] = bs; scores3[2] = ss;
        target = best;
        if (force_evict != -3) target = force_evict;
        info[0] = target;
        scores3[0] = (target == -2) ? s_new : Sc[target];
    }
    if (target >= 0) {
        memcpy(Kc + (size_t)target * d, k_new, sizeof(double) * (size_t)d);
        memcpy(Vc + (size_t)target * d, v_new, sizeof(double) * (size_t)d);
        Sc[target] = s_new;
        pos[target] = p;
    }
    *len = p + 1;
    free(a);
}

/* ------------------------------------------------------------------------
 * Batch drivers: independent units spread over threads, nothing else.
 * ---------------------------------------------------------------------- */
typedef struct {
    int u0, u1;
    const double *Q, *K, *V;
    int n, d; double scale; const double *alphas; int n_alpha;
    int M, R, sel_alpha;
    double *out, *lse, *S; int32_t *kept, *kept_len;
} prefill_job;

static void *prefill_worker(void *arg)
{
    prefill_job *j = (prefill_job *)arg;
    size_t nd = (size_t)j->n * j->d;
    int m = j->n < j->M ? j->n : j->M;
    for (int u = j->u0; u < j->u1; ++u) {
        double *S = j->S + (size_t)u * j->n_alpha * j->n;
        a2sf_oracle_prefill_rows(j->Q + u * nd, j->K + u * nd, j->V + u * nd,
                                 j->n, j->d, j->scale, j->alphas, j->n_alpha, 0, j->n,
                                 j->out ? j->out + u * nd : NULL,
                                 j->lse ? j->lse + (size_t)u * j->n : NULL, S);
        if (j->kept)
            j->kept_len[u] = a2sf_oracle_select(S + (size_t)j->sel_alpha * j->n, j->n, j->M,
                                                j->R, j->kept + (size_t)u * m);
    }
    return NULL;
}

/* Q,K,V [U][n][d]; out [U][n][d] or NULL; lse [U][n] or NULL; S [U][n_alpha][n];
 * kept [U][min(n,M)] or NULL (selection on alphas[sel_alpha]); kept_len [U]. */
int a2sf_oracle_prefill_batch(const double *Q, const double *K, const double *V,
                              int U, int n, int d, double scale,
                              const double *alphas, int n_alpha, int M, int R, int sel_alpha,
                              double *out, double *lse, double *S,
                              int32_t *kept, int32_t *kept_len, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    if (nthreads > U) nthreads = U > 0 ? U : 1;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    prefill_job *jobs = (prefill_job *)malloc(sizeof(prefill_job) * (size_t)nthreads);
    for (int t = 0; t < nthreads; ++t) {
        prefill_job j = { (int)((long)U * t / nthreads), (int)((long)U * (t + 1) / nthreads),
                          Q, K, V, n, d, scale, alphas, n_alpha, M, R, sel_alpha,
                          out, lse, S, kept, kept_len };
        jobs[t] = j;
        pthread_create(&th[t], NULL, prefill_worker, &jobs[t]);
    }
    for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(jobs);
    free(th);
    return nthreads;
}

typedef struct {
    int u0, u1;
    double *Kc, *Vc, *Sc; int32_t *pos, *count, *len;
    const double *q, *k_new, *v_new;
    int d; double scale, alpha; int M, R; const int32_t *force;
    double *out; int32_t *info; double *scores3;
} decode_job;

static void *decode_worker(void *arg)
{
    decode_job *j = (decode_job *)arg;
    size_t Md = (size_t)j->M * j->d;
    for (int u = j->u0; u < j->u1; ++u)
        a2sf_oracle_decode_step(j->Kc + u * Md, j->Vc + u * Md, j->Sc + (size_t)u * j->M,
                                j->pos + (size_t)u * j->M, j->count + u, j->len + u,
                                j->q + (size_t)u * j->d, j->k_new + (size_t)u * j->d,
                                j->v_new + (size_t)u * j->d, j->d, j->scale, j->alpha,
                                j->M, j->R, j->force ? j->force[u] : -3,
                                j->out + (size_t)u * j->d, j->info + 3 * (size_t)u,
                                j->scores3 + 3 * (size_t)u);
    return NULL;
}

/* One step for U units.  Cache arrays [U][M][d] / [U][M] / [U]; q,k_new,v_new,out
 * [U][d]; force [U] or NULL; info [U][3]; scores3 [U][3]. */
int a2sf_oracle_decode_step_batch(double *Kc, double *Vc, double *Sc, int32_t *pos,
                                  int32_t *count, int32_t *len,
                                  const double *q, const double *k_new, const double *v_new,
                                  int U, int d, double scale, double alpha, int M, int R,
                                  const int32_t *force,
                                  double *out, int32_t *info, double *scores3, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    if (nthreads > U) nthreads = U > 0 ? U : 1;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    decode_job *jobs = (decode_job *)malloc(sizeof(decode_job) * (size_t)nthreads);
    for (int t = 0; t < nthreads; ++t) {
        decode_job j = { (int)((long)U * t / nthreads), (int)((long)U * (t + 1) / nthreads),
                         Kc, Vc, Sc, pos, count, len, q, k_new, v_new,
                         d, scale, alpha, M, R, force, out, info, scores3 };
        jobs[t] = j;
        pthread_create(&th[t], NULL, decode_worker, &jobs[t]);
    }
    for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(jobs);
    free(th);
    return nthreads;
}
