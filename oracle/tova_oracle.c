/*
 * TEST INFRASTRUCTURE - CPU checker for the TOVA decode step.
 *
 * A plain, slow, deliberately unoptimised statement of what one decoding step
 * of one transformer layer computes when the layer is run as a bounded
 * multi-state RNN with the TOVA compression policy.  It exists only so that
 * tests, the smoke check and the CPU-baseline leg of the benchmark have
 * something to compare the GPU library with.  It shares no code with the GPU
 * library and must never be called from it.
 *
 * What it follows, step by step and in the paper's order:
 *   - Eq. 6 (Section 3.2): the new (k_t, v_t) is appended to the multi-state
 *     (K_{t-1}, V_{t-1}) first;
 *   - Eq. 4 / Eq. 7: the layer output is Softmax(q_t K_t^T) V_t over ALL rows
 *     of the appended state, including the row that is about to be dropped;
 *   - Section 3.3: g(t) = min(t, k): nothing is dropped while the state has
 *     at most k rows;
 *   - Section 4, Eq. 9 and Algorithm 1: once the appended state has k+1 rows,
 *     the last query's attention weights are averaged over the heads of the
 *     layer, the row with the lowest average is deleted from K and V.
 *
 * Readings where the paper is silent (stated once more in the design notes):
 *   - a scale factor multiplies the logits (the paper omits 1/sqrt(d));
 *   - under grouped-query attention all H query heads are averaged and the one
 *     victim is removed from every KV head;
 *   - ties of the arg-min go to the lowest row index, the new token being the
 *     last row;
 *   - the state is kept in place: the new token takes the victim's row, so
 *     row order is not position order; positions travel with the rows.
 *
 * Other compression policies of the paper, selectable per call (Section 4.1
 * and the ablation in the appendix, Table "lm_ablation"):
 *   - Window: first in, first out - when the state is over capacity the row
 *     holding the earliest position is deleted; the attention weights play no
 *     part;
 *   - "+i" (Window+i, TOVA+i): rows holding the first i positions (0..i-1) are
 *     never deleted; the policy picks among the others.
 *   - TOVA-head (Section 4: the policy "computes the attention scores of each
 *     head separately, and can thus retain different tokens at different
 *     heads"; appendix ablation row TOVA-head): every head keeps its own rows
 *     and drops the row with ITS lowest weight;
 *   - H2O, layer-wise and head-wise (Section 4.1): a window of the most recent
 *     tokens is always kept; among the older rows the one whose attention
 *     weight, summed over all the steps it has been in the state, is lowest
 *     goes.  The number of non-window rows is half the multi-state size unless
 *     the caller says otherwise.
 * Readings for these (the paper gives one paragraph each): a "head" that owns
 * rows is a KV head, and its score for a row is the mean weight of the query
 * heads that read it (for multi-head attention: the head's own weight); a
 * row's accumulated score starts with the weight it received as the new token
 * and grows by its weight at every later step, before the victim of that step
 * is chosen; window membership is "fewer than `recent` positions behind the new
 * token"; ties go to the lowest row index.
 * The layer output of the current step does not depend on the policy (it is
 * computed before the deletion).
 *
 * Precision: every operation is carried out in REAL (float for the parity
 * checker, double for the reference the float build is itself checked with).
 * Sums run in ascending index order; the soft-max divides (no reciprocal).
 *
 * Parity pins (tests marked "not gpu"): textbook soft-max attention in double
 * on tiny states, library causal attention when k >= stream length, the
 * size invariant len_t = min(t, k), a hand-worked 3-row example in exact
 * rational arithmetic, an order-preserving restatement of Algorithm 1, and
 * permutation / shift invariances.  Window and "+i": the closed form of the
 * retained positions (the first i and the most recent k-i), hand-worked
 * traces of the 3-row example, "+0" equal to the plain policy, and the
 * invariant that a protected position is never reported as dropped.
 * Position compression: the gap function's printed examples, "no gap above 10
 * = ordinary rotary attention" against a library routine, invariance under a
 * shift of all positions, and a restatement over the full token history with
 * complex exponentials in double.
 * TOVA-head and H2O: per-head and accumulated-score restatements over the full
 * token history in double (order-preserving lists), hand-worked traces of the
 * 3-row example in exact arithmetic, "one head = the layer policy", H2O with
 * a window as large as the state = Window, accumulated scores = column sums
 * of the textbook causal soft-max matrix while nothing is dropped.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifndef REAL
#define REAL float
#endif

#ifdef _OPENMP
#include <omp.h>
#endif

static REAL real_exp(REAL x) { return sizeof(REAL) == 4 ? (REAL)expf((float)x) : (REAL)exp((double)x); }

/*
 * Attention of the new query over the appended state, for one sequence:
 * weights (Eq. 4) into work[h][0..n] (row n = the new token) and the layer
 * output over all n+1 rows (Eq. 7) into out.  work is [H][cap+1].
 */
static void attend(int H, int Hkv, int D, int cap, REAL scale, int n,
                   const REAL *K, const REAL *V, const REAL *q, const REAL *k_new, const REAL *v_new,
                   REAL *out, REAL *work)
{
    const int m = n + 1;
    const int G = H / Hkv;
    const int ld = cap + 1;
    for (int h = 0; h < H; ++h) {
        const int kv = h / G;
        REAL *p = work + (size_t)h * ld;
        for (int j = 0; j < m; ++j) {
            const REAL *krow = (j < n) ? K + ((size_t)kv * cap + j) * D : k_new + (size_t)kv * D;
            REAL s = 0;
            for (int d = 0; d < D; ++d) s += q[(size_t)h * D + d] * krow[d];
            p[j] = scale * s;
        }
        REAL mx = p[0];
        for (int j = 1; j < m; ++j) if (p[j] > mx) mx = p[j];
        REAL l = 0;
        for (int j = 0; j < m; ++j) { p[j] = real_exp(p[j] - mx); l += p[j]; }
        for (int j = 0; j < m; ++j) p[j] = p[j] / l;
        /* Layer output before any row is dropped (Eq. 7). */
        for (int d = 0; d < D; ++d) {
            REAL o = 0;
            for (int j = 0; j < m; ++j) {
                const REAL *vrow = (j < n) ? V + ((size_t)kv * cap + j) * D : v_new + (size_t)kv * D;
                o += p[j] * vrow[d];
            }
            out[(size_t)h * D + d] = o;
        }
    }

}

/*
 * One token for one sequence.
 *   len      in/out  live rows n (0 <= n <= cap)
 *   pos      in/out  [cap]          original position of each row, -1 if unused
 *   K, V     in/out  [Hkv][cap][D]
 *   q        in      [H][D]
 *   k_new,v_new in   [Hkv][D]
 *   forced   in      -1, or the candidate index (0..cap) to drop instead of
 *                    the arg-min when a drop is due
 *   out      out     [H][D]
 *   evicted_pos out  position dropped; -1 when nothing was dropped
 *   victim   out     candidate index dropped (cap = the new token), -1 if none
 *   argmin   out     the arg-min itself (differs from victim only when forced), -1 if none
 *   gap      out     mean[dropped] - min(mean) (0 unless forced differs); under the
 *                    Window policy 0 if the forced row holds the earliest
 *                    droppable position, else 1; 1e30 if a protected row is forced
 *   policy, keep_first  which row goes once the state is over capacity (see top)
 *   mean_out out     [cap+1] head-averaged weights, or NULL
 *   work     scratch [H+1][cap+1] REAL (weights per head, then their mean)
 */
#define POLICY_TOVA 0
#define POLICY_WINDOW 1

static void drop_and_insert(int H, int Hkv, int D, int cap, int policy, int keep_first,
                            int *len, int *pos, REAL *K, REAL *V,
                            const REAL *k_new, const REAL *v_new,
                            int pos_t, int forced,
                            int *evicted_pos, int *victim, int *argmin, REAL *gap,
                            REAL *mean_out, REAL *work);

static void step_one(int H, int Hkv, int D, int cap, REAL scale, int policy, int keep_first,
                     int *len, int *pos, REAL *K, REAL *V,
                     const REAL *q, const REAL *k_new, const REAL *v_new,
                     int pos_t, int forced,
                     REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                     REAL *mean_out, REAL *work)
{
    attend(H, Hkv, D, cap, scale, *len, K, V, q, k_new, v_new, out, work);
    drop_and_insert(H, Hkv, D, cap, policy, keep_first, len, pos, K, V, k_new, v_new, pos_t, forced,
                    evicted_pos, victim, argmin, gap, mean_out, work);
}

/*
 * The second half of a step: given the weights of the new query over the
 * appended state (work[h][0..n], from attend), keep all rows while the state
 * has room, else pick the row to delete and let the new token take its place.
 * Arguments as for step_one.
 */
static void drop_and_insert(int H, int Hkv, int D, int cap, int policy, int keep_first,
                            int *len, int *pos, REAL *K, REAL *V,
                            const REAL *k_new, const REAL *v_new,
                            int pos_t, int forced,
                            int *evicted_pos, int *victim, int *argmin, REAL *gap,
                            REAL *mean_out, REAL *work)
{
    const int n = *len;          /* rows before the append */
    const int m = n + 1;         /* rows after the append (Eq. 6) */
    const int ld = cap + 1;

    *gap = 0;
    if (m <= cap) {              /* Algorithm 1: num_kv <= cache_max_size -> keep all */
        for (int kv = 0; kv < Hkv; ++kv) {
            memcpy(K + ((size_t)kv * cap + n) * D, k_new + (size_t)kv * D, sizeof(REAL) * D);
            memcpy(V + ((size_t)kv * cap + n) * D, v_new + (size_t)kv * D, sizeof(REAL) * D);
        }
        pos[n] = pos_t;
        *len = m;
        *evicted_pos = -1;
        *victim = -1;
        *argmin = -1;
        if (mean_out) for (int j = 0; j < ld; ++j) mean_out[j] = 0;
        return;
    }

    /* Average the last query's weights over the heads (Algorithm 1). */
    REAL *mean = work + (size_t)H * ld;
    for (int j = 0; j < m; ++j) {
        REAL a = 0;
        for (int h = 0; h < H; ++h) a += work[(size_t)h * ld + j];
        mean[j] = a / (REAL)H;
    }
    if (mean_out) for (int j = 0; j < m; ++j) mean_out[j] = mean[j];
    /* The row to delete, among those not holding one of the first keep_first
     * positions: lowest average (TOVA, Algorithm 1) or earliest position
     * (Window, Section 4.1); lowest index on ties. */
    int jmin = -1;
    for (int j = 0; j < m; ++j) {
        const int pj = (j < n) ? pos[j] : pos_t;
        if (pj < keep_first) continue;
        if (jmin < 0) { jmin = j; continue; }
        const int pmin = (jmin < n) ? pos[jmin] : pos_t;
        if (policy == POLICY_WINDOW ? (pj < pmin) : (mean[j] < mean[jmin])) jmin = j;
    }
    if (jmin < 0) jmin = n;      /* every row is protected: the new token cannot stay */
    int drop = jmin;
    *argmin = jmin;
    if (forced >= 0 && forced < m) {
        drop = forced;
        const int pd = (drop < n) ? pos[drop] : pos_t;
        const int pmin = (jmin < n) ? pos[jmin] : pos_t;
        if (pd < keep_first && drop != jmin) *gap = (REAL)1e30;
        else if (policy == POLICY_WINDOW) *gap = (pd == pmin) ? (REAL)0 : (REAL)1;
        else *gap = mean[drop] - mean[jmin];
    }

    /* Delete row `drop` from K and V (Eq. 9): in place, the new token takes
     * the freed row; dropping the new token itself changes nothing. */
    *victim = drop;
    if (drop < cap) {
        *evicted_pos = pos[drop];
        for (int kv = 0; kv < Hkv; ++kv) {
            memcpy(K + ((size_t)kv * cap + drop) * D, k_new + (size_t)kv * D, sizeof(REAL) * D);
            memcpy(V + ((size_t)kv * cap + drop) * D, v_new + (size_t)kv * D, sizeof(REAL) * D);
        }
        pos[drop] = pos_t;
    } else {
        *evicted_pos = pos_t;
    }
}

/*
 * One token for each of B independent sequences (Algorithm 1 assumes batch 1:
 * sequences never interact).  Layouts: len [B], pos [B][cap],
 * K,V [B][Hkv][cap][D], q/out [B][H][D], k_new/v_new [B][Hkv][D],
 * forced/evicted_pos/victim/argmin/gap [B] (forced may be NULL),
 * mean_out [B][cap+1] or NULL.  Sequences are spread over `nthreads` threads;
 * nothing else is parallel.  Returns 0, or -1 on a bad argument.
 */
int tova_oracle_step_policy(int B, int H, int Hkv, int D, int cap, REAL scale, int policy, int keep_first,
                            int *len, int *pos, REAL *K, REAL *V,
                            const REAL *q, const REAL *k_new, const REAL *v_new,
                            int pos_t, const int *forced,
                            REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                            REAL *mean_out, int nthreads)
{
    if (B < 1 || H < 1 || Hkv < 1 || D < 1 || cap < 1 || H % Hkv != 0) return -1;
    if ((policy != POLICY_TOVA && policy != POLICY_WINDOW) || keep_first < 0) return -1;
    const size_t ld = (size_t)cap + 1;
    if (nthreads < 1) nthreads = 1;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads) schedule(static)
#endif
    for (int b = 0; b < B; ++b) {
        REAL *work = (REAL *)malloc(sizeof(REAL) * (size_t)(H + 1) * ld);
        if (!work) { bad = 1; continue; }
        if (len[b] < 0 || len[b] > cap) { bad = 1; free(work); continue; }
        step_one(H, Hkv, D, cap, scale, policy, keep_first,
                 len + b, pos + (size_t)b * cap,
                 K + (size_t)b * Hkv * cap * D, V + (size_t)b * Hkv * cap * D,
                 q + (size_t)b * H * D, k_new + (size_t)b * Hkv * D, v_new + (size_t)b * Hkv * D,
                 pos_t, forced ? forced[b] : -1,
                 out + (size_t)b * H * D, evicted_pos + b, victim + b, argmin + b, gap + b,
                 mean_out ? mean_out + (size_t)b * ld : NULL, work);
        free(work);
    }
    return bad ? -1 : 0;
}

/* The TOVA policy with no protected positions (the paper's method as is). */
int tova_oracle_step(int B, int H, int Hkv, int D, int cap, REAL scale,
                     int *len, int *pos, REAL *K, REAL *V,
                     const REAL *q, const REAL *k_new, const REAL *v_new,
                     int pos_t, const int *forced,
                     REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                     REAL *mean_out, int nthreads)
{
    return tova_oracle_step_policy(B, H, Hkv, D, cap, scale, POLICY_TOVA, 0, len, pos, K, V, q, k_new, v_new,
                                   pos_t, forced, out, evicted_pos, victim, argmin, gap, mean_out, nthreads);
}

/* ------------------------------------------------------------------------
 * Policies in which rows are owned per unit: a unit is the whole layer (one
 * unit, U = 1) or one KV head (U = Hkv).  TOVA-head, H2O-layer, H2O-head.
 * ------------------------------------------------------------------------ */
#define POLICY_TOVA_HEAD 2
#define POLICY_H2O_LAYER 3
#define POLICY_H2O_HEAD 4

/*
 * One token for one sequence under a unit policy.
 *   len      in/out  live rows n, the same for every unit
 *   pos      in/out  [U][cap]  position held by each row of each unit, -1 if unused
 *   acc      in/out  [U][cap]  H2O: accumulated score of each row (unused otherwise)
 *   K, V     in/out  [Hkv][cap][D]  (row j of KV head kv belongs to unit kv, or to the one unit)
 *   recent   H2O: candidates fewer than `recent` positions behind the new token are never dropped
 *   forced   [U] or NULL: candidate to drop instead of the unit's arg-min (-1: none)
 *   evicted_pos, victim, argmin, gap   [U], as in step_one; gap is measured in the
 *            quantity the policy minimises (weight, or accumulated score)
 *   score_out [U][cap+1] or NULL: that quantity for every candidate
 *   work     scratch [H+1][cap+1]
 */
static void step_units(int H, int Hkv, int D, int cap, REAL scale, int policy, int recent,
                       int *len, int *pos, REAL *acc, REAL *K, REAL *V,
                       const REAL *q, const REAL *k_new, const REAL *v_new,
                       int pos_t, const int *forced,
                       REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                       REAL *score_out, REAL *work)
{
    const int n = *len;
    const int m = n + 1;
    const int G = H / Hkv;
    const int ld = cap + 1;
    const int U = (policy == POLICY_H2O_LAYER) ? 1 : Hkv;
    const int h2o = (policy == POLICY_H2O_LAYER || policy == POLICY_H2O_HEAD);

    attend(H, Hkv, D, cap, scale, n, K, V, q, k_new, v_new, out, work);

    REAL *key = work + (size_t)H * ld;          /* what the unit minimises, per candidate */
    for (int u = 0; u < U; ++u) {
        const int h0 = (U == 1) ? 0 : u * G;    /* query heads that read this unit's rows */
        const int nh = (U == 1) ? H : G;
        const int kv0 = (U == 1) ? 0 : u, kv1 = (U == 1) ? Hkv : u + 1;
        int *upos = pos + (size_t)u * cap;
        REAL *uacc = acc + (size_t)u * cap;
        /* the unit's weight on every candidate: mean over its query heads */
        for (int j = 0; j < m; ++j) {
            REAL a = 0;
            for (int h = h0; h < h0 + nh; ++h) a += work[(size_t)h * ld + j];
            key[j] = a / (REAL)nh;
        }
        if (h2o) {                              /* scores accumulate over the steps (Section 4.1) */
            for (int j = 0; j < n; ++j) { uacc[j] += key[j]; key[j] = uacc[j]; }
            /* key[n]: the new token's score so far is its weight at this step */
        }
        if (score_out) {
            for (int j = 0; j < ld; ++j) score_out[(size_t)u * ld + j] = (j < m) ? key[j] : 0;
        }
        gap[u] = 0;
        if (m <= cap) {                         /* g(t) = min(t, k): keep all */
            for (int kv = kv0; kv < kv1; ++kv) {
                memcpy(K + ((size_t)kv * cap + n) * D, k_new + (size_t)kv * D, sizeof(REAL) * D);
                memcpy(V + ((size_t)kv * cap + n) * D, v_new + (size_t)kv * D, sizeof(REAL) * D);
            }
            upos[n] = pos_t;
            if (h2o) uacc[n] = key[n];
            evicted_pos[u] = -1; victim[u] = -1; argmin[u] = -1;
            continue;
        }
        int jmin = -1;
        for (int j = 0; j < m; ++j) {
            const int pj = (j < n) ? upos[j] : pos_t;
            if (h2o && pos_t - pj < recent) continue;   /* inside the recent window */
            if (jmin < 0 || key[j] < key[jmin]) jmin = j;
        }
        if (jmin < 0) jmin = n;
        int drop = jmin;
        argmin[u] = jmin;
        if (forced && forced[u] >= 0 && forced[u] < m) {
            drop = forced[u];
            const int pd = (drop < n) ? upos[drop] : pos_t;
            if (h2o && pos_t - pd < recent && drop != jmin) gap[u] = (REAL)1e30;
            else gap[u] = key[drop] - key[jmin];
        }
        victim[u] = drop;
        if (drop < cap) {
            evicted_pos[u] = upos[drop];
            for (int kv = kv0; kv < kv1; ++kv) {
                memcpy(K + ((size_t)kv * cap + drop) * D, k_new + (size_t)kv * D, sizeof(REAL) * D);
                memcpy(V + ((size_t)kv * cap + drop) * D, v_new + (size_t)kv * D, sizeof(REAL) * D);
            }
            upos[drop] = pos_t;
            if (h2o) uacc[drop] = key[n];
        } else {
            evicted_pos[u] = pos_t;
        }
    }
    if (m <= cap) *len = m;
}

/*
 * Batch wrapper of step_units.  U = 1 for POLICY_H2O_LAYER, Hkv otherwise.
 * Layouts: len [B], pos [B][U][cap], acc [B][U][cap], K,V [B][Hkv][cap][D],
 * forced/evicted_pos/victim/argmin/gap [B][U] (forced may be NULL),
 * score_out [B][U][cap+1] or NULL.  Returns 0, or -1 on a bad argument.
 */
int tova_oracle_step_units(int B, int H, int Hkv, int D, int cap, REAL scale, int policy, int recent,
                           int *len, int *pos, REAL *acc, REAL *K, REAL *V,
                           const REAL *q, const REAL *k_new, const REAL *v_new,
                           int pos_t, const int *forced,
                           REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                           REAL *score_out, int nthreads)
{
    if (B < 1 || H < 1 || Hkv < 1 || D < 1 || cap < 1 || H % Hkv != 0) return -1;
    if (policy != POLICY_TOVA_HEAD && policy != POLICY_H2O_LAYER && policy != POLICY_H2O_HEAD) return -1;
    const int h2o = policy != POLICY_TOVA_HEAD;
    if (h2o && (recent < 1 || recent > cap)) return -1;
    const size_t ld = (size_t)cap + 1;
    const size_t U = (policy == POLICY_H2O_LAYER) ? 1 : (size_t)Hkv;
    if (nthreads < 1) nthreads = 1;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads) schedule(static)
#endif
    for (int b = 0; b < B; ++b) {
        REAL *work = (REAL *)malloc(sizeof(REAL) * (size_t)(H + 1) * ld);
        if (!work) { bad = 1; continue; }
        if (len[b] < 0 || len[b] > cap) { bad = 1; free(work); continue; }
        step_units(H, Hkv, D, cap, scale, policy, recent,
                   len + b, pos + (size_t)b * U * cap, acc + (size_t)b * U * cap,
                   K + (size_t)b * Hkv * cap * D, V + (size_t)b * Hkv * cap * D,
                   q + (size_t)b * H * D, k_new + (size_t)b * Hkv * D, v_new + (size_t)b * Hkv * D,
                   pos_t, forced ? forced + (size_t)b * U : NULL,
                   out + (size_t)b * H * D, evicted_pos + (size_t)b * U, victim + (size_t)b * U,
                   argmin + (size_t)b * U, gap + (size_t)b * U,
                   score_out ? score_out + (size_t)b * U * ld : NULL, work);
        free(work);
    }
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------------
 * Position compression for streams longer than the training context
 * (Section "Extrapolation with TOVA"): the keys are cached WITHOUT rotary
 * embedding; at every step the retained tokens and the new token, taken in
 * position order, get new positions in which the gap g between neighbours is
 * ln(ln(g)), or g itself while g <= 10; the rotary embedding is then applied
 * with those positions to the cached keys and to the query, and the step
 * proceeds as usual (the un-rotated key of the new token is what is cached).
 * Readings: the new positions accumulate along the chain (p'_{m+1} = p'_m +
 * f(p_{m+1} - p_m)); the earliest retained token sits at 0 - attention depends
 * on differences only, so the origin is immaterial; rotary embedding in the
 * rotate-half form (component d pairs with d + D/2, angle p' * base^(-2d/D)),
 * as in the model families the paper runs; the chain of new positions and the
 * angles are worked out in double, whatever REAL is.
 * ------------------------------------------------------------------------ */
double tova_oracle_compress_gap(int g)
{
    return (g <= 10) ? (double)g : log(log((double)g));
}

/* x[0..D) rotated by position p (rotate-half pairs), into y. */
static void rope_rotate(const REAL *x, REAL *y, int D, double p, double base)
{
    const int half = D / 2;
    for (int d = 0; d < half; ++d) {
        const double ang = p * pow(base, -2.0 * (double)d / (double)D);
        const REAL c = (REAL)cos(ang), s = (REAL)sin(ang);
        const REAL a = x[d], b = x[d + half];
        y[d] = a * c - b * s;
        y[d + half] = b * c + a * s;
    }
}

/*
 * One token for one sequence with position compression.  As step_one, plus:
 *   rope_base      base of the rotary embedding (10000 in the LLaMA family)
 *   cpos_out       [cap+1] or NULL: the new position of every candidate
 *                  (slot order, the new token last)
 *   rot            scratch [Hkv][cap+1][D] + [H][D] REAL
 */
static void step_one_poscomp(int H, int Hkv, int D, int cap, REAL scale, int policy, int keep_first, double rope_base,
                             int *len, int *pos, REAL *K, REAL *V,
                             const REAL *q, const REAL *k_new, const REAL *v_new,
                             int pos_t, int forced,
                             REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                             REAL *mean_out, double *cpos_out, REAL *work, REAL *rot)
{
    const int n = *len, m = n + 1;
    /* candidates in position order: insertion sort of (position, candidate index) */
    int *order = (int *)malloc(sizeof(int) * (size_t)m);
    double *cp = (double *)malloc(sizeof(double) * (size_t)m);
    for (int j = 0; j < m; ++j) {
        const int pj = (j < n) ? pos[j] : pos_t;
        int i = j;
        while (i > 0) {
            const int o = order[i - 1];
            const int po = (o < n) ? pos[o] : pos_t;
            if (po <= pj) break;
            order[i] = o;
            --i;
        }
        order[i] = j;
    }
    /* the chain of compressed positions */
    double acc = 0.0;
    for (int r = 0; r < m; ++r) {
        const int j = order[r];
        if (r > 0) {
            const int jp = order[r - 1];
            const int g = ((j < n) ? pos[j] : pos_t) - ((jp < n) ? pos[jp] : pos_t);
            acc += tova_oracle_compress_gap(g);
        }
        cp[j] = acc;
    }
    if (cpos_out) for (int j = 0; j <= cap; ++j) cpos_out[j] = (j < m) ? cp[j] : 0.0;
    /* rotated copies: keys of the state as [Hkv][cap][D] (stride cap, as attend expects), the new key, the query */
    REAL *Krot = rot;
    REAL *knew_rot = rot + (size_t)Hkv * cap * D;
    REAL *q_rot = knew_rot + (size_t)Hkv * D;
    for (int kv = 0; kv < Hkv; ++kv) {
        for (int j = 0; j < n; ++j)
            rope_rotate(K + ((size_t)kv * cap + j) * D, Krot + ((size_t)kv * cap + j) * D, D, cp[j], rope_base);
        rope_rotate(k_new + (size_t)kv * D, knew_rot + (size_t)kv * D, D, cp[n], rope_base);
    }
    for (int h = 0; h < H; ++h) rope_rotate(q + (size_t)h * D, q_rot + (size_t)h * D, D, cp[n], rope_base);
    attend(H, Hkv, D, cap, scale, n, Krot, V, q_rot, knew_rot, v_new, out, work);
    drop_and_insert(H, Hkv, D, cap, policy, keep_first, len, pos, K, V, k_new, v_new, pos_t, forced,
                    evicted_pos, victim, argmin, gap, mean_out, work);
    free(order);
    free(cp);
}

/* Batch wrapper; layouts as tova_oracle_step_policy, cpos_out [B][cap+1] doubles or NULL. */
int tova_oracle_step_poscomp(int B, int H, int Hkv, int D, int cap, REAL scale, int policy, int keep_first,
                             double rope_base,
                             int *len, int *pos, REAL *K, REAL *V,
                             const REAL *q, const REAL *k_new, const REAL *v_new,
                             int pos_t, const int *forced,
                             REAL *out, int *evicted_pos, int *victim, int *argmin, REAL *gap,
                             REAL *mean_out, double *cpos_out, int nthreads)
{
    if (B < 1 || H < 1 || Hkv < 1 || D < 2 || D % 2 || cap < 1 || H % Hkv != 0 || !(rope_base > 1.0)) return -1;
    if ((policy != POLICY_TOVA && policy != POLICY_WINDOW) || keep_first < 0) return -1;
    const size_t ld = (size_t)cap + 1;
    if (nthreads < 1) nthreads = 1;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads) schedule(static)
#endif
    for (int b = 0; b < B; ++b) {
        REAL *work = (REAL *)malloc(sizeof(REAL) * (size_t)(H + 1) * ld);
        REAL *rot = (REAL *)malloc(sizeof(REAL) * ((size_t)Hkv * ld + (size_t)H) * D);
        if (!work || !rot || len[b] < 0 || len[b] > cap) { bad = 1; free(work); free(rot); continue; }
        step_one_poscomp(H, Hkv, D, cap, scale, policy, keep_first, rope_base,
                         len + b, pos + (size_t)b * cap,
                         K + (size_t)b * Hkv * cap * D, V + (size_t)b * Hkv * cap * D,
                         q + (size_t)b * H * D, k_new + (size_t)b * Hkv * D, v_new + (size_t)b * Hkv * D,
                         pos_t, forced ? forced[b] : -1,
                         out + (size_t)b * H * D, evicted_pos + b, victim + b, argmin + b, gap + b,
                         mean_out ? mean_out + (size_t)b * ld : NULL, cpos_out ? cpos_out + (size_t)b * ld : NULL,
                         work, rot);
        free(work);
        free(rot);
    }
    return bad ? -1 : 0;
}

int tova_oracle_real_bytes(void) { return (int)sizeof(REAL); }

int tova_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
