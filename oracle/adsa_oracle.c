/*
 * CPU oracle for the ADSA decode-attention path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what one
 * layer-step of Adaptive Dynamic Sparse Attention computes, written from the
 * paper's Section 4 (Eq. 1-4 and the cache-update rule of Section 4.2).  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg, and by nothing else: the product path never calls it and shares no code
 * with it.
 *
 * Conventions
 *   - A "stream" is one (batch row, layer, head): its own cache of rows
 *     (pos, k[d], v[d]).  Inputs are float32 arrays holding bf16-exact values;
 *     every sum is accumulated in double.
 *   - Scores (Eq. 2) are rounded to float32 once, then ordered as float32, so
 *     that rows with identical values get identical scores and the position
 *     tie-break is what separates them.
 *   - No blocking, fusion or reordering: each function is the definition
 *     (or the paper's step) written as nested loops.
 *
 * Pins (see tests, marked "not gpu"): dense-attention equivalence when the
 * budget covers the context, brute-force grid-neighbour enumeration,
 * closed forms and hand cases for Eq. 1-2, exhaustive subset search for Eq. 3,
 * set invariants of the update, and the cache sizes printed in Tables 1-2.
 * The attention-mass variant (the comparison method of Section 3.4) is pinned
 * by its own tests: masses add up to the number of steps, subset search for
 * the K highest, a dominant key survives, K = p - 1 evicts the least attended.
 * Image-quality figures (FID, IS, CLIP) are parity unpinned: they need
 * datasets and trained weights.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ADSA_ORACLE_NORM_EPS 1e-8

enum { ADSA_REGION_PREFIX = 0, ADSA_REGION_PREVIOUS = 1, ADSA_REGION_LOCAL = 2, ADSA_REGION_INVALID = -1 };

/* -------------------------------------------------------------------------
 * Section 4.1, the three-region partition [prefix | previous | local].
 *
 * prefix  : the first n_prefix context positions (always kept).
 * local   : image cells that precede the current cell in raster order and lie
 *           in the current grid row or in one of the `rows_back` rows above it.
 *           With rows_back = 1 this is the contiguous span of m = W + c tokens
 *           ending at the previous token, which holds the two neighbours that
 *           Section 3.2 / Fig. 2 show carry the attention mass: the previous
 *           token (g-1) and the token one row up in the same column (g-W).
 * previous: everything else; these are the candidates Eq. 1-3 choose among.
 * A row at or after the current position cannot be in the cache.
 * ------------------------------------------------------------------------- */
int adsa_oracle_region(int pos, int cur_pos, int n_text, int grid_w, int n_prefix, int rows_back)
{
    if (pos < 0 || pos >= cur_pos) return ADSA_REGION_INVALID;
    if (pos < n_prefix) return ADSA_REGION_PREFIX;
    if (pos >= n_text && cur_pos >= n_text) {
        int cell = pos - n_text, cur_cell = cur_pos - n_text;
        int row = cell / grid_w, cur_row = cur_cell / grid_w;
        if (cur_row - row <= rows_back) return ADSA_REGION_LOCAL;
    }
    return ADSA_REGION_PREVIOUS;
}

static double row_norm(const float *x, int d)
{
    double ss = 0.0;
    for (int c = 0; c < d; ++c) ss += (double)x[c] * (double)x[c];
    double n = sqrt(ss);
    return n > ADSA_ORACLE_NORM_EPS ? n : ADSA_ORACLE_NORM_EPS;
}

/* -------------------------------------------------------------------------
 * Eq. 1 and Eq. 2 by definition: S_ij = v_i.v_j / (|v_i| |v_j|) for i != j,
 * S_ii = 0, and S_i = (1/(p-1)) * sum_{j != i} S_ij over the p rows of the
 * "previous" region.  Norms are clamped at 1e-8 so an all-zero row has
 * similarity 0 with everything.  p <= 1 gives S = 0.
 * ------------------------------------------------------------------------- */
void adsa_oracle_score_definition(const float *v, int p, int d, float *score)
{
    for (int i = 0; i < p; ++i) {
        double sum = 0.0;
        double ni = row_norm(v + (size_t)i * d, d);
        for (int j = 0; j < p; ++j) {
            if (j == i) continue; /* S_ii = 0 */
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)v[(size_t)i * d + c] * (double)v[(size_t)j * d + c];
            sum += dot / (ni * row_norm(v + (size_t)j * d, d));
        }
        score[i] = (p > 1) ? (float)(sum / (double)(p - 1)) : 0.0f;
    }
}

/* -------------------------------------------------------------------------
 * The same quantity through the row-sum identity
 *     sum_{j != i} cos(v_i, v_j) = u_i . (sum_j u_j) - u_i . u_i,  u = v/|v|,
 * in O(p d).  It is NOT the oracle of record: it exists so that the cache
 * state of a late step of a large configuration can be produced in reasonable
 * time, and it is itself checked against the definition above.
 * ------------------------------------------------------------------------- */
void adsa_oracle_score_rowsum(const float *v, int p, int d, float *score)
{
    double *s = (double *)calloc((size_t)d, sizeof(double));
    for (int j = 0; j < p; ++j) {
        double nj = row_norm(v + (size_t)j * d, d);
        for (int c = 0; c < d; ++c) s[c] += (double)v[(size_t)j * d + c] / nj;
    }
    for (int i = 0; i < p; ++i) {
        double ni = row_norm(v + (size_t)i * d, d), dot = 0.0, self = 0.0;
        for (int c = 0; c < d; ++c) {
            double u = (double)v[(size_t)i * d + c] / ni;
            dot += u * s[c];
            self += u * u;
        }
        score[i] = (p > 1) ? (float)((dot - self) / (double)(p - 1)) : 0.0f;
    }
    free(s);
}

/* -------------------------------------------------------------------------
 * Eq. 3: the size-K subset with the smallest score sum, i.e. the K lowest
 * scores.  Equal scores are ordered by position, lower position first, which
 * makes the answer unique.  keep[i] = 1 for the chosen rows.
 * ------------------------------------------------------------------------- */
typedef struct { float score; int pos; int idx; } cand_t;

static int cand_less(const void *a, const void *b)
{
    const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
    if (x->score < y->score) return -1;
    if (x->score > y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

void adsa_oracle_select_lowest(const float *score, const int *pos, int p, int K, int *keep)
{
    cand_t *c = (cand_t *)malloc((size_t)(p > 0 ? p : 1) * sizeof(cand_t));
    for (int i = 0; i < p; ++i) { c[i].score = score[i]; c[i].pos = pos[i]; c[i].idx = i; keep[i] = 0; }
    qsort(c, (size_t)p, sizeof(cand_t), cand_less);
    for (int r = 0; r < p && r < K; ++r) keep[c[r].idx] = 1;
    free(c);
}

/* -------------------------------------------------------------------------
 * Attention over a given set of rows (Eq. 4 feeds the gathered K/V into the
 * ordinary softmax attention of Fig. 3): logits q.k_j * scale, softmax with
 * the maximum subtracted, weighted sum of v_j.  With all rows of the context
 * passed in, this is dense causal decode attention.
 * ------------------------------------------------------------------------- */
void adsa_oracle_attend(const float *q, const float *k, const float *v, int n, int d, double scale,
                        double *out, double *weights /* [n] or NULL */)
{
    double *w = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
    double mx = -INFINITY, den = 0.0;
    for (int j = 0; j < n; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += (double)q[c] * (double)k[(size_t)j * d + c];
        w[j] = dot * scale;
        if (w[j] > mx) mx = w[j];
    }
    for (int j = 0; j < n; ++j) { w[j] = exp(w[j] - mx); den += w[j]; }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j < n; ++j) {
        w[j] /= den;
        for (int c = 0; c < d; ++c) out[c] += w[j] * (double)v[(size_t)j * d + c];
    }
    if (weights) memcpy(weights, w, (size_t)n * sizeof(double));
    free(w);
}

/* -------------------------------------------------------------------------
 * One layer-step of one stream, in the paper's order:
 *   1. partition the cached rows (Section 4.1);
 *   2. score the "previous" rows (Eq. 1-2);
 *   3. keep K = min(p, max(0, budget - |prefix| - |local| - 1)) of them
 *      (Eq. 3; the 1 is the new row, which Section 4.2 inserts before
 *      attention runs and which therefore counts toward the budget);
 *   4. attend over prefix + selected + local + the new row (Eq. 4, Fig. 3);
 *   5. the cache becomes exactly that set (Section 4.2: evict, then insert).
 * While the cache has room nothing is evicted and the step is dense
 * attention; once it is full with a fixed budget, exactly the highest-scoring
 * ("most redundant") row goes.
 *
 * score_variant: 0 = Eq. 1-2 by definition (oracle of record), 1 = row-sum identity.
 * Returns 0, or -1 on a malformed cache (bad position) or overflow of cap_rows.
 * ------------------------------------------------------------------------- */
typedef struct {
    int n_text, grid_w, n_prefix, rows_back, score_variant;
    double softmax_scale; /* 0 => 1/sqrt(d) */
} adsa_oracle_params;

int adsa_oracle_layer_step(const adsa_oracle_params *prm, int d, int cap_rows,
                           int *n_live, int *pos, float *k, float *v, /* state, updated in place */
                           const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                           double *out,                      /* [d] */
                           int *n_kept, int *kept_pos,       /* retained cached rows (without the new row) */
                           int *n_evict, int *evict_pos,
                           int *n_cand, int *cand_pos, float *cand_score,
                           double *weights /* [n_kept + 1] (new row last) or NULL */)
{
    int n = *n_live;
    int *region = (int *)malloc((size_t)(n + 1) * sizeof(int));
    int *keep = (int *)malloc((size_t)(n + 1) * sizeof(int));
    float *cv = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    float *gk = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    float *gv = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    int rc = 0, n_pre = 0, n_loc = 0, p = 0;

    /* 1. partition */
    for (int i = 0; i < n; ++i) {
        region[i] = adsa_oracle_region(pos[i], cur_pos, prm->n_text, prm->grid_w, prm->n_prefix, prm->rows_back);
        if (region[i] == ADSA_REGION_INVALID) { rc = -1; goto done; }
        if (region[i] == ADSA_REGION_PREFIX) ++n_pre;
        else if (region[i] == ADSA_REGION_LOCAL) ++n_loc;
        else { cand_pos[p] = pos[i]; memcpy(cv + (size_t)p * d, v + (size_t)i * d, (size_t)d * sizeof(float)); ++p; }
    }
    /* 2. score the candidates */
    if (prm->score_variant == 0) adsa_oracle_score_definition(cv, p, d, cand_score);
    else adsa_oracle_score_rowsum(cv, p, d, cand_score);
    *n_cand = p;
    /* 3. select the K lowest */
    {
        int K = budget - n_pre - n_loc - 1;
        if (K < 0) K = 0;
        if (K > p) K = p;
        adsa_oracle_select_lowest(cand_score, cand_pos, p, K, keep);
    }
    /* 4. gather the retained rows in cache order, the new row last, and attend */
    {
        int m = 0, e = 0, c = 0;
        for (int i = 0; i < n; ++i) {
            int kept = 1;
            if (region[i] == ADSA_REGION_PREVIOUS) kept = keep[c++];
            if (kept) {
                kept_pos[m] = pos[i];
                memcpy(gk + (size_t)m * d, k + (size_t)i * d, (size_t)d * sizeof(float));
                memcpy(gv + (size_t)m * d, v + (size_t)i * d, (size_t)d * sizeof(float));
                ++m;
            } else {
                evict_pos[e++] = pos[i];
            }
        }
        *n_kept = m; *n_evict = e;
        if (m + 1 > cap_rows) { rc = -1; goto done; }
        memcpy(gk + (size_t)m * d, k_new, (size_t)d * sizeof(float));
        memcpy(gv + (size_t)m * d, v_new, (size_t)d * sizeof(float));
        double scale = prm->softmax_scale != 0.0 ? prm->softmax_scale : 1.0 / sqrt((double)d);
        adsa_oracle_attend(q, gk, gv, m + 1, d, scale, out, weights);
        /* 5. the cache is now the retained set plus the new row */
        memcpy(k, gk, (size_t)(m + 1) * d * sizeof(float));
        memcpy(v, gv, (size_t)(m + 1) * d * sizeof(float));
        memcpy(pos, kept_pos, (size_t)m * sizeof(int));
        pos[m] = cur_pos;
        *n_live = m + 1;
    }
done:
    free(region); free(keep); free(cv); free(gk); free(gv);
    return rc;
}

/* -------------------------------------------------------------------------
 * The comparison method of Section 3.4: pruning by attention score, which the
 * paper argues against for image generation (high scores cluster near the
 * current token, so global context is lost).  It is NOT the paper's method;
 * it exists so that the two selection rules can be run side by side on the
 * same cache machinery.  Reading taken here (the paper only names the idea):
 * every cached row carries the attention mass it has received so far, i.e. the
 * sum of its softmax weights over the steps in which it was attended (its own
 * insertion step included); among the "previous" rows the K with the HIGHEST
 * mass are kept, equal masses ordered by position, lower position first.
 * Partition, K, attention and update are those of the step above.
 * ------------------------------------------------------------------------- */
static int cand_more(const void *a, const void *b)
{
    const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

void adsa_oracle_select_highest(const float *score, const int *pos, int p, int K, int *keep)
{
    cand_t *c = (cand_t *)malloc((size_t)(p > 0 ? p : 1) * sizeof(cand_t));
    for (int i = 0; i < p; ++i) { c[i].score = score[i]; c[i].pos = pos[i]; c[i].idx = i; keep[i] = 0; }
    qsort(c, (size_t)p, sizeof(cand_t), cand_more);
    for (int r = 0; r < p && r < K; ++r) keep[c[r].idx] = 1;
    free(c);
}

/* One layer-step of one stream under attention-mass pruning.  mass[i] belongs
 * to cached row i and is updated in place: after the step a retained row's
 * mass has grown by its softmax weight of this step, the new row's mass is its
 * own weight.  Masses are kept as float32 (rounded once per step from a double
 * sum).  cand_score reports the masses the selection saw. */
int adsa_oracle_layer_step_mass(const adsa_oracle_params *prm, int d, int cap_rows,
                                int *n_live, int *pos, float *k, float *v, float *mass,
                                const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                                double *out, int *n_kept, int *kept_pos, int *n_evict, int *evict_pos,
                                int *n_cand, int *cand_pos, float *cand_score)
{
    int n = *n_live;
    int *region = (int *)malloc((size_t)(n + 1) * sizeof(int));
    int *keep = (int *)malloc((size_t)(n + 1) * sizeof(int));
    float *gk = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    float *gv = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    float *gm = (float *)malloc((size_t)(n + 1) * sizeof(float));
    double *w = (double *)malloc((size_t)(n + 1) * sizeof(double));
    int rc = 0, n_pre = 0, n_loc = 0, p = 0;
    for (int i = 0; i < n; ++i) {
        region[i] = adsa_oracle_region(pos[i], cur_pos, prm->n_text, prm->grid_w, prm->n_prefix, prm->rows_back);
        if (region[i] == ADSA_REGION_INVALID) { rc = -1; goto done; }
        if (region[i] == ADSA_REGION_PREFIX) ++n_pre;
        else if (region[i] == ADSA_REGION_LOCAL) ++n_loc;
        else { cand_pos[p] = pos[i]; cand_score[p] = mass[i]; ++p; }
    }
    *n_cand = p;
    {
        int K = budget - n_pre - n_loc - 1;
        if (K < 0) K = 0;
        if (K > p) K = p;
        adsa_oracle_select_highest(cand_score, cand_pos, p, K, keep);
    }
    {
        int m = 0, e = 0, c = 0;
        for (int i = 0; i < n; ++i) {
            int kept = 1;
            if (region[i] == ADSA_REGION_PREVIOUS) kept = keep[c++];
            if (kept) {
                kept_pos[m] = pos[i];
                gm[m] = mass[i];
                memcpy(gk + (size_t)m * d, k + (size_t)i * d, (size_t)d * sizeof(float));
                memcpy(gv + (size_t)m * d, v + (size_t)i * d, (size_t)d * sizeof(float));
                ++m;
            } else {
                evict_pos[e++] = pos[i];
            }
        }
        *n_kept = m; *n_evict = e;
        if (m + 1 > cap_rows) { rc = -1; goto done; }
        memcpy(gk + (size_t)m * d, k_new, (size_t)d * sizeof(float));
        memcpy(gv + (size_t)m * d, v_new, (size_t)d * sizeof(float));
        double scale = prm->softmax_scale != 0.0 ? prm->softmax_scale : 1.0 / sqrt((double)d);
        adsa_oracle_attend(q, gk, gv, m + 1, d, scale, out, w);
        memcpy(k, gk, (size_t)(m + 1) * d * sizeof(float));
        memcpy(v, gv, (size_t)(m + 1) * d * sizeof(float));
        memcpy(pos, kept_pos, (size_t)m * sizeof(int));
        pos[m] = cur_pos;
        for (int j = 0; j < m; ++j) mass[j] = (float)((double)gm[j] + w[j]);
        mass[m] = (float)w[m];
        *n_live = m + 1;
    }
done:
    free(region); free(keep); free(gk); free(gv); free(gm); free(w);
    return rc;
}

int adsa_oracle_layer_step_mass_batch(const adsa_oracle_params *prm, int n_streams, int d, int cap_rows,
                                      int *n_live, int *pos, float *k, float *v, float *mass,
                                      const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                                      double *out, int *n_kept, int *kept_pos, int *n_evict, int *evict_pos,
                                      int *n_cand, int *cand_pos, float *cand_score, int n_threads)
{
    int failed = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : failed)
#endif
    for (int s = 0; s < n_streams; ++s) {
        size_t r = (size_t)s * cap_rows;
        int rc = adsa_oracle_layer_step_mass(prm, d, cap_rows, n_live + s, pos + r, k + r * d, v + r * d, mass + r,
                                             q + (size_t)s * d, k_new + (size_t)s * d, v_new + (size_t)s * d,
                                             cur_pos, budget, out + (size_t)s * d,
                                             n_kept + s, kept_pos + r, n_evict + s, evict_pos + r,
                                             n_cand + s, cand_pos + r, cand_score + r);
        if (rc != 0) ++failed;
    }
    return failed;
}

/* -------------------------------------------------------------------------
 * Granularity variant.  The paper does not say at which granularity V rows are
 * compared (Section 4.1 speaks of "the V of each token").  The default reading
 * is per stream (one head).  This variant compares a token's V over ALL heads of
 * a layer as one vector of n_heads * d elements, so one score per (batch row,
 * token) and the same tokens kept for every head.  The n_heads streams of a
 * batch row are stepped together; their caches must hold the same positions in
 * the same order (they do if they are always stepped together).  Partition, K,
 * attention (per head) and update are those of the per-stream step.
 * Returns 0, -1 on malformed input, -2 if the heads' caches differ.
 * ------------------------------------------------------------------------- */
int adsa_oracle_layer_step_shared(const adsa_oracle_params *prm, int n_heads, int d, int cap_rows,
                                  int *n_live, int *pos, float *k, float *v, /* [n_heads] streams, stride cap_rows */
                                  const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                                  double *out, int *n_kept, int *kept_pos, int *n_evict, int *evict_pos,
                                  int *n_cand, int *cand_pos, float *cand_score)
{
    const int n = n_live[0], D = n_heads * d;
    for (int h = 1; h < n_heads; ++h) {
        if (n_live[h] != n) return -2;
        for (int i = 0; i < n; ++i) if (pos[(size_t)h * cap_rows + i] != pos[i]) return -2;
    }
    int *region = (int *)malloc((size_t)(n + 1) * sizeof(int));
    int *keep = (int *)malloc((size_t)(n + 1) * sizeof(int));
    int *cpos = (int *)malloc((size_t)(n + 1) * sizeof(int));
    float *cscore = (float *)malloc((size_t)(n + 1) * sizeof(float));
    float *cv = (float *)malloc((size_t)(n + 1) * D * sizeof(float));
    float *gk = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    float *gv = (float *)malloc((size_t)(n + 1) * d * sizeof(float));
    int rc = 0, n_pre = 0, n_loc = 0, p = 0;
    for (int i = 0; i < n; ++i) {
        region[i] = adsa_oracle_region(pos[i], cur_pos, prm->n_text, prm->grid_w, prm->n_prefix, prm->rows_back);
        if (region[i] == ADSA_REGION_INVALID) { rc = -1; goto done; }
        if (region[i] == ADSA_REGION_PREFIX) ++n_pre;
        else if (region[i] == ADSA_REGION_LOCAL) ++n_loc;
        else {
            cpos[p] = pos[i];
            for (int h = 0; h < n_heads; ++h)   /* the token's V over all heads, head after head */
                memcpy(cv + (size_t)p * D + (size_t)h * d, v + ((size_t)h * cap_rows + i) * d, (size_t)d * sizeof(float));
            ++p;
        }
    }
    adsa_oracle_score_definition(cv, p, D, cscore);
    {
        int K = budget - n_pre - n_loc - 1;
        if (K < 0) K = 0;
        if (K > p) K = p;
        adsa_oracle_select_lowest(cscore, cpos, p, K, keep);
    }
    for (int h = 0; h < n_heads && rc == 0; ++h) {
        size_t r = (size_t)h * cap_rows;
        int m = 0, e = 0, c = 0;
        for (int i = 0; i < n; ++i) {
            int kept = 1;
            if (region[i] == ADSA_REGION_PREVIOUS) kept = keep[c++];
            if (kept) {
                kept_pos[r + m] = pos[r + i];
                memcpy(gk + (size_t)m * d, k + (r + i) * d, (size_t)d * sizeof(float));
                memcpy(gv + (size_t)m * d, v + (r + i) * d, (size_t)d * sizeof(float));
                ++m;
            } else {
                evict_pos[r + e++] = pos[r + i];
            }
        }
        n_kept[h] = m; n_evict[h] = e; n_cand[h] = p;
        memcpy(cand_pos + r, cpos, (size_t)p * sizeof(int));
        memcpy(cand_score + r, cscore, (size_t)p * sizeof(float));
        if (m + 1 > cap_rows) { rc = -1; break; }
        memcpy(gk + (size_t)m * d, k_new + (size_t)h * d, (size_t)d * sizeof(float));
        memcpy(gv + (size_t)m * d, v_new + (size_t)h * d, (size_t)d * sizeof(float));
        double scale = prm->softmax_scale != 0.0 ? prm->softmax_scale : 1.0 / sqrt((double)d);
        adsa_oracle_attend(q + (size_t)h * d, gk, gv, m + 1, d, scale, out + (size_t)h * d, NULL);
        memcpy(k + r * d, gk, (size_t)(m + 1) * d * sizeof(float));
        memcpy(v + r * d, gv, (size_t)(m + 1) * d * sizeof(float));
        memcpy(pos + r, kept_pos + r, (size_t)m * sizeof(int));
        pos[r + m] = cur_pos;
        n_live[h] = m + 1;
    }
done:
    free(region); free(keep); free(cpos); free(cscore); free(cv); free(gk); free(gv);
    return rc;
}

int adsa_oracle_layer_step_shared_batch(const adsa_oracle_params *prm, int n_rows_batch, int n_heads, int d, int cap_rows,
                                        int *n_live, int *pos, float *k, float *v,
                                        const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                                        double *out, int *n_kept, int *kept_pos, int *n_evict, int *evict_pos,
                                        int *n_cand, int *cand_pos, float *cand_score, int n_threads)
{
    int failed = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : failed)
#endif
    for (int b = 0; b < n_rows_batch; ++b) {
        size_t s0 = (size_t)b * n_heads, r = s0 * cap_rows;
        int rc = adsa_oracle_layer_step_shared(prm, n_heads, d, cap_rows, n_live + s0, pos + r, k + r * d, v + r * d,
                                               q + s0 * d, k_new + s0 * d, v_new + s0 * d, cur_pos, budget, out + s0 * d,
                                               n_kept + s0, kept_pos + r, n_evict + s0, evict_pos + r,
                                               n_cand + s0, cand_pos + r, cand_score + r);
        if (rc != 0) ++failed;
    }
    return failed;
}

/* -------------------------------------------------------------------------
 * Dense causal attention over the rows of the condition (how the text tokens
 * enter the cache before decoding starts; Section 4.2: the method is plain
 * attention while the cache has room): out_i = attention of q_i over rows 0..i.
 * ------------------------------------------------------------------------- */
void adsa_oracle_causal_attend(const float *q, const float *k, const float *v, int n, int d, double scale, double *out)
{
    for (int i = 0; i < n; ++i)
        adsa_oracle_attend(q + (size_t)i * d, k, v, i + 1, d, scale, out + (size_t)i * d, NULL);
}

/* -------------------------------------------------------------------------
 * Two-dimensional rotary position embedding of q or k rows (Section 4.1 notes
 * that RoPE sits on Q and K, which is why V is what gets compared).  The paper
 * does not spell the embedding out; reading taken: elements are rotated in
 * consecutive pairs (2i, 2i+1); the first d/4 pairs turn with the token's grid
 * ROW, the next d/4 pairs with its grid COLUMN, pair i of either half by the
 * angle index * base^(-i / (d/4)); a token of the text condition (pos < n_text)
 * is not rotated.  d must be a multiple of 4.  x: [n][d], pos: [n].
 * ------------------------------------------------------------------------- */
void adsa_oracle_rope_2d(const float *x, const int *pos, int n, int d, int n_text, int grid_w, double base, double *out)
{
    const int quarter = d / 4;
    for (int r = 0; r < n; ++r) {
        const int cell = pos[r] - n_text;
        for (int i = 0; i < d / 2; ++i) {
            double angle = 0.0;
            if (cell >= 0) {
                const int index = i < quarter ? cell / grid_w : cell % grid_w;
                angle = (double)index * pow(base, -(double)(i % quarter) / (double)quarter);
            }
            const double a = x[(size_t)r * d + 2 * i], b = x[(size_t)r * d + 2 * i + 1];
            out[(size_t)r * d + 2 * i] = a * cos(angle) - b * sin(angle);
            out[(size_t)r * d + 2 * i + 1] = a * sin(angle) + b * cos(angle);
        }
    }
}

/* -------------------------------------------------------------------------
 * The pieces of the host model around the attention (Section 5 integrates the
 * method with LlamaGen; the paper defines none of these, they are the published
 * operations of that decoder family).  Parity of a whole generated image is
 * unpinned (no trained weights); each operation is pinned by its definition.
 * ------------------------------------------------------------------------- */

/* Root-mean-square normalisation: y_i = x_i / sqrt(mean_j x_j^2 + eps) * w_i.  x: [rows][dim], w: [dim]. */
void adsa_oracle_rmsnorm(const float *x, const float *w, int rows, int dim, double eps, double *out)
{
    for (int r = 0; r < rows; ++r) {
        double ss = 0.0;
        for (int i = 0; i < dim; ++i) ss += (double)x[(size_t)r * dim + i] * (double)x[(size_t)r * dim + i];
        const double inv = 1.0 / sqrt(ss / (double)dim + eps);
        for (int i = 0; i < dim; ++i) out[(size_t)r * dim + i] = (double)x[(size_t)r * dim + i] * inv * (double)w[i];
    }
}

/* The gated activation of the feed-forward block: out = silu(gate) * up, silu(g) = g / (1 + exp(-g)). */
void adsa_oracle_swiglu(const float *gate, const float *up, long long n, double *out)
{
    for (long long i = 0; i < n; ++i) {
        const double g = gate[i];
        out[i] = g / (1.0 + exp(-g)) * (double)up[i];
    }
}

/* Classifier-free guidance and sampling of the next image token for one image.
 * logits_cond, logits_uncond: [vocab].  Steps: mixed = uncond + scale * (cond - uncond); keep the top_k largest
 * mixed logits (equal logits at the threshold: the lower token id is kept); p_i proportional to
 * exp((mixed_i - max) / temperature) over the kept tokens; the token is the first kept id, in ascending order of
 * id, at which the running sum of p reaches u * (sum of p), u in [0, 1) given by the caller.
 * mixed_out [vocab] (may be NULL) receives the mixed logits, cdf_out [vocab] (may be NULL) the running sum
 * divided by the total at every id (unchanged across ids that are not kept).  Returns the token. */
int adsa_oracle_cfg_sample(const float *logits_cond, const float *logits_uncond, int vocab, double scale, int top_k,
                           double temperature, double u, double *mixed_out, double *cdf_out)
{
    double *mixed = (double *)malloc(sizeof(double) * (size_t)vocab);
    char *kept = (char *)calloc((size_t)vocab, 1);
    for (int i = 0; i < vocab; ++i) mixed[i] = (double)logits_uncond[i] + scale * ((double)logits_cond[i] - (double)logits_uncond[i]);
    if (top_k < 1) top_k = 1;
    if (top_k > vocab) top_k = vocab;
    for (int n = 0; n < top_k; ++n) {            /* pick the largest not yet kept, lowest id first among equals */
        int best = -1;
        for (int i = 0; i < vocab; ++i)
            if (!kept[i] && (best < 0 || mixed[i] > mixed[best])) best = i;
        kept[best] = 1;
    }
    double mx = -INFINITY, total = 0.0;
    for (int i = 0; i < vocab; ++i) if (kept[i] && mixed[i] > mx) mx = mixed[i];
    for (int i = 0; i < vocab; ++i) if (kept[i]) total += exp((mixed[i] - mx) / temperature);
    double run = 0.0;
    int token = -1, last_kept = -1;
    for (int i = 0; i < vocab; ++i) {
        if (kept[i]) {
            run += exp((mixed[i] - mx) / temperature);
            last_kept = i;
            if (token < 0 && run >= u * total) token = i;
        }
        if (cdf_out) cdf_out[i] = run / total;
        if (mixed_out) mixed_out[i] = mixed[i];
    }
    if (token < 0) token = last_kept;            /* rounding at u close to 1 */
    free(mixed);
    free(kept);
    return token;
}

/* The same step for many independent streams.  Arrays carry a leading stream
 * dimension with stride cap_rows (state, lists) or d (q, k_new, v_new, out).
 * Threads split the streams; nothing else is parallel.  Returns the number of
 * streams that failed. */
int adsa_oracle_layer_step_batch(const adsa_oracle_params *prm, int n_streams, int d, int cap_rows,
                                 int *n_live, int *pos, float *k, float *v,
                                 const float *q, const float *k_new, const float *v_new, int cur_pos, int budget,
                                 double *out, int *n_kept, int *kept_pos, int *n_evict, int *evict_pos,
                                 int *n_cand, int *cand_pos, float *cand_score, int n_threads)
{
    int failed = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : failed)
#endif
    for (int s = 0; s < n_streams; ++s) {
        size_t r = (size_t)s * cap_rows;
        int rc = adsa_oracle_layer_step(prm, d, cap_rows, n_live + s, pos + r, k + r * d, v + r * d,
                                        q + (size_t)s * d, k_new + (size_t)s * d, v_new + (size_t)s * d,
                                        cur_pos, budget, out + (size_t)s * d,
                                        n_kept + s, kept_pos + r, n_evict + s, evict_pos + r,
                                        n_cand + s, cand_pos + r, cand_score + r, NULL);
        if (rc != 0) ++failed;
    }
    return failed;
}

int adsa_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
