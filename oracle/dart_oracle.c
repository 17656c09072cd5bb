/*
 * DART token-reduction oracle: TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded fp64 restatement of the duplication-aware
 * token-reduction step of DART (arxiv 2502.11494), written from the paper's
 * definitions.  It exists so that the CUDA library can be checked against
 * something that can be compared with the paper by eye.  It shares no code,
 * header, table or helper with the CUDA path.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.
 *
 * Inputs are bf16 bit patterns (uint16_t) that are widened exactly to fp64;
 * every sum is a plain left-to-right fp64 accumulation; every ordering is a
 * full sort with an explicit total order (value, then token index).
 *
 * Steps (one sample; the batch entry point loops over samples):
 *   scores      Sec. 3.3, footnote on "K-norm": L1 norm of each token's row
 *               of the key matrix; the Euclidean norm needed by Eq. 7.
 *   pivots      Def. 1 + Table 1 caption: the k tokens of maximum K-norm.
 *   similarity  Def. 2, Eq. 7: dup(p_i, x_j) = p_i.x_j / (|p_i| |x_j|).
 *   retention   Eq. 9-10 with a per-pivot threshold set by the budget:
 *               pivot i (rank order) retains its q_i not-yet-retained,
 *               non-pivot tokens of LOWEST dup; eps_i = largest retained dup;
 *               R = P u U_i R_i, |R| = n_keep exactly.
 *   compaction  the retained tokens stay in original order; text tokens
 *               are all kept; hidden rows and position ids are gathered.
 *
 * Readings of points the paper leaves open (ties -> lower index; the r
 * highest-ranked pivots take one extra token when (n_keep - P) % P = r;
 * a zero-norm row has dup 0) are the library's documented readings; the
 * functions whose behaviour rests on such a reading say so below.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_SHAPE (-2)
#define ORACLE_ERR_NOMEM (-6)

/* owner[] codes */
#define OWNER_DROPPED (-1)

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; /* bf16 is the top half of an IEEE binary32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

typedef struct {
    double v;
    int32_t idx;
} keyed_t;

/* descending value, ascending index */
static int cmp_desc(const void *a, const void *b)
{
    const keyed_t *x = (const keyed_t *)a, *y = (const keyed_t *)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/* ascending value, ascending index */
static int cmp_asc(const void *a, const void *b)
{
    const keyed_t *x = (const keyed_t *)a, *y = (const keyed_t *)b;
    if (x->v < y->v) return -1;
    if (x->v > y->v) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/*
 * Scores of the vision tokens of one sample (Sec. 3.3 footnote: K-norm is the
 * L1 norm of the K matrix, taken per token row; Eq. 7 needs the Euclidean norm).
 *   keys   [S, d] bf16 bits, row-major; vision rows are [vis_offset, vis_offset+n_vis)
 *   l1     [n_vis]  sum_c |K[j,c]|
 *   l2     [n_vis]  sqrt(sum_c K[j,c]^2)
 */
int dart_oracle_scores(const uint16_t *keys, int S, int d, int vis_offset, int n_vis,
                       double *l1, double *l2)
{
    if (S < 1 || d < 1 || vis_offset < 0 || n_vis < 0 || vis_offset + n_vis > S) return ORACLE_ERR_SHAPE;
    for (int j = 0; j < n_vis; ++j) {
        const uint16_t *row = keys + (size_t)(vis_offset + j) * (size_t)d;
        double a = 0.0, q = 0.0;
        for (int c = 0; c < d; ++c) {
            double x = bf16_to_f64(row[c]);
            a += fabs(x);
            q += x * x;
        }
        l1[j] = a;
        l2[j] = sqrt(q);
    }
    return ORACLE_OK;
}

/*
 * Pivot tokens (Def. 1; Table 1 caption: chosen by maximum K-norm).
 * The P tokens of largest score, in rank order (rank 0 = largest).
 * largest != 0 : maximum-score pivots (the paper's main setting);
 * largest == 0 : minimum-score pivots (the ablation's "smallest value" variant).
 * Equal scores: the lower token index ranks first (reading; the paper is silent).
 *   gap_out (may be NULL): min over ranks t = 0..P-1 of the relative gap
 *   |s_(t) - s_(t+1)| / |s_(t)| between consecutive tokens in the ranking
 *   (up to and including the gap to the first non-pivot); +inf when P = n_vis
 *   has no successor for the last rank.
 */
int dart_oracle_pivots(const double *score, int n_vis, int P, int largest,
                       int32_t *pivot_idx, double *gap_out)
{
    if (P < 1 || P > n_vis) return ORACLE_ERR_SHAPE;
    keyed_t *k = (keyed_t *)malloc((size_t)n_vis * sizeof *k);
    if (!k) return ORACLE_ERR_NOMEM;
    for (int j = 0; j < n_vis; ++j) {
        k[j].v = score[j];
        k[j].idx = j;
    }
    qsort(k, (size_t)n_vis, sizeof *k, largest ? cmp_desc : cmp_asc);
    for (int i = 0; i < P; ++i) pivot_idx[i] = k[i].idx;
    if (gap_out) {
        double g = INFINITY;
        for (int t = 0; t < P && t + 1 < n_vis; ++t) {
            double den = fabs(k[t].v);
            double rel = den > 0.0 ? fabs(k[t].v - k[t + 1].v) / den : 0.0;
            if (rel < g) g = rel;
        }
        *gap_out = g;
    }
    free(k);
    return ORACLE_OK;
}

/*
 * Duplication scores (Def. 2, Eq. 7): cosine of pivot i and vision token j,
 * dup[i*n_vis + j] = (K_{p_i} . K_j) / (|K_{p_i}| |K_j|).
 * A zero-norm operand gives dup = 0 (reading; Eq. 7 is undefined there).
 */
int dart_oracle_similarity(const uint16_t *keys, int S, int d, int vis_offset, int n_vis,
                           const int32_t *pivot_idx, int P, const double *l2, double *dup)
{
    if (S < 1 || d < 1 || vis_offset < 0 || n_vis < 0 || vis_offset + n_vis > S || P < 1) return ORACLE_ERR_SHAPE;
    for (int i = 0; i < P; ++i) {
        int p = pivot_idx[i];
        if (p < 0 || p >= n_vis) return ORACLE_ERR_SHAPE;
        const uint16_t *prow = keys + (size_t)(vis_offset + p) * (size_t)d;
        for (int j = 0; j < n_vis; ++j) {
            const uint16_t *xrow = keys + (size_t)(vis_offset + j) * (size_t)d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += bf16_to_f64(prow[c]) * bf16_to_f64(xrow[c]);
            double den = l2[p] * l2[j];
            dup[(size_t)i * (size_t)n_vis + j] = den > 0.0 ? dot / den : 0.0;
        }
    }
    return ORACLE_OK;
}

/*
 * Eq. 7 when pivots may be ANY token of the sequence (the paper also tries pivots taken from the text tokens,
 * Sec. 5.4): pivot_idx is still relative to the vision block, so a text token before it has a negative index and
 * one after it an index >= n_vis.  Every norm is computed here from its row; a zero norm gives dup = 0.
 */
int dart_oracle_similarity_any(const uint16_t *keys, int S, int d, int vis_offset, int n_vis,
                               const int32_t *pivot_idx, int P, double *dup)
{
    if (S < 1 || d < 1 || vis_offset < 0 || n_vis < 0 || vis_offset + n_vis > S || P < 1) return ORACLE_ERR_SHAPE;
    for (int i = 0; i < P; ++i) {
        const int s = vis_offset + pivot_idx[i];
        if (s < 0 || s >= S) return ORACLE_ERR_SHAPE;
        const uint16_t *prow = keys + (size_t)s * (size_t)d;
        double pp = 0.0;
        for (int c = 0; c < d; ++c) pp += bf16_to_f64(prow[c]) * bf16_to_f64(prow[c]);
        for (int j = 0; j < n_vis; ++j) {
            const uint16_t *xrow = keys + (size_t)(vis_offset + j) * (size_t)d;
            double dot = 0.0, xx = 0.0;
            for (int c = 0; c < d; ++c) {
                dot += bf16_to_f64(prow[c]) * bf16_to_f64(xrow[c]);
                xx += bf16_to_f64(xrow[c]) * bf16_to_f64(xrow[c]);
            }
            const double den = sqrt(pp) * sqrt(xx);
            dup[(size_t)i * (size_t)n_vis + j] = den > 0.0 ? dot / den : 0.0;
        }
    }
    return ORACLE_OK;
}

/*
 * Retention under the budget (Eq. 9-10; Sec. 1: "retain the vision tokens with the
 * lowest cosine similarity to the pivots"; eps is set per pivot from the ratio).
 *
 *   kept := { p_0 .. p_{P-1} }                         (P subset of R, Eq. 10)
 *   q = (n_keep - P) / P, r = (n_keep - P) % P; q_i = q + 1 for rank i < r, else q
 *   for i = 0 .. P-1 (rank order):
 *       candidates := vision tokens not in kept
 *       order them by (dup[i][j] ascending, j ascending)
 *       R_i := the first q_i;  kept := kept u R_i;  eps_i := max dup over R_i  (Eq. 9)
 *
 * Outputs (any may be NULL except keep):
 *   keep   [n_vis] 1 = retained
 *   owner  [n_vis] -1 dropped, i in [0,P) = retained by pivot i, P + i = is pivot of rank i
 *   eps    [P]     eps_i, NaN when q_i = 0
 *   gap    scalar  min over pivots with q_i > 0 of (dup of the best candidate NOT taken) - eps_i,
 *                  +inf if no pivot leaves a candidate behind
 * The equal split of the budget, the order of the pivots' turns and the exclusion of already
 * retained tokens are readings of the sentence that eps follows from the reduction ratio.
 */
/*
 * With text_pivots != 0 a pivot index outside [0, n_vis) names a text token: it takes its turn like any pivot but is
 * not a vision token, so it is neither marked nor counted: the budget is split as q = (n_keep - Pv) / P,
 * r = (n_keep - Pv) % P with Pv the pivots inside the vision block, and |kept| = n_keep vision tokens as always.
 */
static int retention_quotas(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                            uint8_t *keep, int32_t *owner, double *eps, double *gap_out);

int dart_oracle_retention(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                          uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    return retention_quotas(dup, pivot_idx, n_vis, P, n_keep, 0, keep, owner, eps, gap_out);
}

int dart_oracle_retention_any(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                              uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    return retention_quotas(dup, pivot_idx, n_vis, P, n_keep, 1, keep, owner, eps, gap_out);
}

static int retention_quotas(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                            uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    if (P < 1 || P > n_keep || n_keep > n_vis) return ORACLE_ERR_SHAPE;
    keyed_t *cand = (keyed_t *)malloc((size_t)n_vis * sizeof *cand);
    if (!cand) return ORACLE_ERR_NOMEM;
    memset(keep, 0, (size_t)n_vis);
    if (owner)
        for (int j = 0; j < n_vis; ++j) owner[j] = OWNER_DROPPED;
    int Pv = 0;
    for (int i = 0; i < P; ++i) {
        int p = pivot_idx[i];
        if (text_pivots && (p < 0 || p >= n_vis)) { /* a text token: distinctness among those is the caller's business */
            for (int k = 0; k < i; ++k)
                if (pivot_idx[k] == p) {
                    free(cand);
                    return ORACLE_ERR_SHAPE;
                }
            continue;
        }
        if (p < 0 || p >= n_vis || keep[p]) {
            free(cand);
            return ORACLE_ERR_SHAPE; /* pivots must be distinct vision tokens */
        }
        keep[p] = 1;
        if (owner) owner[p] = P + i;
        ++Pv;
    }
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    double gap = INFINITY;
    for (int i = 0; i < P; ++i) {
        const int qi = q + (i < r ? 1 : 0);
        if (eps) eps[i] = NAN;
        if (qi == 0) continue;
        int m = 0;
        for (int j = 0; j < n_vis; ++j)
            if (!keep[j]) {
                cand[m].v = dup[(size_t)i * (size_t)n_vis + j];
                cand[m].idx = j;
                ++m;
            }
        /* m >= qi always: n_vis - (tokens kept so far) >= n_vis - n_keep + qi */
        qsort(cand, (size_t)m, sizeof *cand, cmp_asc);
        for (int t = 0; t < qi; ++t) {
            keep[cand[t].idx] = 1;
            if (owner) owner[cand[t].idx] = i;
        }
        if (eps) eps[i] = cand[qi - 1].v;
        if (m > qi) {
            double g = cand[qi].v - cand[qi - 1].v;
            if (g < gap) gap = g;
        }
    }
    if (gap_out) *gap_out = gap;
    free(cand);
    return ORACLE_OK;
}

/*
 * Retention with INDEPENDENT pivots (Eq. 9-10 read literally: R = P u U_i R_i, every R_i built from all
 * non-pivot tokens whatever the other pivots took).  Pivot i takes its q_i non-pivot tokens of lowest dup
 * (quotas as in dart_oracle_retention; equal values: lower index first); a token that is lowest for two
 * pivots is retained once, so |R| <= n_keep and the packed length depends on the data.
 *   owner  [n_vis] -1 dropped, i = the first pivot in rank order that took the token, P + i = pivot of rank i
 *   eps    [P]     the largest dup pivot i took, NaN if its quota is 0
 *   gap    scalar  min over pivots of (best dup left behind by that pivot - eps_i), +inf if none
 *   n_kept         |R|
 */
static int retention_union(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                           uint8_t *keep, int32_t *owner, double *eps, double *gap_out, int32_t *n_kept);

int dart_oracle_retention_union(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                                uint8_t *keep, int32_t *owner, double *eps, double *gap_out, int32_t *n_kept)
{
    return retention_union(dup, pivot_idx, n_vis, P, n_keep, 0, keep, owner, eps, gap_out, n_kept);
}

/* The same with pivots that may be text tokens (index outside [0, n_vis), see dart_oracle_retention_any): a text pivot
 * takes its picks like any pivot but is no vision token, so the quotas split n_keep - Pv, Pv = the pivots inside the block. */
int dart_oracle_retention_union_any(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                                    uint8_t *keep, int32_t *owner, double *eps, double *gap_out, int32_t *n_kept)
{
    return retention_union(dup, pivot_idx, n_vis, P, n_keep, 1, keep, owner, eps, gap_out, n_kept);
}

static int retention_union(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                           uint8_t *keep, int32_t *owner, double *eps, double *gap_out, int32_t *n_kept)
{
    if (P < 1 || P > n_keep || n_keep > n_vis) return ORACLE_ERR_SHAPE;
    keyed_t *cand = (keyed_t *)malloc((size_t)n_vis * sizeof *cand);
    uint8_t *is_pivot = (uint8_t *)calloc((size_t)n_vis, 1);
    if (!cand || !is_pivot) {
        free(cand);
        free(is_pivot);
        return ORACLE_ERR_NOMEM;
    }
    memset(keep, 0, (size_t)n_vis);
    if (owner)
        for (int j = 0; j < n_vis; ++j) owner[j] = OWNER_DROPPED;
    int Pv = 0;
    for (int i = 0; i < P; ++i) {
        const int p = pivot_idx[i];
        if (text_pivots && (p < 0 || p >= n_vis)) { /* a text token: only distinctness is checked */
            for (int k = 0; k < i; ++k)
                if (pivot_idx[k] == p) {
                    free(cand);
                    free(is_pivot);
                    return ORACLE_ERR_SHAPE;
                }
            continue;
        }
        if (p < 0 || p >= n_vis || is_pivot[p]) {
            free(cand);
            free(is_pivot);
            return ORACLE_ERR_SHAPE; /* pivots must be distinct vision tokens */
        }
        is_pivot[p] = 1;
        keep[p] = 1;
        if (owner) owner[p] = P + i;
        ++Pv;
    }
    const int q = (n_keep - Pv) / P, r = (n_keep - Pv) % P;
    double gap = INFINITY;
    for (int i = 0; i < P; ++i) {
        const int qi = q + (i < r ? 1 : 0);
        if (eps) eps[i] = NAN;
        if (qi == 0) continue;
        int m = 0;
        for (int j = 0; j < n_vis; ++j)
            if (!is_pivot[j]) { /* every non-pivot token, also those another pivot has taken */
                cand[m].v = dup[(size_t)i * (size_t)n_vis + j];
                cand[m].idx = j;
                ++m;
            }
        qsort(cand, (size_t)m, sizeof *cand, cmp_asc); /* m = n_vis - Pv >= n_keep - Pv >= qi */
        for (int t = 0; t < qi; ++t) {
            const int j = cand[t].idx;
            if (owner && !keep[j]) owner[j] = i;
            keep[j] = 1;
        }
        if (eps) eps[i] = cand[qi - 1].v;
        if (m > qi) {
            const double g = cand[qi].v - cand[qi - 1].v;
            if (g < gap) gap = g;
        }
    }
    int32_t cnt = 0;
    for (int j = 0; j < n_vis; ++j) cnt += keep[j];
    if (n_kept) *n_kept = cnt;
    if (gap_out) *gap_out = gap;
    free(cand);
    free(is_pivot);
    return ORACLE_OK;
}

/*
 * Retention with ONE threshold for all pivots (a second reading of Def. 2 / Eq. 8-9): a token is an
 * eps-duplicate of the pivot set if its dup to SOME pivot exceeds eps, so a token's duplication is its
 * highest dup over the pivots, u_j = max_i dup(p_i, x_j); the n_keep - P non-pivot tokens of lowest u_j are
 * retained (equal values: lower index first), eps = the largest retained u_j, R = P u {x_j : u_j <= eps}.
 *   owner  [n_vis] -1 dropped, i = retained and most similar to pivot i (lowest i on equal dup), P + i = pivot
 *   eps    [P]     the one threshold, repeated; NaN when n_keep = P
 *   gap    scalar  (u of the best token NOT taken) - eps, +inf if none is left behind
 */
static int retention_global(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                            uint8_t *keep, int32_t *owner, double *eps, double *gap_out);

int dart_oracle_retention_global(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                                 uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    return retention_global(dup, pivot_idx, n_vis, P, n_keep, 0, keep, owner, eps, gap_out);
}

/* The same with pivots that may be text tokens (index outside [0, n_vis)): they count among the pivots a token is compared
 * with, but not among the vision tokens kept, so n_keep - Pv non-pivot tokens are retained, Pv = the pivots inside the block. */
int dart_oracle_retention_global_any(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep,
                                     uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    return retention_global(dup, pivot_idx, n_vis, P, n_keep, 1, keep, owner, eps, gap_out);
}

static int retention_global(const double *dup, const int32_t *pivot_idx, int n_vis, int P, int n_keep, int text_pivots,
                            uint8_t *keep, int32_t *owner, double *eps, double *gap_out)
{
    if (P < 1 || P > n_keep || n_keep > n_vis) return ORACLE_ERR_SHAPE;
    keyed_t *cand = (keyed_t *)malloc((size_t)n_vis * sizeof *cand);
    int32_t *nearest = (int32_t *)malloc((size_t)n_vis * sizeof *nearest);
    if (!cand || !nearest) {
        free(cand);
        free(nearest);
        return ORACLE_ERR_NOMEM;
    }
    memset(keep, 0, (size_t)n_vis);
    if (owner)
        for (int j = 0; j < n_vis; ++j) owner[j] = OWNER_DROPPED;
    int Pv = 0;
    for (int i = 0; i < P; ++i) {
        int p = pivot_idx[i];
        if (text_pivots && (p < 0 || p >= n_vis)) { /* a text token: only distinctness is checked */
            for (int k = 0; k < i; ++k)
                if (pivot_idx[k] == p) {
                    free(cand);
                    free(nearest);
                    return ORACLE_ERR_SHAPE;
                }
            continue;
        }
        if (p < 0 || p >= n_vis || keep[p]) {
            free(cand);
            free(nearest);
            return ORACLE_ERR_SHAPE; /* pivots must be distinct vision tokens */
        }
        keep[p] = 1;
        if (owner) owner[p] = P + i;
        ++Pv;
    }
    int m = 0;
    for (int j = 0; j < n_vis; ++j) {
        if (keep[j]) continue;
        double u = dup[j];
        int arg = 0;
        for (int i = 1; i < P; ++i)
            if (dup[(size_t)i * (size_t)n_vis + j] > u) {
                u = dup[(size_t)i * (size_t)n_vis + j];
                arg = i;
            }
        cand[m].v = u;
        cand[m].idx = j;
        nearest[j] = arg;
        ++m;
    }
    const int take = n_keep - Pv;
    qsort(cand, (size_t)m, sizeof *cand, cmp_asc);
    for (int t = 0; t < take; ++t) {
        keep[cand[t].idx] = 1;
        if (owner) owner[cand[t].idx] = nearest[cand[t].idx];
    }
    if (eps)
        for (int i = 0; i < P; ++i) eps[i] = take > 0 ? cand[take - 1].v : NAN;
    if (gap_out) *gap_out = (take > 0 && m > take) ? cand[take].v - cand[take - 1].v : INFINITY;
    free(cand);
    free(nearest);
    return ORACLE_OK;
}

/*
 * Pivots from both modalities (Sec. 5.4 finds that pivots from either modality alone do worse; the pivot-selection
 * table's caption uses "4 visual and 4 text tokens"): the Pv vision tokens and the Pt text tokens of largest (or
 * smallest) score, each group ranked like dart_oracle_pivots (equal scores: lower sequence position first).
 *   score_all [S] the score of EVERY token of the sample (K-norm of its key row)
 *   pivot_idx [Pv + Pt] relative to the vision block (a text token before it is negative, one after it >= n_vis):
 *             the vision pivots in rank order, then the text pivots in rank order (reading: the paper does not say in
 *             which order pivots of different modality take their turns)
 * Needs Pv <= n_vis and Pt <= S - n_vis.
 */
int dart_oracle_pivots_mixed(const double *score_all, int S, int vis_offset, int n_vis, int Pv, int Pt, int largest,
                             int32_t *pivot_idx)
{
    if (S < 1 || vis_offset < 0 || n_vis < 0 || vis_offset + n_vis > S || Pv < 0 || Pt < 0 || Pv > n_vis || Pt > S - n_vis)
        return ORACLE_ERR_SHAPE;
    keyed_t *t = (keyed_t *)malloc((size_t)S * sizeof *t);
    if (!t) return ORACLE_ERR_NOMEM;
    int m = 0;
    for (int j = 0; j < n_vis; ++j) {
        t[m].v = score_all[vis_offset + j];
        t[m].idx = j;
        ++m;
    }
    qsort(t, (size_t)m, sizeof *t, largest ? cmp_desc : cmp_asc);
    for (int i = 0; i < Pv; ++i) pivot_idx[i] = t[i].idx;
    m = 0;
    for (int s = 0; s < S; ++s) {
        if (s >= vis_offset && s < vis_offset + n_vis) continue;
        t[m].v = score_all[s];
        t[m].idx = s - vis_offset; /* ascending with the sequence position, so ties go to the earlier token */
        ++m;
    }
    qsort(t, (size_t)m, sizeof *t, largest ? cmp_desc : cmp_asc);
    for (int i = 0; i < Pt; ++i) pivot_idx[Pv + i] = t[i].idx;
    free(t);
    return ORACLE_OK;
}

/*
 * The output of SplitMix64 (Steele, Lea, Flood: "Fast splittable pseudorandom number generators", OOPSLA 2014) for the
 * state `state` AFTER its increment by the golden gamma: the generator's next() is mix(state += gamma).
 */
static uint64_t splitmix64_mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* The k-th output (k = 0, 1, ...) of a SplitMix64 generator seeded with `seed`: a counter-based form of the same sequence. */
uint64_t dart_oracle_splitmix64(uint64_t seed, uint64_t k) { return splitmix64_mix(seed + (k + 1) * 0x9E3779B97F4A7C15ull); }

/*
 * Random pivots (Sec. 5.2 also draws the pivots at random, five seeds): P distinct vision tokens of sample b, uniformly at
 * random without replacement.  Every token gets a 32-bit ticket, the upper half of output number (b * 2^32 + j) of a
 * SplitMix64 generator seeded with `seed`; the P tokens with the smallest tickets are the pivots, smallest first, equal
 * tickets to the lower index.  (Any P-subset is equally likely because the tickets are exchangeable.)
 */
int dart_oracle_pivots_random(uint64_t seed, int b, int n_vis, int P, int32_t *pivot_idx)
{
    if (n_vis < 1 || P < 1 || P > n_vis || b < 0) return ORACLE_ERR_SHAPE;
    keyed_t *t = (keyed_t *)malloc((size_t)n_vis * sizeof *t);
    if (!t) return ORACLE_ERR_NOMEM;
    for (int j = 0; j < n_vis; ++j) {
        t[j].v = (double)(uint32_t)(dart_oracle_splitmix64(seed, ((uint64_t)b << 32) | (uint32_t)j) >> 32);
        t[j].idx = j;
    }
    qsort(t, (size_t)n_vis, sizeof *t, cmp_asc);
    for (int i = 0; i < P; ++i) pivot_idx[i] = t[i].idx;
    free(t);
    return ORACLE_OK;
}

/*
 * Row gather by a packed index list: out[b, t, :] = src[b, idx[b, t], :] (bit copies of rows of `row_elems`
 * 16-bit words).  This is how a cache kept per token (the key and value rows of the layers already run) follows
 * the shortened sequence: the paper counts the KV cache of the retained tokens only (Table 2).
 */
int dart_oracle_gather_rows(const uint16_t *src, const int32_t *idx, int B, int S, int S_out, int row_elems,
                            uint16_t *out)
{
    if (B < 0 || S < 1 || S_out < 0 || row_elems < 1) return ORACLE_ERR_SHAPE;
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < S_out; ++t) {
            const int32_t s = idx[(size_t)b * S_out + t];
            if (s < 0 || s >= S) return ORACLE_ERR_SHAPE;
            memcpy(out + ((size_t)b * S_out + t) * (size_t)row_elems, src + ((size_t)b * S + s) * (size_t)row_elems,
                   (size_t)row_elems * sizeof(uint16_t));
        }
    return ORACLE_OK;
}

/*
 * Sequence shortening (Table 1 caption: tokens are pruned after layer K; the remaining
 * layers see a dense, shorter sequence).  Kept rows stay in original order:
 *   out_idx    = [0, vis_offset) ++ sorted{vis_offset + j : keep[j]} ++ [vis_offset + n_vis, S)
 *   out_pos[t] = pos_in[out_idx[t]]   (pos_in NULL means pos_in[s] = s)
 *   out_hidden[t, :] = hidden[out_idx[t], :]   (bit copy of the bf16 row)
 * Returns the packed length S_out through *S_out_p.
 */
int dart_oracle_compact(const uint8_t *keep, const uint16_t *hidden, const int64_t *pos_in,
                        int S, int d, int vis_offset, int n_vis,
                        uint16_t *out_hidden, int32_t *out_idx, int64_t *out_pos, int *S_out_p)
{
    if (S < 1 || d < 1 || vis_offset < 0 || n_vis < 0 || vis_offset + n_vis > S) return ORACLE_ERR_SHAPE;
    int t = 0;
    for (int s = 0; s < S; ++s) {
        int is_vis = (s >= vis_offset && s < vis_offset + n_vis);
        if (is_vis && !keep[s - vis_offset]) continue;
        out_idx[t] = s;
        out_pos[t] = pos_in ? pos_in[s] : (int64_t)s;
        if (out_hidden && hidden)
            memcpy(out_hidden + (size_t)t * (size_t)d, hidden + (size_t)s * (size_t)d, (size_t)d * sizeof(uint16_t));
        ++t;
    }
    if (S_out_p) *S_out_p = t;
    return ORACLE_OK;
}

/*
 * The whole step over a batch of independent samples (the paper's step has no
 * cross-sample term).  hidden/keys are [B, S, d] bf16 bits in host memory; keys == NULL
 * means the hidden states are scored and compared.  pos_in is [B, S] or NULL.
 * norm_kind: 1 = L1 score (the paper's K-norm), 2 = Euclidean score.
 * Per-sample debug outputs (each may be NULL):
 *   l1, l2 [B, n_vis]; pivot_idx [B, P]; dup [B, P, n_vis]; keep [B, n_vis];
 *   owner [B, n_vis]; eps [B, P]; pivot_gap [B]; retain_gap [B].
 * Packed outputs: out_hidden [B, S_out, d], out_idx [B, S_out], out_pos [B, S_out],
 * S_out = S - n_vis + n_keep.
 * pivots_in: NULL, or [B, P] distinct vision-relative indices that replace the pivot step (their
 * order is the order of the pivots' turns); the retention step rejects repeated or out-of-range ones.
 * rule: 0 = one threshold per pivot from equal quotas (dart_oracle_retention), 1 = one threshold for all
 * (dart_oracle_retention_global), 2 = independent pivots (dart_oracle_retention_union): the packed length of a
 * sample then depends on its data, the outputs are packed WITHOUT padding (sample b's rows start at row
 * cu_seqlens_out[b] of out_hidden / out_idx / out_pos, whose capacity stays B * S_out rows) and
 * cu_seqlens_out [B + 1] is required.
 * cosine_on_hidden: the paper ranks pivots by the K-norm but defines dup on "tokens" (Def. 2) without saying
 * which tensor represents them.  0: the key rows (one tensor for both); 1: the pivots are still chosen by the
 * key rows' scores, Eq. 7 is evaluated on the hidden rows.  Then l1_out holds the key rows' L1 scores and
 * l2_out the HIDDEN rows' Euclidean norms (Eq. 7's denominators).  Ignored when keys is NULL.
 * text_pivots: entries of pivots_in outside [0, n_vis) name text tokens (index relative to the vision block);
 * see dart_oracle_similarity_any and the dart_oracle_retention*_any functions.  Needs pivots_in or pivot_source 1.
 * pivot_source (without pivots_in): 0 = the n_pivot vision tokens of best score; 1 = n_pivot - n_text_pivots vision
 * tokens and n_text_pivots text tokens of best score (dart_oracle_pivots_mixed; implies text_pivots); 2 = random
 * vision tokens (dart_oracle_pivots_random with `seed` and the sample's number b).
 */
int dart_oracle_reduce_ex(const uint16_t *hidden, const uint16_t *keys, const int64_t *pos_in,
                          const int32_t *pivots_in,
                          int B, int S, int d, int vis_offset, int n_vis, int n_pivot, int n_keep,
                          int norm_kind, int largest, int rule, int cosine_on_hidden, int text_pivots,
                          int pivot_source, int n_text_pivots, uint64_t seed,
                          uint16_t *out_hidden, int32_t *out_idx, int64_t *out_pos,
                          double *l1_out, double *l2_out, int32_t *pivot_out, double *dup_out,
                          uint8_t *keep_out, int32_t *owner_out, double *eps_out,
                          double *pivot_gap_out, double *retain_gap_out, int32_t *cu_seqlens_out)
{
    if (B < 0 || S < 1 || d < 1 || vis_offset < 0 || n_vis < 1 || vis_offset + n_vis > S) return ORACLE_ERR_SHAPE;
    if (n_pivot < 1 || n_pivot > n_keep || n_keep > n_vis) return ORACLE_ERR_SHAPE;
    if (norm_kind != 1 && norm_kind != 2) return ORACLE_ERR_SHAPE;
    if (rule != 0 && rule != 1 && rule != 2) return ORACLE_ERR_SHAPE;
    if (rule == 2 && !cu_seqlens_out) return ORACLE_ERR_SHAPE;
    if (pivot_source < 0 || pivot_source > 2 || (pivot_source && pivots_in)) return ORACLE_ERR_SHAPE;
    if (pivot_source == 1) {
        if (n_text_pivots < 0 || n_text_pivots > n_pivot || n_text_pivots > S - n_vis || n_pivot - n_text_pivots > n_vis) return ORACLE_ERR_SHAPE;
        text_pivots = 1;
    }
    if (text_pivots && !pivots_in && pivot_source != 1) return ORACLE_ERR_SHAPE; /* text pivots come from the caller or from source 1 */
    const int P = n_pivot, S_out = S - n_vis + n_keep;
    double *all1 = (double *)malloc((size_t)S * sizeof(double));
    double *all2 = (double *)malloc((size_t)S * sizeof(double));
    double *l1 = (double *)malloc((size_t)n_vis * sizeof(double));
    double *l2 = (double *)malloc((size_t)n_vis * sizeof(double));
    double *hl1 = (double *)malloc((size_t)n_vis * sizeof(double));
    double *dup = (double *)malloc((size_t)P * (size_t)n_vis * sizeof(double));
    int32_t *piv = (int32_t *)malloc((size_t)P * sizeof(int32_t));
    uint8_t *keep = (uint8_t *)malloc((size_t)n_vis);
    int rc = ORACLE_OK;
    if (!l1 || !l2 || !hl1 || !dup || !piv || !keep || !all1 || !all2) rc = ORACLE_ERR_NOMEM;
    size_t cu = 0; /* rows packed so far (rule 2) */
    if (cu_seqlens_out) cu_seqlens_out[0] = 0;
    for (int b = 0; b < B && rc == ORACLE_OK; ++b) {
        const uint16_t *h = hidden + (size_t)b * (size_t)S * (size_t)d;
        const uint16_t *k = keys ? keys + (size_t)b * (size_t)S * (size_t)d : h;
        const int64_t *pos = pos_in ? pos_in + (size_t)b * (size_t)S : NULL;
        double pgap = 0.0, rgap = 0.0;
        int so = 0;
        rc = dart_oracle_scores(k, S, d, vis_offset, n_vis, l1, l2);
        if (rc) break;
        if (pivots_in) { /* the caller names the pivots and their order (Sec. 5.2 compares several ways to choose them) */
            memcpy(piv, pivots_in + (size_t)b * P, (size_t)P * sizeof(int32_t));
            pgap = INFINITY; /* nothing is ranked, so no ranking can be close */
        } else if (pivot_source == 1) { /* both modalities: the scores of all S tokens */
            rc = dart_oracle_scores(k, S, d, 0, S, all1, all2);
            if (rc) break;
            rc = dart_oracle_pivots_mixed(norm_kind == 1 ? all1 : all2, S, vis_offset, n_vis, P - n_text_pivots, n_text_pivots, largest, piv);
            if (rc) break;
            pgap = 0.0; /* the gaps of the two rankings are not tracked: compare under tolerance */
        } else if (pivot_source == 2) {
            rc = dart_oracle_pivots_random(seed, b, n_vis, P, piv);
            if (rc) break;
            pgap = INFINITY; /* integer tickets: nothing can be close */
        } else {
            rc = dart_oracle_pivots(norm_kind == 1 ? l1 : l2, n_vis, P, largest, piv, &pgap);
            if (rc) break;
        }
        if (cosine_on_hidden && keys) {
            /* the pivots are ranked by the key states, but the tokens that are compared are the hidden states */
            rc = dart_oracle_scores(h, S, d, vis_offset, n_vis, hl1, l2);
            if (rc) break;
        }
        if (text_pivots)
            rc = dart_oracle_similarity_any((cosine_on_hidden && keys) ? h : k, S, d, vis_offset, n_vis, piv, P, dup);
        else
            rc = dart_oracle_similarity((cosine_on_hidden && keys) ? h : k, S, d, vis_offset, n_vis, piv, P, l2, dup);
        if (rc) break;
        if (rule == 2)
            rc = (text_pivots ? dart_oracle_retention_union_any : dart_oracle_retention_union)(
                dup, piv, n_vis, P, n_keep, keep, owner_out ? owner_out + (size_t)b * n_vis : NULL,
                eps_out ? eps_out + (size_t)b * P : NULL, &rgap, NULL);
        else if (rule == 1)
            rc = (text_pivots ? dart_oracle_retention_global_any : dart_oracle_retention_global)(
                dup, piv, n_vis, P, n_keep, keep, owner_out ? owner_out + (size_t)b * n_vis : NULL,
                eps_out ? eps_out + (size_t)b * P : NULL, &rgap);
        else
            rc = (text_pivots ? dart_oracle_retention_any : dart_oracle_retention)(
                dup, piv, n_vis, P, n_keep, keep, owner_out ? owner_out + (size_t)b * n_vis : NULL,
                eps_out ? eps_out + (size_t)b * P : NULL, &rgap);
        if (rc) break;
        const size_t row0 = rule == 2 ? cu : (size_t)b * (size_t)S_out;
        rc = dart_oracle_compact(keep, h, pos, S, d, vis_offset, n_vis, out_hidden ? out_hidden + row0 * (size_t)d : NULL,
                                 out_idx + row0, out_pos + row0, &so);
        if (rc) break;
        if (rule == 2 ? so > S_out : so != S_out) {
            rc = ORACLE_ERR_SHAPE;
            break;
        }
        cu += (size_t)so;
        if (cu_seqlens_out) cu_seqlens_out[b + 1] = (int32_t)cu;
        if (l1_out) memcpy(l1_out + (size_t)b * n_vis, l1, (size_t)n_vis * sizeof(double));
        if (l2_out) memcpy(l2_out + (size_t)b * n_vis, l2, (size_t)n_vis * sizeof(double));
        if (pivot_out) memcpy(pivot_out + (size_t)b * P, piv, (size_t)P * sizeof(int32_t));
        if (dup_out) memcpy(dup_out + (size_t)b * P * n_vis, dup, (size_t)P * (size_t)n_vis * sizeof(double));
        if (keep_out) memcpy(keep_out + (size_t)b * n_vis, keep, (size_t)n_vis);
        if (pivot_gap_out) pivot_gap_out[b] = pgap;
        if (retain_gap_out) retain_gap_out[b] = rgap;
    }
    free(l1);
    free(l2);
    free(hl1);
    free(dup);
    free(piv);
    free(keep);
    free(all1);
    free(all2);
    return rc;
}

/* The step with pivots chosen by score (the paper's main setting). */
int dart_oracle_reduce(const uint16_t *hidden, const uint16_t *keys, const int64_t *pos_in,
                       int B, int S, int d, int vis_offset, int n_vis, int n_pivot, int n_keep,
                       int norm_kind, int largest,
                       uint16_t *out_hidden, int32_t *out_idx, int64_t *out_pos,
                       double *l1_out, double *l2_out, int32_t *pivot_out, double *dup_out,
                       uint8_t *keep_out, int32_t *owner_out, double *eps_out,
                       double *pivot_gap_out, double *retain_gap_out)
{
    return dart_oracle_reduce_ex(hidden, keys, pos_in, NULL, B, S, d, vis_offset, n_vis, n_pivot, n_keep, norm_kind,
                                 largest, 0, 0, 0, 0, 0, 0, out_hidden, out_idx, out_pos, l1_out, l2_out, pivot_out, dup_out, keep_out,
                                 owner_out, eps_out, pivot_gap_out, retain_gap_out, NULL);
}
