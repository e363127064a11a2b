/*
 * CPU oracle, part 1: the candidate space as plain integer combinatorics.
 * TEST INFRASTRUCTURE -- see orc.h.  No cost arithmetic lives here.
 *
 * Follows the paper's Section "Planner" (execution plan search: DP/PP parallelism,
 * batch distribution, layer distribution) and Algorithm 1 (get_parallel_strategy).
 */
#include "orc.h"

#include <string.h>

/* Binomial coefficient by Pascal's rule with saturating addition.  Rows up to
 * ORC_BINOM_ROWS, columns up to ORC_BINOM_COLS; C(n,k) with both k and n-k beyond the
 * columns is far above 2^64 and reported as saturated. */
#define ORC_BINOM_ROWS 4096
#define ORC_BINOM_COLS 128
uint64_t orc_binom(int n, int k) {
    static uint64_t tab[ORC_BINOM_ROWS + 1][ORC_BINOM_COLS + 1];
    static int ready = 0;
    if (!ready) {
        for (int i = 0; i <= ORC_BINOM_ROWS; i++) {
            for (int j = 0; j <= ORC_BINOM_COLS; j++) {
                if (j == 0) tab[i][j] = 1;
                else if (i == 0) tab[i][j] = 0;
                else {
                    uint64_t a = tab[i - 1][j - 1], b = tab[i - 1][j];
                    tab[i][j] = (a > UINT64_MAX - b) ? UINT64_MAX : a + b;
                }
            }
        }
        ready = 1;
    }
    if (k < 0 || n < 0 || k > n) return 0;
    if (n - k < k) k = n - k;
    if (n > ORC_BINOM_ROWS || k > ORC_BINOM_COLS) return UINT64_MAX;
    return tab[n][k];
}

/*
 * Combinatorial number system, colexicographic order: the t-subset c[0]<...<c[t-1]
 * has rank sum_{u=1..t} C(c[u-1], u).  Unranking is greedy from the largest element:
 * take the largest c with C(c,u) <= rank.
 */
void orc_unrank_subset(uint64_t rank, int t, int *c) {
    for (int u = t; u >= 1; u--) {
        int v = u - 1; /* C(u-1,u) = 0 <= rank always holds */
        while (orc_binom(v + 1, u) <= rank) v++;
        c[u - 1] = v;
        rank -= orc_binom(v, u);
    }
}

uint64_t orc_rank_subset(int t, const int *c) {
    uint64_t r = 0;
    for (int u = 1; u <= t; u++) r += orc_binom(c[u - 1], u);
    return r;
}

/*
 * Parallel strategies (Algorithm 1, get_parallel_strategy; Section "Planner", DP/PP
 * parallelism: use all surviving nodes, asymmetric pipelines allowed, DP degree and
 * pipeline depth limited to ranges).  Reading of integer_partition: all partitions of
 * the survivor count into dp parts (non-decreasing stage counts) with every part in
 * [pp_lo, min(pp_hi, L)], for dp ascending, tuples in lexicographic order.
 */
typedef struct {
    int dp, lo, hi, max_out, n;
    int32_t *dp_out, *stages_out;
    int32_t cur[ORC_MAX_PIPES];
} strat_rec;

static void strat_fill(strat_rec *r, int pos, int remaining, int min_part) {
    if (pos == r->dp) {
        if (remaining != 0) return;
        if (r->n < r->max_out) {
            r->dp_out[r->n] = r->dp;
            memset(&r->stages_out[(size_t)r->n * ORC_MAX_PIPES], 0, sizeof(int32_t) * ORC_MAX_PIPES);
            memcpy(&r->stages_out[(size_t)r->n * ORC_MAX_PIPES], r->cur, sizeof(int32_t) * r->dp);
        }
        r->n++;
        return;
    }
    for (int s = min_part; s <= r->hi; s++) {
        int left = r->dp - pos - 1;
        if (remaining - s < (int64_t)left * s) break; /* later parts are >= s */
        r->cur[pos] = s;
        strat_fill(r, pos + 1, remaining - s, s);
    }
}

int orc_strategies(int n_surv, int dp_lo, int dp_hi, int pp_lo, int pp_hi, int L,
                   int max_out, int32_t *dp_out, int32_t *stages_out) {
    strat_rec r;
    r.n = 0;
    r.max_out = max_out;
    r.dp_out = dp_out;
    r.stages_out = stages_out;
    r.lo = pp_lo < 1 ? 1 : pp_lo;
    r.hi = pp_hi < L ? pp_hi : L;
    for (int dp = (dp_lo < 1 ? 1 : dp_lo); dp <= dp_hi && dp <= ORC_MAX_PIPES; dp++) {
        r.dp = dp;
        strat_fill(&r, 0, n_surv, r.lo);
    }
    return r.n;
}

/*
 * Micro-batch distribution (Section "Planner", batch distribution: pre-allocate in
 * proportion to the nodes of each pipeline, hand out what is left one by one; the sum
 * is the global batch, Definition 1 (iii)).
 *   REMAINDER: base_p = floor(G*S_p/N'), R = G - sum base_p; beta ranks the R-subset of
 *              pipelines that receive one more (rank 0 = the first R pipelines).
 *   FULL:      beta ranks every composition of G into dp positive parts.
 */
static void split_base(int G, int n_surv, int dp, const int32_t *stages, int32_t *base, int *R) {
    int sum = 0;
    for (int p = 0; p < dp; p++) {
        base[p] = (int32_t)(((int64_t)G * stages[p]) / n_surv);
        sum += base[p];
    }
    *R = G - sum;
}

uint64_t orc_split_count(int batch_mode, int G, int n_surv, int dp, const int32_t *stages) {
    if (batch_mode == ORC_BATCH_REMAINDER) {
        int32_t base[ORC_MAX_PIPES];
        int R;
        split_base(G, n_surv, dp, stages, base, &R);
        return orc_binom(dp, R);
    }
    return orc_binom(G - 1, dp - 1);
}

int orc_split_unrank(int batch_mode, int G, int n_surv, int dp, const int32_t *stages,
                     uint64_t beta, int32_t *micro_out) {
    int c[ORC_MAX_PIPES];
    if (batch_mode == ORC_BATCH_REMAINDER) {
        int32_t base[ORC_MAX_PIPES];
        int R;
        split_base(G, n_surv, dp, stages, base, &R);
        orc_unrank_subset(beta, R, c);
        for (int p = 0; p < dp; p++) micro_out[p] = base[p];
        for (int u = 0; u < R; u++) micro_out[c[u]] += 1;
    } else {
        /* composition <-> (dp-1)-subset of cut positions {1..G-1} */
        orc_unrank_subset(beta, dp - 1, c);
        int prev = 0;
        for (int p = 0; p < dp - 1; p++) {
            int cut = c[p] + 1;
            micro_out[p] = cut - prev;
            prev = cut;
        }
        micro_out[dp - 1] = G - prev;
    }
    for (int p = 0; p < dp; p++)
        if (micro_out[p] < 1) return 0;
    return 1;
}

/*
 * Layer distribution (Section "Planner", layer distribution: split evenly first, then
 * enumerate every placement of the r = L mod S leftover layers, C(S, r) of them).
 *   REMAINDER: n_i = floor(L/S) + [i in subset(kappa)], subsets of r stages.
 *   FULL:      every composition of L into S positive parts, C(L-1, S-1) of them,
 *              as (S-1)-subsets of the cut positions {1..L-1}.
 * Returns the count K of enumerated compositions (0 in MINMAX mode).
 */
uint64_t orc_layer_count(int layer_mode, int L, int S) {
    if (layer_mode == ORC_LAYERS_REMAINDER) return orc_binom(S, L % S);
    if (layer_mode == ORC_LAYERS_FULL) return orc_binom(L - 1, S - 1);
    return 0;
}

void orc_layer_unrank(int layer_mode, int L, int S, uint64_t kappa, int32_t *cuts_out) {
    int c[ORC_MAX_LAYERS];
    cuts_out[0] = 0;
    if (layer_mode == ORC_LAYERS_REMAINDER) {
        int q = L / S, r = L % S;
        int extra[ORC_MAX_STAGES];
        memset(extra, 0, sizeof(extra));
        orc_unrank_subset(kappa, r, c);
        for (int u = 0; u < r; u++) extra[c[u]] = 1;
        for (int i = 0; i < S; i++) cuts_out[i + 1] = cuts_out[i] + q + extra[i];
    } else {
        orc_unrank_subset(kappa, S - 1, c);
        for (int i = 0; i < S - 1; i++) cuts_out[i + 1] = c[i] + 1;
        cuts_out[S] = L;
    }
}
