/*
 * CPU oracle, weight-transfer part -- TEST INFRASTRUCTURE, not the product.
 *
 * Section "Restorer", paragraph "Weight Transfer": after a dynamic-parallelism plan has
 * been chosen, every surviving device takes over one position of the new plan.  The
 * N x N matrix Cost[i][j] is what device i would have to fetch to serve position j, and
 * the migration scheme is the perfect matching of least total cost (Kuhn-Munkres).
 *
 * Reading taken where the paper is silent: the cost of a (device, position) pair is the
 * number of bytes of model state -- parameters plus optimizer state, per layer -- of the
 * layers that position j holds and device i does not hold yet; layers that device i
 * holds and position j does not need are dropped for free.  With one unit per layer this
 * gives the two values of the paper's worked example (0 and 1).
 *
 * All arithmetic here is integer, so every result is exact in both cost modes.
 */
#include <stdlib.h>
#include <string.h>

#include "orc.h"

/*
 * Cost matrix of the matching, row-major [n][n]: row = surviving device (its old layer
 * range [old_lo, old_hi)), column = position of the new plan (layer range [new_lo, new_hi)).
 * w[l] = bytes of model state of layer l.  Written layer by layer, as the definition reads.
 */
void orc_transfer_cost_matrix(int L, const int64_t *w, int n, const int32_t *old_lo, const int32_t *old_hi,
                              const int32_t *new_lo, const int32_t *new_hi, int64_t *cost) {
    (void)L;
    for (int i = 0; i < n; i++)
        for (int j = 0; j < n; j++) {
            int64_t c = 0;
            for (int l = new_lo[j]; l < new_hi[j]; l++) {
                int held = l >= old_lo[i] && l < old_hi[i];
                if (!held) c += w[l];
            }
            cost[(size_t)i * n + j] = c;
        }
}

/*
 * Minimum-cost perfect matching of an n x n integer matrix (Kuhn-Munkres, in the
 * potentials / shortest-augmenting-path form: rows are added one at a time; for each new
 * row a cheapest alternating path to a free column is grown column by column over the
 * reduced costs cost[i][j] - u[i] - v[j], the potentials are shifted so that the tree
 * edges stay tight, and the matching is flipped along the path).  O(n^3).
 * row_of_col[j] = row matched to column j.  Returns the total cost.
 */
int64_t orc_assign(int n, const int64_t *cost, int32_t *row_of_col) {
    const int64_t INF = INT64_MAX / 4;
    int64_t *u = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));     /* row potentials     */
    int64_t *v = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));     /* column potentials  */
    int64_t *slack = (int64_t *)malloc(((size_t)n + 1) * sizeof(int64_t));
    int *match = (int *)malloc(((size_t)n + 1) * sizeof(int));            /* row of column, -1 = free; column n = root */
    int *prev = (int *)malloc(((size_t)n + 1) * sizeof(int));             /* previous column on the path */
    char *in_tree = (char *)malloc((size_t)n + 1);
    for (int j = 0; j <= n; j++) match[j] = -1;
    for (int r = 0; r < n; r++) {
        /* the virtual column n holds the new row; grow the tree from it */
        match[n] = r;
        for (int j = 0; j <= n; j++) { slack[j] = INF; in_tree[j] = 0; prev[j] = n; }
        int col = n;
        do {
            in_tree[col] = 1;
            int row = match[col];
            int64_t delta = INF;
            int next = -1;
            for (int j = 0; j < n; j++) {
                if (in_tree[j]) continue;
                int64_t red = cost[(size_t)row * n + j] - u[row] - v[j];
                if (red < slack[j]) { slack[j] = red; prev[j] = col; }
                if (slack[j] < delta) { delta = slack[j]; next = j; }
            }
            for (int j = 0; j <= n; j++) {
                if (in_tree[j]) { u[match[j]] += delta; v[j] -= delta; }
                else slack[j] -= delta;
            }
            col = next;
        } while (match[col] >= 0);
        /* flip the matching along the path back to the root */
        while (col != n) {
            int p = prev[col];
            match[col] = match[p];
            col = p;
        }
    }
    int64_t total = 0;
    for (int j = 0; j < n; j++) {
        row_of_col[j] = match[j];
        total += cost[(size_t)match[j] * n + j];
    }
    free(u); free(v); free(slack); free(match); free(prev); free(in_tree);
    return total;
}

/* The same minimum by trying every permutation (n <= 10); pins orc_assign. */
int64_t orc_assign_brute(int n, const int64_t *cost) {
    int perm[16];
    if (n > 10) return -1;
    for (int j = 0; j < n; j++) perm[j] = j;
    int64_t best = INT64_MAX;
    for (;;) {
        int64_t t = 0;
        for (int j = 0; j < n; j++) t += cost[(size_t)perm[j] * n + j];
        if (t < best) best = t;
        /* next permutation in lexicographic order */
        int i = n - 2;
        while (i >= 0 && perm[i] > perm[i + 1]) i--;
        if (i < 0) break;
        int k = n - 1;
        while (perm[k] < perm[i]) k--;
        int s = perm[i]; perm[i] = perm[k]; perm[k] = s;
        for (int a = i + 1, b = n - 1; a < b; a++, b--) { s = perm[a]; perm[a] = perm[b]; perm[b] = s; }
    }
    return best;
}

/*
 * Section "Restorer", Asymmetric Communication: every model layer is a vertex; two layers
 * are joined when some device holds both (then their data-parallel all-reduces cannot run
 * at the same time); a greedy colouring gives the communication rounds, layers of one
 * colour synchronise in parallel.  stage_of[p * L + l] = stage of pipeline p that holds
 * layer l (device = (pipeline, stage)).  Greedy in layer order: a layer takes the least
 * colour that none of its already coloured neighbours has.  Returns the number of colours;
 * colour[l] in 0..rounds-1.  O(L^2 * dp).
 */
int orc_comm_rounds(int L, int dp, const int32_t *stage_of, int32_t *colour) {
    int rounds = 0;
    for (int l = 0; l < L; l++) {
        char used[ORC_MAX_LAYERS + 1];
        memset(used, 0, sizeof(used));
        for (int k = 0; k < l; k++) {
            int adjacent = 0;
            for (int p = 0; p < dp; p++)
                if (stage_of[(size_t)p * L + l] == stage_of[(size_t)p * L + k]) adjacent = 1;
            if (adjacent) used[colour[k]] = 1;
        }
        int c = 0;
        while (used[c]) c++;
        colour[l] = c;
        if (c + 1 > rounds) rounds = c + 1;
    }
    return rounds;
}

/*
 * Communication domains of a plan: maximal runs of layers that sit on the same device in
 * every pipeline, i.e. the distinct tuples (stage in pipeline 1, ..., stage in pipeline dp).
 * One all-reduce group is set up per domain (the paper's example counts 4 of them in the
 * symmetric and 6 in the asymmetric layout of its figure).
 */
int orc_comm_domains(int L, int dp, const int32_t *stage_of) {
    int n = 0;
    for (int l = 0; l < L; l++) {
        int fresh = l == 0;
        for (int p = 0; p < dp && !fresh; p++)
            if (stage_of[(size_t)p * L + l] != stage_of[(size_t)p * L + l - 1]) fresh = 1;
        n += fresh;
    }
    return n;
}
