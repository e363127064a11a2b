/*
 * CPU oracle, part 2: the unified performance model and the exhaustive plan search.
 * TEST INFRASTRUCTURE -- see orc.h.  Shares no code with the CUDA path.
 *
 * Compiled twice: -DORC_INT=0 gives the *_f64 entry points (IEEE double, every written
 * operation rounded once, compile with -ffp-contract=off), -DORC_INT=1 gives *_i64
 * (integer nanoseconds, every division floors).  Bytes are int64 in both.
 *
 * Sources in the paper: Section "Estimator" (time estimator: symmetric closed form,
 * step time = slowest pipeline, the start/end transition recurrence, the data-rerouting
 * step times for one and for several failures; memory estimator: the peak-memory
 * decomposition), Section "Planner" with Algorithm 1 (what is enumerated and that the
 * plan with the least estimated time is kept), Section "Limitations of Backup-free
 * Methods" (redundant computation, prose only).  Readings taken where the paper gives
 * no formula are stated at each function.
 */
#include "orc.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#if ORC_INT
typedef int64_t num_t;
#define NUM_INF INT64_MAX
#define NAME(x) x##_i64
#else
typedef double num_t;
#define NUM_INF ((double)INFINITY)
#define NAME(x) x##_f64
#endif

static num_t nmax(num_t a, num_t b) { return a > b ? a : b; }

/* ------------------------------------------------------------------ profile */

typedef struct {
    const orc_profile *p;
    int L;
    int schedule;      /* ORC_SCHED_*: order of the computations on every stage */
    num_t PF[ORC_MAX_LAYERS + 1], PB[ORC_MAX_LAYERS + 1];   /* time prefix sums  */
    int64_t PA[ORC_MAX_LAYERS + 1], PP[ORC_MAX_LAYERS + 1], PO[ORC_MAX_LAYERS + 1];
} model;

/* Prefix sums, accumulated left to right (PF[0]=0, PF[l+1]=PF[l]+f[l]). */
static void model_init(model *M, const orc_profile *p, int schedule) {
    M->p = p;
    M->L = p->L;
    M->schedule = schedule;
    M->PF[0] = 0; M->PB[0] = 0; M->PA[0] = 0; M->PP[0] = 0; M->PO[0] = 0;
    for (int l = 0; l < p->L; l++) {
#if ORC_INT
        M->PF[l + 1] = M->PF[l] + p->fwd_ns_i[l];
        M->PB[l + 1] = M->PB[l] + p->bwd_ns_i[l];
#else
        M->PF[l + 1] = M->PF[l] + p->fwd_ns[l];
        M->PB[l + 1] = M->PB[l] + p->bwd_ns[l];
#endif
        M->PA[l + 1] = M->PA[l] + p->act_bytes[l];
        M->PP[l + 1] = M->PP[l] + p->param_bytes[l];
        M->PO[l + 1] = M->PO[l] + p->opt_bytes[l];
    }
}

/* One pipeline stage holding layers [lo, hi). */
typedef struct {
    num_t F, B;        /* forward / backward time per micro-batch                 */
    int64_t A;         /* activation bytes stored per in-flight micro-batch       */
    int64_t stat;      /* parameters + gradients (= parameters) + optimizer state */
    int64_t G;         /* gradient bytes synchronised among data-parallel peers   */
    int64_t X;         /* bytes sent to the next stage per micro-batch            */
} stage_t;

static stage_t stage_of(const model *M, int lo, int hi) {
    stage_t s;
    s.F = M->PF[hi] - M->PF[lo];
    s.B = M->PB[hi] - M->PB[lo];
    s.A = M->PA[hi] - M->PA[lo];
    s.stat = (M->PP[hi] - M->PP[lo]) * 2 + (M->PO[hi] - M->PO[lo]);
    s.G = M->PP[hi] - M->PP[lo];
    s.X = M->p->p2p_bytes[hi - 1];
    return s;
}

/* ------------------------------------------------------------ memory estimator */

/*
 * Peak memory of stage i of S (Section "Estimator", memory estimator: static memory
 * N_l (m_p + m_o + m_g) with m_g = m_p, plus (N_pp - i) micro-batches of activations
 * in flight, stage index from 0).  Per-layer bytes are summed over the stage instead
 * of using per-layer averages; the in-flight count is capped by the number of
 * micro-batches the pipeline runs (only matters when m < S).  The (N_pp - i) count is
 * that of the 1F1B order; under the all-forward-all-backward order (every stage runs its
 * m forwards before its first backward) all m micro-batches are in flight at the peak.
 */
static int64_t stage_peak_memory(const stage_t *s, int i, int S, int m, int schedule) {
    int inflight = S - i;
    if (m < inflight) inflight = m;
    if (schedule == ORC_SCHED_GPIPE) inflight = m;
    return s->stat + (int64_t)inflight * s->A;
}

/* ---------------------------------------------------------------- time estimator */

/*
 * Pipeline time by the start/end recurrence (Section "Estimator", the transition
 * equation): the j-th computation of stage i starts when both the previous computation
 * of the same stage and the computation it depends on in the neighbouring stage have
 * ended; a forward depends on the same micro-batch's forward one stage earlier, a
 * backward on the same micro-batch's backward one stage later (on its own forward at
 * the last stage).  The order of computations per stage -- the paper's f_2, "profiled
 * from the actual execution order" -- is one of
 *   ORC_SCHED_1F1B   non-interleaved 1F1B: w = min(S-1-i, m) warm-up forwards, then
 *                    forward/backward pairs, then the remaining backwards;
 *   ORC_SCHED_GPIPE  all forwards F_0..F_{m-1}, then all backwards B_0..B_{m-1}.
 * A transfer time xt[i] is paid on the boundary between stages i and i+1 in both
 * directions.
 *
 * Plain event simulation: sweep the stages and let each advance through its list while
 * the dependency of its next computation is known.
 */
static num_t pipe_time(int S, int m, const num_t *F, const num_t *B, const num_t *xt, int schedule) {
    const int n_ops = 2 * m;
    char *kind = (char *)malloc((size_t)S * n_ops);            /* 0 forward, 1 backward */
    int *mb = (int *)malloc(sizeof(int) * (size_t)S * n_ops);
    num_t *endF = (num_t *)malloc(sizeof(num_t) * (size_t)S * m);
    num_t *endB = (num_t *)malloc(sizeof(num_t) * (size_t)S * m);
    char *doneF = (char *)calloc((size_t)S * m, 1);
    char *doneB = (char *)calloc((size_t)S * m, 1);
    num_t clock[ORC_MAX_STAGES];
    int pos[ORC_MAX_STAGES];

    for (int i = 0; i < S; i++) {
        int w = S - 1 - i;
        if (w > m) w = m;
        if (schedule == ORC_SCHED_GPIPE) w = m;   /* every forward is a "warm-up" forward */
        int n = 0;
        for (int j = 0; j < w; j++) { kind[i * n_ops + n] = 0; mb[i * n_ops + n] = j; n++; }
        for (int k = 0; k < m - w; k++) {
            kind[i * n_ops + n] = 0; mb[i * n_ops + n] = w + k; n++;
            kind[i * n_ops + n] = 1; mb[i * n_ops + n] = k; n++;
        }
        for (int j = m - w; j < m; j++) { kind[i * n_ops + n] = 1; mb[i * n_ops + n] = j; n++; }
        clock[i] = 0;
        pos[i] = 0;
    }

    long remaining = (long)S * n_ops;
    while (remaining > 0) {
        long before = remaining;
        for (int i = 0; i < S; i++) {
            while (pos[i] < n_ops) {
                int j = mb[i * n_ops + pos[i]];
                num_t start, end;
                if (kind[i * n_ops + pos[i]] == 0) {
                    if (i > 0) {
                        if (!doneF[(i - 1) * m + j]) break;
                        start = nmax(clock[i], endF[(i - 1) * m + j] + xt[i - 1]);
                    } else {
                        start = nmax(clock[i], (num_t)0);
                    }
                    end = start + F[i];
                    endF[i * m + j] = end;
                    doneF[i * m + j] = 1;
                } else {
                    if (i < S - 1) {
                        if (!doneB[(i + 1) * m + j]) break;
                        start = nmax(clock[i], endB[(i + 1) * m + j] + xt[i]);
                    } else {
                        if (!doneF[i * m + j]) break;
                        start = nmax(clock[i], endF[i * m + j]);
                    }
                    end = start + B[i];
                    endB[i * m + j] = end;
                    doneB[i * m + j] = 1;
                }
                clock[i] = end;
                pos[i]++;
                remaining--;
            }
        }
        if (remaining == before) break; /* cannot happen for a valid 1F1B order */
    }
    num_t t = (remaining == 0) ? 0 : NUM_INF;
    if (remaining == 0)
        for (int i = 0; i < S; i++) t = nmax(t, clock[i]);
    free(kind); free(mb); free(endF); free(endB); free(doneF); free(doneB);
    return t;
}

/* Bandwidth of the link between two devices: intra-node if they share a node. */
static int64_t link_bw(const orc_profile *p, int dev_a, int dev_b) {
    return (dev_a / p->devices_per_node == dev_b / p->devices_per_node) ? p->bw_intra : p->bw_inter;
}

/* Activation transfer time over one stage boundary (north-star term "P2P activation
 * transfer"; the paper's equations carry no such term). */
static num_t transfer_time(int64_t bytes, int64_t bw) {
#if ORC_INT
    return bytes / bw;
#else
    return (double)bytes / (double)bw;
#endif
}

/*
 * Gradient synchronisation time of one stage among n data-parallel peers (the paper
 * says the step consists of pipeline time plus synchronisation, Section "Performance
 * Modeling", and gives no formula): ring all-reduce lower bound 2 (n-1) G / (n bw).
 * The links used are the inter-node tier whenever the fault-free job spans more than
 * one node.
 */
static num_t sync_time(const orc_profile *p, int64_t G, int n) {
    if (n <= 1) return 0;
    int64_t bw = (p->n_dp * p->n_pp > p->devices_per_node) ? p->bw_inter : p->bw_intra;
#if ORC_INT
    return (2 * (int64_t)(n - 1) * G) / ((int64_t)n * bw);
#else
    return ((2.0 * (double)(n - 1)) * (double)G) / ((double)n * (double)bw);
#endif
}

/*
 * One pipeline: S stages given explicitly, m micro-batches, devices devs[0..S-1],
 * n_sync[i] peers synchronising stage i.  feasible <=> every stage fits in memory,
 * m >= 1.  cost = pipeline time + max over stages of the synchronisation time.
 * Also returns the bare pipeline time.
 */
static void pipe_eval(const model *M, int S, const stage_t *st, int m, const int *devs,
                      const int *n_sync, num_t *cost, num_t *t_pipe_out, int *feasible) {
    num_t F[ORC_MAX_STAGES], B[ORC_MAX_STAGES], xt[ORC_MAX_STAGES];
    *cost = NUM_INF;
    if (t_pipe_out) *t_pipe_out = NUM_INF;
    *feasible = 0;
    if (m < 1) return;
    for (int i = 0; i < S; i++)
        if (stage_peak_memory(&st[i], i, S, m, M->schedule) > M->p->mem_capacity_bytes) return;
    for (int i = 0; i < S; i++) {
        F[i] = st[i].F;
        B[i] = st[i].B;
        xt[i] = (i < S - 1) ? transfer_time(st[i].X, link_bw(M->p, devs[i], devs[i + 1])) : 0;
    }
    num_t t_pipe = pipe_time(S, m, F, B, xt, M->schedule);
    num_t t_sync = 0;
    for (int i = 0; i < S; i++) t_sync = nmax(t_sync, sync_time(M->p, st[i].G, n_sync[i]));
    *cost = t_pipe + t_sync;
    if (t_pipe_out) *t_pipe_out = t_pipe;
    *feasible = 1;
}

/* A pipeline given by its layer cuts (cuts[0]=0 < ... < cuts[S]=L). */
static void pipe_from_cuts(const model *M, int S, const int32_t *cuts, int m, const int *devs,
                           int n_sync_all, num_t *cost, int *feasible) {
    stage_t st[ORC_MAX_STAGES];
    int n_sync[ORC_MAX_STAGES];
    *cost = NUM_INF;
    *feasible = 0;
    for (int i = 0; i < S; i++) {
        if (cuts[i + 1] <= cuts[i]) return; /* every stage needs a layer */
        st[i] = stage_of(M, cuts[i], cuts[i + 1]);
        n_sync[i] = n_sync_all;
    }
    pipe_eval(M, S, st, m, devs, n_sync, cost, NULL, feasible);
}

/* ------------------------------------------------------- min-max layer partition */

/*
 * Contiguous partition of the L layers into S stages minimising the largest stage
 * work W(k,l) = forward + backward time of layers [k,l), subject to each stage fitting
 * in memory at its position (textbook DP; not in the paper, one extra candidate per
 * pipeline):  D[l][1] = W(0,l);  D[l][s] = min_k max(D[k][s-1], W(k,l)).
 * Backtracking takes the smallest k that attains D[l][s].  Returns 0 if no partition
 * is memory-feasible.
 */
static int minmax_partition(const model *M, int S, int m, int32_t *cuts, num_t *value) {
    const int L = M->L;
    static num_t D[ORC_MAX_LAYERS + 1][ORC_MAX_STAGES + 1];
    for (int l = 0; l <= L; l++)
        for (int s = 0; s <= S; s++) D[l][s] = NUM_INF;
    for (int s = 1; s <= S; s++) {
        for (int l = s; l <= L; l++) {
            int k_lo = (s == 1) ? 0 : s - 1, k_hi = (s == 1) ? 0 : l - 1;
            num_t best = NUM_INF;
            for (int k = k_lo; k <= k_hi; k++) {
                stage_t st = stage_of(M, k, l);
                if (stage_peak_memory(&st, s - 1, S, m, M->schedule) > M->p->mem_capacity_bytes) continue;
                num_t W = st.F + st.B;
                num_t prev = (s == 1) ? 0 : D[k][s - 1];
                if (prev == NUM_INF) continue;
                num_t v = nmax(prev, W);
                if (v < best) best = v;
            }
            D[l][s] = best;
        }
    }
    if (value) *value = D[L][S];
    if (D[L][S] == NUM_INF) return 0;
    int l = L;
    cuts[S] = L;
    for (int s = S; s >= 2; s--) {
        int found = -1;
        for (int k = s - 1; k <= l - 1; k++) {
            stage_t st = stage_of(M, k, l);
            if (stage_peak_memory(&st, s - 1, S, m, M->schedule) > M->p->mem_capacity_bytes) continue;
            if (D[k][s - 1] == NUM_INF) continue;
            if (nmax(D[k][s - 1], st.F + st.B) == D[l][s]) { found = k; break; }
        }
        cuts[s - 1] = found;
        l = found;
    }
    cuts[0] = 0;
    return 1;
}

/* ------------------------------------------------------------------ data rerouting */

/*
 * Data rerouting (Section "Estimator", the single-failure and the multi-failure step
 * time): the failed devices' micro-batches are spread evenly over the data-parallel
 * peers of the same stage.  F_i = failed devices in stage i (device d sits in pipeline
 * d / N_pp, stage d mod N_pp).  Unrecoverable when a stage keeps no peer (F_i >= N_dp).
 * With non-uniform stages the factor (T_f + T_b) of the printed formula becomes the
 * stage's own forward + backward time, and the (N_pp + N_m - 1)(T_f + T_b) part becomes
 * the recurrence's pipeline time of the unchanged base configuration:
 *   cost = t_pipe(base) + sum_i [F_i>0] N_m F_i (F_i^st + B_i^st) / (N_dp - F_i)
 *          + max_i sync_i(N_dp - F_i peers).
 */
static void reroute_eval(const model *M, const uint32_t *failed, int n_failed,
                         num_t *cost, int *feasible) {
    const orc_profile *p = M->p;
    const int S = p->n_pp, m = p->n_micro;
    int Fcnt[ORC_MAX_STAGES];
    stage_t st[ORC_MAX_STAGES];
    int devs[ORC_MAX_STAGES], n_sync[ORC_MAX_STAGES];
    *cost = NUM_INF;
    *feasible = 0;
    memset(Fcnt, 0, sizeof(Fcnt));
    for (int f = 0; f < n_failed; f++) Fcnt[failed[f] % S]++;
    for (int i = 0; i < S; i++)
        if (Fcnt[i] >= p->n_dp) return;
    for (int i = 0; i < S; i++) {
        st[i] = stage_of(M, p->base_cuts[i], p->base_cuts[i + 1]);
        devs[i] = i; /* pipeline 0's devices */
        n_sync[i] = p->n_dp - Fcnt[i];
    }
    num_t with_sync, base;
    int ok;
    pipe_eval(M, S, st, m, devs, n_sync, &with_sync, &base, &ok);
    if (!ok) return;
    num_t extra = 0;
    for (int i = 0; i < S; i++) {
        if (Fcnt[i] > 0) {
#if ORC_INT
            extra = extra + ((int64_t)(m * Fcnt[i]) * (st[i].F + st[i].B)) / (int64_t)(p->n_dp - Fcnt[i]);
#else
            extra = extra + ((double)(m * Fcnt[i]) * (st[i].F + st[i].B)) / (double)(p->n_dp - Fcnt[i]);
#endif
        }
    }
    num_t t_sync = 0;
    for (int i = 0; i < S; i++) t_sync = nmax(t_sync, sync_time(p, st[i].G, n_sync[i]));
    *cost = (base + extra) + t_sync;
    *feasible = 1;
}

/* ------------------------------------------------------------ redundant computation */

/*
 * Redundant computation (Section "Limitations of Backup-free Methods": every node keeps
 * a replica of its successor, at nearly twice the computation and memory; prose only).
 * Reading: in each pipeline a failed stage's layers are taken over by its predecessor
 * (no wrap-around: stage 0 has no predecessor; a failed stage whose predecessor failed
 * too has lost its replica) -- the pipeline shrinks to its surviving devices.  Every
 * stage but the last also carries its successor's work: F'_i = F_i + F_{i+1}, likewise
 * B, static bytes and activation bytes.  Gradient sync stays that of the stage's own
 * parameters among N_dp peers.  cost = slowest pipeline; all pipelines carry the
 * overhead, failed or not.  stages_out[k] receives the stage count of pipeline k.
 */
static void redundant_eval(const model *M, const uint32_t *failed, int n_failed,
                           num_t *cost, int *feasible, uint16_t *stages_out) {
    const orc_profile *p = M->p;
    const int S0 = p->n_pp, m = p->n_micro;
    num_t worst = 0;
    *cost = NUM_INF;
    *feasible = 0;
    for (int k = 0; k < p->n_dp; k++) {
        char dead[ORC_MAX_STAGES];
        memset(dead, 0, sizeof(dead));
        for (int f = 0; f < n_failed; f++)
            if ((int)(failed[f] / S0) == k) dead[failed[f] % S0] = 1;
        if (dead[0]) return;
        for (int i = 1; i < S0; i++)
            if (dead[i] && dead[i - 1]) return;
        /* merged cuts over the surviving devices */
        int32_t cuts[ORC_MAX_STAGES + 1];
        int devs[ORC_MAX_STAGES], n_sync[ORC_MAX_STAGES];
        int S = 0;
        cuts[0] = 0;
        for (int i = 0; i < S0; i++) {
            if (dead[i]) continue;
            int hi = p->base_cuts[i + 1];
            if (i + 1 < S0 && dead[i + 1]) hi = p->base_cuts[i + 2];
            devs[S] = k * S0 + i;
            n_sync[S] = p->n_dp;
            cuts[S + 1] = hi;
            S++;
        }
        stage_t own[ORC_MAX_STAGES], st[ORC_MAX_STAGES];
        for (int i = 0; i < S; i++) own[i] = stage_of(M, cuts[i], cuts[i + 1]);
        for (int i = 0; i < S; i++) {
            st[i] = own[i];
            if (i < S - 1) {
                st[i].F = own[i].F + own[i + 1].F;
                st[i].B = own[i].B + own[i + 1].B;
                st[i].A = own[i].A + own[i + 1].A;
                st[i].stat = own[i].stat + own[i + 1].stat;
            }
        }
        num_t c;
        int ok;
        pipe_eval(M, S, st, m, devs, n_sync, &c, NULL, &ok);
        if (!ok) return;
        worst = nmax(worst, c);
        if (stages_out) stages_out[k] = (uint16_t)S;
    }
    *cost = worst;
    *feasible = 1;
}

/* -------------------------------------------------------------- dynamic parallelism */

/*
 * The candidate space of dynamic parallelism for one failure set (Section "Planner").
 * Survivors, ascending by id, are handed out in consecutive blocks: pipeline p of a
 * strategy owns survivors off_p .. off_p+S_p-1, stage i sits on survivor off_p+i.
 *
 * A segment is one (strategy, pipeline, micro-batch count); its candidates are the
 * layer compositions kappa = 0..K-1 followed by the min-max partition (kappa = K), or
 * the min-max partition alone when K exceeds kappa_cap or in MINMAX mode.  Candidate
 * indices run segment-major in the order strategy, pipeline, micro-batch count.
 */
typedef struct {
    int strategy, pipe, S, m, off, dp;
    uint64_t K;       /* enumerated compositions in this segment (0 if min-max only) */
    uint64_t count;   /* candidates: K+1 or 1 */
    uint64_t first;   /* index of its first candidate */
} segment;

typedef struct {
    model M;
    orc_opts o;
    int n_surv, G;
    int surv[ORC_MAX_PIPES * ORC_MAX_STAGES];
    int n_strat;
    int32_t *dp;       /* [n_strat] */
    int32_t *stages;   /* [n_strat][ORC_MAX_PIPES] */
    int n_seg;
    segment *seg;
    int *seg_begin;    /* [n_strat+1] first segment of each strategy */
    uint64_t n_cand;
} space;

static int micro_range(const space *sp, int si, int p, int *m_lo, int *m_hi) {
    int dp = sp->dp[si];
    const int32_t *st = &sp->stages[(size_t)si * ORC_MAX_PIPES];
    if (sp->o.batch_mode == ORC_BATCH_REMAINDER) {
        int sum = 0, base_p = 0;
        for (int q = 0; q < dp; q++) {
            int b = (int)(((int64_t)sp->G * st[q]) / sp->n_surv);
            sum += b;
            if (q == p) base_p = b;
        }
        int R = sp->G - sum;
        *m_lo = base_p;
        *m_hi = base_p + (R > 0 ? 1 : 0);
    } else {
        *m_lo = 1;
        *m_hi = sp->G - dp + 1;
    }
    return *m_hi >= *m_lo;
}

static int space_build(space *sp, const orc_profile *prof, const orc_opts *o,
                       const uint32_t *failed, int n_failed) {
    memset(sp, 0, sizeof(*sp));
    model_init(&sp->M, prof, o->schedule);
    sp->o = *o;
    int N = prof->n_dp * prof->n_pp;
    sp->G = prof->n_dp * prof->n_micro;
    for (int d = 0; d < N; d++) {
        int is_failed = 0;
        for (int f = 0; f < n_failed; f++)
            if ((int)failed[f] == d) is_failed = 1;
        if (!is_failed) sp->surv[sp->n_surv++] = d;
    }
    int n = orc_strategies(sp->n_surv, o->dp_lo, o->dp_hi, o->pp_lo, o->pp_hi, prof->L, 0, NULL, NULL);
    sp->n_strat = n;
    sp->dp = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n + 1));
    sp->stages = (int32_t *)malloc(sizeof(int32_t) * ORC_MAX_PIPES * (size_t)(n + 1));
    orc_strategies(sp->n_surv, o->dp_lo, o->dp_hi, o->pp_lo, o->pp_hi, prof->L, n, sp->dp, sp->stages);
    /* count, then fill, the segments */
    for (int pass = 0; pass < 2; pass++) {
        int ns = 0;
        uint64_t first = 0;
        for (int si = 0; si < n; si++) {
            if (pass) sp->seg_begin[si] = ns;
            int off = 0;
            for (int p = 0; p < sp->dp[si]; p++) {
                int S = sp->stages[(size_t)si * ORC_MAX_PIPES + p];
                int m_lo, m_hi;
                if (micro_range(sp, si, p, &m_lo, &m_hi)) {
                    for (int m = m_lo; m <= m_hi; m++) {
                        if (pass) {
                            segment *g = &sp->seg[ns];
                            g->strategy = si; g->pipe = p; g->S = S; g->m = m; g->off = off;
                            g->dp = sp->dp[si];
                            uint64_t K = orc_layer_count(o->layer_mode, prof->L, S);
                            if (o->layer_mode == ORC_LAYERS_MINMAX || K > o->kappa_cap) { g->K = 0; g->count = 1; }
                            else { g->K = K; g->count = K + 1; }
                            g->first = first;
                            first += g->count;
                        }
                        ns++;
                    }
                }
                off += S;
            }
        }
        if (!pass) {
            sp->n_seg = ns;
            sp->seg = (segment *)malloc(sizeof(segment) * (size_t)(ns + 1));
            sp->seg_begin = (int *)malloc(sizeof(int) * (size_t)(n + 1));
        } else {
            sp->seg_begin[n] = ns;
            sp->n_cand = first;
        }
    }
    return 0;
}

static void space_free(space *sp) {
    free(sp->dp); free(sp->stages); free(sp->seg); free(sp->seg_begin);
}

/* Layer cuts of candidate kappa of a segment; returns 0 if the min-max slot is infeasible. */
static int segment_cuts(const space *sp, const segment *g, uint64_t kappa, int32_t *cuts) {
    if (kappa < g->K) {
        orc_layer_unrank(sp->o.layer_mode, sp->M.L, g->S, kappa, cuts);
        return 1;
    }
    return minmax_partition(&sp->M, g->S, g->m, cuts, NULL);
}

/* Cost and feasibility of one pipeline-plan (segment, kappa). */
static void segment_eval(const space *sp, const segment *g, uint64_t kappa, num_t *cost, int *feasible) {
    int32_t cuts[ORC_MAX_STAGES + 1];
    int devs[ORC_MAX_STAGES];
    *cost = NUM_INF;
    *feasible = 0;
    if (g->m < 1) return;
    if (!segment_cuts(sp, g, kappa, cuts)) return;
    for (int i = 0; i < g->S; i++) devs[i] = sp->surv[g->off + i];
    pipe_from_cuts(&sp->M, g->S, cuts, g->m, devs, g->dp, cost, feasible);
}

static const segment *find_segment(const space *sp, int si, int p, int m) {
    for (int s = sp->seg_begin[si]; s < sp->seg_begin[si + 1]; s++)
        if (sp->seg[s].pipe == p && sp->seg[s].m == m) return &sp->seg[s];
    return NULL;
}

/* Step 1 of the search: the least feasible cost of every segment (malloc'ed, n_seg entries). */
static num_t *segment_minima(const space *sp) {
    num_t *best = (num_t *)malloc(sizeof(num_t) * (size_t)(sp->n_seg + 1));
    for (int s = 0; s < sp->n_seg; s++) {
        const segment *g = &sp->seg[s];
        num_t b = NUM_INF;
        for (uint64_t kappa = 0; kappa < g->count; kappa++) {
            num_t c; int ok;
            segment_eval(sp, g, kappa, &c, &ok);
            if (ok && c < b) b = c;
        }
        best[s] = b;
    }
    return best;
}

/*
 * Search over dynamic-parallelism plans (Algorithm 1, get_execution_plan: keep the plan
 * with the least estimated time; step time = slowest pipeline).  A plan is the tuple
 * (strategy, split rank beta, kappa_1..kappa_dp).  Selected: the feasible plan of least
 * cost, ties to the lexicographically smallest tuple.  Because feasibility and
 * "cost <= T" are per-pipeline conditions this is found in three plain steps:
 *   1. best[segment] = min over feasible kappa of the pipeline cost;
 *   2. T(strategy, beta) = max over pipelines of best[...]; T* = min, first on ties;
 *   3. for the winner, kappa_p = the lowest kappa that is feasible with cost <= T*.
 */
static void dynpar_search(const space *sp, orc_plan *out) {
    num_t *best = segment_minima(sp);
    num_t Tstar = NUM_INF;
    int win_si = -1;
    uint64_t win_beta = 0;
    int32_t win_micro[ORC_MAX_PIPES];
    for (int si = 0; si < sp->n_strat; si++) {
        int dp = sp->dp[si];
        const int32_t *st = &sp->stages[(size_t)si * ORC_MAX_PIPES];
        uint64_t n_split = orc_split_count(sp->o.batch_mode, sp->G, sp->n_surv, dp, st);
        for (uint64_t beta = 0; beta < n_split; beta++) {
            int32_t micro[ORC_MAX_PIPES];
            if (!orc_split_unrank(sp->o.batch_mode, sp->G, sp->n_surv, dp, st, beta, micro)) continue;
            num_t T = 0;
            for (int p = 0; p < dp; p++) {
                const segment *g = find_segment(sp, si, p, micro[p]);
                num_t b = g ? best[g - sp->seg] : NUM_INF;
                T = nmax(T, b);
            }
            if (T < Tstar) {
                Tstar = T; win_si = si; win_beta = beta;
                memcpy(win_micro, micro, sizeof(int32_t) * dp);
            }
        }
    }
    memset(out, 0, sizeof(*out));
    out->policy = ORC_DYNPAR;
    if (win_si < 0) { free(best); return; }
    out->feasible = 1;
#if ORC_INT
    out->cost_ns = Tstar;
#else
    out->cost = Tstar;
#endif
    out->strategy = (uint32_t)win_si;
    out->n_pipes = (uint32_t)sp->dp[win_si];
    out->split_rank = win_beta;
    for (int p = 0; p < sp->dp[win_si]; p++) {
        const segment *g = find_segment(sp, win_si, p, win_micro[p]);
        out->stages[p] = (uint16_t)g->S;
        out->micro[p] = (uint16_t)win_micro[p];
        for (uint64_t kappa = 0; kappa < g->count; kappa++) {
            num_t c; int ok;
            segment_eval(sp, g, kappa, &c, &ok);
            if (ok && c <= Tstar) { out->kappa[p] = kappa; break; }
        }
    }
    free(best);
}

/*
 * The same search as the definition reads: every tuple of the full product is
 * evaluated from scratch, in lexicographic order, keeping the first strict minimum.
 * Exponential; for tiny inputs only (checks the three-step rule above).
 */
static void dynpar_search_flat(const space *sp, orc_plan *out, uint64_t *n_flat) {
    num_t Tstar = NUM_INF;
    uint64_t visited = 0;
    memset(out, 0, sizeof(*out));
    out->policy = ORC_DYNPAR;
    for (int si = 0; si < sp->n_strat; si++) {
        int dp = sp->dp[si];
        const int32_t *st = &sp->stages[(size_t)si * ORC_MAX_PIPES];
        uint64_t n_split = orc_split_count(sp->o.batch_mode, sp->G, sp->n_surv, dp, st);
        for (uint64_t beta = 0; beta < n_split; beta++) {
            int32_t micro[ORC_MAX_PIPES];
            int split_ok = orc_split_unrank(sp->o.batch_mode, sp->G, sp->n_surv, dp, st, beta, micro);
            const segment *g[ORC_MAX_PIPES];
            uint64_t kap[ORC_MAX_PIPES];
            int usable = split_ok;
            for (int p = 0; p < dp && usable; p++) {
                g[p] = find_segment(sp, si, p, micro[p]);
                if (!g[p]) usable = 0;
                kap[p] = 0;
            }
            if (!usable) continue;
            for (;;) {
                num_t T = 0;
                int all_ok = 1;
                for (int p = 0; p < dp; p++) {
                    num_t c; int ok;
                    segment_eval(sp, g[p], kap[p], &c, &ok);
                    if (!ok) all_ok = 0;
                    T = nmax(T, c);
                }
                visited++;
                if (all_ok && T < Tstar) {
                    Tstar = T;
                    out->feasible = 1;
                    out->strategy = (uint32_t)si;
                    out->n_pipes = (uint32_t)dp;
                    out->split_rank = beta;
                    for (int p = 0; p < dp; p++) {
                        out->stages[p] = (uint16_t)g[p]->S;
                        out->micro[p] = (uint16_t)micro[p];
                        out->kappa[p] = kap[p];
                    }
                    for (int p = dp; p < ORC_MAX_PIPES; p++) { out->stages[p] = 0; out->micro[p] = 0; out->kappa[p] = 0; }
                }
                /* next tuple, last pipeline fastest */
                int p = dp - 1;
                while (p >= 0) {
                    if (++kap[p] < g[p]->count) break;
                    kap[p] = 0;
                    p--;
                }
                if (p < 0) break;
            }
        }
    }
#if ORC_INT
    out->cost_ns = out->feasible ? Tstar : 0;
#else
    out->cost = out->feasible ? Tstar : 0;
#endif
    if (n_flat) *n_flat = visited;
}

/* ------------------------------------------------------------------- entry points */

static void set_cost(orc_plan *pl, num_t c) {
#if ORC_INT
    pl->cost_ns = c;
#else
    pl->cost = c;
#endif
}
static num_t get_cost(const orc_plan *pl) {
#if ORC_INT
    return pl->cost_ns;
#else
    return pl->cost;
#endif
}

/* Pipeline time of explicit stage times (tests pin this against the closed form). */
double NAME(orc_pipe_time)(int S, int m, const double *F, const double *B, const double *xt, int schedule) {
    num_t f[ORC_MAX_STAGES], b[ORC_MAX_STAGES], x[ORC_MAX_STAGES];
    for (int i = 0; i < S; i++) { f[i] = (num_t)F[i]; b[i] = (num_t)B[i]; x[i] = (num_t)xt[i]; }
    return (double)pipe_time(S, m, f, b, x, schedule);
}

/* One pipeline from layer cuts on explicit devices; cost as double (exact for the
 * integer build below 2^53). Returns feasibility; peak memory per stage optional. */
int NAME(orc_pipe)(const orc_profile *prof, int S, const int32_t *cuts, int m, const int32_t *devs,
                   int n_sync, double *cost, int64_t *cost_ns, int64_t *peak_mem /* [S] or NULL */, int schedule) {
    model M;
    model_init(&M, prof, schedule);
    num_t c; int ok;
    int d[ORC_MAX_STAGES];
    for (int i = 0; i < S; i++) d[i] = devs[i];
    pipe_from_cuts(&M, S, cuts, m, d, n_sync, &c, &ok);
    if (peak_mem)
        for (int i = 0; i < S; i++) {
            stage_t st = stage_of(&M, cuts[i], cuts[i + 1]);
            peak_mem[i] = stage_peak_memory(&st, i, S, m, schedule);
        }
    if (cost) *cost = ok ? (double)c : INFINITY;
    if (cost_ns) *cost_ns = ok ? (int64_t)c : INT64_MAX;
    return ok;
}

int NAME(orc_minmax)(const orc_profile *prof, int S, int m, int32_t *cuts, double *value, int schedule) {
    model M;
    model_init(&M, prof, schedule);
    num_t v;
    int ok = minmax_partition(&M, S, m, cuts, &v);
    if (value) *value = ok ? (double)v : INFINITY;
    return ok;
}

/* Candidate count of the dynamic-parallelism space; optional strategy / segment counts. */
uint64_t NAME(orc_count)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                         int32_t *n_strategies, int32_t *n_segments) {
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    uint64_t n = sp.n_cand;
    if (n_strategies) *n_strategies = sp.n_strat;
    if (n_segments) *n_segments = sp.n_seg;
    space_free(&sp);
    return n;
}

/* Cost / feasibility of candidates [first, first+count) or of the listed indices. */
void NAME(orc_eval)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                    uint64_t first, uint64_t count, const uint64_t *idx,
                    double *cost, int64_t *cost_ns, uint8_t *feasible) {
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    for (uint64_t t = 0; t < count; t++) {
        uint64_t e = idx ? idx[t] : first + t;
        num_t c = NUM_INF; int ok = 0;
        if (e < sp.n_cand) {
            int lo = 0, hi = sp.n_seg - 1;
            while (lo < hi) {
                int mid = (lo + hi + 1) / 2;
                if (sp.seg[mid].first <= e) lo = mid; else hi = mid - 1;
            }
            segment_eval(&sp, &sp.seg[lo], e - sp.seg[lo].first, &c, &ok);
        }
        if (cost) cost[t] = ok ? (double)c : INFINITY;
        if (cost_ns) cost_ns[t] = ok ? (int64_t)c : INT64_MAX;
        if (feasible) feasible[t] = (uint8_t)ok;
    }
    space_free(&sp);
}

/* Describe segment s of the space (tests use it to walk the candidate order). */
int NAME(orc_segment)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                      int s, int32_t *desc /* strategy,pipe,S,m,off,dp */, uint64_t *K, uint64_t *first) {
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    int ok = s >= 0 && s < sp.n_seg;
    if (ok) {
        const segment *g = &sp.seg[s];
        desc[0] = g->strategy; desc[1] = g->pipe; desc[2] = g->S; desc[3] = g->m; desc[4] = g->off; desc[5] = g->dp;
        *K = g->K; *first = g->first;
    }
    space_free(&sp);
    return ok;
}

/* One policy's best plan. */
void NAME(orc_search_policy)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                             int policy, int flat, orc_plan *out, uint64_t *n_flat) {
    memset(out, 0, sizeof(*out));
    out->policy = policy;
    if (policy == ORC_DYNPAR) {
        space sp;
        space_build(&sp, prof, o, failed, n_failed);
        if (flat) dynpar_search_flat(&sp, out, n_flat);
        else dynpar_search(&sp, out);
        space_free(&sp);
        return;
    }
    model M;
    model_init(&M, prof, o ? o->schedule : ORC_SCHED_1F1B);
    num_t c; int ok;
    out->n_pipes = (uint32_t)prof->n_dp;
    for (int k = 0; k < prof->n_dp; k++) { out->stages[k] = (uint16_t)prof->n_pp; out->micro[k] = (uint16_t)prof->n_micro; }
    if (policy == ORC_REROUTE) reroute_eval(&M, failed, n_failed, &c, &ok);
    else redundant_eval(&M, failed, n_failed, &c, &ok, out->stages);
    out->feasible = ok;
    set_cost(out, ok ? c : 0);
}

/*
 * The whole search for one failure set: every policy, then the least cost, ties to the
 * lowest policy id (rerouting < redundant computation < dynamic parallelism, i.e. the
 * cheaper transition wins a tie).  per_policy[3] optional.  Returns 1 if any plan is
 * feasible.
 */
int NAME(orc_search)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                     orc_plan *best, orc_plan *per_policy) {
    orc_plan pl[3];
    int win = -1;
    for (int pol = 0; pol < 3; pol++) {
        NAME(orc_search_policy)(prof, o, failed, n_failed, pol, 0, &pl[pol], NULL);
        if (pl[pol].feasible && (win < 0 || get_cost(&pl[pol]) < get_cost(&pl[win]))) win = pol;
    }
    if (per_policy) memcpy(per_policy, pl, sizeof(pl));
    if (win < 0) { memset(best, 0, sizeof(*best)); return 0; }
    *best = pl[win];
    return 1;
}

/* Layer cuts of every pipeline of a plan, concatenated (sum of stages+1 entries). */
int NAME(orc_decode)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                     const orc_plan *pl, int32_t *cuts_out) {
    int n = 0;
    if (pl->policy == ORC_DYNPAR) {
        space sp;
        space_build(&sp, prof, o, failed, n_failed);
        for (uint32_t p = 0; p < pl->n_pipes; p++) {
            const segment *g = find_segment(&sp, (int)pl->strategy, (int)p, pl->micro[p]);
            if (!g || !segment_cuts(&sp, g, pl->kappa[p], &cuts_out[n])) { space_free(&sp); return -1; }
            n += g->S + 1;
        }
        space_free(&sp);
        return n;
    }
    const int S0 = prof->n_pp;
    for (int k = 0; k < prof->n_dp; k++) {
        char dead[ORC_MAX_STAGES];
        memset(dead, 0, sizeof(dead));
        if (pl->policy == ORC_REDUNDANT)
            for (int f = 0; f < n_failed; f++)
                if ((int)(failed[f] / S0) == k) dead[failed[f] % S0] = 1;
        cuts_out[n++] = 0;
        for (int i = 0; i < S0; i++) {
            if (dead[i]) continue;
            int hi = prof->base_cuts[i + 1];
            if (i + 1 < S0 && dead[i + 1]) hi = prof->base_cuts[i + 2];
            cuts_out[n++] = hi;
        }
    }
    return n;
}

/* ------------------------------------------------- transition time, full objective */

/*
 * Shortlist of dynamic-parallelism plans for the full objective.  The pairs (strategy,
 * split) are ordered by their step time T(strategy, split), ties by position in the
 * enumeration; the first k feasible ones are kept.  Each is completed the same way the
 * search completes its winner: kappa_p = the lowest kappa that is feasible with pipeline
 * cost <= T of that pair.  (Reading: the paper ranks plans by the product of throughput
 * and effective-time ratio but gives no procedure for the coupled problem; the transfer
 * cost couples the pipelines, so only a shortlist by step time is re-scored.)
 */
typedef struct { num_t T; int si; uint64_t beta; uint64_t order; } pair_t;

static int pair_cmp(const void *a, const void *b) {
    const pair_t *x = (const pair_t *)a, *y = (const pair_t *)b;
    if (x->T < y->T) return -1;
    if (x->T > y->T) return 1;
    return x->order < y->order ? -1 : (x->order > y->order ? 1 : 0);
}

static int dynpar_shortlist(const space *sp, int k, orc_plan *plans) {
    num_t *best = segment_minima(sp);
    size_t cap = 1024, n = 0;
    pair_t *pairs = (pair_t *)malloc(cap * sizeof(pair_t));
    uint64_t order = 0;
    for (int si = 0; si < sp->n_strat; si++) {
        int dp = sp->dp[si];
        const int32_t *st = &sp->stages[(size_t)si * ORC_MAX_PIPES];
        uint64_t n_split = orc_split_count(sp->o.batch_mode, sp->G, sp->n_surv, dp, st);
        for (uint64_t beta = 0; beta < n_split; beta++, order++) {
            int32_t micro[ORC_MAX_PIPES];
            if (!orc_split_unrank(sp->o.batch_mode, sp->G, sp->n_surv, dp, st, beta, micro)) continue;
            num_t T = 0;
            for (int p = 0; p < dp; p++) {
                const segment *g = find_segment(sp, si, p, micro[p]);
                num_t b = g ? best[g - sp->seg] : NUM_INF;
                T = nmax(T, b);
            }
            if (!(T < NUM_INF)) continue;
            if (n == cap) { cap *= 2; pairs = (pair_t *)realloc(pairs, cap * sizeof(pair_t)); }
            pairs[n].T = T; pairs[n].si = si; pairs[n].beta = beta; pairs[n].order = order;
            n++;
        }
    }
    qsort(pairs, n, sizeof(pair_t), pair_cmp);
    int kept = 0;
    for (size_t t = 0; t < n && kept < k; t++, kept++) {
        orc_plan *out = &plans[kept];
        int si = pairs[t].si;
        int dp = sp->dp[si];
        int32_t micro[ORC_MAX_PIPES];
        memset(out, 0, sizeof(*out));
        orc_split_unrank(sp->o.batch_mode, sp->G, sp->n_surv, dp, &sp->stages[(size_t)si * ORC_MAX_PIPES],
                         pairs[t].beta, micro);
        out->policy = ORC_DYNPAR;
        out->feasible = 1;
#if ORC_INT
        out->cost_ns = pairs[t].T;
#else
        out->cost = pairs[t].T;
#endif
        out->strategy = (uint32_t)si;
        out->n_pipes = (uint32_t)dp;
        out->split_rank = pairs[t].beta;
        for (int p = 0; p < dp; p++) {
            const segment *g = find_segment(sp, si, p, micro[p]);
            out->stages[p] = (uint16_t)g->S;
            out->micro[p] = (uint16_t)micro[p];
            for (uint64_t kappa = 0; kappa < g->count; kappa++) {
                num_t c; int ok;
                segment_eval(sp, g, kappa, &c, &ok);
                if (ok && c <= pairs[t].T) { out->kappa[p] = kappa; break; }
            }
        }
    }
    free(pairs);
    free(best);
    return kept;
}

/*
 * Bytes moved by the cheapest migration into a dynamic-parallelism plan (Section
 * "Restorer", Weight Transfer).  Survivor u (ascending device id, device = pipeline *
 * n_pp + stage) still holds the layers of its old stage; position j = off_p + i of the
 * plan needs the layers of stage i of pipeline p.  assign[j] = index of the survivor that
 * takes position j.
 */
static int64_t plan_transfer_bytes(const space *sp, const orc_plan *pl, int32_t *assign) {
    const orc_profile *pr = sp->M.p;
    int n = sp->n_surv;
    int32_t *olo = (int32_t *)malloc(sizeof(int32_t) * 4 * (size_t)n);
    int32_t *ohi = olo + n, *nlo = ohi + n, *nhi = nlo + n;
    int64_t *w = (int64_t *)malloc(sizeof(int64_t) * (size_t)pr->L);
    for (int l = 0; l < pr->L; l++) w[l] = pr->param_bytes[l] + pr->opt_bytes[l];
    for (int u = 0; u < n; u++) {
        int stage = sp->surv[u] % pr->n_pp;
        olo[u] = pr->base_cuts[stage];
        ohi[u] = pr->base_cuts[stage + 1];
    }
    int j = 0;
    for (uint32_t p = 0; p < pl->n_pipes; p++) {
        int32_t cuts[ORC_MAX_STAGES + 1];
        const segment *g = find_segment(sp, (int)pl->strategy, (int)p, pl->micro[p]);
        segment_cuts(sp, g, pl->kappa[p], cuts);
        for (int i = 0; i < g->S; i++, j++) { nlo[j] = cuts[i]; nhi[j] = cuts[i + 1]; }
    }
    int64_t *cost = (int64_t *)malloc(sizeof(int64_t) * (size_t)n * (size_t)n);
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    orc_transfer_cost_matrix(pr->L, w, n, olo, ohi, nlo, nhi, cost);
    int64_t total = orc_assign(n, cost, tmp);
    if (assign) memcpy(assign, tmp, sizeof(int32_t) * (size_t)n);
    free(cost); free(tmp); free(w); free(olo);
    return total;
}

/*
 * Objective of one candidate next state (Section "Problem Formulation", the arg max over
 * the next state): throughput B / t_step times the effective-time ratio
 * t_state / (t_trans + t_state), where t_trans + t_state = t_gap is the same for every
 * plan.  B and t_gap are constants of the arg max, so plans are ranked by
 *     (t_gap - t_trans) / t_step  =  training steps completed before the next fault.
 * Transition time (Section "Estimator"): search cost is overlapped with training and not
 * charged; restart overhead is a constant of the training scale; the weight transfer is
 * the matched bytes over the transfer bandwidth (reading: the paper gives no formula for
 * the time of the transfer, only that its amount is minimised).  Rerouting and redundant
 * computation need no reconstruction: transition time 0.
 * _f64: one IEEE operation per written operation.  _i64: the quotient bytes / bandwidth
 * floors and two objectives are compared exactly as fractions.
 */
/*
 * Step time of a dynamic-parallelism plan with the asymmetric synchronisation of Section
 * "Restorer" (Asymmetric Communication): the slowest pipeline (without a synchronisation
 * term of its own) plus the all-reduce rounds of the coloured layer graph.  Reading (the
 * paper gives the rounds, not their time): the all-reduce of layer l over the dp pipelines
 * takes the ring lower bound 2(n-1) * params(l) / (n * bw_sync), a round lasts as long as
 * its largest layer, rounds run one after the other (summed in colour order).
 */
static num_t plan_async_step(const space *sp, const orc_plan *pl, int *rounds_out, int *domains_out, num_t *t_sync_out) {
    const orc_profile *pr = sp->M.p;
    int L = pr->L, dp = (int)pl->n_pipes;
    int32_t *stage_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)dp * (size_t)L);
    int32_t colour[ORC_MAX_LAYERS];
    num_t t_pipe = 0;
    for (int p = 0; p < dp; p++) {
        int32_t cuts[ORC_MAX_STAGES + 1];
        int devs[ORC_MAX_STAGES];
        const segment *g = find_segment(sp, (int)pl->strategy, p, pl->micro[p]);
        segment_cuts(sp, g, pl->kappa[p], cuts);
        for (int i = 0; i < g->S; i++) {
            devs[i] = sp->surv[g->off + i];
            for (int l = cuts[i]; l < cuts[i + 1]; l++) stage_of[(size_t)p * L + l] = i;
        }
        num_t c; int ok;
        pipe_from_cuts(&sp->M, g->S, cuts, g->m, devs, 1 /* no peers: bare pipeline time */, &c, &ok);
        t_pipe = nmax(t_pipe, c);
    }
    int rounds = orc_comm_rounds(L, dp, stage_of, colour);
    num_t t_sync = 0;
    for (int c = 0; c < rounds; c++) {
        num_t longest = 0;
        for (int l = 0; l < L; l++)
            if (colour[l] == c) longest = nmax(longest, sync_time(pr, pr->param_bytes[l], dp));
        t_sync = t_sync + longest;
    }
    if (rounds_out) *rounds_out = rounds;
    if (domains_out) *domains_out = orc_comm_domains(L, dp, stage_of);
    if (t_sync_out) *t_sync_out = t_sync;
    free(stage_of);
    return t_pipe + t_sync;
}

typedef struct { num_t numer, denom; } frac_t;

static int frac_greater(frac_t a, frac_t b) {   /* a > b, both denominators > 0 */
#if ORC_INT
    return (__int128)a.numer * (__int128)b.denom > (__int128)b.numer * (__int128)a.denom;
#else
    return a.numer / a.denom > b.numer / b.denom;
#endif
}

int NAME(orc_search_objective)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                               const orc_objective *q, orc_plan *best, orc_transition *tr,
                               int32_t *assign /* [n_surv] or NULL */,
                               orc_plan *short_plans /* [topk] or NULL */, int64_t *short_bytes /* [topk] or NULL */,
                               int32_t *short_rounds /* [topk] or NULL */, int32_t *n_short /* or NULL */) {
#if ORC_INT
    const num_t t_gap = q->t_gap_ns, t_restart = q->t_restart_ns;
#else
    const num_t t_gap = q->t_gap, t_restart = q->t_restart;
#endif
    int k = q->topk < 1 ? 1 : q->topk;
    orc_plan *plans = (orc_plan *)calloc((size_t)k + 2, sizeof(orc_plan));
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    int32_t *asg = (int32_t *)malloc(sizeof(int32_t) * (size_t)(sp.n_surv + 1));
    int have = 0;
    frac_t best_j = {0, 1};
    memset(best, 0, sizeof(*best));
    memset(tr, 0, sizeof(*tr));
    tr->n_surv = sp.n_surv;
    tr->rank = -1;
    /* policies without reconstruction, in policy order */
    for (int pol = 0; pol < 2; pol++) {
        orc_plan pl;
        NAME(orc_search_policy)(prof, o, failed, n_failed, pol, 0, &pl, NULL);
        if (!pl.feasible) continue;
        frac_t j = {t_gap, get_cost(&pl)};
        if (!have || frac_greater(j, best_j)) {
            have = 1; best_j = j; *best = pl;
            tr->policy = pol; tr->feasible = 1; tr->rank = -1; tr->xfer_bytes = 0;
            tr->t_trans = 0; tr->t_trans_ns = 0;
        }
    }
    int ns = dynpar_shortlist(&sp, k, plans);
    if (n_short) *n_short = ns;
    for (int r = 0; r < ns; r++) {
        int64_t bytes = plan_transfer_bytes(&sp, &plans[r], asg);
        int rounds = 0, domains = 0;
        num_t t_sync = 0;
        if (q->sync_rounds) set_cost(&plans[r], plan_async_step(&sp, &plans[r], &rounds, &domains, &t_sync));
        if (short_plans) short_plans[r] = plans[r];
        if (short_bytes) short_bytes[r] = bytes;
        if (short_rounds) short_rounds[r] = rounds;
#if ORC_INT
        num_t t_trans = t_restart + bytes / q->bw_xfer;
#else
        num_t t_trans = t_restart + (double)bytes / (double)q->bw_xfer;
#endif
        frac_t j = {t_gap - t_trans, get_cost(&plans[r])};
        if (!have || frac_greater(j, best_j)) {
            have = 1; best_j = j; *best = plans[r];
            tr->policy = ORC_DYNPAR; tr->feasible = 1; tr->rank = r; tr->xfer_bytes = bytes;
            tr->rounds = rounds; tr->domains = domains;
#if ORC_INT
            tr->t_trans_ns = t_trans; tr->t_trans = 0;
            tr->t_sync_ns = t_sync; tr->t_sync = 0;
#else
            tr->t_trans = t_trans; tr->t_trans_ns = 0;
            tr->t_sync = t_sync; tr->t_sync_ns = 0;
#endif
            if (assign) memcpy(assign, asg, sizeof(int32_t) * (size_t)sp.n_surv);
        }
    }
    if (have) tr->objective = (double)best_j.numer / (double)best_j.denom;
    free(asg);
    free(plans);
    space_free(&sp);
    return have;
}

/* Transfer bytes and matching of one given dynamic-parallelism plan. */
int64_t NAME(orc_plan_transfer)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                                const orc_plan *pl, int32_t *assign /* [n_surv] or NULL */) {
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    int64_t b = plan_transfer_bytes(&sp, pl, assign);
    space_free(&sp);
    return b;
}

/* Asymmetric-synchronisation step time of one given dynamic-parallelism plan. */
double NAME(orc_plan_async_step)(const orc_profile *prof, const orc_opts *o, const uint32_t *failed, int n_failed,
                                 const orc_plan *pl, int32_t *rounds, int32_t *domains, double *t_sync) {
    space sp;
    space_build(&sp, prof, o, failed, n_failed);
    int r = 0, d = 0;
    num_t ts = 0;
    num_t t = plan_async_step(&sp, pl, &r, &d, &ts);
    if (rounds) *rounds = r;
    if (domains) *domains = d;
    if (t_sync) *t_sync = (double)ts;
    space_free(&sp);
    return (double)t;
}
