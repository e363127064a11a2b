/*
 * CPU oracle for the execution-plan search -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded restatement of the paper's performance model and of
 * the exhaustive search over recovery plans.  It shares no code with the CUDA path and
 * is used only by the tests, the smoke check and the bench's CPU-baseline leg.
 *
 * Every function cites the passage of the paper it follows (section / equation /
 * algorithm).  Where the paper is silent, the reading taken is stated at the function.
 *
 * Two numeric builds of the model exist side by side: suffix _f64 (IEEE double, one
 * rounding per written operation, no contraction) and suffix _i64 (integer nanoseconds,
 * every division floors).  Bytes are always int64.
 */
#ifndef ORC_H
#define ORC_H

#include <stdint.h>

#define ORC_MAX_PIPES 16
#define ORC_MAX_STAGES 64
#define ORC_MAX_LAYERS 128

enum { ORC_REROUTE = 0, ORC_REDUNDANT = 1, ORC_DYNPAR = 2 };
enum { ORC_LAYERS_FULL = 0, ORC_LAYERS_REMAINDER = 1, ORC_LAYERS_MINMAX = 2 };
enum { ORC_BATCH_FULL = 0, ORC_BATCH_REMAINDER = 1 };
/* Order of the computations on every stage: the dependency map f_2 of the transition equation
 * (Section "Estimator").  1F1B = non-interleaved one-forward-one-backward; GPIPE = all forwards
 * of the iteration, then all backwards. */
enum { ORC_SCHED_1F1B = 0, ORC_SCHED_GPIPE = 1 };

typedef struct {
    int32_t L, n_dp, n_pp, n_micro;
    const double *fwd_ns, *bwd_ns;       /* [L] per micro-batch            */
    const int64_t *fwd_ns_i, *bwd_ns_i;  /* [L] same, integer nanoseconds  */
    const int64_t *act_bytes, *param_bytes, *opt_bytes, *p2p_bytes; /* [L] */
    const int32_t *base_cuts;            /* [n_pp+1]                       */
    int64_t mem_capacity_bytes;
    int32_t devices_per_node;
    int64_t bw_intra, bw_inter;          /* bytes per nanosecond           */
} orc_profile;

typedef struct {
    int32_t dp_lo, dp_hi, pp_lo, pp_hi;
    int32_t layer_mode, batch_mode;
    uint64_t kappa_cap;
    int32_t schedule;   /* ORC_SCHED_* */
} orc_opts;

typedef struct {
    int32_t policy, feasible;
    double cost;      /* _f64 build; 0 in the _i64 build */
    int64_t cost_ns;  /* _i64 build; 0 in the _f64 build */
    uint32_t strategy, n_pipes;
    uint64_t split_rank;
    uint16_t stages[ORC_MAX_PIPES], micro[ORC_MAX_PIPES];
    uint64_t kappa[ORC_MAX_PIPES];
} orc_plan;

/* The paper's full objective (Section "Problem Formulation"): throughput of the next state
 * times the share of the time until the next fault that is spent training.  */
typedef struct {
    int32_t topk;                    /* dynamic-parallelism plans that are re-scored, >= 1   */
    int32_t sync_rounds;             /* 1: step time of a shortlisted plan = slowest pipeline +
                                        all-reduce rounds of the coloured layer graph         */
    double t_gap, t_restart;         /* ns between two faults / restart overhead (_f64)     */
    int64_t t_gap_ns, t_restart_ns;  /* the same as integers (_i64)                         */
    int64_t bw_xfer;                 /* bytes per ns available to the weight transfer       */
} orc_objective;

typedef struct {
    int32_t policy, feasible;
    int32_t rank;                    /* position of the chosen plan in the shortlist, -1 for the other policies */
    int32_t n_surv;
    int64_t xfer_bytes;              /* bytes moved by the cheapest migration scheme        */
    double t_trans;                  /* transition time, _f64                               */
    int64_t t_trans_ns;              /* transition time, _i64                               */
    double objective;                /* steps completed before the next fault               */
    int32_t rounds, domains;         /* communication rounds / domains of the chosen plan (sync_rounds = 1) */
    double t_sync;                   /* time of those rounds, _f64                          */
    int64_t t_sync_ns;               /* _i64                                                */
} orc_transition;

/* ---- orc_restore.c: weight-transfer matching (integer) ---- */
void orc_transfer_cost_matrix(int L, const int64_t *w, int n, const int32_t *old_lo, const int32_t *old_hi,
                              const int32_t *new_lo, const int32_t *new_hi, int64_t *cost /* [n][n] */);
int64_t orc_assign(int n, const int64_t *cost, int32_t *row_of_col);
int64_t orc_assign_brute(int n, const int64_t *cost);
int orc_comm_rounds(int L, int dp, const int32_t *stage_of /* [dp][L] */, int32_t *colour /* [L] */);
int orc_comm_domains(int L, int dp, const int32_t *stage_of);

/* ---- orc_enum.c: integer combinatorics (no cost arithmetic) ---- */
uint64_t orc_binom(int n, int k);                       /* saturates at UINT64_MAX */
void orc_unrank_subset(uint64_t rank, int t, int *c);   /* colex, c[0]<...<c[t-1]  */
uint64_t orc_rank_subset(int t, const int *c);
int orc_strategies(int n_surv, int dp_lo, int dp_hi, int pp_lo, int pp_hi, int L,
                   int max_out, int32_t *dp_out, int32_t *stages_out /* [max_out][ORC_MAX_PIPES] */);
uint64_t orc_split_count(int batch_mode, int G, int n_surv, int dp, const int32_t *stages);
int orc_split_unrank(int batch_mode, int G, int n_surv, int dp, const int32_t *stages,
                     uint64_t beta, int32_t *micro_out);
uint64_t orc_layer_count(int layer_mode, int L, int S);  /* K of the enumerated part  */
void orc_layer_unrank(int layer_mode, int L, int S, uint64_t kappa, int32_t *cuts_out /* [S+1] */);

#endif
