/*
 * chameleon.h -- C ABI of the B200-native execution-plan search.
 *
 * The library answers the question the paper's decision center answers when a device
 * fails (Chameleon, Section "Performance Modeling": given the current state, determine
 * the next execution plan with the least step time; Section "Planner", Algorithm 1):
 * enumerate the candidate recovery plans under each backup-free policy -- data
 * rerouting, redundant computation, dynamic parallelism -- evaluate the unified
 * performance model (Section "Estimator": step time and peak memory) on every
 * candidate, and return the feasible plan with the least estimated iteration time.
 *
 * Everything is computed by hand-written CUDA kernels for sm_100a on the stream given
 * to cm_create; the host side only builds small descriptor tables (strategies,
 * segments) from the failure set.  There is no CPU fallback: without an sm_100 device
 * cm_create fails with CM_ECUDA.
 *
 * Conventions
 *  - Every call returns a cm_status and never throws, aborts or prints.  On error the
 *    out-parameters are untouched; cm_last_error(ctx) holds a message.
 *  - "HOST" / "DEVICE" at a pointer says where the memory lives.  The caller owns every
 *    buffer it passes; the library owns cm_ctx and cm_space objects until they are
 *    destroyed / freed.
 *  - All device work is enqueued on the context's stream (independent kernels of the search
 *    pass may run on streams the library owns, forked from and joined back into the
 *    context's stream, so ordering as seen from that stream is unchanged).  Calls that return results to
 *    the host (cm_select, cm_search_batch, cm_decode_plan) synchronise that stream
 *    before returning; cm_load_profile, cm_enumerate and cm_evaluate only enqueue.
 *  - A cm_ctx is not thread-safe; distinct contexts are independent.
 *  - Times are nanoseconds, sizes are bytes, bandwidths are bytes per nanosecond
 *    (numerically GB/s).  Device d of the fault-free N_dp x N_pp grid is stage
 *    d mod N_pp of pipeline d / N_pp and sits on node d / devices_per_node.
 */
#ifndef CHAMELEON_H
#define CHAMELEON_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CM_MAX_PIPES 16    /* data-parallel pipelines of a plan            */
#define CM_MAX_STAGES 64   /* stages of one pipeline                       */
#define CM_MAX_LAYERS 128  /* model layers in a profile                    */
#define CM_MAX_MICRO 4096  /* global micro-batches per iteration (N_dp*N_m) */
#define CM_MAX_SHORTLIST 16 /* dynamic-parallelism plans re-scored by the full objective */
#define CM_MAX_MATCH 256   /* devices in one weight-transfer matching      */

typedef struct cm_ctx cm_ctx;     /* device buffers, profile copy, tables               */
typedef struct cm_space cm_space; /* implicit candidate space of one (policy, failure set) */

typedef enum {
    CM_OK = 0,
    CM_EINVAL = 1,      /* bad argument (message says which)                         */
    CM_ENOPROFILE = 2,  /* cm_load_profile has not been called                       */
    CM_EOVERFLOW = 3,   /* a candidate / split count does not fit the index type     */
    CM_ENOFEASIBLE = 4, /* cm_select: no feasible plan in the given spaces           */
    CM_ECUDA = 5,       /* CUDA runtime error or no sm_100 device                    */
    CM_ENOMEM = 6,
    CM_ETIMEOUT = 7     /* reserved: no kernel of this library waits on another      */
} cm_status;

/* Policies in ascending order of transition cost (Section "Performance Modeling":
 * rerouting needs no reconstruction, dynamic parallelism moves weights and restarts),
 * so that breaking a cost tie by the lowest id picks the cheapest transition. */
typedef enum { CM_REROUTE = 0, CM_REDUNDANT = 1, CM_DYNPAR = 2 } cm_policy;

/* Arithmetic of the time estimator: IEEE double with one rounding per operation of the
 * model, or integer nanoseconds where every division floors (fully reproducible). */
typedef enum { CM_COST_FP64 = 0, CM_COST_INT64NS = 1 } cm_cost_mode;

/* Layer distribution (Section "Planner"): FULL = every composition of the L layers into
 * S non-empty stages; REMAINDER = even split, then every placement of the L mod S
 * leftover layers (C(S, L mod S) of them, the paper's rule); MINMAX = only the
 * contiguous partition that minimises the largest stage time.  FULL and REMAINDER add
 * that min-max partition as one more candidate per pipeline. */
typedef enum { CM_LAYERS_FULL = 0, CM_LAYERS_REMAINDER = 1, CM_LAYERS_MINMAX = 2 } cm_layer_mode;

/* Micro-batch distribution (Section "Planner"): REMAINDER = proportional to the nodes
 * of each pipeline, every way of handing out the leftover micro-batches one each;
 * FULL = every composition of the global micro-batch count into positive parts. */
typedef enum { CM_BATCH_FULL = 0, CM_BATCH_REMAINDER = 1 } cm_batch_mode;

/* The profile the paper's profiler delivers (Section "System Design", monitoring:
 * execution time, HBM usage, parallel configuration) plus the link tiers.  All pointers
 * are HOST memory and are copied by cm_load_profile. */
typedef struct {
    int32_t L, n_dp, n_pp, n_micro;     /* layers; fault-free grid; micro-batches per pipeline */
    const double *fwd_ns, *bwd_ns;      /* [L] time per micro-batch (fp64 mode)                */
    const int64_t *fwd_ns_i, *bwd_ns_i; /* [L] the same in whole nanoseconds (int64 mode)      */
    const int64_t *act_bytes;           /* [L] activations stored per in-flight micro-batch    */
    const int64_t *param_bytes;         /* [L] parameters; gradients take the same             */
    const int64_t *opt_bytes;           /* [L] optimizer state                                 */
    const int64_t *p2p_bytes;           /* [L] bytes crossing a stage boundary after layer l   */
    const int32_t *base_cuts;           /* [n_pp+1] fault-free layer->stage cuts, 0 .. L       */
    int64_t mem_capacity_bytes;         /* per device                                          */
    int32_t devices_per_node;
    int64_t bw_intra_Bpns, bw_inter_Bpns;
} cm_profile;

/* Order of the computations on every stage: the dependency map f_2 of the start/end transition
 * equation (Section "Estimator": "f_1(i), f_2(j) ... can be profiled from the actual execution
 * order").  1F1B = non-interleaved one-forward-one-backward (min(S-1-i, m) warm-up forwards,
 * forward/backward pairs, the remaining backwards; min(S-i, m) micro-batches of activations in
 * flight at stage i, the paper's memory estimator).  GPIPE = all m forwards of the iteration,
 * then all m backwards; all m micro-batches are in flight at every stage.  The order applies
 * to every policy: rerouting and redundant computation are timed under it as well. */
typedef enum { CM_SCHED_1F1B = 0, CM_SCHED_GPIPE = 1 } cm_schedule;

/* Search window (Algorithm 1 inputs R_dp, R_pp) and enumeration modes.  A pipeline whose
 * enumerated layer compositions outnumber kappa_cap contributes only its min-max
 * partition. */
typedef struct {
    int32_t dp_lo, dp_hi, pp_lo, pp_hi;
    cm_layer_mode lm;
    cm_batch_mode bm;
    uint64_t kappa_cap;
    cm_cost_mode cost;
    cm_schedule sched;
} cm_enum_opts;

/* An execution plan (Definition 1: policy, parallel configuration, data distribution,
 * layer distribution).  stages[p], micro[p], kappa[p] describe pipeline p: its stage
 * count, its micro-batches per iteration and the rank of its layer composition (for
 * CM_DYNPAR; kappa equal to the enumerated count means the min-max partition).
 * cost is filled in fp64 mode, cost_ns in int64 mode; the other is 0. */
typedef struct {
    int32_t policy, feasible;
    double cost;
    int64_t cost_ns;
    uint32_t strategy, n_pipes;
    uint64_t split_rank;
    uint16_t stages[CM_MAX_PIPES], micro[CM_MAX_PIPES];
    uint64_t kappa[CM_MAX_PIPES];
} cm_plan;

/* Create a context on a CUDA device.  cuda_stream is a cudaStream_t owned by the caller
 * (NULL = the default stream); all work of this context is enqueued on it.
 * CM_ECUDA if the device is not compute capability 10.x. */
cm_status cm_create(cm_ctx **out, int cuda_device, void *cuda_stream);
cm_status cm_destroy(cm_ctx *ctx);

/* Copy a profile to the device and build the per-layer prefix sums the estimators read
 * (Section "Estimator": stage time and stage memory are sums over the stage's layers).
 * Validates: 1 <= L <= CM_MAX_LAYERS, 1 <= n_pp <= min(L, CM_MAX_STAGES),
 * 1 <= n_dp <= CM_MAX_PIPES, n_dp*n_micro <= CM_MAX_MICRO, finite non-negative times,
 * non-negative bytes, positive bandwidths and capacity, base_cuts strictly increasing
 * from 0 to L.  May be called again to replace the profile. */
cm_status cm_load_profile(cm_ctx *ctx, const cm_profile *profile);

/* Describe the candidate space of one policy for one failure set (HOST failed_ids,
 * distinct, each < n_dp*n_pp; n_failed may be 0).  For CM_DYNPAR the space is
 * (Section "Planner"): every strategy (dp, S_1<=...<=S_dp) that uses all survivors
 * within the window, every micro-batch split, every layer composition per pipeline;
 * *n_candidates counts pipeline-plans (strategy, pipeline, micro-batch count, layer
 * composition) in segment-major order.  CM_REROUTE and CM_REDUNDANT have one candidate.
 * Nothing is stored per candidate: plans are unranked from their index on the device.
 * opts may be NULL for the one-candidate policies (fp64 is then assumed). */
cm_status cm_enumerate(cm_ctx *ctx, cm_policy policy, const uint32_t *failed_ids, int32_t n_failed,
                       const cm_enum_opts *opts, cm_space **out, uint64_t *n_candidates);

/* Evaluate candidates first .. first+count-1 of a space, or the count indices listed in
 * DEVICE idx_dev (NULL = contiguous).  Writes, for each, the pipeline cost (pipeline
 * time by the start/end recurrence of Section "Estimator" plus gradient-sync time) and
 * the memory-feasibility flag (peak-memory formula of Section "Estimator") into the
 * caller's DEVICE buffers; any of them may be NULL.  Infeasible candidates get
 * +infinity / INT64_MAX and flag 0; that is not an error.  cost_dev is written in fp64
 * mode, cost_ns_dev in int64 mode (the other buffer is left untouched).  Enqueues only. */
cm_status cm_evaluate(cm_ctx *ctx, const cm_space *space, uint64_t first, uint64_t count,
                      const uint64_t *idx_dev, double *cost_dev, int64_t *cost_ns_dev,
                      uint8_t *feasible_dev);

/* Search the given spaces (Algorithm 1, get_execution_plan: keep the plan with the
 * least estimated time; step time = slowest pipeline) and write the best plan to HOST
 * *best: least cost, ties to the lexicographically smallest plan tuple within a policy
 * and to the lowest policy id across policies.  CM_ENOFEASIBLE (best->feasible = 0) if
 * nothing fits in memory.  All spaces must share one cost mode.  Synchronises. */
cm_status cm_select(cm_ctx *ctx, cm_space *const *spaces, int32_t n_spaces, cm_plan *best);

/* Layer cuts of every pipeline of a plan found in this space, concatenated into HOST
 * cuts_out (sum over pipelines of stages[p]+1 entries, each pipeline 0 .. L). */
cm_status cm_decode_plan(cm_ctx *ctx, const cm_space *space, const cm_plan *plan, int32_t *cuts_out);

cm_status cm_space_free(cm_space *space);

/* The whole search for B failure sets in one launch sequence (the paper pre-computes
 * the plans for potential failure scenarios, Section "Planner"): scenario b fails
 * failed_ids[offsets[b] .. offsets[b+1]-1] (HOST).  All three policies are searched for
 * every scenario.  best_per_scenario: HOST [B]; best_per_policy: HOST [B*3] or NULL;
 * a scenario without a feasible plan gets feasible = 0 and the call still returns
 * CM_OK.  If latency_us (HOST [B]) is not NULL the scenarios are searched one at a
 * time and latency_us[b] is the wall time of scenario b from descriptor build to its
 * plan on the host; results are identical either way.  Synchronises. */
cm_status cm_search_batch(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                          const cm_enum_opts *opts, cm_plan *best_per_scenario,
                          cm_plan *best_per_policy, float *latency_us);

/* The same search split in two, for callers that search one set of scenarios repeatedly
 * (and for timing the kernels with the descriptors already resident in device memory):
 * cm_batch_prepare builds the descriptor tables of B failure sets, copies them to the
 * device and computes the min-max partitions they need; cm_batch_search runs the launch
 * sequence over a prepared batch and returns the plans as cm_search_batch does
 * (synchronises); cm_batch_free releases it.  A batch belongs to the profile that was
 * loaded when it was prepared. */
typedef struct cm_batch cm_batch;
cm_status cm_batch_prepare(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                           const cm_enum_opts *opts, cm_batch **out, uint64_t *n_candidates);
cm_status cm_batch_search(cm_ctx *ctx, cm_batch *batch, cm_plan *best_per_scenario,
                          cm_plan *best_per_policy);
cm_status cm_batch_free(cm_batch *batch);

/* The paper has no counterpart to this call: it exists for callers that must not allocate.
 * A failure handler may run while the training framework's caching allocator holds all
 * free device memory, on a path where the device-wide synchronisation of an allocation
 * is unaffordable, or in a process whose memory budget was fixed at start-up.  Such a
 * caller builds its candidate space beforehand with cm_enumerate (that does allocate)
 * and later calls this function, which allocates nothing on host or device.
 *
 * Evaluates candidates first .. first+count-1 of a CM_DYNPAR space exactly as cm_evaluate
 * does and reduces them on the device to the least cost and the lowest candidate index
 * that attains it, written to the caller's DEVICE buffers: best_cost_dev in fp64 mode,
 * best_cost_ns_dev in int64 mode (the other is left untouched; any pointer may be NULL),
 * best_index_dev = UINT64_MAX and cost = +infinity / INT64_MAX if no candidate of the
 * range is memory-feasible.  Enqueues on the context's stream and returns.
 *
 * Limits and rules: count must be 1 .. CM_NOALLOC_MAX_CANDIDATES (larger ranges are
 * rejected with CM_EINVAL; split them).  The block partials of the reduction live in a
 * fixed 64 KB array inside the library, one per GPU, shared by every call on that GPU:
 * two calls that overlap on the device (different streams or contexts) race on it, so
 * serialise them.  The first call on a device looks up the array's address; make that
 * call before starting any stream capture. */
#define CM_NOALLOC_MAX_CANDIDATES 524288
cm_status cm_evaluate_argmin_noalloc(cm_ctx *ctx, const cm_space *space, uint64_t first, uint64_t count,
                                     double *best_cost_dev, int64_t *best_cost_ns_dev,
                                     uint64_t *best_index_dev);

/* ---------------------------------------------------------------------------------
 * Full objective: transition time included.
 *
 * Section "Problem Formulation" ranks a candidate next state by
 *     throughput * effective-time ratio = (B / t_step) * t_state / (t_trans + t_state),
 * where t_trans + t_state (the time between two faults, t_gap) does not depend on the plan.
 * B and t_gap being constants of the arg max, plans are ranked by
 *     (t_gap - t_trans) / t_step,   the training steps completed before the next fault.
 * Section "Estimator": rerouting (and redundant computation) need no reconstruction,
 * t_trans = 0; for dynamic parallelism t_trans = restart overhead + weight transfer (the
 * search itself is overlapped with training).  Section "Restorer", Weight Transfer: the
 * survivors are matched to the positions of the new plan by a minimum-cost perfect
 * matching over Cost[i][j] = model state (parameters + optimizer bytes per layer, from the
 * loaded profile) of the layers position j holds and device i does not hold yet; the
 * transfer takes (matched bytes) / bw_xfer.
 *
 * The transfer couples the pipelines of a plan, so it is applied to a shortlist: the
 * `topk` (strategy, split) pairs of least step time (ties: enumeration order), each
 * completed with the lowest layer compositions that meet its own step time.  The winner
 * is the candidate of greatest objective among rerouting, redundant computation and the
 * shortlist, ties to the lower policy id, then to the earlier shortlist rank.  fp64 mode
 * computes t_trans = t_restart + bytes / bw and the objective with one IEEE operation each;
 * int64 mode floors bytes / bw and compares objectives exactly as fractions.
 *
 * sync_rounds = 1 (Section "Restorer", Asymmetric Communication): when pipelines cut the
 * model differently, the all-reduce of a layer spans different stages in different
 * pipelines and two layers that share a device in any pipeline cannot synchronise at the
 * same time.  Layers are vertices, such pairs edges; a greedy colouring in layer order
 * (least colour no coloured neighbour has) gives the communication rounds.  A shortlisted
 * plan is then timed as  slowest pipeline (without a synchronisation term of its own)
 * + sum over rounds of the longest all-reduce of the round, the all-reduce of layer l over
 * the dp pipelines taking 2 (dp-1) params(l) / (dp * bw_sync) as in the search's model;
 * that step time replaces the search's in plan.cost / cost_ns and in the objective.
 * Communication domains = maximal runs of layers held by the same device in every pipeline.
 * --------------------------------------------------------------------------------- */
typedef struct {
    int32_t topk;              /* 1 .. CM_MAX_SHORTLIST                                   */
    int32_t sync_rounds;       /* 0: step time as the search computes it; 1: asymmetric
                                  synchronisation rounds (above)                           */
    double t_gap_ns;           /* time between two faults (fp64 mode), finite, > 0          */
    double t_restart_ns;       /* restart overhead of a reconstruction (fp64 mode), >= 0     */
    int64_t t_gap_ns_i;        /* the same, integer nanoseconds (int64 mode)                */
    int64_t t_restart_ns_i;
    int64_t bw_xfer_Bpns;      /* bandwidth of the weight transfer, bytes per ns, > 0       */
} cm_objective_opts;

typedef struct {
    int32_t policy, feasible;
    int32_t rank;              /* shortlist rank of the chosen plan, -1 for the other policies */
    int32_t n_survivors;
    int64_t xfer_bytes;        /* bytes moved by the cheapest migration (0 without one)     */
    double t_trans;            /* transition time, ns (fp64 mode; 0 in int64 mode)          */
    int64_t t_trans_ns;        /* transition time, ns (int64 mode; 0 in fp64 mode)          */
    double objective;          /* steps before the next fault (int64 mode: numerator / denominator rounded once) */
    int32_t rounds, domains;   /* sync_rounds = 1, dynamic parallelism: communication rounds and
                                  communication domains of the chosen plan; 0 otherwise     */
    double t_sync;             /* time of those rounds, ns (fp64 mode)                      */
    int64_t t_sync_ns;         /* time of those rounds, ns (int64 mode)                     */
    uint16_t assign[CM_MAX_MATCH]; /* dynamic parallelism: position j (pipeline-major, stage-minor) ->
                                      index, among the survivors in ascending id order, of the device
                                      that takes it; zeros otherwise                         */
} cm_transition;

/* The search of cm_search_batch followed by the re-scoring above, for B failure sets.
 * failed_ids / offsets / opts as for cm_search_batch (HOST).  best[B] and trans[B] (HOST,
 * caller-owned) receive the chosen plan (plan.cost / cost_ns = its step time) and its
 * transition.  shortlist (HOST [B * topk], may be NULL) receives the shortlisted plans in
 * rank order, shortlist_bytes (HOST [B * topk], may be NULL) their matched bytes,
 * shortlist_rounds (HOST [B * topk], may be NULL) their communication rounds (0 unless
 * sync_rounds = 1); unused slots have feasible = 0, bytes = -1, rounds = 0.  Several
 * matchings of one plan can be optimal: assign[] is one of them, xfer_bytes is unique.
 * Errors: CM_EINVAL (bad options; more than CM_MAX_MATCH devices in the profile's grid),
 * CM_ENOPROFILE, CM_EOVERFLOW, CM_ENOMEM, CM_ECUDA.  A scenario without any feasible plan
 * has best[b].feasible = 0 and is not an error of the batch.  Synchronises the stream. */
cm_status cm_search_objective(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                              const cm_enum_opts *opts, const cm_objective_opts *objective,
                              cm_plan *best, cm_transition *trans, cm_plan *shortlist,
                              int64_t *shortlist_bytes, int32_t *shortlist_rounds);

/* Transition time the full objective charges a reconstruction that moves xfer_bytes of model
 * state (Section "Estimator", state-transition overhead = restart + weight transfer):
 * fp64 mode t_restart_ns + bytes / bw_xfer (one IEEE operation each), int64 mode
 * t_restart_ns_i + floor(bytes / bw_xfer) -- the very routine the objective kernel applies, so a
 * caller can price the shortlisted plans that were not chosen from the shortlist_bytes of
 * cm_search_objective without restating the rule.  All pointers HOST; n values; either output
 * may be NULL; an entry of -1 (empty shortlist slot) gives -1.  No device work.
 * CM_EINVAL on NULL options, negative n or a non-positive bandwidth. */
cm_status cm_transition_time(const cm_objective_opts *objective, int32_t n, const int64_t *xfer_bytes,
                             double *t_trans_ns, int64_t *t_trans_ns_i);

/* The host-side descriptor builder alone, for one failure set and the dynamic-parallelism
 * policy (Algorithm 1, get_parallel_strategy; Section "Planner", batch and layer
 * distribution): no CUDA call is made, so it also runs on a machine without a GPU.
 * HOST out[8]: [0] candidates (pipeline-plans)  [1] strategies  [2] segments
 * [3] (strategy, split) pairs  [4] surviving devices  [5] launch classes  [6] buckets
 * [7] node boundaries between neighbouring survivors.  Errors as cm_load_profile /
 * cm_enumerate (CM_EINVAL, CM_EOVERFLOW). */
cm_status cm_host_describe(const cm_profile *profile, const uint32_t *failed_ids, int32_t n_failed,
                           const cm_enum_opts *opts, uint64_t out[8]);

/* Arithmetic of the integer-nanosecond mode.  Its inputs are integers and the model only adds,
 * takes maxima and floors quotients, so every value is an integer; as long as all of them
 * stay below 2^53 a double holds them exactly, and 64-bit floating-point adds issue faster
 * on this GPU than 64-bit integer adds.  cm_load_profile bounds the largest value the loaded
 * profile can produce (all work of all micro-batches, rerouted and redundant load included,
 * plus every transfer in sequence plus the longest synchronisation); below 2^52 the integer
 * mode is evaluated in double arithmetic with floored quotients, bit-identical to the integer
 * kernels, otherwise in 64-bit integer arithmetic.  cm_set_int64_arithmetic(ctx, 1) forces the
 * integer kernels for batches and spaces built afterwards, (ctx, 0) restores the default;
 * cm_int64_runs_in_fp64 returns 1 if the integer mode of the loaded profile currently runs in
 * double arithmetic. */
cm_status cm_set_int64_arithmetic(cm_ctx *ctx, int native);
int cm_int64_runs_in_fp64(const cm_ctx *ctx);

/* Per-failure searches (cm_search_batch with latency_us): everything but the failed ids and the
 * node-crossing bits of a one-scenario search depends only on the survivor count and the
 * options, so the context keeps a prepared batch per (survivor count, options) resident (at most
 * 64; dropped by cm_load_profile) and a search patches those few bytes.  From its second use on,
 * such a batch replays its launch sequence as a CUDA graph, captured on a library-owned stream
 * and launched on the context's stream; cm_last_stats then reports the whole device time but
 * not the per-phase times ([8], [11], [12] stay 0).  cm_set_latency_graphs(ctx, 0) keeps the
 * plain launches (default 1).  Results are identical either way.  The first search for a
 * survivor count builds its batch and the second captures its graph (1 to 2 ms each on the
 * 32-device workload); a caller that wants the short path at failure time searches any failure
 * set of each expected size twice beforehand. */
cm_status cm_set_latency_graphs(cm_ctx *ctx, int on);

/* Memory screen (on by default).  Whether a layer composition fits in memory depends on the
 * stage count, the micro-batches in flight and the composition itself -- not on which devices
 * failed, the link tiers or the cost mode (Section "Estimator", memory estimator).  The context
 * therefore lists, once per profile and (layer mode, stages, micro-batches), the memory-feasible
 * compositions in ascending order, and the search and tie-break passes walk those lists instead
 * of all enumerated compositions (segments of more than 2^20 compositions are walked in full).
 * The first search that meets a new (stages, micro-batches) pair builds its list: one small copy
 * each way, one kernel and a stream synchronisation.  Results are identical either way; candidate
 * indices, cm_evaluate and cm_decode_plan are unaffected; cm_last_stats [0] still counts every
 * enumerated pipeline-plan and [16] those whose recurrence ran.  cm_set_memory_screen(ctx, 0)
 * makes batches and spaces built afterwards test every composition inside the search pass. */
cm_status cm_set_memory_screen(cm_ctx *ctx, int on);

/* Micro-batch pairs (on by default).  A pipeline of a strategy appears with two micro-batch
 * counts, m and m + 1 (the two shares the remainder rule leaves it; consecutive counts under the
 * full split enumeration).  Under the 1F1B order the recurrences of the two coincide in every
 * round before the ramp-down of the shorter one -- whether micro-batch m exists shows first in
 * round m -- so for pipelines of up to 48 stages with m >= stages one thread evaluates both: the
 * common rounds once, then the two tails (shallow pipelines, up to 16 stages, where a group of
 * them holds enough plans to be worth a launch of its own).  Same operations on the same values: results are
 * bit-identical; cm_last_stats [1] counts the recurrence cells that actually ran.
 * cm_set_micro_batch_pairs(ctx, 0) makes batches and spaces built afterwards evaluate every
 * segment on its own. */
cm_status cm_set_micro_batch_pairs(cm_ctx *ctx, int on);

/* Pipeline reuse (on by default).  The strategies of one survivor count have pipelines in
 * common: the stage tuples (30, 31, ..) and (30, 32, ..) both start with 30 stages over the first
 * 30 survivors, with the same micro-batch counts and the same number of data-parallel peers.
 * Such a pipeline has the same candidates with the same costs whatever strategy it is part of
 * (Section "Estimator": a pipeline's time and memory are functions of its own stages, links and
 * micro-batches), so its least cost is searched once per scenario and the other strategies take
 * the result.  Results are identical; cm_last_stats [0] still counts every pipeline-plan of the
 * search space, [16] those whose recurrence ran.  cm_set_pipeline_reuse(ctx, 0) makes batches and
 * spaces built afterwards search every (strategy, pipeline) on its own. */
cm_status cm_set_pipeline_reuse(cm_ctx *ctx, int on);

/* Sharing (off by default): in a batch, failure sets that leave the same number of survivors
 * with node boundaries at the same places among them have identical dynamic-parallelism
 * searches -- survivors are placed in consecutive blocks and nothing else of the failure set
 * enters that policy's model.  With sharing on, cm_search_batch / cm_batch_prepare search
 * such scenarios once and copy the result; rerouting and redundant computation are always
 * evaluated per scenario.  In a batch of more than one scenario the pipelines are shared as
 * well: the least time of a pipeline over its layer compositions depends on its stages, its
 * micro-batches, the data-parallel peers of its strategy and the link tiers of its stage
 * boundaries only (Section "Estimator"), so the distinct such tuples of the batch are found on
 * the device (one small device->host copy and one synchronisation of the context's stream per
 * prepared batch) and each is searched once (as one half of a micro-batch pair where two distinct
 * pipelines differ only by one micro-batch).  A single failure set searched through the latency
 * path of cm_search_batch has its duplicate pipelines removed on the host when enough work is
 * saved to pay for launching its sequence directly instead of replaying the resident graph.
 * Results are identical either way; cm_last_stats
 * [0] then counts only the plans of the scenarios that were searched and [16] only the plans
 * whose recurrence ran.  cm_cache_build always shares. */
cm_status cm_set_sharing(cm_ctx *ctx, int on);

/* Device time and work of the objective pass of the last cm_search_objective (HOST out[8]):
 * [0] shortlist kernel, ns  [1] completing the shortlisted plans (tie-break kernels), ns
 * [2] matching kernel (and, with sync_rounds, the rounds kernel), ns  [3] objective kernel, ns  [4] matchings solved (only counted when
 * shortlist_bytes was asked for)  [5] kernels launched  [6] bytes copied device->host
 * [7] sum of [0..3].  cm_last_stats describes the search that ran before it. */
cm_status cm_objective_stats(const cm_ctx *ctx, uint64_t out[8]);

/* Weight-transfer matchings over explicit layer ranges (Section "Restorer", Weight
 * Transfer), using the per-layer model state of the loaded profile.  Problem q has
 * sizes[q] devices (1 .. CM_MAX_MATCH); device i holds layers [old_lo[q][i], old_hi[q][i]),
 * position j needs [new_lo[q][j], new_hi[q][j]) (all HOST, row stride CM_MAX_MATCH, values
 * 0 .. L, empty ranges allowed).  total[q] (HOST) = bytes of the cheapest perfect matching;
 * assign (HOST [n_problems][CM_MAX_MATCH], may be NULL): device index matched to position j.
 * Errors: CM_EINVAL, CM_ENOPROFILE, CM_ENOMEM, CM_ECUDA.  Synchronises the stream. */
cm_status cm_transfer_matching(cm_ctx *ctx, int32_t n_problems, const int32_t *sizes,
                               const uint8_t *old_lo, const uint8_t *old_hi,
                               const uint8_t *new_lo, const uint8_t *new_hi,
                               int64_t *total, uint16_t *assign);

/* ---------------------------------------------------------------------------------
 * Plan cache (Section "Planner", last paragraph: the best plans for the loss of 1 to k
 * devices are computed and cached during fault-free training, so that the decision at
 * failure time is a lookup).  The cache holds the result of the search for EVERY failure
 * set of at most max_failures devices (the empty set included) of the loaded profile's
 * grid; entries are addressed by the set's size and combinatorial rank.
 *
 * cm_cache_build: max_failures 0 .. 16; the number of sets may not exceed 2^20
 * (CM_EOVERFLOW).  Runs cm_search_batch over all
 * sets, 4096 at a time, on the context's stream (synchronises).  The cache is a HOST object
 * owned by the caller until cm_cache_free; it keeps no reference to device memory and stays
 * valid when the profile is reloaded (its plans then describe the old profile).
 * cm_cache_lookup: failed_ids in any order (HOST); best and per_policy[3] (may be NULL) are
 * HOST out-parameters; exactly what cm_search_batch returns for that set.  Errors:
 * CM_EINVAL (id out of range, duplicate ids), CM_ENOFEASIBLE if the set is larger than the
 * cache covers (the caller searches it instead).  Thread-safe for concurrent lookups.
 * --------------------------------------------------------------------------------- */
typedef struct cm_cache cm_cache;
cm_status cm_cache_build(cm_ctx *ctx, int32_t max_failures, const cm_enum_opts *opts, cm_cache **out,
                         uint64_t *n_scenarios);
cm_status cm_cache_lookup(const cm_cache *cache, const uint32_t *failed_ids, int32_t n_failed,
                          cm_plan *best, cm_plan *per_policy);
cm_status cm_cache_free(cm_cache *cache);

/* Work counters of the last cm_select / cm_search_batch / cm_batch_search on this
 * context (HOST out[24]):
 *  [0] pipeline-plans evaluated by the search pass   [1] recurrence cells simulated by it
 *      (2 * stages * micro-batches per memory-feasible plan, counted on the device)
 *  [2] pipeline-plans re-evaluated by the tie-break pass   [3] kernels launched
 *  [4] device time of the whole launch sequence, ns (CUDA events on the context's stream)
 *  [5] segments  [6] strategies  [7] micro-batch splits reduced
 *  [8] device time of the search-pass cost kernel(s) alone, ns   [9] bytes copied host->device
 *  [10] bytes copied device->host   [11] device time of the tie-break kernel(s), ns
 *  [12] launches of the search-pass cost kernel   [13] host time building descriptor tables, ns
 *  [14] host time enqueueing the launch sequence, ns   [15] host time waiting for the stream, ns
 *  [16] pipeline-plans whose recurrence ran, i.e. that are searched in their own right ([19]) and
 *       passed the memory estimator (Section "Estimator", memory estimator)
 *  [17] host time spent listing memory-feasible compositions (inside [13]; includes one stream
 *       synchronisation when a new (stages, micro-batches) pair is met), ns
 *  [18] host time packing and uploading the descriptor tables, buffer allocation included, ns
 *  [19] pipeline-plans of [0] that are searched in their own right: [0] - [19] belong to pipelines
 *       that another strategy of the same survivor count has as well and take its result
 *       (cm_set_pipeline_reuse); [19] - [16] were rejected by the memory estimator (with sharing
 *       on, [16] also leaves out what other scenarios' segments already covered)
 *  [20..23] reserved, 0. */
cm_status cm_last_stats(const cm_ctx *ctx, uint64_t out[24]);

const char *cm_strerror(cm_status status);
const char *cm_last_error(const cm_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* CHAMELEON_H */
