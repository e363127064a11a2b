// Internal layout shared by the host-side descriptor builder and the kernels.
// Nothing here is part of the C ABI.
#pragma once

#include <cstdint>
#include <string>
#include <cuda_runtime.h>

#include "chameleon.h"

namespace cm {

constexpr int kMaxL = CM_MAX_LAYERS;
constexpr int kMaxS = CM_MAX_STAGES;
constexpr int kMaxP = CM_MAX_PIPES;
constexpr int kBinomCols = 64;          // binomial table columns 0..64
constexpr int kTile = 128;              // layer compositions per CTA in the tie-break kernels
constexpr uint64_t kSat = ~0ull;        // saturated binomial

// Per-layer prefix arrays, built on the device by cm_prefix_kernel and staged into shared
// memory by every kernel that evaluates stages.  PS = 2*params + optimizer (static bytes).
struct DevProfile {
    int32_t L, n_dp, n_pp, n_micro;
    int32_t devices_per_node, G;
    int32_t intval, pad;   // 1: the double arrays hold the integer-nanosecond values (see cm_load_profile)
    int64_t cap, bw_intra, bw_inter, bw_sync;
    double PFd[kMaxL + 1], PBd[kMaxL + 1];
    int64_t PFi[kMaxL + 1], PBi[kMaxL + 1];
    int64_t PA[kMaxL + 1], PS[kMaxL + 1], PP[kMaxL + 1];
    int64_t PW[kMaxL + 1];  // parameters + optimizer state: what a migration moves per layer
    double XTd[2][kMaxL];   // transfer time of the boundary after layer l: [0] intra, [1] inter
    int64_t XTi[2][kMaxL];
    int32_t base_cuts[kMaxS + 1];
    // raw inputs (kept for the prefix kernel)
    double fwd[kMaxL], bwd[kMaxL];
    int64_t fwd_i[kMaxL], bwd_i[kMaxL], act[kMaxL], par[kMaxL], opt[kMaxL], p2p[kMaxL];
};

// The descriptor tables are TEMPLATES keyed by the survivor count: which strategies exist,
// how micro-batches split and how many layer compositions a pipeline has depend only on
// how many devices survive, not on which.  A failure scenario adds just its failed ids
// and one bit per pair of neighbouring survivors ("do they sit on different nodes?"),
// from which a pipeline's link tiers are cut out on the device.
//
// One template segment = (strategy, pipeline, micro-batch count): its candidates are the
// layer compositions kappa = 0..K-1 followed by the min-max partition, or the min-max
// partition alone (K = 0).
struct TSeg {              // 32 bytes
    uint64_t cand_first;   // index of its first candidate within one scenario's space
    uint64_t K;            // enumerated compositions
    uint16_t S, m, n_sync; // stages, micro-batches, data-parallel peers of the strategy
    uint16_t off;          // survivor index of the pipeline's first stage
    uint32_t feas_first;   // its memory-feasible candidates, ascending, as a range of the feasible-
    uint32_t feas_count;   //   composition pool (kNoFeasList: none was built, all K+1 are walked)
};
// Whether a layer composition fits in memory depends on (stages, micro-batches, composition)
// only -- not on the failure scenario, the link tiers or the cost mode (Section "Estimator",
// memory estimator).  So the feasible compositions of every (S, m) are listed once per profile
// and the search pass and the tie-break pass walk that list instead of all K + 1 candidates.
constexpr uint32_t kNoFeasList = 0xffffffffu;
constexpr uint64_t kFeasMaxK = 1ull << 20;   // larger segments are walked unscreened

// One parallel strategy of a template.
struct Strat {
    uint64_t split_first;  // first split item of this strategy within its template
    uint64_t n_split;      // micro-batch splits
    uint32_t seg_first;    // its first template segment (global row of the TSeg table)
    uint16_t dp, n_m;      // pipelines; micro-batch values per pipeline (segments per pipeline)
    uint16_t R, pad;       // REMAINDER mode: pipelines that receive one more
    uint16_t S[kMaxP], m_lo[kMaxP];
};

struct Tmpl {
    uint64_t n_split_total;  // split items over all its strategies
    uint64_t n_cand;         // candidates of one scenario
    uint32_t strat_first, n_strat;
    uint32_t tseg_first, n_tseg;
    uint32_t scen_first, n_scen;   // its scenarios, as a range of the tmpl_scen list
    uint32_t n_red, pad;           // blocks of the split reduction per scenario
};

// One failure scenario of a batch.  Its segments own rows seg_base .. seg_base+n_tseg-1 of
// the per-segment result array, in template order.
struct Scen {              // 32 bytes
    uint32_t tmpl, seg_base;
    uint32_t failed_first, n_failed;   // into the failed-id array
    uint32_t cross_first, red_first;   // into the node-crossing bit words; first reduction block
    uint32_t policy_mask;
    uint32_t rep;                      // scenario whose dynamic-parallelism search this one shares (itself if none)
};

// Work layout of the search pass: all segments of a batch that share (stages,
// micro-batches) form a bucket; its pipeline-plans are flattened segment-major
// (index = segment-in-bucket * count + kappa) and cut into chunks of kChunk plans, one CTA
// each.  Lanes of a warp therefore run recurrences of identical shape.
constexpr int kChunk = 128;
constexpr int kRegStagesMax = 16;   // deepest pipeline the register-resident kernel is built for
struct Bucket {
    uint64_t count;        // candidates per segment (K+1 or 1)
    uint64_t chunk_first;  // first chunk of the bucket within its launch class
    uint32_t list_first;   // its template segments, as a range of the bucket_tseg list
    uint32_t n_tseg;
    uint32_t tmpl, n_seg;  // n_seg = n_tseg * scenarios of the template
    uint16_t S, m;
    uint32_t feas_first;   // count = length of this list if there is one (kNoFeasList: count = K+1 or 1)
    // 1: every segment of the bucket stands for TWO template segments, itself (m micro-batches) and
    // the next row (the same pipeline with m + 1): their recurrences share all rounds before the
    // ramp-down, so one thread evaluates both (sim_rounds_pair, sim_regs_pair).  Built only where the two have
    // the same feasible compositions: 1F1B with m >= S, where a stage holds min(S - i, m) = S - i
    // micro-batches in flight either way (Section "Estimator", memory estimator), and only for
    // template buckets (with shared segments the distinct ones are searched singly: pairing
    // (m, m+1) and (m+1, m+2) heads would search the middle one twice).
    uint32_t pair, pad;
};
constexpr int kPairStagesMin = kRegStagesMax + 1, kPairStagesMax = 48;   // depths whose transposed kernel evaluates pairs (shallow ones: all)

// Segments shared between scenarios.  The least cost of a segment over its layer compositions
// depends on its stages, micro-batches, data-parallel peers and the link tiers of its S-1
// boundaries -- not on the scenario or the strategy it belongs to (Section "Estimator": a
// pipeline's time is a function of its own stages and links).  With sharing on, the segments
// of a batch are keyed by exactly that, every distinct key is searched once, and the other
// rows copy the result.  A class = (S, m, peers); within a class the key is the tier word,
// found in an open-addressing table; a bucket with tmpl == kSharedBucket walks a range of the
// (scenario, template segment) list of the distinct segments of one class.
constexpr uint32_t kSharedBucket = 0xffffffffu;
constexpr uint32_t kNoSegClass = 0xffffffffu;   // template segment that is not searched (no micro-batches, nothing fits)
// Micro-batch pairs among shared segments.  Classes of pair heads are formed at non-overlapping
// micro-batch counts (m, m+1), (m+2, m+3), .. of a (stages, peers) group; a head of such a class
// is keyed in the class's table and searched together with its next row.  Every other row first
// looks its tier up in the pair class that would hold it as a head (its own m) and in the one
// that would hold it as a second row (m - 1); only if neither has it is it keyed in the class of
// single segments of its m.  So every distinct (stages, m, peers, tiers) is searched once.
constexpr uint32_t kPartnerSeg = 0xfffffffeu;   // second row of a keyed pair head: takes the row after its head's representative
constexpr uint32_t kSecondRowFlag = 0x80000000u;   // in slot_of: the row after the slot's representative holds this row's result
struct USegClass {
    uint32_t tab_first, tab_mask;   // its table: slots tab_first .. tab_first + tab_mask (a power of two of them)
    uint32_t list_first, pad;       // its distinct segments: list entries list_first .. list_first + count - 1
};
struct USegDev {
    const USegClass *cls;
    const uint32_t *tseg_cls;       // class of every template segment (kNoSegClass: none; kPartnerSeg: rides with the row before)
    const uint32_t *look_head;      // per template segment that is not a keyed pair head: the pair class of its own m, or kNoSegClass
    const uint32_t *look_part;      //   and the pair class of m - 1
    unsigned long long *tab;        // tier words, all-ones = empty
    uint32_t *rep;                  // per slot: lowest row with that key
    uint32_t *slot_of;              // per row: its slot (kNoSegClass: none)
    uint32_t *count;                // per class: distinct segments; count[n_cls]: probes that found no slot (never)
    uint2 *list;                    // (scenario, template segment) of every distinct segment, by class
    uint32_t n_cls, n_rep_scen;
    uint32_t n_pair_cls;            // classes 0 .. n_pair_cls-1 are the pair classes
};

// Buckets that one kernel instantiation handles.  Plan-major classes cut a bucket's
// flattened plans (segment-in-bucket * count + kappa) into chunks of kChunk; the
// transposed class cuts its (kappa, group of 32 segments) warp items into chunks of 4.
enum { CM_CLASS_REGS = 0, CM_CLASS_WIDE_UNI = 1, CM_CLASS_WIDE_LANE = 2, CM_CLASS_SHORT = 3, CM_CLASS_SOLO = 4, CM_CLASS_WARP = 5,
       CM_CLASS_WIDE_PAIR = 6, CM_CLASS_REGS_PAIR = 7, CM_CLASS_WIDE_LANE_PAIR = 8 };
// CM_CLASS_WIDE_PAIR / CM_CLASS_WIDE_LANE_PAIR / CM_CLASS_REGS_PAIR: micro-batch pairs (Bucket::pair) in the
// transposed layout (cm_cost_pair_kernel), the per-lane layout (cm_cost_lane_pair_kernel) and the
// register-resident one (cm_cost_regs_pair_kernel).
constexpr uint64_t kRegsPairMinPlans = 8192;   // shallow pairs are formed where a group has at least this many plans;
                                               // smaller batches stay with the one launch for every shallow depth
// CM_CLASS_WARP: the pipelines deeper than kRegStagesMax of a batch that has so few plans there (after the memory
// screen) that a thread per plan would leave the GPU waiting on a handful of long dependent chains: a warp per plan
// in lock step, every depth in one launch.
constexpr uint64_t kWarpPlansMax = 4096;   // deep plans of a batch up to which they are evaluated a warp per plan
// CM_CLASS_SHORT: pipelines of at most kRegStagesMax stages with fewer micro-batches than warm-up slots (m < S-1).
// CM_CLASS_SOLO: segments deeper than kRegStagesMax whose only candidate is the min-max partition.
// One plan is one dependent chain (2*S*m cells, ~100 us in a single thread); a warp walks it in
// lock step instead, stages over the lanes, four segments per CTA, every depth in one launch.
constexpr int kWideStagesMax = 48;  // deepest pipeline with clock AND pending state in registers (deeper: pending forwards in shared memory)
// Stage counts of the deep-pipeline kernels, cut into ranges that compile as separate
// translation units (the build script passes the same pairs to cm_cost_deep.cu).
#define CM_DEEP_RANGES(X) X(17, 28) X(29, 34) X(35, 41) X(42, 48) X(49, 56) X(57, 64)
constexpr int kUniMinSegments = 22; // fewer segments in a bucket (or left over after full warps of 32): the per-lane kernel
                                    // is faster than a transposed warp that is two-thirds empty
constexpr int kAnyMaxChunks = 4096; // shallow classes smaller than this together: one launch for all depths
struct LaunchClass {
    int kind, stages;
    uint64_t chunk_begin;  // first chunk of the class in its kind's chunk numbering
    uint32_t bucket_begin, bucket_end;
    uint64_t n_chunks;
    uint32_t uni_items, pad;   // transposed class: consecutive warp items one warp takes (1..kUniItemsMax)
};
constexpr int kUniItemsMax = 8;
constexpr int kUniBatchStagesMax = 28;     // deeper transposed classes keep one item per warp
constexpr uint64_t kUniMinChunks = 4096;   // keep at least this many CTAs (about ten waves) in a class before batching items

// (cost, index) pair carried through the hierarchical argmin of the split reduction.
struct Partial {
    uint64_t cost_bits;     // cost as an order-preserving 64-bit pattern (inf = infeasible)
    uint64_t item;          // split item index within the scenario
};

// Per-scenario winner of the split reduction, decoded for the tie-break pass.
struct Winner {
    uint64_t cost_bits;
    uint64_t item;
    uint32_t strat, dp;     // global strategy row; pipelines
    uint32_t seg[kMaxP];    // global segment row of every pipeline
    uint16_t micro[kMaxP];
    uint32_t scen, pad;     // scenario it belongs to (a shortlist holds several records per scenario)
};

struct BatchDev {
    const Scen *scen;
    const Tmpl *tmpl;
    const Strat *strat;
    const TSeg *tseg;
    const uint32_t *failed;
    const uint64_t *cross;        // per scenario: bit j = survivors j and j+1 sit on different nodes
    const uint32_t *tmpl_scen;    // scenario ids grouped by template
    const Bucket *bucket;         // search-pass work layout
    const uint32_t *bucket_tseg;  // template segment rows grouped by bucket
    const uint32_t *feas;         // feasible-composition pool of the context
    const uint2 *useg;            // distinct segments of a batch searched with sharing (buckets with tmpl == kSharedBucket)
    // Strategies of one survivor count repeat pipelines: the same stages over the same survivors with
    // the same micro-batches and peers (the tuples (30,31,..) and (30,32,..) start with the same
    // pipeline).  Such template segments have the same candidates with the same costs in every
    // scenario, so only the first of them -- tseg_canon[t] == t -- is searched; the others take its
    // per-segment minimum afterwards (cm_dup_copy_kernel).  NULL: the batch has no duplicates.
    const uint32_t *tseg_canon;
    uint32_t n_rep_scen;          // scenarios that own result rows (entries of tmpl_scen in use)
    uint64_t *seg_best;     // [n_seg] min cost over kappa, order-preserving bits
    const uint32_t *red_scen;  // [n_red_blocks] scenario of every block of the split reduction
    Partial *partial;       // [n_red_blocks]
    Winner *winner;         // [B]
    uint64_t *kappa_sel;    // [B][kMaxP] lowest kappa with cost <= T*
    uint64_t *pol_cost;     // [B][2] rerouting / redundant cost bits
    uint16_t *rc_stages;    // [B][kMaxP] stage counts of the redundant-computation plan
    cm_plan *plans;         // [B][4]: per policy, then the overall best
    unsigned long long *counters;  // [0] cells simulated in pass 1, [1] plans in pass 2
    int32_t B, mode;
    uint32_t n_rows;             // rows of seg_best over all scenarios
    // 1: integer-nanosecond mode evaluated in double arithmetic on integer-valued inputs; every
    // cost on the device is then a double bit pattern and becomes an integer only on the way out
    uint32_t intval;
    uint64_t n_tiles;
    uint32_t max_tiles_per_seg, n_red_blocks;
    uint32_t dp_max;
    uint32_t max_red_per_scen;   // most blocks of the split reduction any scenario has
    int32_t layer_mode, batch_mode;
};

struct Tables {
    const DevProfile *prof;
    const uint64_t *binom;      // [rows][kBinomCols+1], saturating
    int32_t binom_rows;
    uint8_t *mm_cuts;           // [slots][kMaxS+1], min-max partitions; mm_cuts[slot][0]=255: infeasible
    int32_t mm_stride_m;        // slot = (S-1)*mm_stride_m + m
    int32_t sched;              // cm_schedule of the batch / space these tables serve
    __host__ __device__ uint32_t mm_slot(int S, int m) const { return (uint32_t)((S - 1) * mm_stride_m + m); }
};

// Full objective (transition time included): per scenario a shortlist of the `topk` best
// (strategy, split) pairs by step time, each completed to a plan and matched against the old
// placement.  Slot = scenario * topk + rank.
constexpr int kMaxShort = CM_MAX_SHORTLIST;
constexpr int kMaxMatch = CM_MAX_MATCH;
struct ObjDev {
    int32_t topk, sync_rounds;
    double t_gap, t_restart;
    int64_t t_gap_i, t_restart_i, bw_xfer;
    Winner *short_win;        // [B*topk]
    uint64_t *short_kappa;    // [B*topk][kMaxP]
    int64_t *short_bytes;     // [B*topk] bytes moved by the cheapest migration, -1 = empty slot
    uint16_t *short_assign;   // [B*topk][kMaxMatch] position -> survivor index
    uint64_t *short_step;     // [B*topk][2] step time / time of the rounds under asymmetric synchronisation (cost bits)
    int32_t *short_rounds;    // [B*topk][2] communication rounds, communication domains
    cm_plan *short_plans;     // [B*topk] or NULL
    cm_plan *best;            // [B]
    cm_transition *trans;     // [B]
};

// Transition time of a reconstruction that moves `bytes` of model state (Section "Estimator",
// state-transition overhead: restart + weight transfer; the search itself overlaps training).
// One routine for the objective kernel and for cm_transition_time on the host.
__host__ __device__ inline double transition_time_f64(double t_restart, long long bytes, long long bw) {
    return t_restart + (double)bytes / (double)bw;
}
__host__ __device__ inline long long transition_time_i64(long long t_restart, long long bytes, long long bw) {
    return t_restart + bytes / bw;
}

// Integer-nanosecond mode runs the long long instantiations unless the batch evaluates it in
// double arithmetic on integer-valued inputs (BatchDev::intval).
inline bool native_i64(const BatchDev &b) { return b.mode == CM_COST_INT64NS && !b.intval; }

// launchers (cm_kernels.cu); all enqueue on the stream and return the launch error
cudaError_t launch_prefix(DevProfile *prof, cudaStream_t st);
cudaError_t launch_minmax(const Tables &t, const uint32_t *keys_dev, int n_keys, int mode, cudaStream_t st);   // order: t.sched
// feasible compositions of n_keys (S << 16 | m) keys: list of key q written at pool + first[q]
// (room for K[q] + 1 entries), its length to count[q]
cudaError_t launch_feasible(const Tables &t, int layer_mode, const uint32_t *keys_dev, const uint64_t *K_dev,
                            const uint32_t *first_dev, int n_keys, uint32_t *pool, uint32_t *count_dev, cudaStream_t st);
cudaError_t launch_policies(const Tables &t, const BatchDev &b, int n_dp, cudaStream_t st);
// segments shared between scenarios: key every row and list the distinct ones (tab, rep, count
// cleared by the caller); after the search pass, give every other row its representative's result
cudaError_t launch_useg_keys(const BatchDev &b, const USegDev &u, cudaStream_t st);   // three launches
cudaError_t launch_useg_copy(const BatchDev &b, const USegDev &u, cudaStream_t st);
cudaError_t launch_dup_copy(const BatchDev &b, cudaStream_t st);   // duplicate template segments take their first occurrence's minimum
// Tiles of a segment that the tie-break kernels take side by side (grid.y); the rest is
// walked serially inside the CTA.  A single scenario gets every tile its own CTA (lowest
// latency), a large batch about one CTA per (scenario, pipeline): most of those stop after
// their first tile anyway, and an idle CTA per tile would cost more than the work.
inline unsigned tiebreak_grid_y(uint64_t nx, uint32_t max_tiles) {
    const uint64_t target = 2048;   // CTAs worth launching
    uint64_t y = nx ? (target + nx - 1) / nx : 1;
    if (y > max_tiles) y = max_tiles;
    if (y > 65535) y = 65535;
    return (unsigned)(y ? y : 1);
}

// side streams (may be NULL / 0): launch classes are independent of one another, so they are
// spread over the caller's stream and the side streams and joined again before returning
constexpr int kSideStreams = 7;
struct SideStreams {
    cudaStream_t stream[kSideStreams];
    cudaEvent_t fork, join[kSideStreams];
    int n;
};
cudaError_t launch_cost_pass1(const Tables &t, const BatchDev &b, const LaunchClass *classes, int n_classes,
                              cudaStream_t st, const SideStreams *side, int *launches);
cudaError_t launch_split_reduce(const Tables &t, const BatchDev &b, cudaStream_t st);
// deep_elsewhere: winners' pipelines deeper than kRegStagesMax are completed by another kernel
// (the per-depth ones, or the lock-step one below), this one leaves them alone
cudaError_t launch_cost_pass2(const Tables &t, const BatchDev &b, cudaStream_t st, bool deep_elsewhere_all = false);
// Tie-break pass for few winners (one failure at a time): a warp per layer composition walks the
// pipeline in lock step, every depth above kRegStagesMax in one launch.
constexpr uint64_t kWarpTieMaxPairs = 64;   // (scenario, pipeline) pairs up to which the lock-step tie-break is used
cudaError_t launch_tiebreak_warp(const Tables &t, const BatchDev &b, cudaStream_t st);
cudaError_t launch_tiebreak_wide(const Tables &t, const BatchDev &b, uint64_t stage_mask, cudaStream_t st,
                                 const SideStreams *side, int *launches);
cudaError_t launch_finalize(const Tables &t, const BatchDev &b, cudaStream_t st);
// single_policy < 0: candidates of the dynamic-parallelism segments; otherwise the one
// candidate of that policy (its cost must already be in pol_cost of scenario 0)
cudaError_t launch_evaluate(const Tables &t, const BatchDev &b, uint64_t n_cand, int single_policy,
                            uint64_t first, uint64_t count, const uint64_t *idx, double *cost,
                            int64_t *cost_ns, uint8_t *feas, cudaStream_t st);
// cm_restore.cu
cudaError_t launch_shortlist(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st);
cudaError_t launch_plan_matching(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st);
cudaError_t launch_plan_rounds(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st);
cudaError_t launch_objective(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st);
// stand-alone matchings over explicit layer ranges ([n_problems][kMaxMatch] each)
cudaError_t launch_range_matching(const Tables &t, int n_problems, const int32_t *sizes, const uint8_t *old_lo,
                                  const uint8_t *old_hi, const uint8_t *new_lo, const uint8_t *new_hi,
                                  int64_t *total, uint16_t *assign, cudaStream_t st);
cudaError_t launch_pick(const cm_plan *const *plans_dev, int n, cm_plan *out_dev, int mode, cudaStream_t st);

// What an entry point implemented outside cm_api.cu needs to know about a space.
struct SpaceView {
    Tables tb;
    BatchDev bd;
    uint64_t n_cand;
    cudaStream_t stream;
    int device, policy;
};

}  // namespace cm

struct cm_ctx;
struct cm_space;
cm_status cm_internal_space_view(cm_ctx *ctx, const cm_space *space, cm::SpaceView *out);
cm_status cm_internal_fail(cm_ctx *ctx, cm_status status, const std::string &message);
int cm_internal_set_sharing(cm_ctx *ctx, int on);   // returns the previous setting
int cm_internal_grid_devices(const cm_ctx *ctx);   // n_dp * n_pp of the loaded profile, 0 without one
