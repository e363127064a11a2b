// C ABI of the plan search: context, profile upload, host-side descriptor builder
// (strategies, segments, survivor placement) and the launch sequences.
//
// The host never evaluates the cost model.  It only turns a failure set into small
// integer tables -- which (dp, S_1<=...<=S_dp) strategies exist, which survivor sits
// on which stage, how many layer compositions each pipeline has -- and the kernels in
// cm_kernels.cu do the rest from plan indices.
#include <algorithm>
#include <chrono>
#include <map>
#include <unordered_map>
#include <memory>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "cm_internal.h"

using namespace cm;

// ------------------------------------------------------------------ small utilities
namespace {

template <typename T> struct PinnedVec {   // host staging that async copies can read
    T *p = nullptr;
    size_t n = 0, cap = 0;
    ~PinnedVec() { if (p) cudaFreeHost(p); }
    bool reserve(size_t want) {
        if (want <= cap) return true;
        size_t nc = std::max(want, cap * 2 + 16);
        T *q = nullptr;
        if (cudaHostAlloc((void **)&q, nc * sizeof(T), cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); return false; }
        if (n) memcpy(q, p, n * sizeof(T));
        if (p) cudaFreeHost(p);
        p = q;
        cap = nc;
        return true;
    }
    bool push(const T &v) { if (n == cap && !reserve(n + 1)) return false; p[n++] = v; return true; }
    bool resize(size_t m) { if (!reserve(m)) return false; n = m; return true; }
    void clear() { n = 0; }
    T &operator[](size_t i) { return p[i]; }
    const T &operator[](size_t i) const { return p[i]; }
    size_t size() const { return n; }
    T &back() { return p[n - 1]; }
};

template <typename T> struct DevBuf {
    T *p = nullptr;
    size_t cap = 0;
    ~DevBuf() { if (p) cudaFree(p); }
    bool reserve(size_t want) {
        if (want <= cap) return true;
        size_t nc = std::max(want, cap + cap / 2 + 16);
        T *q = nullptr;
        if (cudaMalloc((void **)&q, nc * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return false; }
        if (p) cudaFree(p);
        p = q;
        cap = nc;
        return true;
    }
};

inline uint64_t sat_add(uint64_t a, uint64_t b) { return a > kSat - b ? kSat : a + b; }

inline uint64_t now_ns() {
    return (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

}  // namespace

// One batch of failure scenarios: host tables, device mirrors, result buffers.
// All descriptor tables are small (templates per survivor count plus ~100 bytes per
// scenario), so they are packed into one pinned arena and reach the device in one copy.
struct Batch {
    std::vector<Scen> scen;
    std::vector<Tmpl> tmpl;
    std::vector<Strat> strat;
    std::vector<TSeg> tseg;
    std::vector<uint32_t> failed, red_scen, keys, tmpl_scen, bucket_tseg;
    std::vector<uint32_t> tseg_canon;      // first template segment with the same (stages, micro-batches, peers, offset): itself if none before
    uint32_t n_dup = 0;                    // template segments that are not their own first occurrence
    size_t off_canon = 0;
    std::vector<uint64_t> cross;
    std::vector<Bucket> bucket;
    std::vector<LaunchClass> classes;
    std::vector<int> tmpl_of_nsurv;        // survivor count -> template, -1 = not built
    PinnedVec<unsigned char> arena;        // host image of the tables
    DevBuf<unsigned char> d_arena;
    size_t off_scen = 0, off_tmpl = 0, off_strat = 0, off_tseg = 0, off_failed = 0, off_red = 0, off_keys = 0,
           off_tmpl_scen = 0, off_bucket_tseg = 0, off_cross = 0, off_bucket = 0;
    PinnedVec<cm_plan> plans_host;
    DevBuf<uint64_t> d_seg_best, d_kappa_sel, d_pol_cost;
    DevBuf<Partial> d_partial;
    DevBuf<Winner> d_winner;
    DevBuf<uint16_t> d_rc_stages;
    DevBuf<cm_plan> d_plans;
    // full objective: shortlist slots (scenario-major) and per-scenario results
    DevBuf<Winner> d_short_win;
    DevBuf<uint64_t> d_short_kappa;
    DevBuf<int64_t> d_short_bytes;
    DevBuf<uint16_t> d_short_assign;
    DevBuf<uint64_t> d_short_step;
    DevBuf<int32_t> d_short_rounds;
    PinnedVec<int32_t> short_rounds_host;
    DevBuf<cm_plan> d_short_plans, d_obj_best;
    DevBuf<cm_transition> d_trans;
    PinnedVec<cm_plan> obj_best_host, short_plans_host;
    PinnedVec<cm_transition> trans_host;
    PinnedVec<int64_t> short_bytes_host;
    cm_enum_opts opts{};
    uint32_t policy_mask = 0;
    uint64_t n_cand = 0, n_tiles = 0, n_split = 0;
    uint64_t n_cand_own = 0;               // candidates of the template segments that are searched in their own right
    std::vector<uint64_t> tmpl_cand_own;   // the same per template (one scenario)
    uint64_t n_rows = 0;                   // rows of seg_best over all scenarios
    uint32_t max_tiles_per_seg = 0, dp_max = 0;
    int B = 0;
    bool intval = false;                   // integer mode evaluated in double arithmetic (fixed when the batch is built)
    uint64_t profile_gen = 0;              // generation of the profile the tables describe (see cm_ctx::profile_gen)
    bool mm_launched = false;              // the min-max partitions of `keys` were already enqueued (with the feasible lists)
    // Segments shared between scenarios (sharing on, more than one scenario): classes = distinct
    // (stages, micro-batches, peers), their table and list regions, the class of every template
    // segment; the buckets are laid out in upload_batch, once the device has counted the distinct
    // segments of every class.
    bool useg = false;
    struct USegInfo { uint16_t S, m, n_sync, pair; uint64_t K; uint32_t feas_first, feas_count; uint64_t rows; };
    // Role of every template segment in the search pass: on its own, head of a micro-batch pair
    // (evaluated together with the next row), or that next row.
    enum : uint8_t { kAlone = 0, kPairHead = 1, kPairPartner = 2 };
    std::vector<uint8_t> role;
    std::vector<USegInfo> ucls_info;
    std::vector<USegClass> ucls;
    std::vector<uint32_t> tseg_cls, look_head, look_part;
    uint32_t n_pair_cls = 0;
    size_t off_ucls = 0, off_tseg_cls = 0, off_look_head = 0, off_look_part = 0;
    uint64_t utab_slots = 0, ulist_len = 0;
    DevBuf<unsigned long long> d_utab;
    DevBuf<uint32_t> d_urep, d_slot_of, d_ucount;
    DevBuf<uint2> d_useg;
    PinnedVec<uint32_t> ucount_host;
    // A resident one-scenario batch searched with shared segments keeps its template buckets (the
    // replayed graph uses them) and lays the shared ones out beside them, per search.
    const Bucket *bucket_override = nullptr;
    uint64_t single_cells = 0;            // recurrence cells of the one scenario's search pass, every segment on its own
    DevBuf<Bucket> d_alt_bucket;
    PinnedVec<unsigned char> alt_stage;   // slot_of | rep | list | buckets, staged for the copies
};

struct cm_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    bool has_profile = false;
    // Bumped by every cm_load_profile.  Descriptor tables (a cm_space, a cm_batch) are stamped with
    // the generation they were built under: their segment shapes, min-max keys and candidate
    // counts describe that profile's L and G, so they are refused once another profile is loaded.
    uint64_t profile_gen = 0;
    DevBuf<unsigned char> d_scratch;  // small per-call device scratch (cm_select, cm_transfer_matching): grown, never shrunk
    DevProfile hp{};                  // host copy: scalars, raw inputs, base cuts
    DevProfile *d_prof = nullptr;
    // The integer-nanosecond mode normally runs in double arithmetic: its inputs are integers,
    // the recurrence only adds and takes maxima, so every value is an integer that a double
    // holds exactly as long as it stays below 2^53 -- and 64-bit floating-point adds issue
    // faster on this GPU than 64-bit integer adds, which are pairs of 32-bit operations.
    // d_prof53 is the profile with integer-valued double arrays; exact53 says whether the
    // loaded profile keeps every intermediate below 2^52 (otherwise, or when the caller asks
    // for it, the long long kernels run).
    DevProfile *d_prof53 = nullptr;
    bool exact53 = false, force_native_i64 = false;
    std::vector<uint64_t> binom;      // [rows][kBinomCols+1]
    int binom_rows = 0;
    uint64_t *d_binom = nullptr;
    // min-max cuts per (cost mode, execution order): the partition depends on the arithmetic of
    // the stage times and, through the memory check, on the micro-batches in flight
    static constexpr int kMmTables = 4;
    static int mm_index(const cm_enum_opts &o) { return (int)o.cost * 2 + (int)o.sched; }
    uint8_t *d_mm[kMmTables] = {nullptr, nullptr, nullptr, nullptr};
    std::vector<uint8_t> mm_done[kMmTables];
    int mm_stride_m = 0;
    // Memory-feasible layer compositions per (layer mode, stages, micro-batches), listed once per
    // profile (cm_feasible_kernel) into one device pool that only grows; key = S << 16 | m.
    struct FeasEntry { uint32_t first, count; uint64_t K; };
    std::map<uint32_t, FeasEntry> feas[6];   // [layer mode * 2 + execution order]
    DevBuf<uint32_t> d_feas;
    size_t feas_used = 0;
    PinnedVec<unsigned char> feas_stage;      // keys, K, offsets out; counts back
    DevBuf<unsigned char> d_feas_stage;
    bool screen = true;               // walk only the listed feasible compositions (cm_set_memory_screen)
    bool dedup = true;                // search a pipeline that several strategies of a survivor count share once (cm_set_pipeline_reuse)
    bool pairs = true;                // one recurrence for a pipeline's m and m+1 micro-batch variants (cm_set_micro_batch_pairs)
    Batch batch;                      // reused by cm_search_batch
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ev_obj[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // phases of the objective pass
    uint64_t obj_stats[8] = {0};
    bool share = false;               // search scenarios with identical dynamic-parallelism spaces once
    // One-scenario searches (per-failure latency): everything but the failed ids and the
    // node-crossing bits depends only on the survivor count and the options, so a prepared
    // batch per (survivor count, options) stays resident and a search patches those few bytes.
    // From its second use on, such a batch replays its launch sequence as a CUDA graph (captured
    // on a library-owned stream, launched on the caller's): same kernels, same arguments, one
    // submission instead of a dozen.
    struct Single {
        int n_surv = 0;
        cm_enum_opts opts{};
        bool intval = false;
        std::unique_ptr<Batch> batch;
        cudaGraphExec_t exec = nullptr;
        bool graph_failed = false;
        int launches = 0;
        ~Single() { if (exec) cudaGraphExecDestroy(exec); }
    };
    std::vector<std::unique_ptr<Single>> single;
    cudaStream_t graph_stream = nullptr;
    bool use_graphs = true;
    // the two one-plan policies do not depend on the dynamic-parallelism search: they run beside it
    cudaStream_t pol_stream = nullptr;
    cudaEvent_t pol_fork = nullptr, pol_join = nullptr;
    SideStreams side{};               // library-owned streams for independent launch classes
    uint64_t stats[24] = {0};
    std::string err;
};

struct cm_space {
    cm_ctx *ctx = nullptr;
    int policy = 0;
    Batch batch;
    std::vector<uint32_t> failed;
};

struct cm_batch {
    cm_ctx *ctx = nullptr;
    Batch batch;
    int prep_launches = 0;
};

namespace {

cm_status fail(cm_ctx *c, cm_status s, const std::string &msg) {
    if (c) c->err = msg;
    return s;
}

// Tables built under an earlier profile describe another L and G: refuse them.
bool stale(const cm_ctx *c, const Batch &bt) { return bt.profile_gen != c->profile_gen; }
const char *const kStaleMsg = "space or batch was built for an earlier profile: enumerate / prepare it again after cm_load_profile";

// No exception may cross the C ABI (the host side uses std::vector / std::string / std::map).
cm_status api_caught(cm_ctx *c, cm_status s) noexcept {
    if (c) {
        try { c->err = s == CM_ENOMEM ? "host memory exhausted" : "internal error (unexpected exception)"; } catch (...) {}
    }
    return s;
}
#define CM_API_BEGIN try {
#define CM_API_END(ctx)                                                           \
    }                                                                             \
    catch (const std::bad_alloc &) { return api_caught((ctx), CM_ENOMEM); }       \
    catch (...) { return api_caught((ctx), CM_EINVAL); }

#define CM_CUDA(ctx, expr)                                                                       \
    do {                                                                                         \
        cudaError_t e_ = (expr);                                                                 \
        if (e_ != cudaSuccess) {                                                                 \
            cudaGetLastError();                                                                  \
            return fail((ctx), CM_ECUDA, std::string(#expr) + ": " + cudaGetErrorString(e_));    \
        }                                                                                        \
    } while (0)

uint64_t hbinom(const cm_ctx *c, int n, int k) {
    if (k < 0 || n < 0 || k > n) return 0;
    if (n >= c->binom_rows || k > kBinomCols) return kSat;
    return c->binom[(size_t)n * (kBinomCols + 1) + k];
}

// Strategies (Algorithm 1, get_parallel_strategy): non-decreasing stage counts that use
// every survivor, dp ascending, tuples in lexicographic order.
void enum_strategies(int n_surv, int dp_lo, int dp_hi, int lo, int hi,
                     std::vector<std::vector<uint16_t>> &out) {
    std::vector<uint16_t> cur;
    struct Rec {
        static void go(int dp, int pos, int remaining, int min_part, int hi, std::vector<uint16_t> &cur,
                       std::vector<std::vector<uint16_t>> &out) {
            if (pos == dp) {
                if (remaining == 0) out.push_back(cur);
                return;
            }
            const int left = dp - pos - 1;
            for (int s = min_part; s <= hi; ++s) {
                if (remaining - s < left * s) break;            // later parts are >= s
                if (remaining - s > left * hi) continue;        // later parts are <= hi
                cur.push_back((uint16_t)s);
                go(dp, pos + 1, remaining - s, s, hi, cur, out);
                cur.pop_back();
            }
        }
    };
    for (int dp = dp_lo; dp <= dp_hi; ++dp) Rec::go(dp, 0, n_surv, lo, hi, cur, out);
}

cm_status check_opts(cm_ctx *ctx, const cm_enum_opts *o) {
    if (!o) return fail(ctx, CM_EINVAL, "opts is NULL");
    if (o->dp_lo > o->dp_hi || o->pp_lo > o->pp_hi) return fail(ctx, CM_EINVAL, "empty dp/pp window");
    if (o->dp_hi > CM_MAX_PIPES) return fail(ctx, CM_EINVAL, "dp_hi exceeds CM_MAX_PIPES");
    if (o->pp_hi > CM_MAX_STAGES) return fail(ctx, CM_EINVAL, "pp_hi exceeds CM_MAX_STAGES");
    if (o->lm < CM_LAYERS_FULL || o->lm > CM_LAYERS_MINMAX) return fail(ctx, CM_EINVAL, "bad layer mode");
    if (o->bm < CM_BATCH_FULL || o->bm > CM_BATCH_REMAINDER) return fail(ctx, CM_EINVAL, "bad batch mode");
    if (o->cost < CM_COST_FP64 || o->cost > CM_COST_INT64NS) return fail(ctx, CM_EINVAL, "bad cost mode");
    if (o->sched < CM_SCHED_1F1B || o->sched > CM_SCHED_GPIPE) return fail(ctx, CM_EINVAL, "bad execution order");
    return CM_OK;
}

// Work layout of the search pass: the template segments of every template are grouped by
// (stages, micro-batches) into buckets (a bucket's segments are its template segments
// times the template's scenarios), buckets grouped into launch classes: one per
// (kernel kind, stage count); the short-pipeline and the one-plan kinds pool every depth in one class.
struct PreBucket { uint32_t tmpl, list_first, n_tseg; uint16_t S, m; uint64_t count; uint32_t n_seg; int kind; uint32_t feas_first; uint32_t pair; };

// Micro-batch pairs (Bucket::pair): template segment t and t+1 are the same pipeline with m and
// m+1 micro-batches (the two shares the remainder rule of Section "Planner" leaves a pipeline;
// consecutive counts under the full split enumeration).  They pair up where one recurrence can
// serve both and both walk the same compositions: 1F1B, a depth of the deep-pipeline kernels,
// a choice of compositions, m >= S, equal feasible-list lengths.
void mark_pairs(const cm_ctx *ctx, Batch &bt) {
    bt.role.assign(bt.tseg.size(), Batch::kAlone);
    if (!ctx->pairs || bt.opts.sched != CM_SCHED_1F1B) return;
    for (const Tmpl &tp : bt.tmpl)
        for (uint32_t i = 0; i + 1 < tp.n_tseg; ++i) {
            const uint32_t t = tp.tseg_first + i;
            if (bt.role[t] != Batch::kAlone) continue;
            if (bt.tseg_canon[t] != t || bt.tseg_canon[t + 1] != t + 1) continue;   // a duplicate is not searched at all
            const TSeg &a = bt.tseg[t], &b = bt.tseg[t + 1];
            const bool same_pipe = a.S == b.S && a.off == b.off && a.n_sync == b.n_sync && a.K == b.K && b.m == a.m + 1 &&
                                   b.cand_first == a.cand_first + (a.K ? a.K + 1 : 1);
            if (!same_pipe || a.S > kPairStagesMax || a.m < a.S) continue;
            if (a.S >= kPairStagesMin && a.K == 0) continue;   // (a deep one-plan segment is walked by a warp)
            if ((a.feas_first == kNoFeasList) != (b.feas_first == kNoFeasList) || a.feas_count != b.feas_count) continue;
            if (a.feas_first != kNoFeasList && a.feas_count == 0) continue;
            bt.role[t] = Batch::kPairHead;
            bt.role[t + 1] = Batch::kPairPartner;
        }
}

// Kernel kind of a bucket.  by_warp: the batch has so few deep plans that they go a warp per plan.
int bucket_kind(bool by_warp, int S, int m, uint64_t n_seg, uint64_t K) {
    if (S <= kRegStagesMax) return m >= S - 1 ? (int)CM_CLASS_REGS : (int)CM_CLASS_SHORT;
    if (K == 0) return (int)CM_CLASS_SOLO;   // the min-max partition is the only candidate there is
    if (by_warp) return (int)CM_CLASS_WARP;
    if (S <= kWideStagesMax) return n_seg >= (uint64_t)kUniMinSegments ? (int)CM_CLASS_WIDE_UNI : (int)CM_CLASS_WIDE_LANE;
    return (int)CM_CLASS_WIDE_UNI;           // deeper than kWideStagesMax: the transposed layout only
}

cm_status layout_buckets(cm_ctx *ctx, Batch &bt, const std::vector<PreBucket> &pre);

cm_status build_buckets(cm_ctx *ctx, Batch &bt) {
    bt.bucket.clear();
    bt.classes.clear();
    bt.bucket_tseg.clear();
    using Pre = PreBucket;
    std::vector<Pre> pre;
    std::vector<uint8_t> role = bt.role;   // pairs too few for the transposed kernel are dissolved here, for this layout only
    // plans of the deep pipelines that have a choice of composition, over the whole batch
    uint64_t deep_plans = 0;
    for (const Tmpl &tp : bt.tmpl)
        for (uint32_t i = 0; i < tp.n_tseg && tp.n_scen; ++i) {
            const TSeg &g = bt.tseg[tp.tseg_first + i];
            if (bt.tseg_canon[tp.tseg_first + i] != tp.tseg_first + i) continue;
            if (g.S > kRegStagesMax && g.K > 0 && g.m >= 1)
                deep_plans += (g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : g.K + 1) * tp.n_scen;
        }
    const bool by_warp = deep_plans <= kWarpPlansMax;
    auto kind_of = [by_warp](int S, int m, uint64_t n_seg, uint64_t K, uint64_t) { return bucket_kind(by_warp, S, m, n_seg, K); };
    std::vector<uint32_t> idx;
    for (size_t t = 0; t < bt.tmpl.size(); ++t) {
        const Tmpl &tp = bt.tmpl[t];
        if (tp.n_scen == 0 || tp.n_tseg == 0) continue;
        // which micro-batch pairs this layout keeps: deep ones where the group of pair heads goes to
        // the transposed or the per-lane kernel (not where the batch's few deep plans go a warp per
        // plan), shallow ones where the group holds enough plans to be worth a launch of its own
        {
            std::unordered_map<uint32_t, uint32_t> heads;   // (S << 16 | m) -> pair heads of the template
            for (uint32_t i = 0; i < tp.n_tseg; ++i)
                if (role[tp.tseg_first + i] == Batch::kPairHead) {
                    const TSeg &g = bt.tseg[tp.tseg_first + i];
                    ++heads[((uint32_t)g.S << 16) | g.m];
                }
            for (uint32_t i = 0; i < tp.n_tseg; ++i)
                if (role[tp.tseg_first + i] == Batch::kPairHead) {
                    const TSeg &g = bt.tseg[tp.tseg_first + i];
                    const uint64_t n_pairs = (uint64_t)heads[((uint32_t)g.S << 16) | g.m] * tp.n_scen;
                    const uint64_t count = g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : (g.K ? g.K + 1 : 1);
                    const int kind = bucket_kind(by_warp, g.S, g.m, n_pairs, g.K);
                    const bool keep = g.S <= kRegStagesMax ? n_pairs * count >= kRegsPairMinPlans
                                                           : kind == CM_CLASS_WIDE_UNI || kind == CM_CLASS_WIDE_LANE;
                    if (!keep)
                        role[tp.tseg_first + i] = role[tp.tseg_first + i + 1] = Batch::kAlone;
                }
        }
        idx.clear();
        for (uint32_t i = 0; i < tp.n_tseg; ++i)
            if (role[tp.tseg_first + i] != Batch::kPairPartner && bt.tseg_canon[tp.tseg_first + i] == tp.tseg_first + i)
                idx.push_back(tp.tseg_first + i);
        std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) {
            const TSeg &x = bt.tseg[a], &y = bt.tseg[b];
            return x.S != y.S ? x.S < y.S : x.m != y.m ? x.m < y.m : role[a] < role[b];
        });
        for (size_t i = 0; i < idx.size();) {
            size_t j = i;
            const TSeg &g = bt.tseg[idx[i]];
            const uint32_t pair = role[idx[i]] == Batch::kPairHead ? 1u : 0u;
            while (j < idx.size() && bt.tseg[idx[j]].S == g.S && bt.tseg[idx[j]].m == g.m && role[idx[j]] == role[idx[i]]) ++j;
            if (g.m >= 1) {   // m = 0 cannot be feasible: no work is scheduled
                const uint64_t n_seg = (uint64_t)(j - i) * tp.n_scen;
                if (n_seg >= (1ull << 31)) return fail(ctx, CM_EOVERFLOW, "too many segments in one bucket");
                // candidates the search pass walks per segment: the listed feasible ones, or all
                const uint64_t count = g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : (g.K ? g.K + 1 : 1);
                if (count == 0) { i = j; continue; }   // nothing fits in memory: the segments stay infeasible
                // The transposed kernel gives every 32 segments a warp per composition, full or
                // not.  With one scenario the segments are few: what does not fill most of a
                // last warp goes to the per-lane kernel, which wastes no lane.
                size_t cut = j;
                if (tp.n_scen == 1 && kind_of(g.S, g.m, n_seg, g.K, count) == CM_CLASS_WIDE_UNI) {
                    const size_t rest = (j - i) % 32;
                    if (rest > 0 && rest < (size_t)kUniMinSegments) cut = j - rest;
                }
                for (int part = 0; part < 2; ++part) {
                    const size_t p0 = part ? cut : i, p1 = part ? j : cut;
                    if (p1 <= p0) continue;
                    const uint64_t ns = (uint64_t)(p1 - p0) * tp.n_scen;
                    Pre q{(uint32_t)t, (uint32_t)bt.bucket_tseg.size(), (uint32_t)(p1 - p0), g.S, g.m,
                          count, (uint32_t)ns,
                          !pair ? kind_of(g.S, g.m, ns, g.K, count)
                          : g.S <= kRegStagesMax ? (int)CM_CLASS_REGS_PAIR
                          : kind_of(g.S, g.m, ns, g.K, count) == CM_CLASS_WIDE_UNI ? (int)CM_CLASS_WIDE_PAIR : (int)CM_CLASS_WIDE_LANE_PAIR,
                          g.feas_first, pair};
                    for (size_t k = p0; k < p1; ++k) bt.bucket_tseg.push_back(idx[k]);
                    pre.push_back(q);
                }
            }
            i = j;
        }
    }
    return layout_buckets(ctx, bt, pre);
}

// Buckets and launch classes from the collected (template or shared-list) segment groups.
cm_status layout_buckets(cm_ctx *ctx, Batch &bt, const std::vector<PreBucket> &pre) {
    using Pre = PreBucket;
    for (int kind = CM_CLASS_REGS; kind <= CM_CLASS_WIDE_LANE_PAIR; ++kind) {
        uint64_t kind_chunks = 0;   // chunks are numbered through all classes of a kind
        const bool pooled_kind = kind == CM_CLASS_SHORT || kind == CM_CLASS_SOLO || kind == CM_CLASS_WARP;   // every depth in one class
        LaunchClass pooled{kind, 0, 0, (uint32_t)bt.bucket.size(), (uint32_t)bt.bucket.size(), 0, 1, 0};
        for (int S = 1; S <= CM_MAX_STAGES; ++S) {
            LaunchClass cls{kind, S, kind_chunks, (uint32_t)bt.bucket.size(), (uint32_t)bt.bucket.size(), 0, 1, 0};
            LaunchClass &c = pooled_kind ? pooled : cls;
            const bool transposed = kind == CM_CLASS_WIDE_UNI || kind == CM_CLASS_WIDE_PAIR;
            if (transposed) {
                // a warp of the transposed kernel takes several consecutive items once the class
                // is large enough to fill the GPU anyway
                uint64_t items = 0;
                for (const Pre &q : pre)
                    if (q.kind == kind && q.S == S) items += q.count * ((q.n_seg + 31) / 32);
                const uint64_t per = items / ((uint64_t)(kChunk / 32) * kUniMinChunks);
                c.uni_items = S <= kUniBatchStagesMax ? (uint32_t)std::min<uint64_t>(std::max<uint64_t>(per, 1), kUniItemsMax) : 1u;
            }
            for (const Pre &q : pre) {
                if (q.kind != kind || q.S != S) continue;
                Bucket bk{};
                bk.count = q.count;
                bk.chunk_first = c.chunk_begin + c.n_chunks;
                bk.list_first = q.list_first;
                bk.n_tseg = q.n_tseg;
                bk.tmpl = q.tmpl;
                bk.n_seg = q.n_seg;
                bk.S = q.S;
                bk.m = q.m;
                bk.feas_first = q.feas_first;
                bk.pair = q.pair;
                if (transposed) {
                    const uint64_t items = bk.count * ((bk.n_seg + 31) / 32);
                    const uint64_t per_cta = (uint64_t)(kChunk / 32) * c.uni_items;
                    c.n_chunks += (items + per_cta - 1) / per_cta;
                } else if (kind == CM_CLASS_SOLO) {
                    c.n_chunks += ((uint64_t)bk.n_seg + kChunk / 32 - 1) / (kChunk / 32);   // a warp per segment
                } else if (kind == CM_CLASS_WARP) {
                    c.n_chunks += (bk.count * bk.n_seg + kChunk / 32 - 1) / (kChunk / 32);   // a warp per plan
                } else {
                    c.n_chunks += (bk.count * bk.n_seg + kChunk - 1) / kChunk;
                }
                bt.bucket.push_back(bk);
                c.bucket_end = (uint32_t)bt.bucket.size();
            }
            if (!pooled_kind && cls.n_chunks) { bt.classes.push_back(cls); kind_chunks += cls.n_chunks; }
        }
        if (pooled_kind && pooled.n_chunks) bt.classes.push_back(pooled);
    }
    for (const LaunchClass &c : bt.classes)
        if (c.n_chunks >= (1ull << 44)) return fail(ctx, CM_EOVERFLOW, "candidate count does not fit the index type");
    return CM_OK;
}

// Segments shared between scenarios, host part 1: the classes (stages, micro-batches, peers) of
// the template segments that are searched, with room for every row in the class's table (twice
// the rows, a power of two) and list.  The bucket table gets two placeholder entries per class:
// its real content follows once the device has counted the distinct segments.
constexpr size_t kSharedBucketsPerClass = 2;   // transposed part and per-lane remainder
void assign_segment_classes(Batch &bt) {
    bt.tseg_cls.assign(bt.tseg.size(), kNoSegClass);
    bt.look_head.assign(bt.tseg.size(), kNoSegClass);
    bt.look_part.assign(bt.tseg.size(), kNoSegClass);
    bt.ucls_info.clear();
    bt.ucls.clear();
    auto searched = [&](const TSeg &g) {
        const uint32_t t = (uint32_t)(&g - bt.tseg.data());
        return bt.tseg_canon[t] == t && g.m >= 1 && !(g.feas_first != kNoFeasList && g.feas_count == 0);
    };
    auto key_of = [](const TSeg &g, uint16_t m) { return ((uint64_t)g.S << 32) | ((uint64_t)m << 16) | g.n_sync; };
    // pair classes first: the micro-batch counts at which pair heads occur, per (stages, peers),
    // taken greedily from the lowest so that no two pair classes overlap
    std::map<uint64_t, uint32_t> pair_ids, single_ids;
    {
        std::map<std::pair<uint32_t, uint16_t>, const TSeg *> by_group;   // ((S << 16 | peers), m)
        for (const Tmpl &tp : bt.tmpl) {
            if (tp.n_scen == 0) continue;
            for (uint32_t i = 0; i < tp.n_tseg; ++i) {
                const TSeg &g = bt.tseg[tp.tseg_first + i];
                if (bt.role[tp.tseg_first + i] == Batch::kPairHead && searched(g))
                    by_group.emplace(std::make_pair(((uint32_t)g.S << 16) | g.n_sync, g.m), &g);
            }
        }
        uint32_t group = 0xffffffffu;
        int last_start = -2;
        for (const auto &e : by_group) {
            if (e.first.first != group) { group = e.first.first; last_start = -2; }
            const int m = e.first.second;
            if (m == last_start + 1) continue;   // covered as the second count of the pair class before
            last_start = m;
            const TSeg &g = *e.second;
            pair_ids.emplace(key_of(g, g.m), (uint32_t)bt.ucls_info.size());
            bt.ucls_info.push_back(Batch::USegInfo{g.S, g.m, g.n_sync, 1, g.K, g.feas_first, g.feas_count, 0});
        }
    }
    bt.n_pair_cls = (uint32_t)bt.ucls_info.size();
    for (const Tmpl &tp : bt.tmpl) {
        if (tp.n_scen == 0) continue;
        for (uint32_t i = 0; i < tp.n_tseg; ++i) {
            const uint32_t t = tp.tseg_first + i;
            const TSeg &g = bt.tseg[t];
            if (!searched(g) || bt.tseg_cls[t] == kPartnerSeg) continue;
            auto own = pair_ids.find(key_of(g, g.m));
            if (bt.role[t] == Batch::kPairHead && own != pair_ids.end()) {
                bt.tseg_cls[t] = own->second;        // keyed as a pair head; the next row rides with it
                bt.tseg_cls[t + 1] = kPartnerSeg;
                bt.ucls_info[own->second].rows += tp.n_scen;
                continue;
            }
            if (own != pair_ids.end()) bt.look_head[t] = own->second;
            if (g.m >= 1) {
                auto before = pair_ids.find(key_of(g, (uint16_t)(g.m - 1)));
                if (before != pair_ids.end()) bt.look_part[t] = before->second;
            }
            auto it = single_ids.find(key_of(g, g.m));
            if (it == single_ids.end()) {
                it = single_ids.emplace(key_of(g, g.m), (uint32_t)bt.ucls_info.size()).first;
                bt.ucls_info.push_back(Batch::USegInfo{g.S, g.m, g.n_sync, 0, g.K, g.feas_first, g.feas_count, 0});
            }
            bt.ucls_info[it->second].rows += tp.n_scen;
            bt.tseg_cls[t] = it->second;
        }
    }
}

cm_status build_segment_classes(cm_ctx *ctx, Batch &bt) {
    assign_segment_classes(bt);
    uint64_t slots = 0, list = 0;
    for (const Batch::USegInfo &u : bt.ucls_info) {
        uint64_t cap = 64;
        while (cap < 2 * u.rows) cap <<= 1;
        bt.ucls.push_back(USegClass{(uint32_t)slots, (uint32_t)(cap - 1), (uint32_t)list, 0});
        slots += cap;
        list += u.rows;
        if (slots >= (1ull << 31)) return fail(ctx, CM_EOVERFLOW, "batch too large for the index type");
    }
    bt.utab_slots = slots;
    bt.ulist_len = list;
    bt.bucket.assign(std::max<size_t>(kSharedBucketsPerClass * bt.ucls_info.size(), 1), Bucket{});
    bt.classes.clear();
    bt.bucket_tseg.clear();
    return CM_OK;
}

// Host part 2: one bucket per class over its list of distinct segments (counted on the device).
// What does not fill most of a last transposed warp goes to the per-lane kernel.
cm_status build_shared_buckets(cm_ctx *ctx, Batch &bt, const uint32_t *n_distinct) {
    const size_t room = bt.bucket.size();
    bt.bucket.clear();
    bt.classes.clear();
    std::vector<PreBucket> pre;
    auto count_of = [](const Batch::USegInfo &u) {
        return u.feas_first != kNoFeasList ? (uint64_t)u.feas_count : (u.K ? u.K + 1 : 1);
    };
    uint64_t deep_plans = 0;
    for (size_t c = 0; c < bt.ucls_info.size(); ++c) {
        const Batch::USegInfo &u = bt.ucls_info[c];
        if (u.S > kRegStagesMax && u.K > 0) deep_plans += count_of(u) * n_distinct[c] * (u.pair ? 2 : 1);
    }
    const bool by_warp = deep_plans <= kWarpPlansMax;
    for (size_t c = 0; c < bt.ucls_info.size(); ++c) {
        const Batch::USegInfo &u = bt.ucls_info[c];
        const uint32_t n = n_distinct[c];
        if (n == 0) continue;
        if (n > u.rows) return fail(ctx, CM_ECUDA, "internal: more distinct segments than rows");
        uint32_t cut = n;
        if (bucket_kind(by_warp, u.S, u.m, n, u.K) == CM_CLASS_WIDE_UNI && u.S <= kWideStagesMax) {
            const uint32_t rest = n % 32;
            if (rest > 0 && rest < (uint32_t)kUniMinSegments) cut = n - rest;
        }
        for (int part = 0; part < 2; ++part) {
            const uint32_t p0 = part ? cut : 0, p1 = part ? n : cut;
            if (p1 <= p0) continue;
            const int kind = bucket_kind(by_warp, u.S, u.m, p1 - p0, u.K);
            const uint32_t first = bt.ucls[c].list_first + p0;
            if (!u.pair) {
                pre.push_back(PreBucket{kSharedBucket, first, 0, u.S, u.m, count_of(u), p1 - p0, kind, u.feas_first, 0});
            } else if (kind == CM_CLASS_REGS || kind == CM_CLASS_WIDE_UNI || kind == CM_CLASS_WIDE_LANE) {
                const int pk = kind == CM_CLASS_REGS ? CM_CLASS_REGS_PAIR : kind == CM_CLASS_WIDE_UNI ? CM_CLASS_WIDE_PAIR : CM_CLASS_WIDE_LANE_PAIR;
                pre.push_back(PreBucket{kSharedBucket, first, 0, u.S, u.m, count_of(u), p1 - p0, pk, u.feas_first, 1});
            } else {
                // a kernel without a pair form (the batch's few deep plans go a warp per plan): the
                // heads as they are, and their next rows (m + 1, the same compositions) through the same list
                pre.push_back(PreBucket{kSharedBucket, first, 0, u.S, u.m, count_of(u), p1 - p0, kind, u.feas_first, 0});
                pre.push_back(PreBucket{kSharedBucket, first, 0, u.S, (uint16_t)(u.m + 1), count_of(u), p1 - p0,
                                        bucket_kind(by_warp, u.S, u.m + 1, p1 - p0, u.K), u.feas_first, 2});
            }
        }
    }
    cm_status s = layout_buckets(ctx, bt, pre);
    if (s == CM_OK && bt.bucket.size() > room) return fail(ctx, CM_ECUDA, "internal: bucket table outgrew its room");
    return s;
}

// The template of a survivor count (Algorithm 1, get_parallel_strategy, plus the batch
// and layer distribution rules of Section "Planner"): strategies, their micro-batch split
// ranges and one template segment per (strategy, pipeline, micro-batch count).
cm_status build_template(cm_ctx *ctx, Batch &bt, int n_surv, uint32_t *out) {
    const DevProfile &hp = ctx->hp;
    const cm_enum_opts &o = bt.opts;
    const int L = hp.L, G = hp.G;
    const int dp_lo = std::max(1, (int)o.dp_lo), dp_hi = std::min((int)o.dp_hi, CM_MAX_PIPES);
    const int pp_lo = std::max(1, (int)o.pp_lo), pp_hi = std::min(std::min((int)o.pp_hi, L), CM_MAX_STAGES);
    std::vector<uint8_t> &mm_done = ctx->mm_done[cm_ctx::mm_index(o)];
    Tmpl tp{};
    tp.strat_first = (uint32_t)bt.strat.size();
    tp.tseg_first = (uint32_t)bt.tseg.size();
    std::vector<std::vector<uint16_t>> strategies;
    if (n_surv > 0 && pp_lo <= pp_hi) enum_strategies(n_surv, dp_lo, dp_hi, pp_lo, pp_hi, strategies);
    uint64_t split_first = 0, cand = 0;
    for (const auto &tuple : strategies) {
        Strat st{};
        const int dp = (int)tuple.size();
        st.dp = (uint16_t)dp;
        st.seg_first = (uint32_t)bt.tseg.size();
        st.split_first = split_first;
        bt.dp_max = std::max<uint32_t>(bt.dp_max, (uint32_t)dp);
        int sum = 0;
        for (int p = 0; p < dp; ++p) {
            st.S[p] = tuple[p];
            if (o.bm == CM_BATCH_REMAINDER) {
                st.m_lo[p] = (uint16_t)(((int64_t)G * tuple[p]) / n_surv);
                sum += st.m_lo[p];
            } else {
                st.m_lo[p] = 1;
            }
        }
        if (o.bm == CM_BATCH_REMAINDER) {
            st.R = (uint16_t)(G - sum);
            st.n_m = st.R > 0 ? 2 : 1;
            st.n_split = hbinom(ctx, dp, st.R);
        } else {
            st.R = 0;
            st.n_m = (uint16_t)(G >= dp ? G - dp + 1 : 0);
            st.n_split = G >= dp ? hbinom(ctx, G - 1, dp - 1) : 0;
        }
        if (st.n_split == kSat) return fail(ctx, CM_EOVERFLOW, "micro-batch split count overflows 64 bits");
        split_first = sat_add(split_first, st.n_split);
        if (split_first >= (1ull << 62)) return fail(ctx, CM_EOVERFLOW, "too many micro-batch splits");
        int off = 0;
        for (int p = 0; p < dp; ++p) {
            const int S = tuple[p];
            uint64_t K = 0;
            if (o.lm == CM_LAYERS_REMAINDER) K = hbinom(ctx, S, L % S);
            else if (o.lm == CM_LAYERS_FULL) K = hbinom(ctx, L - 1, S - 1);
            if (o.lm == CM_LAYERS_MINMAX || K > o.kappa_cap) K = 0;
            if (K >= (1ull << 62)) return fail(ctx, CM_EOVERFLOW, "layer composition count overflows");
            for (int mi = 0; mi < st.n_m; ++mi) {
                TSeg g{};
                g.S = (uint16_t)S;
                g.m = (uint16_t)(st.m_lo[p] + mi);
                g.n_sync = (uint16_t)dp;
                g.off = (uint16_t)off;
                g.K = K;
                g.feas_first = kNoFeasList;
                g.feas_count = 0;
                g.cand_first = cand;
                const uint64_t count = K ? K + 1 : 1;
                const uint64_t tiles = (count + kTile - 1) / kTile;
                cand = sat_add(cand, count);
                if (cand >= (1ull << 62)) return fail(ctx, CM_EOVERFLOW, "candidate count does not fit the index type");
                if (tiles > 0x7fffffffu) return fail(ctx, CM_EOVERFLOW, "segment too large");
                bt.max_tiles_per_seg = std::max(bt.max_tiles_per_seg, (uint32_t)tiles);
                const uint32_t slot = (uint32_t)((S - 1) * ctx->mm_stride_m + g.m);
                if (g.m >= 1 && !mm_done[slot]) {
                    mm_done[slot] = 1;
                    bt.keys.push_back(((uint32_t)S << 16) | g.m);
                }
                bt.tseg.push_back(g);
            }
            off += S;
        }
        bt.strat.push_back(st);
    }
    tp.n_strat = (uint32_t)bt.strat.size() - tp.strat_first;
    tp.n_tseg = (uint32_t)bt.tseg.size() - tp.tseg_first;
    // pipelines that strategies of this survivor count have in common: searched once (BatchDev::tseg_canon)
    {
        std::unordered_map<uint64_t, uint32_t> first_of;
        first_of.reserve(2 * (size_t)tp.n_tseg);
        uint64_t own = 0;
        bt.tseg_canon.resize(bt.tseg.size());
        for (uint32_t i = 0; i < tp.n_tseg; ++i) {
            const uint32_t t = tp.tseg_first + i;
            const TSeg &g = bt.tseg[t];
            const uint64_t key = ((uint64_t)g.S << 48) | ((uint64_t)g.m << 32) | ((uint64_t)g.n_sync << 16) | g.off;
            const uint32_t c = ctx->dedup ? first_of.emplace(key, t).first->second : t;
            bt.tseg_canon[t] = c;
            if (c != t) ++bt.n_dup;
            else own = sat_add(own, g.K ? g.K + 1 : 1);
        }
        bt.tmpl_cand_own.resize(bt.tmpl.size() + 1, 0);
        bt.tmpl_cand_own[bt.tmpl.size()] = own;
    }
    tp.n_split_total = split_first;
    tp.n_cand = cand;
    tp.n_red = split_first ? (uint32_t)std::min<uint64_t>((split_first + 1023) / 1024, 64) : 0;
    *out = (uint32_t)bt.tmpl.size();
    bt.tmpl.push_back(tp);
    return CM_OK;
}

Tables tables(const cm_ctx *ctx, const Batch &bt);

// Grow the feasible-composition pool to hold `want` entries, keeping its contents.  The pool's
// address changes, and captured launch sequences carry the old one: they are dropped and
// captured again at their next use.
cm_status grow_feas_pool(cm_ctx *ctx, size_t want) {
    if (want <= ctx->d_feas.cap) return CM_OK;
    size_t nc = std::max<size_t>(want, std::max<size_t>(ctx->d_feas.cap * 2, 1u << 20));
    uint32_t *q = nullptr;
    CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (cudaMalloc((void **)&q, nc * sizeof(uint32_t)) != cudaSuccess) { cudaGetLastError(); return fail(ctx, CM_ENOMEM, "device memory"); }
    if (ctx->feas_used) {
        cudaError_t e = cudaMemcpyAsync(q, ctx->d_feas.p, ctx->feas_used * sizeof(uint32_t), cudaMemcpyDeviceToDevice, ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
        if (e != cudaSuccess) { cudaFree(q); cudaGetLastError(); return fail(ctx, CM_ECUDA, cudaGetErrorString(e)); }
    }
    if (ctx->d_feas.p) cudaFree(ctx->d_feas.p);
    ctx->d_feas.p = q;
    ctx->d_feas.cap = nc;
    for (auto &e : ctx->single)
        if (e->exec) { cudaGraphExecDestroy(e->exec); e->exec = nullptr; }
    return CM_OK;
}

// Point every template segment at the list of its memory-feasible candidates, building the
// lists this context has not built yet (Section "Estimator", memory estimator: feasibility is
// a function of stages, micro-batches and composition only).  New lists cost one small copy
// each way, the min-max partitions they end with, one kernel and a synchronisation -- once
// per (layer mode, stages, micro-batches) and profile.
cm_status ensure_feasible_lists(cm_ctx *ctx, Batch &bt) {
    const int lm = bt.opts.lm;
    if (lm == CM_LAYERS_MINMAX) return CM_OK;
    std::map<uint32_t, cm_ctx::FeasEntry> &known = ctx->feas[lm * 2 + (int)bt.opts.sched];
    std::vector<uint32_t> new_keys;
    std::vector<uint64_t> new_K;
    std::vector<uint32_t> new_first;
    size_t used = ctx->feas_used;
    for (const TSeg &g : bt.tseg) {
        if (g.K == 0 || g.K > kFeasMaxK || g.m < 1) continue;
        const uint32_t key = ((uint32_t)g.S << 16) | g.m;
        if (known.count(key)) continue;
        if (used + g.K + 1 >= 0xfffffff0ull) break;   // pool offsets are 32-bit: later keys stay unscreened
        known[key] = cm_ctx::FeasEntry{(uint32_t)used, kNoFeasList, g.K};   // count filled in below
        new_keys.push_back(key);
        new_K.push_back(g.K);
        new_first.push_back((uint32_t)used);
        used += g.K + 1;
    }
    if (!new_keys.empty()) {
        auto undo = [&]() { for (uint32_t k : new_keys) known.erase(k); };
        cm_status s = grow_feas_pool(ctx, used);
        if (s != CM_OK) { undo(); return s; }
        const size_t n = new_keys.size(), n_mm = bt.keys.size();
        // staging layout: K (8n) | keys (4n) | first (4n) | min-max keys (4 n_mm) | counts (4n, device -> host)
        const size_t off_key = 8 * n, off_first = off_key + 4 * n, off_mm = off_first + 4 * n, off_cnt = off_mm + 4 * n_mm;
        const size_t bytes = off_cnt + 4 * n;
        if (!ctx->feas_stage.resize(bytes) || !ctx->d_feas_stage.reserve(bytes)) { undo(); return fail(ctx, CM_ENOMEM, "memory"); }
        unsigned char *h = ctx->feas_stage.p, *d = ctx->d_feas_stage.p;
        memcpy(h, new_K.data(), 8 * n);
        memcpy(h + off_key, new_keys.data(), 4 * n);
        memcpy(h + off_first, new_first.data(), 4 * n);
        if (n_mm) memcpy(h + off_mm, bt.keys.data(), 4 * n_mm);
        const Tables tb = tables(ctx, bt);
        cudaError_t e = cudaMemcpyAsync(d, h, off_cnt, cudaMemcpyHostToDevice, ctx->stream);
        if (e == cudaSuccess && n_mm)
            e = launch_minmax(tb, (const uint32_t *)(d + off_mm), (int)n_mm, bt.intval ? CM_COST_FP64 : bt.opts.cost, ctx->stream);
        if (e == cudaSuccess)
            e = launch_feasible(tb, lm, (const uint32_t *)(d + off_key), (const uint64_t *)d, (const uint32_t *)(d + off_first),
                                (int)n, ctx->d_feas.p, (uint32_t *)(d + off_cnt), ctx->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(h + off_cnt, d + off_cnt, 4 * n, cudaMemcpyDeviceToHost, ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
        if (e != cudaSuccess) { cudaGetLastError(); undo(); return fail(ctx, CM_ECUDA, std::string("feasible-composition lists: ") + cudaGetErrorString(e)); }
        bt.mm_launched = n_mm > 0;
        const uint32_t *cnt = (const uint32_t *)(h + off_cnt);
        for (size_t q = 0; q < n; ++q) known[new_keys[q]].count = cnt[q];
        ctx->feas_used = used;
        ctx->stats[9] += off_cnt;
        ctx->stats[10] += 4 * n;
    }
    for (TSeg &g : bt.tseg) {
        if (g.K == 0 || g.K > kFeasMaxK || g.m < 1) continue;
        auto it = known.find(((uint32_t)g.S << 16) | g.m);
        if (it == known.end() || it->second.count == kNoFeasList) continue;
        g.feas_first = it->second.first;
        g.feas_count = it->second.count;
    }
    return CM_OK;
}

// Build the descriptor tables of a batch on the host: integers only, no cost arithmetic.
cm_status build_batch(cm_ctx *ctx, Batch &bt, const uint32_t *failed_ids, const int32_t *offsets, int B,
                      const cm_enum_opts &o, uint32_t policy_mask) {
    const DevProfile &hp = ctx->hp;
    const int N = hp.n_dp * hp.n_pp;
    bt.scen.clear(); bt.tmpl.clear(); bt.strat.clear(); bt.tseg.clear(); bt.failed.clear(); bt.red_scen.clear();
    bt.keys.clear(); bt.tmpl_scen.clear(); bt.cross.clear(); bt.tseg_canon.clear();
    bt.n_dup = 0;
    bt.opts = o;
    bt.profile_gen = ctx->profile_gen;
    bt.intval = o.cost == CM_COST_INT64NS && ctx->exact53 && !ctx->force_native_i64;
    bt.policy_mask = policy_mask;
    bt.n_cand = bt.n_tiles = bt.n_split = bt.n_rows = 0;
    bt.n_cand_own = 0;
    bt.tmpl_cand_own.assign(1, 0);   // template 0 has no strategies
    bt.max_tiles_per_seg = 0;
    bt.dp_max = 0;
    bt.B = B;
    bt.tmpl_of_nsurv.assign((size_t)N + 1, -1);
    bt.tmpl.push_back(Tmpl{});   // template 0: no strategies (scenarios without a dynamic-parallelism search)
    const int cross_words = (N + 63) / 64 + 1;
    std::vector<char> dead(N);
    std::map<std::string, uint32_t> seen;   // sharing: (node-crossing string, survivor count) -> first scenario
    bt.scen.reserve(B);
    bt.cross.reserve((size_t)B * cross_words);

    for (int b = 0; b < B; ++b) {
        const int f0 = offsets[b], f1 = offsets[b + 1];
        if (f1 < f0) return fail(ctx, CM_EINVAL, "offsets must be non-decreasing");
        Scen sc{};
        sc.failed_first = (uint32_t)bt.failed.size();
        sc.n_failed = (uint32_t)(f1 - f0);
        sc.policy_mask = policy_mask;
        bool bad = false;
        for (int f = f0; f < f1; ++f) {
            const uint32_t d = failed_ids[f];
            if (d >= (uint32_t)N || dead[d]) { bad = true; break; }
            dead[d] = 1;
            bt.failed.push_back(d);
        }
        if (bad) {
            const bool range = std::any_of(failed_ids + f0, failed_ids + f1, [&](uint32_t d) { return d >= (uint32_t)N; });
            for (int f = f0; f < f1; ++f) if (failed_ids[f] < (uint32_t)N) dead[failed_ids[f]] = 0;
            return fail(ctx, CM_EINVAL, range ? "failed device id out of range" : "failed device ids must be distinct");
        }
        // survivors ascending; bit j: survivors j and j+1 sit on different nodes
        sc.cross_first = (uint32_t)bt.cross.size();
        bt.cross.resize(bt.cross.size() + cross_words, 0);
        uint64_t *cw = bt.cross.data() + sc.cross_first;
        int n_surv = 0, prev_node = -1;
        for (int d = 0; d < N; ++d) {
            if (dead[d]) continue;
            const int node = d / hp.devices_per_node;
            if (n_surv > 0 && node != prev_node) cw[(n_surv - 1) >> 6] |= 1ull << ((n_surv - 1) & 63);
            prev_node = node;
            ++n_surv;
        }
        for (int f = f0; f < f1; ++f) dead[failed_ids[f]] = 0;
        sc.rep = (uint32_t)b;
        if (policy_mask & (1u << CM_DYNPAR)) {
            // The dynamic-parallelism space of a scenario is a function of how many devices survive
            // and of where node boundaries fall among them (survivors are placed in consecutive
            // blocks; which device failed enters nowhere else).  With sharing on, scenarios that
            // agree in both are searched once and the others point at that result.
            if (ctx->share) {
                std::string key((const char *)cw, sizeof(uint64_t) * cross_words);
                key.append((const char *)&n_surv, sizeof(n_surv));
                auto it = seen.find(key);
                if (it != seen.end()) {
                    const Scen &r = bt.scen[it->second];
                    sc.rep = it->second;
                    sc.tmpl = r.tmpl;
                    sc.cross_first = r.cross_first;
                    bt.cross.resize(bt.cross.size() - cross_words);
                    bt.scen.push_back(sc);
                    continue;
                }
                seen.emplace(std::move(key), (uint32_t)b);
            }
            int t = bt.tmpl_of_nsurv[n_surv];
            if (t < 0) {
                uint32_t nt = 0;
                cm_status s = build_template(ctx, bt, n_surv, &nt);
                if (s != CM_OK) return s;
                t = (int)nt;
                bt.tmpl_of_nsurv[n_surv] = t;
            }
            sc.tmpl = (uint32_t)t;
        }
        bt.tmpl[sc.tmpl].n_scen++;
        bt.scen.push_back(sc);
    }
    // scenarios grouped by template; result rows and reduction blocks per scenario
    uint32_t first = 0;
    for (Tmpl &tp : bt.tmpl) { tp.scen_first = first; first += tp.n_scen; tp.n_scen = 0; }
    bt.tmpl_scen.resize(B);
    uint64_t rows = 0, red = 0;
    for (int b = 0; b < B; ++b) {
        Scen &sc = bt.scen[b];
        Tmpl &tp = bt.tmpl[sc.tmpl];
        if (sc.rep != (uint32_t)b) {   // shares the rows of an earlier scenario; nothing of its own to search
            sc.seg_base = bt.scen[sc.rep].seg_base;
            sc.red_first = 0;
            continue;
        }
        bt.tmpl_scen[tp.scen_first + tp.n_scen++] = (uint32_t)b;
        sc.seg_base = (uint32_t)rows;
        sc.red_first = (uint32_t)red;
        rows += tp.n_tseg;
        red += tp.n_red;
        for (uint32_t r = 0; r < tp.n_red; ++r) bt.red_scen.push_back((uint32_t)b);
        bt.n_cand = sat_add(bt.n_cand, tp.n_cand);
        bt.n_cand_own = sat_add(bt.n_cand_own, bt.tmpl_cand_own[sc.tmpl]);
        bt.n_split = sat_add(bt.n_split, tp.n_split_total);
        if (rows >= (1ull << 31) || red >= (1ull << 31) || bt.n_cand >= (1ull << 62))
            return fail(ctx, CM_EOVERFLOW, "batch too large for the index type");
    }
    bt.n_rows = rows;
    bt.n_tiles = bt.max_tiles_per_seg ? 1 : 0;   // only "is there anything to tie-break" matters
    bt.mm_launched = false;
    if (ctx->d_prof && ctx->screen) {   // (a context without a device only describes: cm_host_describe)
        const uint64_t t0 = now_ns();
        cm_status s = ensure_feasible_lists(ctx, bt);
        ctx->stats[17] += now_ns() - t0;
        if (s != CM_OK) return s;
    }
    // With sharing on, a batch of several scenarios also shares SEGMENTS: the distinct (stages,
    // micro-batches, peers, link tiers) are found on the device once the tables are there.
    mark_pairs(ctx, bt);
    bt.useg = ctx->share && ctx->d_prof && B > 1 && (policy_mask & (1u << CM_DYNPAR)) && rows > 0;
    if (bt.useg) return build_segment_classes(ctx, bt);
    bt.ucls.clear();
    bt.tseg_cls.clear();
    bt.look_head.clear();
    bt.look_part.clear();
    return build_buckets(ctx, bt);
}

// Pack the host tables into the pinned arena (16-byte aligned sections).
template <typename T>
size_t arena_put(PinnedVec<unsigned char> &arena, const std::vector<T> &v, bool &ok) {
    const size_t off = (arena.size() + 15) & ~(size_t)15;
    const size_t bytes = std::max<size_t>(v.size(), 1) * sizeof(T);
    if (!arena.resize(off + bytes)) { ok = false; return off; }
    if (!v.empty()) memcpy(arena.p + off, v.data(), v.size() * sizeof(T));
    return off;
}

BatchDev dev_view(const cm_ctx *ctx, Batch &bt) {
    BatchDev v{};
    const unsigned char *a = bt.d_arena.p;
    v.scen = (const Scen *)(a + bt.off_scen); v.tmpl = (const Tmpl *)(a + bt.off_tmpl);
    v.strat = (const Strat *)(a + bt.off_strat); v.tseg = (const TSeg *)(a + bt.off_tseg);
    v.failed = (const uint32_t *)(a + bt.off_failed); v.cross = (const uint64_t *)(a + bt.off_cross);
    v.tmpl_scen = (const uint32_t *)(a + bt.off_tmpl_scen);
    v.bucket = bt.bucket_override ? bt.bucket_override : (const Bucket *)(a + bt.off_bucket);
    v.bucket_tseg = (const uint32_t *)(a + bt.off_bucket_tseg); v.red_scen = (const uint32_t *)(a + bt.off_red);
    v.feas = ctx->d_feas.p;
    v.useg = bt.d_useg.p;
    v.tseg_canon = bt.n_dup ? (const uint32_t *)(a + bt.off_canon) : nullptr;
    v.n_rep_scen = 0;
    for (const Tmpl &tp : bt.tmpl) v.n_rep_scen += tp.n_scen;
    v.seg_best = bt.d_seg_best.p; v.partial = bt.d_partial.p;
    v.winner = bt.d_winner.p; v.kappa_sel = bt.d_kappa_sel.p; v.pol_cost = bt.d_pol_cost.p;
    v.rc_stages = bt.d_rc_stages.p; v.plans = bt.d_plans.p;
    v.counters = reinterpret_cast<unsigned long long *>(bt.d_seg_best.p + bt.n_rows);
    v.B = bt.B; v.mode = bt.opts.cost; v.intval = bt.intval ? 1u : 0u;
    v.n_rows = (uint32_t)bt.n_rows;
    v.n_tiles = bt.n_tiles; v.max_tiles_per_seg = bt.max_tiles_per_seg;
    v.n_red_blocks = (uint32_t)bt.red_scen.size(); v.dp_max = bt.dp_max;
    v.max_red_per_scen = 0;
    for (const Tmpl &tp : bt.tmpl) v.max_red_per_scen = std::max(v.max_red_per_scen, tp.n_scen ? tp.n_red : 0u);
    v.layer_mode = bt.opts.lm; v.batch_mode = bt.opts.bm;
    return v;
}

USegDev useg_view(const Batch &bt) {
    USegDev u{};
    u.cls = (const USegClass *)(bt.d_arena.p + bt.off_ucls);
    u.tseg_cls = (const uint32_t *)(bt.d_arena.p + bt.off_tseg_cls);
    u.look_head = (const uint32_t *)(bt.d_arena.p + bt.off_look_head);
    u.look_part = (const uint32_t *)(bt.d_arena.p + bt.off_look_part);
    u.n_pair_cls = bt.n_pair_cls;
    u.tab = bt.d_utab.p; u.rep = bt.d_urep.p; u.slot_of = bt.d_slot_of.p; u.count = bt.d_ucount.p; u.list = bt.d_useg.p;
    u.n_cls = (uint32_t)bt.ucls.size();
    u.n_rep_scen = 0;
    for (const Tmpl &tp : bt.tmpl) u.n_rep_scen += tp.n_scen;
    return u;
}

Tables tables(const cm_ctx *ctx, const Batch &bt) {
    Tables t{};
    t.prof = bt.intval ? ctx->d_prof53 : ctx->d_prof; t.binom = ctx->d_binom; t.binom_rows = ctx->binom_rows;
    t.mm_cuts = ctx->d_mm[cm_ctx::mm_index(bt.opts)]; t.mm_stride_m = ctx->mm_stride_m;
    t.sched = (int32_t)bt.opts.sched;
    return t;
}

Tables tables_plain(const cm_ctx *ctx) {   // for kernels that only read the byte prefix sums
    Tables t{};
    t.prof = ctx->d_prof; t.binom = ctx->d_binom; t.binom_rows = ctx->binom_rows;
    t.mm_cuts = ctx->d_mm[0]; t.mm_stride_m = ctx->mm_stride_m;
    return t;
}

// Copy the tables of a batch to the device (one copy) and run the min-max partitions it needs.
cm_status upload_batch(cm_ctx *ctx, Batch &bt, int *launches) {
    struct Timer { cm_ctx *c; uint64_t t0; ~Timer() { c->stats[18] += now_ns() - t0; } } timer{ctx, now_ns()};
    bool ok = true;
    bt.arena.clear();
    bt.off_scen = arena_put(bt.arena, bt.scen, ok);
    bt.off_tmpl = arena_put(bt.arena, bt.tmpl, ok);
    bt.off_strat = arena_put(bt.arena, bt.strat, ok);
    bt.off_tseg = arena_put(bt.arena, bt.tseg, ok);
    bt.off_failed = arena_put(bt.arena, bt.failed, ok);
    bt.off_red = arena_put(bt.arena, bt.red_scen, ok);
    bt.off_keys = arena_put(bt.arena, bt.keys, ok);
    bt.off_tmpl_scen = arena_put(bt.arena, bt.tmpl_scen, ok);
    bt.off_bucket_tseg = arena_put(bt.arena, bt.bucket_tseg, ok);
    bt.off_cross = arena_put(bt.arena, bt.cross, ok);
    bt.off_canon = arena_put(bt.arena, bt.tseg_canon, ok);
    bt.off_ucls = arena_put(bt.arena, bt.ucls, ok);
    bt.off_tseg_cls = arena_put(bt.arena, bt.tseg_cls, ok);
    bt.off_look_head = arena_put(bt.arena, bt.look_head, ok);
    bt.off_look_part = arena_put(bt.arena, bt.look_part, ok);
    bt.off_bucket = arena_put(bt.arena, bt.bucket, ok);
    if (!ok) return fail(ctx, CM_ENOMEM, "host memory");
    if (!bt.d_arena.reserve(bt.arena.size())) return fail(ctx, CM_ENOMEM, "device memory");
    CM_CUDA(ctx, cudaMemcpyAsync(bt.d_arena.p, bt.arena.p, bt.arena.size(), cudaMemcpyHostToDevice, ctx->stream));
    ctx->stats[9] += bt.arena.size();
    const size_t B = std::max(bt.B, 1);
    ok = bt.d_seg_best.reserve(bt.n_rows + 4) &&   // + the four work counters, cleared by the same memset
         bt.d_partial.reserve(std::max<size_t>(bt.red_scen.size(), 1)) && bt.d_winner.reserve(B) &&
         bt.d_kappa_sel.reserve(B * kMaxP) && bt.d_pol_cost.reserve(B * 2) &&
         bt.d_rc_stages.reserve(B * kMaxP) && bt.d_plans.reserve(B * 4 + 1);   // + room for the counters
    if (!ok) return fail(ctx, CM_ENOMEM, "device memory");
    if (bt.keys.size() && !bt.mm_launched) {
        CM_CUDA(ctx, launch_minmax(tables(ctx, bt), (const uint32_t *)(bt.d_arena.p + bt.off_keys),
                                   (int)bt.keys.size(), bt.intval ? CM_COST_FP64 : bt.opts.cost, ctx->stream));
        if (launches) ++*launches;
    }
    if (bt.useg) {
        // key every row, list the distinct segments, count them per class; the counts decide the
        // work layout, so they come back (one small copy, one synchronisation) before the buckets
        // are laid out and their table -- the last section of the arena -- is copied again
        const size_t n_cls = bt.ucls.size();
        ok = bt.d_utab.reserve(std::max<uint64_t>(bt.utab_slots, 1)) && bt.d_urep.reserve(std::max<uint64_t>(bt.utab_slots, 1)) &&
             bt.d_slot_of.reserve(std::max<uint64_t>(bt.n_rows, 1)) && bt.d_ucount.reserve(n_cls + 1) &&
             bt.d_useg.reserve(std::max<uint64_t>(bt.ulist_len, 1)) && bt.ucount_host.resize(n_cls + 1);
        if (!ok) return fail(ctx, CM_ENOMEM, "memory");
        CM_CUDA(ctx, cudaMemsetAsync(bt.d_utab.p, 0xFF, bt.utab_slots * sizeof(unsigned long long), ctx->stream));
        CM_CUDA(ctx, cudaMemsetAsync(bt.d_urep.p, 0xFF, bt.utab_slots * sizeof(uint32_t), ctx->stream));
        CM_CUDA(ctx, cudaMemsetAsync(bt.d_ucount.p, 0, (n_cls + 1) * sizeof(uint32_t), ctx->stream));
        CM_CUDA(ctx, launch_useg_keys(dev_view(ctx, bt), useg_view(bt), ctx->stream));
        if (launches) *launches += 3;
        CM_CUDA(ctx, cudaMemcpyAsync(bt.ucount_host.p, bt.d_ucount.p, (n_cls + 1) * sizeof(uint32_t), cudaMemcpyDeviceToHost, ctx->stream));
        CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        ctx->stats[10] += (n_cls + 1) * sizeof(uint32_t);
        if (bt.ucount_host[n_cls] != 0) return fail(ctx, CM_ECUDA, "internal: segment table full");
        cm_status s = build_shared_buckets(ctx, bt, bt.ucount_host.p);
        if (s != CM_OK) return s;
        if (!bt.bucket.empty()) {
            memcpy(bt.arena.p + bt.off_bucket, bt.bucket.data(), bt.bucket.size() * sizeof(Bucket));
            CM_CUDA(ctx, cudaMemcpyAsync(bt.d_arena.p + bt.off_bucket, bt.arena.p + bt.off_bucket, bt.bucket.size() * sizeof(Bucket),
                                         cudaMemcpyHostToDevice, ctx->stream));
            ctx->stats[9] += bt.bucket.size() * sizeof(Bucket);
        }
    }
    return CM_OK;
}

// Enqueue the launch sequence of a search on `st`: clear, the two one-plan policies, search
// pass, split reduction, tie-break pass, finalize, plans back to the host.  phase_events: record
// the events between the phases (not while the sequence is being captured into a graph).
cm_status enqueue_search(cm_ctx *ctx, Batch &bt, cudaStream_t st, bool phase_events, int *launches_out, int *cost_launches_out) {
    const Tables tb = tables(ctx, bt);
    const BatchDev bd = dev_view(ctx, bt);
    int launches = 0, cost_launches = 0;
    // per-segment minima start at all-ones (above every cost); so do the work counters, which
    // therefore read "value - 1" until cm_finalize_kernel adds the one back
    CM_CUDA(ctx, cudaMemsetAsync(bt.d_seg_best.p, 0xFF, (bt.n_rows + 4) * sizeof(uint64_t), st));
    const bool policies = (bt.policy_mask & ((1u << CM_REROUTE) | (1u << CM_REDUNDANT))) != 0;
    const bool beside = policies && (bt.policy_mask & (1u << CM_DYNPAR)) && ctx->pol_stream;
    if (policies) {
        if (beside) {
            CM_CUDA(ctx, cudaEventRecord(ctx->pol_fork, st));
            CM_CUDA(ctx, cudaStreamWaitEvent(ctx->pol_stream, ctx->pol_fork, 0));
        }
        CM_CUDA(ctx, launch_policies(tb, bd, ctx->hp.n_dp, beside ? ctx->pol_stream : st));
        if (beside) CM_CUDA(ctx, cudaEventRecord(ctx->pol_join, ctx->pol_stream));
        ++launches;
    }
    if (bt.policy_mask & (1u << CM_DYNPAR)) {
        if (phase_events) CM_CUDA(ctx, cudaEventRecord(ctx->ev[2], st));
        CM_CUDA(ctx, launch_cost_pass1(tb, bd, bt.classes.data(), (int)bt.classes.size(), st, &ctx->side, &cost_launches));
        launches += cost_launches;
        if (bt.useg) {   // rows that share a segment take its representative's minimum
            CM_CUDA(ctx, launch_useg_copy(bd, useg_view(bt), st));
            ++launches;
        }
        if (bt.n_dup) {  // pipelines that strategies have in common were searched once
            CM_CUDA(ctx, launch_dup_copy(bd, st));
            ++launches;
        }
        if (phase_events) CM_CUDA(ctx, cudaEventRecord(ctx->ev[3], st));
        CM_CUDA(ctx, launch_split_reduce(tb, bd, st));
        launches += (bd.n_red_blocks && bd.max_red_per_scen > 1) ? 2 : 1;
        if (phase_events) CM_CUDA(ctx, cudaEventRecord(ctx->ev[4], st));
        if (bt.n_tiles) {
            bool deep = false;
            for (const TSeg &g : bt.tseg) deep = deep || (g.S > kRegStagesMax && g.K > 0);
            // few winners (a failure handled on its own): the lock-step kernel completes every deep
            // pipeline in one launch; many: one plan per lane, a kernel per depth
            const bool by_warp = deep && (uint64_t)bt.B * bt.dp_max <= kWarpTieMaxPairs;
            CM_CUDA(ctx, launch_cost_pass2(tb, bd, st, by_warp));
            ++launches;
            if (by_warp) {
                CM_CUDA(ctx, launch_tiebreak_warp(tb, bd, st));
                ++launches;
            } else if (deep) {
                uint64_t stage_mask = 0;
                for (const TSeg &g : bt.tseg) stage_mask |= 1ull << (g.S & 63);
                CM_CUDA(ctx, launch_tiebreak_wide(tb, bd, stage_mask, st, &ctx->side, &launches));
            }
        }
        if (phase_events) CM_CUDA(ctx, cudaEventRecord(ctx->ev[5], st));
    }
    if (beside) CM_CUDA(ctx, cudaStreamWaitEvent(st, ctx->pol_join, 0));
    CM_CUDA(ctx, launch_finalize(tb, bd, st));
    ++launches;
    if (phase_events) CM_CUDA(ctx, cudaEventRecord(ctx->ev[1], st));
    const size_t back_bytes = (size_t)bt.B * 4 * sizeof(cm_plan) + 4 * sizeof(unsigned long long);
    CM_CUDA(ctx, cudaMemcpyAsync(bt.plans_host.p, bt.d_plans.p, back_bytes, cudaMemcpyDeviceToHost, st));
    *launches_out = launches;
    *cost_launches_out = cost_launches;
    return CM_OK;
}

// The search over an uploaded batch; results land in bt.plans_host ([B][4]) after the stream is
// synchronised.  `single`: a resident one-scenario entry whose sequence may replay as a graph.
cm_status run_batch(cm_ctx *ctx, Batch &bt, int launches_so_far, cm_ctx::Single *single = nullptr) {
    cudaStream_t st = ctx->stream;
    int launches = 0, cost_launches = 0;
    const size_t back_bytes = (size_t)bt.B * 4 * sizeof(cm_plan) + 4 * sizeof(unsigned long long);
    if (!bt.plans_host.resize((size_t)bt.B * 4 + 1)) return fail(ctx, CM_ENOMEM, "host memory");
    const uint64_t h_enqueue = now_ns();
    bool replay = false;
    if (single && ctx->use_graphs && ctx->graph_stream && !single->graph_failed) {
        if (!single->exec) {
            // capture the sequence once; any failure leaves the entry on the plain path for good
            cudaGraph_t graph = nullptr;
            bool ok = cudaStreamBeginCapture(ctx->graph_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
            if (ok) {
                const cm_status cs = enqueue_search(ctx, bt, ctx->graph_stream, false, &single->launches, &cost_launches);
                const cudaError_t ce = cudaStreamEndCapture(ctx->graph_stream, &graph);
                ok = cs == CM_OK && ce == cudaSuccess && graph;
            }
            if (ok) ok = cudaGraphInstantiate(&single->exec, graph, 0) == cudaSuccess;
            if (graph) cudaGraphDestroy(graph);
            if (!ok) { cudaGetLastError(); single->exec = nullptr; single->graph_failed = true; ctx->err.clear(); }
        }
        replay = single->exec != nullptr;
    }
    CM_CUDA(ctx, cudaEventRecord(ctx->ev[0], st));
    if (replay) {
        CM_CUDA(ctx, cudaGraphLaunch(single->exec, st));
        CM_CUDA(ctx, cudaEventRecord(ctx->ev[1], st));
        launches = single->launches;
    } else {
        cm_status s = enqueue_search(ctx, bt, st, true, &launches, &cost_launches);
        if (s != CM_OK) return s;
    }
    launches += launches_so_far;
    const uint64_t h_wait = now_ns();
    CM_CUDA(ctx, cudaStreamSynchronize(st));
    ctx->stats[14] += h_wait - h_enqueue;
    ctx->stats[15] += now_ns() - h_wait;
    float ms = 0.f;
    CM_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]));
    if (!replay && (bt.policy_mask & (1u << CM_DYNPAR))) {
        float ms_cost = 0.f, ms_tie = 0.f;
        CM_CUDA(ctx, cudaEventElapsedTime(&ms_cost, ctx->ev[2], ctx->ev[3]));
        CM_CUDA(ctx, cudaEventElapsedTime(&ms_tie, ctx->ev[4], ctx->ev[5]));
        ctx->stats[8] += (uint64_t)((double)ms_cost * 1e6);
        ctx->stats[11] += (uint64_t)((double)ms_tie * 1e6);
        ctx->stats[12] += (uint64_t)cost_launches;
    }
    ctx->stats[10] += back_bytes;
    const unsigned long long *counters_host = reinterpret_cast<const unsigned long long *>(bt.plans_host.p + (size_t)bt.B * 4);
    ctx->stats[0] += (bt.policy_mask & (1u << CM_DYNPAR)) ? bt.n_cand : 0;
    ctx->stats[19] += (bt.policy_mask & (1u << CM_DYNPAR)) ? bt.n_cand_own : 0;
    ctx->stats[1] += counters_host[0];
    ctx->stats[2] += counters_host[1];
    ctx->stats[16] += counters_host[2];
    ctx->stats[3] += (uint64_t)launches;
    ctx->stats[4] += (uint64_t)((double)ms * 1e6);
    ctx->stats[5] += bt.n_rows;
    ctx->stats[6] += bt.strat.size();
    ctx->stats[7] += bt.n_split;
    return CM_OK;
}

// One resident scenario searched with its duplicate segments removed (sharing on).  A single
// failure set repeats pipelines too: strategies share stage counts, and a pipeline that starts a
// whole number of nodes further on sees the same link tiers.  The few hundred template segments
// are keyed on the host (class, tier word), sorted, and the distinct ones laid out as shared
// buckets beside the template buckets; the sequence is launched directly (its grids change from
// failure to failure, so the resident graph does not fit).  *done = false: too little would be
// saved to pay for the direct launches -- the caller replays the graph as usual.
constexpr uint64_t kShareSingleMinCells = 250000000ull;   // recurrence cells that sharing must save (~70 us of search pass)
cm_status run_single_shared(cm_ctx *ctx, Batch &bt, int launches_so_far, bool *done) {
    *done = false;
    if (bt.B != 1 || !(bt.policy_mask & (1u << CM_DYNPAR)) || bt.scen.empty()) return CM_OK;
    const Scen &sc = bt.scen[0];
    const Tmpl &tp = bt.tmpl[sc.tmpl];
    if (tp.n_tseg < 2) return CM_OK;
    if (bt.tseg_cls.size() != bt.tseg.size()) {   // once per resident batch
        assign_segment_classes(bt);
        bt.single_cells = 0;
        for (uint32_t i = 0; i < tp.n_tseg; ++i) {
            const TSeg &g = bt.tseg[tp.tseg_first + i];
            if (bt.tseg_cls[tp.tseg_first + i] == kNoSegClass) continue;
            bt.single_cells += (g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : (g.K ? g.K + 1 : 1)) * 2ull * g.S * g.m;
        }
    }
    if (bt.single_cells < kShareSingleMinCells) return CM_OK;   // not even all of its cells would be worth it
    const size_t n_cls = bt.ucls_info.size();
    // The same keying as cm_useg_key_kernel, on the host: the heads of the pair classes first, then
    // every other row, which joins a pair that holds its tier (as head: its own m; as second row:
    // m - 1) before it is keyed among the single segments.  `joined`: slot_of value of such a row.
    struct Key { uint32_t cls; uint64_t tier; uint32_t row; uint32_t joined; };
    std::vector<Key> heads, others;
    heads.reserve(tp.n_tseg);
    others.reserve(tp.n_tseg);
    const uint64_t *words = bt.cross.data() + sc.cross_first;
    auto single_cells_of = [&](const TSeg &g) {
        return (g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : (g.K ? g.K + 1 : 1)) * 2ull * g.S * g.m;
    };
    uint64_t all_cells = 0, distinct_cells = 0;
    for (uint32_t i = 0; i < tp.n_tseg; ++i) {
        const uint32_t c = bt.tseg_cls[tp.tseg_first + i];
        if (c == kNoSegClass) continue;
        const TSeg &g = bt.tseg[tp.tseg_first + i];
        all_cells += single_cells_of(g);
        if (c == kPartnerSeg) continue;
        const int w = g.off >> 6, sh = g.off & 63, n = g.S - 1;
        uint64_t v = words[w] >> sh;
        if (sh) v |= words[w + 1] << (64 - sh);
        (c < bt.n_pair_cls ? heads : others).push_back(Key{c, v & ((1ull << n) - 1ull), i, kNoSegClass});
    }
    auto by_key = [](const Key &a, const Key &b) {
        return a.cls != b.cls ? a.cls < b.cls : a.tier != b.tier ? a.tier < b.tier : a.row < b.row;
    };
    auto same_key = [](const Key &a, const Key &b) { return a.cls == b.cls && a.tier == b.tier; };
    std::sort(heads.begin(), heads.end(), by_key);
    std::vector<Key> pair_reps;   // distinct pair heads, sorted by (class, tier); index = their slot
    for (size_t i = 0; i < heads.size(); ++i)
        if (i == 0 || !same_key(heads[i], heads[i - 1])) pair_reps.push_back(heads[i]);
    auto find_pair = [&](uint32_t cls, uint64_t tier) -> uint32_t {
        if (cls == kNoSegClass) return kNoSegClass;
        const Key probe{cls, tier, 0, 0};
        auto it = std::lower_bound(pair_reps.begin(), pair_reps.end(), probe, [](const Key &a, const Key &b) {
            return a.cls != b.cls ? a.cls < b.cls : a.tier < b.tier;
        });
        return it != pair_reps.end() && same_key(*it, probe) ? (uint32_t)(it - pair_reps.begin()) : kNoSegClass;
    };
    std::vector<Key> singles;
    singles.reserve(others.size());
    for (Key &k : others) {
        const uint32_t t = tp.tseg_first + k.row;
        uint32_t at = find_pair(bt.look_head[t], k.tier);
        if (at == kNoSegClass) {
            at = find_pair(bt.look_part[t], k.tier);
            if (at != kNoSegClass) at |= kSecondRowFlag;
        }
        k.joined = at;
        if (at == kNoSegClass) singles.push_back(k);
    }
    std::sort(singles.begin(), singles.end(), by_key);
    auto cells_of = [&](uint32_t c) {
        const Batch::USegInfo &u = bt.ucls_info[c];
        const uint64_t count = u.feas_first != kNoFeasList ? (uint64_t)u.feas_count : (u.K ? u.K + 1 : 1);
        return count * (u.pair ? 2ull * u.S * (u.m + 1) + 3ull * u.S * (u.S - 1) / 2 : 2ull * u.S * u.m);
    };
    std::vector<uint32_t> counts(n_cls + 1, 0);
    size_t n_distinct = pair_reps.size();
    for (const Key &k : pair_reps) { distinct_cells += cells_of(k.cls); ++counts[k.cls]; }
    for (size_t i = 0; i < singles.size(); ++i)
        if (i == 0 || !same_key(singles[i], singles[i - 1])) { distinct_cells += cells_of(singles[i].cls); ++counts[singles[i].cls]; ++n_distinct; }
    if (all_cells < distinct_cells + kShareSingleMinCells) return CM_OK;

    // staging: slot_of [rows] | rep [distinct] | list [distinct] | buckets [2 per class]
    const size_t rows = bt.n_rows, max_buckets = std::max<size_t>(kSharedBucketsPerClass * n_cls, 1);
    const size_t off_rep = 4 * rows, off_list = (off_rep + 4 * n_distinct + 7) & ~(size_t)7;
    const size_t off_bk = (off_list + 8 * n_distinct + 15) & ~(size_t)15, bytes = off_bk + max_buckets * sizeof(Bucket);
    bool ok = bt.alt_stage.resize(bytes) && bt.d_slot_of.reserve(std::max<size_t>(rows, 1)) && bt.d_urep.reserve(std::max<size_t>(n_distinct, 1)) &&
              bt.d_useg.reserve(std::max<size_t>(n_distinct, 1)) && bt.d_alt_bucket.reserve(max_buckets);
    if (!ok) return fail(ctx, CM_ENOMEM, "memory");
    uint32_t *slot_of = (uint32_t *)bt.alt_stage.p, *rep = (uint32_t *)(bt.alt_stage.p + off_rep);
    uint2 *list = (uint2 *)(bt.alt_stage.p + off_list);
    std::fill(slot_of, slot_of + rows, kNoSegClass);
    bt.ucls.assign(n_cls, USegClass{0, 0, 0, 0});
    uint32_t first_of = 0;
    for (size_t c = 0; c < n_cls; ++c) { bt.ucls[c].list_first = first_of; first_of += counts[c]; }
    // slots (= list positions): the distinct pair heads, then the distinct single segments; pair
    // classes have the lower class numbers, so the positions follow the class regions
    uint32_t u = 0;
    for (size_t i = 0; i < heads.size(); ++i) {
        if (i == 0 || !same_key(heads[i], heads[i - 1])) {
            rep[u] = sc.seg_base + heads[i].row;
            list[u] = make_uint2(0u, tp.tseg_first + heads[i].row);
            ++u;
        }
        slot_of[sc.seg_base + heads[i].row] = u - 1;
        slot_of[sc.seg_base + heads[i].row + 1] = kPartnerSeg;
    }
    for (const Key &k : others)
        if (k.joined != kNoSegClass) slot_of[sc.seg_base + k.row] = k.joined;
    for (size_t i = 0; i < singles.size(); ++i) {
        if (i == 0 || !same_key(singles[i], singles[i - 1])) {
            rep[u] = sc.seg_base + singles[i].row;
            list[u] = make_uint2(0u, tp.tseg_first + singles[i].row);
            ++u;
        }
        slot_of[sc.seg_base + singles[i].row] = u - 1;
    }
    std::vector<Bucket> keep_buckets;
    std::vector<LaunchClass> keep_classes;
    keep_buckets.swap(bt.bucket);
    keep_classes.swap(bt.classes);
    bt.bucket.assign(max_buckets, Bucket{});
    cm_status s = build_shared_buckets(ctx, bt, counts.data());
    cudaError_t e = cudaSuccess;
    if (s == CM_OK) {
        if (!bt.bucket.empty()) memcpy(bt.alt_stage.p + off_bk, bt.bucket.data(), bt.bucket.size() * sizeof(Bucket));
        cudaStream_t st = ctx->stream;
        e = cudaMemcpyAsync(bt.d_slot_of.p, slot_of, 4 * rows, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && n_distinct) e = cudaMemcpyAsync(bt.d_urep.p, rep, 4 * n_distinct, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && n_distinct) e = cudaMemcpyAsync(bt.d_useg.p, list, 8 * n_distinct, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && !bt.bucket.empty())
            e = cudaMemcpyAsync(bt.d_alt_bucket.p, bt.alt_stage.p + off_bk, bt.bucket.size() * sizeof(Bucket), cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) {
            ctx->stats[9] += 4 * rows + 12 * n_distinct + bt.bucket.size() * sizeof(Bucket);
            bt.bucket_override = bt.d_alt_bucket.p;
            bt.useg = true;
            s = run_batch(ctx, bt, launches_so_far, nullptr);
            *done = s == CM_OK;
        }
    }
    bt.useg = false;
    bt.bucket_override = nullptr;
    bt.bucket.swap(keep_buckets);
    bt.classes.swap(keep_classes);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ctx, CM_ECUDA, std::string("shared segments: ") + cudaGetErrorString(e)); }
    return s;
}

// Keys of min-max partitions that were scheduled but never computed must be asked for
// again by the next batch.
void forget_keys(cm_ctx *ctx, Batch &bt) {
    std::vector<uint8_t> &done = ctx->mm_done[cm_ctx::mm_index(bt.opts)];
    for (size_t i = 0; i < bt.keys.size(); ++i) {
        const uint32_t S = bt.keys[i] >> 16, m = bt.keys[i] & 0xffffu;
        done[(size_t)(S - 1) * ctx->mm_stride_m + m] = 0;
    }
    bt.keys.clear();
}

// A pipeline-plan index that the winner kernel leaves untouched means "not found";
// it cannot happen for a feasible winner, but never hand it to the caller as a rank.
void scrub(cm_plan &pl) {
    for (int p = 0; p < CM_MAX_PIPES; ++p)
        if (pl.kappa[p] == ~0ull) { pl.kappa[p] = 0; pl.feasible = 0; }
}

// A prepared one-scenario batch for this failure set: found among the context's resident ones
// (same survivor count, same options, same arithmetic) and patched, or built and uploaded.
// *entry: the resident entry that was reused (its launch sequence may replay as a graph), NULL
// if the batch was just built.
cm_status single_batch(cm_ctx *ctx, const uint32_t *ids, int n, const cm_enum_opts &o, uint32_t mask, Batch **out,
                       int *launches, cm_ctx::Single **entry) {
    const DevProfile &hp = ctx->hp;
    const int N = hp.n_dp * hp.n_pp;
    const int32_t off[2] = {0, n};
    const bool intval = o.cost == CM_COST_INT64NS && ctx->exact53 && !ctx->force_native_i64;
    // distinct ids in range (the builder checks the same; here it decides the survivor count)
    bool ok = n <= N;
    for (int i = 0; i < n && ok; ++i) {
        ok = ids[i] < (uint32_t)N;
        for (int j = 0; j < i && ok; ++j) ok = ids[j] != ids[i];
    }
    cm_ctx::Single *hit = nullptr;
    if (ok)
        for (auto &e : ctx->single)
            if (e->n_surv == N - n && e->intval == intval && memcmp(&e->opts, &o, sizeof(o)) == 0) { hit = e.get(); break; }
    *entry = hit;
    if (!hit) {
        // (also the path of malformed sets: the builder produces the error)
        std::unique_ptr<Batch> b(new (std::nothrow) Batch());
        if (!b) return fail(ctx, CM_ENOMEM, "host memory");
        cm_status s = build_batch(ctx, *b, ids, off, 1, o, mask);
        if (s == CM_OK) s = upload_batch(ctx, *b, launches);
        if (s != CM_OK) { cudaStreamSynchronize(ctx->stream); forget_keys(ctx, *b); return s; }
        if (ctx->single.size() >= 64) {   // bounded: start over rather than grow without limit
            cudaStreamSynchronize(ctx->stream);
            ctx->single.clear();
        }
        std::unique_ptr<cm_ctx::Single> e(new (std::nothrow) cm_ctx::Single());
        if (!e) return fail(ctx, CM_ENOMEM, "host memory");
        e->n_surv = N - n; e->opts = o; e->intval = intval; e->batch = std::move(b);
        *out = e->batch.get();
        ctx->single.push_back(std::move(e));
        return CM_OK;
    }
    Batch &bt = *hit->batch;
    // patch what depends on WHICH devices failed: the ids and the node-crossing bits
    const size_t cross_words = bt.cross.size();
    std::fill(bt.cross.begin(), bt.cross.end(), 0ull);
    int n_surv = 0, prev_node = -1, f = 0;
    uint32_t sorted[CM_MAX_PIPES * CM_MAX_STAGES];
    for (int i = 0; i < n; ++i) { bt.failed[i] = ids[i]; sorted[i] = ids[i]; }
    std::sort(sorted, sorted + n);
    for (int d = 0; d < N; ++d) {
        if (f < n && sorted[f] == (uint32_t)d) { ++f; continue; }
        const int node = d / hp.devices_per_node;
        if (n_surv > 0 && node != prev_node) bt.cross[(n_surv - 1) >> 6] |= 1ull << ((n_surv - 1) & 63);
        prev_node = node;
        ++n_surv;
    }
    if (n) memcpy(bt.arena.p + bt.off_failed, bt.failed.data(), sizeof(uint32_t) * n);
    memcpy(bt.arena.p + bt.off_cross, bt.cross.data(), sizeof(uint64_t) * cross_words);
    if (n) CM_CUDA(ctx, cudaMemcpyAsync(bt.d_arena.p + bt.off_failed, bt.arena.p + bt.off_failed, sizeof(uint32_t) * n, cudaMemcpyHostToDevice, ctx->stream));
    CM_CUDA(ctx, cudaMemcpyAsync(bt.d_arena.p + bt.off_cross, bt.arena.p + bt.off_cross, sizeof(uint64_t) * cross_words, cudaMemcpyHostToDevice, ctx->stream));
    ctx->stats[9] += sizeof(uint32_t) * n + sizeof(uint64_t) * cross_words;
    *out = &bt;
    return CM_OK;
}

}  // namespace

// Accessors for entry points that live in other translation units.
cm_status cm_internal_fail(cm_ctx *ctx, cm_status status, const std::string &message) { return fail(ctx, status, message); }

int cm_internal_set_sharing(cm_ctx *ctx, int on) {
    const int before = ctx->share ? 1 : 0;
    ctx->share = on != 0;
    return before;
}

int cm_internal_grid_devices(const cm_ctx *ctx) { return ctx && ctx->has_profile ? ctx->hp.n_dp * ctx->hp.n_pp : 0; }

cm_status cm_internal_space_view(cm_ctx *ctx, const cm_space *space, SpaceView *out) {
    if (!space || space->ctx != ctx) return fail(ctx, CM_EINVAL, "space does not belong to this context");
    Batch &bt = const_cast<Batch &>(space->batch);
    if (stale(ctx, bt)) return fail(ctx, CM_EINVAL, kStaleMsg);
    out->tb = tables(ctx, bt);
    out->bd = dev_view(ctx, bt);
    out->n_cand = space->policy == CM_DYNPAR ? bt.n_cand : 1;
    out->stream = ctx->stream;
    out->device = ctx->device;
    out->policy = space->policy;
    return CM_OK;
}

// ------------------------------------------------------------------------- C ABI
extern "C" {

const char *cm_strerror(cm_status s) {
    switch (s) {
    case CM_OK: return "ok";
    case CM_EINVAL: return "invalid argument";
    case CM_ENOPROFILE: return "no profile loaded";
    case CM_EOVERFLOW: return "count overflows the index type";
    case CM_ENOFEASIBLE: return "no feasible plan";
    case CM_ECUDA: return "CUDA error";
    case CM_ENOMEM: return "out of memory";
    case CM_ETIMEOUT: return "timeout";
    }
    return "unknown status";
}

const char *cm_last_error(const cm_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

cm_status cm_create(cm_ctx **out, int cuda_device, void *cuda_stream) {
    if (!out) return CM_EINVAL;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || cuda_device < 0 || cuda_device >= n) { cudaGetLastError(); return CM_ECUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess) { cudaGetLastError(); return CM_ECUDA; }
    if (prop.major != 10) return CM_ECUDA;   // kernels are built for sm_100a only; no fallback
    if (cudaSetDevice(cuda_device) != cudaSuccess) { cudaGetLastError(); return CM_ECUDA; }
    cm_ctx *c = new (std::nothrow) cm_ctx();
    if (!c) return CM_ENOMEM;
    c->device = cuda_device;
    c->stream = (cudaStream_t)cuda_stream;
    bool ok = true;
    for (int i = 0; i < 6; ++i) ok = ok && cudaEventCreate(&c->ev[i]) == cudaSuccess;
    for (int i = 0; i < 5; ++i) ok = ok && cudaEventCreate(&c->ev_obj[i]) == cudaSuccess;
    if (cudaStreamCreateWithFlags(&c->graph_stream, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); c->graph_stream = nullptr; }
    if (cudaStreamCreateWithFlags(&c->pol_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->pol_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->pol_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        if (c->pol_stream) cudaStreamDestroy(c->pol_stream);
        c->pol_stream = nullptr;
    }
    ok = ok && cudaEventCreateWithFlags(&c->side.fork, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < kSideStreams && ok; ++i) {
        ok = cudaStreamCreateWithFlags(&c->side.stream[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->side.join[i], cudaEventDisableTiming) == cudaSuccess;
        if (ok) c->side.n = i + 1;
    }
    ok = ok && c->d_scratch.reserve(sizeof(cm_plan *) * 64 + sizeof(cm_plan));   // what cm_select needs
    // the feasible-composition pool and its staging are allocated here, not at the first search:
    // a pinned allocation costs milliseconds, which a failure handler should not pay
    ok = ok && c->d_feas.reserve(1u << 20) && c->feas_stage.reserve(1u << 16) && c->d_feas_stage.reserve(1u << 16);
    if (!ok || cudaMalloc((void **)&c->d_prof, sizeof(DevProfile)) != cudaSuccess ||
        cudaMalloc((void **)&c->d_prof53, sizeof(DevProfile)) != cudaSuccess) {
        if (c->d_prof) cudaFree(c->d_prof);
        cudaGetLastError();
        delete c;
        return CM_ECUDA;
    }
    *out = c;
    return CM_OK;
}

cm_status cm_destroy(cm_ctx *c) {
    if (!c) return CM_EINVAL;
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    for (int i = 0; i < 6; ++i)
        if (c->ev[i]) cudaEventDestroy(c->ev[i]);
    for (int i = 0; i < 5; ++i)
        if (c->ev_obj[i]) cudaEventDestroy(c->ev_obj[i]);
    c->single.clear();
    if (c->graph_stream) cudaStreamDestroy(c->graph_stream);
    if (c->pol_stream) { cudaStreamSynchronize(c->pol_stream); cudaStreamDestroy(c->pol_stream); }
    if (c->pol_fork) cudaEventDestroy(c->pol_fork);
    if (c->pol_join) cudaEventDestroy(c->pol_join);
    for (int i = 0; i < kSideStreams; ++i) {
        if (c->side.stream[i]) { cudaStreamSynchronize(c->side.stream[i]); cudaStreamDestroy(c->side.stream[i]); }
        if (c->side.join[i]) cudaEventDestroy(c->side.join[i]);
    }
    if (c->side.fork) cudaEventDestroy(c->side.fork);
    if (c->d_prof) cudaFree(c->d_prof);
    if (c->d_prof53) cudaFree(c->d_prof53);
    if (c->d_binom) cudaFree(c->d_binom);
    for (int i = 0; i < cm_ctx::kMmTables; ++i)
        if (c->d_mm[i]) cudaFree(c->d_mm[i]);
    delete c;
    return CM_OK;
}

// Host half of cm_load_profile: validation, the host copy of the profile, the binomial table,
// the bound that decides the arithmetic of the integer mode.  No CUDA call.
static cm_status load_profile_host(cm_ctx *ctx, const cm_profile *p) {
    if (!p) return fail(ctx, CM_EINVAL, "profile is NULL");
    if (p->L < 1 || p->L > CM_MAX_LAYERS) return fail(ctx, CM_EINVAL, "L out of range");
    if (p->n_pp < 1 || p->n_pp > std::min(p->L, CM_MAX_STAGES)) return fail(ctx, CM_EINVAL, "n_pp out of range");
    if (p->n_dp < 1 || p->n_dp > CM_MAX_PIPES) return fail(ctx, CM_EINVAL, "n_dp out of range");
    if (p->n_micro < 1 || (int64_t)p->n_dp * p->n_micro > CM_MAX_MICRO) return fail(ctx, CM_EINVAL, "n_micro out of range");
    if (!p->fwd_ns || !p->bwd_ns || !p->fwd_ns_i || !p->bwd_ns_i || !p->act_bytes || !p->param_bytes ||
        !p->opt_bytes || !p->p2p_bytes || !p->base_cuts)
        return fail(ctx, CM_EINVAL, "profile array is NULL");
    if (p->mem_capacity_bytes <= 0 || p->devices_per_node < 1 || p->bw_intra_Bpns <= 0 || p->bw_inter_Bpns <= 0)
        return fail(ctx, CM_EINVAL, "capacity, devices_per_node and bandwidths must be positive");
    for (int l = 0; l < p->L; ++l) {
        if (!(p->fwd_ns[l] >= 0.0) || !(p->bwd_ns[l] >= 0.0) || !std::isfinite(p->fwd_ns[l]) || !std::isfinite(p->bwd_ns[l]))
            return fail(ctx, CM_EINVAL, "layer times must be finite and non-negative");
        if (p->fwd_ns_i[l] < 0 || p->bwd_ns_i[l] < 0 || p->fwd_ns_i[l] > (1ll << 40) || p->bwd_ns_i[l] > (1ll << 40))
            return fail(ctx, CM_EINVAL, "integer layer times out of range");
        if (p->act_bytes[l] < 0 || p->param_bytes[l] < 0 || p->opt_bytes[l] < 0 || p->p2p_bytes[l] < 0 ||
            p->act_bytes[l] > (1ll << 44) || p->param_bytes[l] > (1ll << 44) || p->opt_bytes[l] > (1ll << 44))
            return fail(ctx, CM_EINVAL, "layer bytes out of range");
    }
    if (p->base_cuts[0] != 0 || p->base_cuts[p->n_pp] != p->L) return fail(ctx, CM_EINVAL, "base_cuts must run from 0 to L");
    for (int i = 0; i < p->n_pp; ++i)
        if (p->base_cuts[i + 1] <= p->base_cuts[i]) return fail(ctx, CM_EINVAL, "base_cuts must be strictly increasing");

    DevProfile &h = ctx->hp;
    memset(&h, 0, sizeof(h));
    h.L = p->L; h.n_dp = p->n_dp; h.n_pp = p->n_pp; h.n_micro = p->n_micro;
    h.devices_per_node = p->devices_per_node;
    h.G = p->n_dp * p->n_micro;
    h.cap = p->mem_capacity_bytes; h.bw_intra = p->bw_intra_Bpns; h.bw_inter = p->bw_inter_Bpns;
    // gradient all-reduce runs over the inter-node tier as soon as the job spans nodes
    h.bw_sync = (p->n_dp * p->n_pp > p->devices_per_node) ? p->bw_inter_Bpns : p->bw_intra_Bpns;
    for (int l = 0; l < p->L; ++l) {
        h.fwd[l] = p->fwd_ns[l]; h.bwd[l] = p->bwd_ns[l];
        h.fwd_i[l] = p->fwd_ns_i[l]; h.bwd_i[l] = p->bwd_ns_i[l];
        h.act[l] = p->act_bytes[l]; h.par[l] = p->param_bytes[l]; h.opt[l] = p->opt_bytes[l]; h.p2p[l] = p->p2p_bytes[l];
    }
    for (int i = 0; i <= p->n_pp; ++i) h.base_cuts[i] = p->base_cuts[i];
    {
        // Largest value the integer mode can form: all work of all micro-batches in sequence
        // (rerouted and redundant load included: at most three times that), every transfer of
        // every micro-batch in sequence, the longest synchronisation.
        double work = 0.0, xfer = 0.0, params = 0.0;
        const double bw_min = (double)std::min(h.bw_intra, h.bw_inter);
        for (int l = 0; l < h.L; ++l) {
            work += (double)h.fwd_i[l] + (double)h.bwd_i[l];
            xfer = std::max(xfer, (double)h.p2p[l] / bw_min);
            params += (double)h.par[l];
        }
        const double bound = 3.0 * h.G * work + 2.0 * h.G * CM_MAX_STAGES * xfer + 2.0 * params / bw_min;
        ctx->exact53 = bound < 4503599627370496.0;   // 2^52
    }
    // saturating Pascal triangle: rows cover layers, stages, pipelines and micro-batches
    const int rows = std::max(CM_MAX_LAYERS, h.G) + 1;
    ctx->binom.assign((size_t)rows * (kBinomCols + 1), 0);
    for (int n = 0; n < rows; ++n)
        for (int k = 0; k <= kBinomCols; ++k) {
            uint64_t v;
            if (k == 0) v = 1;
            else if (n == 0) v = 0;
            else v = sat_add(ctx->binom[(size_t)(n - 1) * (kBinomCols + 1) + k - 1], ctx->binom[(size_t)(n - 1) * (kBinomCols + 1) + k]);
            ctx->binom[(size_t)n * (kBinomCols + 1) + k] = v;
        }
    ctx->binom_rows = rows;
    // min-max partition table, one row per (stages, micro-batches), per cost mode
    ctx->mm_stride_m = h.G + 2;
    const size_t slots = (size_t)CM_MAX_STAGES * ctx->mm_stride_m;
    for (int i = 0; i < cm_ctx::kMmTables; ++i) ctx->mm_done[i].assign(slots, 0);
    return CM_OK;
}

cm_status cm_load_profile(cm_ctx *ctx, const cm_profile *p) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));   // nothing may still read the old profile
    ctx->has_profile = false;
    ++ctx->profile_gen;                                  // spaces and batches of the old profile are refused from here on
    ctx->single.clear();                                 // prepared one-scenario batches describe the old profile
    for (auto &f : ctx->feas) f.clear();                 // so do the feasible-composition lists
    ctx->feas_used = 0;
    cm_status s = load_profile_host(ctx, p);
    if (s != CM_OK) return s;
    DevProfile &h = ctx->hp;
    h.intval = 1;
    CM_CUDA(ctx, cudaMemcpyAsync(ctx->d_prof53, &h, sizeof(h), cudaMemcpyHostToDevice, ctx->stream));
    CM_CUDA(ctx, launch_prefix(ctx->d_prof53, ctx->stream));
    CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));   // the next copy reuses the host image
    h.intval = 0;
    CM_CUDA(ctx, cudaMemcpyAsync(ctx->d_prof, &h, sizeof(h), cudaMemcpyHostToDevice, ctx->stream));
    CM_CUDA(ctx, launch_prefix(ctx->d_prof, ctx->stream));
    if (ctx->d_binom) { cudaFree(ctx->d_binom); ctx->d_binom = nullptr; }
    CM_CUDA(ctx, cudaMalloc((void **)&ctx->d_binom, ctx->binom.size() * sizeof(uint64_t)));
    CM_CUDA(ctx, cudaMemcpyAsync(ctx->d_binom, ctx->binom.data(), ctx->binom.size() * sizeof(uint64_t), cudaMemcpyHostToDevice, ctx->stream));
    const size_t slots = (size_t)CM_MAX_STAGES * ctx->mm_stride_m;
    for (int i = 0; i < cm_ctx::kMmTables; ++i) {
        if (ctx->d_mm[i]) { cudaFree(ctx->d_mm[i]); ctx->d_mm[i] = nullptr; }
        CM_CUDA(ctx, cudaMalloc((void **)&ctx->d_mm[i], slots * (kMaxS + 1)));
        CM_CUDA(ctx, cudaMemsetAsync(ctx->d_mm[i], 0xFF, slots * (kMaxS + 1), ctx->stream));
    }
    CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));   // ctx->hp / binom may change on the next load
    ctx->has_profile = true;
    return CM_OK;
    CM_API_END(ctx)
}

// The descriptor builder alone, for one failure set, without a GPU (no CUDA call is made).
cm_status cm_host_describe(const cm_profile *p, const uint32_t *failed_ids, int32_t n_failed,
                           const cm_enum_opts *opts, uint64_t out[8]) {
    if (!p || !opts || !out || n_failed < 0 || (n_failed > 0 && !failed_ids)) return CM_EINVAL;
    CM_API_BEGIN
    cm_ctx ctx;   // plain host object: nothing here touches the device
    cm_status s = load_profile_host(&ctx, p);
    if (s == CM_OK) s = check_opts(&ctx, opts);
    if (s != CM_OK) return s;
    Batch bt;
    const int32_t offsets[2] = {0, n_failed};
    s = build_batch(&ctx, bt, failed_ids, offsets, 1, *opts, 1u << CM_DYNPAR);
    if (s != CM_OK) return s;
    const Tmpl &tp = bt.tmpl[bt.scen[0].tmpl];
    uint64_t crossings = 0;
    for (uint64_t w : bt.cross) crossings += (uint64_t)__builtin_popcountll(w);
    out[0] = bt.n_cand;
    out[1] = tp.n_strat;
    out[2] = tp.n_tseg;
    out[3] = tp.n_split_total;
    out[4] = (uint64_t)(ctx.hp.n_dp * ctx.hp.n_pp - n_failed);
    out[5] = bt.classes.size();
    out[6] = bt.bucket.size();
    out[7] = crossings;
    return CM_OK;
    CM_API_END(nullptr)
}

cm_status cm_enumerate(cm_ctx *ctx, cm_policy policy, const uint32_t *failed_ids, int32_t n_failed,
                       const cm_enum_opts *opts, cm_space **out, uint64_t *n_candidates) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!ctx->has_profile) return fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (!out) return fail(ctx, CM_EINVAL, "out is NULL");
    if (policy < CM_REROUTE || policy > CM_DYNPAR) return fail(ctx, CM_EINVAL, "bad policy");
    if (n_failed < 0 || (n_failed > 0 && !failed_ids)) return fail(ctx, CM_EINVAL, "bad failure set");
    cm_enum_opts o{};
    if (opts) o = *opts;
    else if (policy == CM_DYNPAR) return fail(ctx, CM_EINVAL, "opts is NULL");
    else { o.dp_lo = o.dp_hi = 1; o.pp_lo = o.pp_hi = 1; o.lm = CM_LAYERS_MINMAX; o.bm = CM_BATCH_REMAINDER; o.cost = CM_COST_FP64; }
    cm_status s = check_opts(ctx, &o);
    if (s != CM_OK) return s;
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    std::unique_ptr<cm_space> sp(new (std::nothrow) cm_space());   // released on every error path, a thrown one included
    if (!sp) return fail(ctx, CM_ENOMEM, "host memory");
    sp->ctx = ctx;
    sp->policy = policy;
    sp->failed.assign(failed_ids, failed_ids + n_failed);
    const int32_t offsets[2] = {0, n_failed};
    s = build_batch(ctx, sp->batch, failed_ids, offsets, 1, o, 1u << policy);
    if (s == CM_OK) s = upload_batch(ctx, sp->batch, nullptr);
    if (s == CM_OK && policy != CM_DYNPAR) {
        // the one candidate of these policies is evaluated right away so that
        // cm_evaluate can hand its cost out
        cudaError_t e = launch_policies(tables(ctx, sp->batch), dev_view(ctx, sp->batch), ctx->hp.n_dp, ctx->stream);
        if (e != cudaSuccess) s = fail(ctx, CM_ECUDA, cudaGetErrorString(e));
    }
    if (s != CM_OK) {
        cudaStreamSynchronize(ctx->stream);
        forget_keys(ctx, sp->batch);
        return s;
    }
    if (n_candidates) *n_candidates = policy == CM_DYNPAR ? sp->batch.n_cand : 1;
    *out = sp.release();
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_space_free(cm_space *sp) {
    if (!sp) return CM_EINVAL;
    cudaSetDevice(sp->ctx->device);
    cudaStreamSynchronize(sp->ctx->stream);   // queued copies still read its host tables
    delete sp;
    return CM_OK;
}

cm_status cm_evaluate(cm_ctx *ctx, const cm_space *space, uint64_t first, uint64_t count,
                      const uint64_t *idx_dev, double *cost_dev, int64_t *cost_ns_dev, uint8_t *feasible_dev) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!space || space->ctx != ctx) return fail(ctx, CM_EINVAL, "space does not belong to this context");
    // one thread per candidate, 128 per block, the block count a 31-bit grid dimension
    if (count > 0x7fffffffull * 128ull) return fail(ctx, CM_EINVAL, "count too large: at most (2^31 - 1) * 128 candidates per call");
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    Batch &bt = const_cast<Batch &>(space->batch);
    if (stale(ctx, bt)) return fail(ctx, CM_EINVAL, kStaleMsg);
    const uint64_t n_cand = space->policy == CM_DYNPAR ? bt.n_cand : 1;
    if (!idx_dev && (first > n_cand || count > n_cand - first)) return fail(ctx, CM_EINVAL, "candidate range out of bounds");
    CM_CUDA(ctx, launch_evaluate(tables(ctx, bt), dev_view(ctx, bt), n_cand,
                                 space->policy == CM_DYNPAR ? -1 : space->policy, first, count, idx_dev,
                                 cost_dev, cost_ns_dev, feasible_dev, ctx->stream));
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_select(cm_ctx *ctx, cm_space *const *spaces, int32_t n_spaces, cm_plan *best) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!spaces || n_spaces < 1 || n_spaces > 64 || !best) return fail(ctx, CM_EINVAL, "bad arguments");
    for (int i = 0; i < n_spaces; ++i) {
        if (!spaces[i] || spaces[i]->ctx != ctx) return fail(ctx, CM_EINVAL, "space does not belong to this context");
        if (stale(ctx, spaces[i]->batch)) return fail(ctx, CM_EINVAL, kStaleMsg);
        if (spaces[i]->batch.opts.cost != spaces[0]->batch.opts.cost) return fail(ctx, CM_EINVAL, "spaces mix cost modes");
    }
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(ctx->stats, 0, sizeof(ctx->stats));
    const int mode = spaces[0]->batch.opts.cost;
    std::vector<const cm_plan *> ptrs(n_spaces);
    for (int i = 0; i < n_spaces; ++i) {
        cm_status s = run_batch(ctx, spaces[i]->batch, 0);
        if (s != CM_OK) return s;
        ptrs[i] = spaces[i]->batch.d_plans.p + spaces[i]->policy;
    }
    // best over the spaces, on the device as well (scratch of the context: 64 pointers and a plan
    // were reserved by cm_create, so this call allocates nothing)
    if (!ctx->d_scratch.reserve(sizeof(cm_plan *) * 64 + sizeof(cm_plan))) return fail(ctx, CM_ENOMEM, "device memory");
    const cm_plan **d_ptrs = reinterpret_cast<const cm_plan **>(ctx->d_scratch.p);
    cm_plan *d_out = reinterpret_cast<cm_plan *>(ctx->d_scratch.p + sizeof(cm_plan *) * 64);
    cm_plan result;
    cudaError_t e = cudaMemcpyAsync(d_ptrs, ptrs.data(), sizeof(cm_plan *) * n_spaces, cudaMemcpyHostToDevice, ctx->stream);
    if (e == cudaSuccess) e = launch_pick(d_ptrs, n_spaces, d_out, mode, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&result, d_out, sizeof(cm_plan), cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ctx, CM_ECUDA, cudaGetErrorString(e)); }
    ctx->stats[3] += 1;
    scrub(result);
    *best = result;
    if (!result.feasible) return fail(ctx, CM_ENOFEASIBLE, "no feasible plan in the given spaces");
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_search_batch(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                          const cm_enum_opts *opts, cm_plan *best_per_scenario, cm_plan *best_per_policy,
                          float *latency_us) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!ctx->has_profile) return fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (B < 0 || !offsets || !best_per_scenario || (offsets[B] > 0 && !failed_ids)) return fail(ctx, CM_EINVAL, "bad arguments");
    cm_status s = check_opts(ctx, opts);
    if (s != CM_OK) return s;
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(ctx->stats, 0, sizeof(ctx->stats));
    if (B == 0) return CM_OK;
    const uint32_t mask = (1u << CM_REROUTE) | (1u << CM_REDUNDANT) | (1u << CM_DYNPAR);
    Batch &bt = ctx->batch;
    auto copy_out = [&](int b_dst, int b_src) {
        for (int pol = 0; pol < 3; ++pol) {
            cm_plan pl = bt.plans_host[(size_t)b_src * 4 + pol];
            scrub(pl);
            if (best_per_policy) best_per_policy[(size_t)b_dst * 3 + pol] = pl;
        }
        cm_plan pl = bt.plans_host[(size_t)b_src * 4 + 3];
        scrub(pl);
        best_per_scenario[b_dst] = pl;
    };
    if (!latency_us) {
        int launches = 0;
        const uint64_t h0 = now_ns();
        if ((s = build_batch(ctx, bt, failed_ids, offsets, B, *opts, mask)) != CM_OK) { forget_keys(ctx, bt); return s; }
        ctx->stats[13] += now_ns() - h0;
        if ((s = upload_batch(ctx, bt, &launches)) != CM_OK) { forget_keys(ctx, bt); return s; }
        if ((s = run_batch(ctx, bt, launches)) != CM_OK) return s;
        for (int b = 0; b < B; ++b) copy_out(b, b);
        return CM_OK;
    }
    for (int b = 0; b < B; ++b) {
        const auto t0 = std::chrono::steady_clock::now();
        int launches = 0;
        const uint64_t h0 = now_ns();
        Batch *sb = nullptr;
        cm_ctx::Single *entry = nullptr;
        if ((s = single_batch(ctx, failed_ids + offsets[b], offsets[b + 1] - offsets[b], *opts, mask, &sb, &launches, &entry)) != CM_OK) return s;
        ctx->stats[13] += now_ns() - h0;
        bool done = false;
        if (ctx->share) {
            const uint64_t h1 = now_ns();
            s = run_single_shared(ctx, *sb, launches, &done);
            if (!done) ctx->stats[13] += now_ns() - h1;   // (the keys were built and found not worth using)
            if (s != CM_OK) return s;
        }
        if (!done && (s = run_batch(ctx, *sb, launches, entry)) != CM_OK) return s;
        for (int pol = 0; pol < 3; ++pol) {
            cm_plan pl = sb->plans_host[pol];
            scrub(pl);
            if (best_per_policy) best_per_policy[(size_t)b * 3 + pol] = pl;
        }
        cm_plan pl = sb->plans_host[3];
        scrub(pl);
        best_per_scenario[b] = pl;
        const auto t1 = std::chrono::steady_clock::now();
        latency_us[b] = (float)std::chrono::duration<double, std::micro>(t1 - t0).count();
    }
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_search_objective(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                              const cm_enum_opts *opts, const cm_objective_opts *objective,
                              cm_plan *best, cm_transition *trans, cm_plan *shortlist, int64_t *shortlist_bytes,
                              int32_t *shortlist_rounds) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!ctx->has_profile) return fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (B < 0 || !offsets || !best || !trans || !objective || (offsets[B] > 0 && !failed_ids))
        return fail(ctx, CM_EINVAL, "bad arguments");
    cm_status s = check_opts(ctx, opts);
    if (s != CM_OK) return s;
    const cm_objective_opts &q = *objective;
    if (q.topk < 1 || q.topk > CM_MAX_SHORTLIST) return fail(ctx, CM_EINVAL, "topk must be 1 .. CM_MAX_SHORTLIST");
    if (q.bw_xfer_Bpns <= 0) return fail(ctx, CM_EINVAL, "transfer bandwidth must be positive");
    if (q.sync_rounds != 0 && q.sync_rounds != 1) return fail(ctx, CM_EINVAL, "sync_rounds must be 0 or 1");
    if (!(q.t_gap_ns > 0.0) || !std::isfinite(q.t_gap_ns) || !(q.t_restart_ns >= 0.0) || !std::isfinite(q.t_restart_ns) ||
        q.t_gap_ns_i <= 0 || q.t_restart_ns_i < 0 || q.t_gap_ns_i > (1ll << 60) || q.t_restart_ns_i > (1ll << 60))
        return fail(ctx, CM_EINVAL, "fault gap must be positive and finite, restart overhead non-negative");
    if (ctx->hp.n_dp * ctx->hp.n_pp > CM_MAX_MATCH) return fail(ctx, CM_EINVAL, "more than CM_MAX_MATCH devices");
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(ctx->stats, 0, sizeof(ctx->stats));
    memset(ctx->obj_stats, 0, sizeof(ctx->obj_stats));
    if (B == 0) return CM_OK;
    const uint32_t mask = (1u << CM_REROUTE) | (1u << CM_REDUNDANT) | (1u << CM_DYNPAR);
    Batch &bt = ctx->batch;
    int launches = 0;
    const uint64_t h0 = now_ns();
    if ((s = build_batch(ctx, bt, failed_ids, offsets, B, *opts, mask)) != CM_OK) { forget_keys(ctx, bt); return s; }
    ctx->stats[13] += now_ns() - h0;
    if ((s = upload_batch(ctx, bt, &launches)) != CM_OK) { forget_keys(ctx, bt); return s; }
    if ((s = run_batch(ctx, bt, launches)) != CM_OK) return s;

    // the objective pass works on what the search left on the device
    const size_t slots = (size_t)B * q.topk;
    bool ok = bt.d_short_win.reserve(slots) && bt.d_short_kappa.reserve(slots * kMaxP) && bt.d_short_bytes.reserve(slots) &&
              bt.d_short_assign.reserve(slots * kMaxMatch) && bt.d_short_plans.reserve(slots) &&
              bt.d_short_step.reserve(slots * 2) && bt.d_short_rounds.reserve(slots * 2) &&
              bt.d_obj_best.reserve(B) && bt.d_trans.reserve(B);
    if (!ok) return fail(ctx, CM_ENOMEM, "device memory");
    ok = bt.obj_best_host.resize(B) && bt.trans_host.resize(B) && bt.short_plans_host.resize(slots) &&
         bt.short_bytes_host.resize(slots) && bt.short_rounds_host.resize(slots * 2);
    if (!ok) return fail(ctx, CM_ENOMEM, "host memory");
    const Tables tb = tables(ctx, bt);
    const BatchDev bd = dev_view(ctx, bt);
    ObjDev od{};
    od.topk = q.topk;
    od.sync_rounds = q.sync_rounds;
    od.short_step = bt.d_short_step.p; od.short_rounds = bt.d_short_rounds.p;
    od.t_gap = q.t_gap_ns; od.t_restart = q.t_restart_ns;
    od.t_gap_i = q.t_gap_ns_i; od.t_restart_i = q.t_restart_ns_i; od.bw_xfer = q.bw_xfer_Bpns;
    od.short_win = bt.d_short_win.p; od.short_kappa = bt.d_short_kappa.p; od.short_bytes = bt.d_short_bytes.p;
    od.short_assign = bt.d_short_assign.p; od.short_plans = shortlist ? bt.d_short_plans.p : nullptr;
    od.best = bt.d_obj_best.p; od.trans = bt.d_trans.p;
    cudaStream_t st = ctx->stream;
    int obj_launches = 0;
    CM_CUDA(ctx, cudaEventRecord(ctx->ev_obj[0], st));
    CM_CUDA(ctx, launch_shortlist(tb, bd, od, st));
    ++obj_launches;
    CM_CUDA(ctx, cudaEventRecord(ctx->ev_obj[1], st));
    if (bt.n_tiles) {
        // the tie-break kernels complete every shortlisted pair exactly as they complete the winner
        BatchDev sd = bd;
        sd.winner = od.short_win;
        sd.kappa_sel = od.short_kappa;
        sd.B = (int32_t)slots;
        CM_CUDA(ctx, launch_cost_pass2(tb, sd, st));
        ++obj_launches;
        uint64_t stage_mask = 0;
        for (const TSeg &g : bt.tseg) stage_mask |= 1ull << (g.S & 63);
        CM_CUDA(ctx, launch_tiebreak_wide(tb, sd, stage_mask, st, &ctx->side, &obj_launches));
    }
    CM_CUDA(ctx, cudaEventRecord(ctx->ev_obj[2], st));
    CM_CUDA(ctx, launch_plan_matching(tb, bd, od, st));
    ++obj_launches;
    if (q.sync_rounds) {
        CM_CUDA(ctx, launch_plan_rounds(tb, bd, od, st));
        ++obj_launches;
    }
    CM_CUDA(ctx, cudaEventRecord(ctx->ev_obj[3], st));
    CM_CUDA(ctx, launch_objective(tb, bd, od, st));
    ++obj_launches;
    CM_CUDA(ctx, cudaEventRecord(ctx->ev_obj[4], st));
    size_t back = 0;
    CM_CUDA(ctx, cudaMemcpyAsync(bt.obj_best_host.p, bt.d_obj_best.p, sizeof(cm_plan) * B, cudaMemcpyDeviceToHost, st));
    CM_CUDA(ctx, cudaMemcpyAsync(bt.trans_host.p, bt.d_trans.p, sizeof(cm_transition) * B, cudaMemcpyDeviceToHost, st));
    back += (sizeof(cm_plan) + sizeof(cm_transition)) * (size_t)B;
    if (shortlist) {
        CM_CUDA(ctx, cudaMemcpyAsync(bt.short_plans_host.p, bt.d_short_plans.p, sizeof(cm_plan) * slots, cudaMemcpyDeviceToHost, st));
        back += sizeof(cm_plan) * slots;
    }
    if (shortlist_bytes) {
        CM_CUDA(ctx, cudaMemcpyAsync(bt.short_bytes_host.p, bt.d_short_bytes.p, sizeof(int64_t) * slots, cudaMemcpyDeviceToHost, st));
        back += sizeof(int64_t) * slots;
    }
    if (shortlist_rounds && q.sync_rounds) {
        CM_CUDA(ctx, cudaMemcpyAsync(bt.short_rounds_host.p, bt.d_short_rounds.p, sizeof(int32_t) * 2 * slots, cudaMemcpyDeviceToHost, st));
        back += sizeof(int32_t) * 2 * slots;
    }
    CM_CUDA(ctx, cudaStreamSynchronize(st));
    for (int i = 0; i < 4; ++i) {
        float ms = 0.f;
        CM_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev_obj[i], ctx->ev_obj[i + 1]));
        ctx->obj_stats[i] = (uint64_t)((double)ms * 1e6);
        ctx->obj_stats[7] += ctx->obj_stats[i];
    }
    ctx->obj_stats[5] = (uint64_t)obj_launches;
    ctx->obj_stats[6] = back;
    for (int b = 0; b < B; ++b) {
        cm_plan pl = bt.obj_best_host[b];
        scrub(pl);
        best[b] = pl;
        trans[b] = bt.trans_host[b];
        if (!pl.feasible) trans[b].feasible = 0;
    }
    uint64_t solved = 0;
    for (size_t i = 0; i < slots; ++i) {
        if (shortlist) { cm_plan pl = bt.short_plans_host[i]; scrub(pl); shortlist[i] = pl; }
        if (shortlist_bytes) { shortlist_bytes[i] = bt.short_bytes_host[i]; solved += bt.short_bytes_host[i] >= 0; }
        if (shortlist_rounds) shortlist_rounds[i] = q.sync_rounds ? bt.short_rounds_host[i * 2] : 0;
    }
    ctx->obj_stats[4] = solved;
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_set_int64_arithmetic(cm_ctx *ctx, int native) {
    if (!ctx) return CM_EINVAL;
    ctx->force_native_i64 = native != 0;
    return CM_OK;
}

int cm_int64_runs_in_fp64(const cm_ctx *ctx) {
    return ctx && ctx->has_profile && ctx->exact53 && !ctx->force_native_i64 ? 1 : 0;
}

cm_status cm_set_latency_graphs(cm_ctx *ctx, int on) {
    if (!ctx) return CM_EINVAL;
    ctx->use_graphs = on != 0;
    return CM_OK;
}

cm_status cm_set_memory_screen(cm_ctx *ctx, int on) {
    if (!ctx) return CM_EINVAL;
    ctx->screen = on != 0;
    return CM_OK;
}

cm_status cm_set_micro_batch_pairs(cm_ctx *ctx, int on) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if ((on != 0) != ctx->pairs) {
        // resident one-scenario batches were laid out under the other setting
        if (ctx->stream) cudaStreamSynchronize(ctx->stream);
        ctx->single.clear();
    }
    ctx->pairs = on != 0;
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_set_pipeline_reuse(cm_ctx *ctx, int on) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if ((on != 0) != ctx->dedup) {
        // resident one-scenario batches were laid out under the other setting
        if (ctx->stream) cudaStreamSynchronize(ctx->stream);
        ctx->single.clear();
    }
    ctx->dedup = on != 0;
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_set_sharing(cm_ctx *ctx, int on) {
    if (!ctx) return CM_EINVAL;
    cm_internal_set_sharing(ctx, on);
    return CM_OK;
}

cm_status cm_transition_time(const cm_objective_opts *objective, int32_t n, const int64_t *xfer_bytes,
                             double *t_trans_ns, int64_t *t_trans_ns_i) {
    if (!objective || n < 0 || (n > 0 && !xfer_bytes) || objective->bw_xfer_Bpns <= 0) return CM_EINVAL;
    for (int i = 0; i < n; ++i) {
        const bool used = xfer_bytes[i] >= 0;   // -1 marks an empty shortlist slot
        if (t_trans_ns) t_trans_ns[i] = used ? transition_time_f64(objective->t_restart_ns, xfer_bytes[i], objective->bw_xfer_Bpns) : -1.0;
        if (t_trans_ns_i) t_trans_ns_i[i] = used ? transition_time_i64(objective->t_restart_ns_i, xfer_bytes[i], objective->bw_xfer_Bpns) : -1;
    }
    return CM_OK;
}

cm_status cm_objective_stats(const cm_ctx *ctx, uint64_t out[8]) {
    if (!ctx || !out) return CM_EINVAL;
    memcpy(out, ctx->obj_stats, sizeof(ctx->obj_stats));
    return CM_OK;
}

cm_status cm_transfer_matching(cm_ctx *ctx, int32_t n_problems, const int32_t *sizes, const uint8_t *old_lo,
                               const uint8_t *old_hi, const uint8_t *new_lo, const uint8_t *new_hi,
                               int64_t *total, uint16_t *assign) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!ctx->has_profile) return fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (n_problems < 0 || (n_problems > 0 && (!sizes || !old_lo || !old_hi || !new_lo || !new_hi || !total)))
        return fail(ctx, CM_EINVAL, "bad arguments");
    if (n_problems == 0) return CM_OK;
    const int L = ctx->hp.L;
    for (int q = 0; q < n_problems; ++q) {
        if (sizes[q] < 1 || sizes[q] > CM_MAX_MATCH) return fail(ctx, CM_EINVAL, "problem size must be 1 .. CM_MAX_MATCH");
        for (int j = 0; j < sizes[q]; ++j) {
            const size_t i = (size_t)q * CM_MAX_MATCH + j;
            if (old_lo[i] > L || old_hi[i] > L || new_lo[i] > L || new_hi[i] > L) return fail(ctx, CM_EINVAL, "layer index above L");
        }
    }
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    const size_t rows = (size_t)n_problems * CM_MAX_MATCH;
    const size_t off_sizes = 0, off_rng = ((size_t)n_problems * sizeof(int32_t) + 15) & ~(size_t)15;
    const size_t off_total = (off_rng + 4 * rows + 15) & ~(size_t)15, off_assign = off_total + (size_t)n_problems * sizeof(int64_t);
    const size_t bytes = off_assign + rows * sizeof(uint16_t);
    // scratch of the context: allocated when a call needs more than any call before it, kept afterwards
    CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));   // growing frees the old block: nothing may still use it
    if (!ctx->d_scratch.reserve(bytes)) return fail(ctx, CM_ENOMEM, "device memory");
    unsigned char *d = ctx->d_scratch.p;
    cudaStream_t st = ctx->stream;
    cudaError_t e = cudaMemcpyAsync(d + off_sizes, sizes, (size_t)n_problems * sizeof(int32_t), cudaMemcpyHostToDevice, st);
    const uint8_t *src[4] = {old_lo, old_hi, new_lo, new_hi};
    for (int a = 0; a < 4 && e == cudaSuccess; ++a)
        e = cudaMemcpyAsync(d + off_rng + a * rows, src[a], rows, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = launch_range_matching(tables_plain(ctx), n_problems, (const int32_t *)(d + off_sizes), d + off_rng,
                                  d + off_rng + rows, d + off_rng + 2 * rows, d + off_rng + 3 * rows,
                                  (int64_t *)(d + off_total), (uint16_t *)(d + off_assign), st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(total, d + off_total, (size_t)n_problems * sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && assign) e = cudaMemcpyAsync(assign, d + off_assign, rows * sizeof(uint16_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(ctx, CM_ECUDA, cudaGetErrorString(e)); }
    for (int q = 0; q < n_problems; ++q)
        if (total[q] < 0) return fail(ctx, CM_ECUDA, "matching iteration did not terminate");
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_batch_prepare(cm_ctx *ctx, const uint32_t *failed_ids, const int32_t *offsets, int32_t B,
                           const cm_enum_opts *opts, cm_batch **out, uint64_t *n_candidates) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!ctx->has_profile) return fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (B < 0 || !offsets || !out || (offsets[B] > 0 && !failed_ids)) return fail(ctx, CM_EINVAL, "bad arguments");
    cm_status s = check_opts(ctx, opts);
    if (s != CM_OK) return s;
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    std::unique_ptr<cm_batch> bp(new (std::nothrow) cm_batch());
    if (!bp) return fail(ctx, CM_ENOMEM, "host memory");
    bp->ctx = ctx;
    memset(ctx->stats, 0, sizeof(ctx->stats));
    const uint32_t mask = (1u << CM_REROUTE) | (1u << CM_REDUNDANT) | (1u << CM_DYNPAR);
    s = build_batch(ctx, bp->batch, failed_ids, offsets, B, *opts, mask);
    if (s == CM_OK) s = upload_batch(ctx, bp->batch, &bp->prep_launches);
    if (s != CM_OK) {
        cudaStreamSynchronize(ctx->stream);
        forget_keys(ctx, bp->batch);
        return s;
    }
    if (n_candidates) *n_candidates = bp->batch.n_cand;
    *out = bp.release();
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_batch_search(cm_ctx *ctx, cm_batch *bp, cm_plan *best_per_scenario, cm_plan *best_per_policy) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!bp || bp->ctx != ctx || !best_per_scenario) return fail(ctx, CM_EINVAL, "bad arguments");
    if (stale(ctx, bp->batch)) return fail(ctx, CM_EINVAL, kStaleMsg);
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(ctx->stats, 0, sizeof(ctx->stats));
    Batch &bt = bp->batch;
    if (bt.B == 0) return CM_OK;
    cm_status s = run_batch(ctx, bt, 0);
    if (s != CM_OK) return s;
    for (int b = 0; b < bt.B; ++b) {
        for (int pol = 0; pol < 3 && best_per_policy; ++pol) {
            cm_plan pl = bt.plans_host[(size_t)b * 4 + pol];
            scrub(pl);
            best_per_policy[(size_t)b * 3 + pol] = pl;
        }
        cm_plan pl = bt.plans_host[(size_t)b * 4 + 3];
        scrub(pl);
        best_per_scenario[b] = pl;
    }
    return CM_OK;
    CM_API_END(ctx)
}

cm_status cm_batch_free(cm_batch *bp) {
    if (!bp) return CM_EINVAL;
    cudaSetDevice(bp->ctx->device);
    cudaStreamSynchronize(bp->ctx->stream);
    delete bp;
    return CM_OK;
}

cm_status cm_last_stats(const cm_ctx *ctx, uint64_t out[24]) {
    if (!ctx || !out) return CM_EINVAL;
    memcpy(out, ctx->stats, sizeof(ctx->stats));
    return CM_OK;
}

cm_status cm_decode_plan(cm_ctx *ctx, const cm_space *space, const cm_plan *plan, int32_t *cuts_out) {
    if (!ctx) return CM_EINVAL;
    CM_API_BEGIN
    if (!space || space->ctx != ctx || !plan || !cuts_out) return fail(ctx, CM_EINVAL, "bad arguments");
    if (stale(ctx, space->batch)) return fail(ctx, CM_EINVAL, kStaleMsg);
    if (plan->policy != space->policy) return fail(ctx, CM_EINVAL, "plan was not found in this space");
    const DevProfile &hp = ctx->hp;
    CM_CUDA(ctx, cudaSetDevice(ctx->device));
    std::vector<int32_t> cuts;
    if (space->policy != CM_DYNPAR) {
        const int S0 = hp.n_pp;
        for (int k = 0; k < hp.n_dp; ++k) {
            std::vector<char> dead(S0, 0);
            if (space->policy == CM_REDUNDANT)
                for (uint32_t d : space->failed)
                    if ((int)(d / S0) == k) dead[d % S0] = 1;
            cuts.push_back(0);
            for (int i = 0; i < S0; ++i) {
                if (dead[i]) continue;
                int hi = hp.base_cuts[i + 1];
                if (i + 1 < S0 && dead[i + 1]) hi = hp.base_cuts[i + 2];
                cuts.push_back(hi);
            }
        }
    } else {
        const Batch &bt = space->batch;
        const Tmpl &tp = bt.tmpl[bt.scen[0].tmpl];
        if (plan->strategy >= tp.n_strat) return fail(ctx, CM_EINVAL, "strategy index out of range");
        const Strat &st = bt.strat[tp.strat_first + plan->strategy];
        if (plan->n_pipes != st.dp) return fail(ctx, CM_EINVAL, "plan does not match its strategy");
        for (int p = 0; p < st.dp; ++p) {
            const int S = st.S[p], L = hp.L;
            const int off = (int)plan->micro[p] - (int)st.m_lo[p];
            if (plan->stages[p] != S || off < 0 || off >= st.n_m) return fail(ctx, CM_EINVAL, "plan does not match its strategy");
            const TSeg &g = bt.tseg[st.seg_first + p * st.n_m + off];
            const uint64_t kappa = plan->kappa[p];
            if (kappa > g.K) return fail(ctx, CM_EINVAL, "layer composition rank out of range");
            if (kappa < g.K) {
                // combinadic unranking, the same rule the kernels apply
                auto unrank = [&](uint64_t rank, int n, int t, std::vector<int> &c) {
                    c.assign(t, 0);
                    int v = n;
                    for (int u = t; u >= 1; --u) {
                        uint64_t b;
                        do { --v; b = hbinom(ctx, v, u); } while (b > rank);
                        rank -= b;
                        c[u - 1] = v;
                    }
                };
                std::vector<int> c;
                cuts.push_back(0);
                if (bt.opts.lm == CM_LAYERS_REMAINDER) {
                    unrank(kappa, S, L % S, c);
                    std::vector<char> extra(S, 0);
                    for (int v : c) extra[v] = 1;
                    int acc = 0;
                    for (int i = 0; i < S; ++i) { acc += L / S + extra[i]; cuts.push_back(acc); }
                } else {
                    unrank(kappa, L - 1, S - 1, c);
                    for (int i = 0; i < S - 1; ++i) cuts.push_back(c[i] + 1);
                    cuts.push_back(L);
                }
            } else {
                uint8_t row[kMaxS + 1];
                CM_CUDA(ctx, cudaMemcpyAsync(row, ctx->d_mm[cm_ctx::mm_index(bt.opts)] + ((size_t)(S - 1) * ctx->mm_stride_m + g.m) * (kMaxS + 1), kMaxS + 1,
                                             cudaMemcpyDeviceToHost, ctx->stream));
                CM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
                if (row[0] != 0) return fail(ctx, CM_EINVAL, "min-max partition of this pipeline is infeasible");
                for (int i = 0; i <= S; ++i) cuts.push_back(row[i]);
            }
        }
    }
    memcpy(cuts_out, cuts.data(), cuts.size() * sizeof(int32_t));
    return CM_OK;
    CM_API_END(ctx)
}

}  // extern "C"
