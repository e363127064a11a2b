// Device-side building blocks of the plan search: numeric traits for the two cost
// modes, the shared-memory copy of the profile, combinadic unranking, the per-stage
// sums with the memory check, and the 1F1B start/end recurrence.
#pragma once

#include <type_traits>

#include "cm_internal.h"

namespace cm {

// ----------------------------------------------------------------------------------
// Cost arithmetic.  T = double: IEEE, one rounding per written operation (compile with
// --fmad=false).  T = long long: integer nanoseconds, divisions floor.  Costs are never
// negative, so their 64-bit patterns order like the values and a plain unsigned
// atomicMin implements "least cost"; infeasible is +inf / INT64_MAX.
// ----------------------------------------------------------------------------------
template <typename T> struct Num;

template <> struct Num<double> {
    static __device__ __forceinline__ double inf() { return __longlong_as_double(0x7FF0000000000000LL); }
    static __device__ __forceinline__ uint64_t bits(double x) { return (uint64_t)__double_as_longlong(x); }
    static __device__ __forceinline__ double from_bits(uint64_t b) { return __longlong_as_double((long long)b); }
    static __device__ __forceinline__ const double *PF(const DevProfile *p) { return p->PFd; }
    static __device__ __forceinline__ const double *PB(const DevProfile *p) { return p->PBd; }
    static __device__ __forceinline__ const double *XT(const DevProfile *p, int tier) { return p->XTd[tier]; }
    // intval: the values are integer nanoseconds held in doubles; quotients floor as in the
    // integer mode (sums and maxima of such values are exact below 2^53)
    static __device__ __forceinline__ double sync(int64_t G, int n, int64_t bw, int intval) {
        if (n <= 1) return 0.0;
        if (intval) return (double)((2LL * (long long)(n - 1) * (long long)G) / ((long long)n * (long long)bw));
        return ((2.0 * (double)(n - 1)) * (double)G) / ((double)n * (double)bw);
    }
    static __device__ __forceinline__ double reroute_extra(int mF, double fb, int peers, int intval) {
        if (intval) return (double)(((long long)mF * (long long)fb) / (long long)peers);
        return ((double)mF * fb) / (double)peers;
    }
};

template <> struct Num<long long> {
    static __device__ __forceinline__ long long inf() { return 0x7FFFFFFFFFFFFFFFLL; }
    static __device__ __forceinline__ uint64_t bits(long long x) { return (uint64_t)x; }
    static __device__ __forceinline__ long long from_bits(uint64_t b) { return (long long)b; }
    static __device__ __forceinline__ const long long *PF(const DevProfile *p) { return (const long long *)p->PFi; }
    static __device__ __forceinline__ const long long *PB(const DevProfile *p) { return (const long long *)p->PBi; }
    static __device__ __forceinline__ const long long *XT(const DevProfile *p, int tier) { return (const long long *)p->XTi[tier]; }
    static __device__ __forceinline__ long long sync(int64_t G, int n, int64_t bw, int) {
        if (n <= 1) return 0;
        return (2LL * (long long)(n - 1) * (long long)G) / ((long long)n * (long long)bw);
    }
    static __device__ __forceinline__ long long reroute_extra(int mF, long long fb, int peers, int) {
        return ((long long)mF * fb) / (long long)peers;
    }
};

constexpr uint64_t kInfBitsF64 = 0x7FF0000000000000ull;
constexpr uint64_t kInfBitsI64 = 0x7FFFFFFFFFFFFFFFull;
// "infeasible" in the bit patterns a batch carries on the device
__host__ __device__ __forceinline__ uint64_t batch_inf_bits(const BatchDev &b) {
    return (b.mode == CM_COST_INT64NS && !b.intval) ? kInfBitsI64 : kInfBitsF64;
}
// integer nanoseconds of a cost bit pattern of a batch in integer mode
__device__ __forceinline__ int64_t batch_cost_ns(const BatchDev &b, uint64_t bits) {
    if (!b.intval) return (int64_t)bits;
    return bits >= kInfBitsF64 ? (int64_t)kInfBitsI64 : (int64_t)__longlong_as_double((long long)bits);
}
template <typename T> __device__ __forceinline__ uint64_t inf_bits() { return Num<T>::bits(Num<T>::inf()); }

template <typename T> __device__ __forceinline__ T tmax(T a, T b) { return a > b ? a : b; }

// ----------------------------------------------------------------------------------
// Profile in shared memory: prefix sums over layers, so that any stage [lo,hi) costs a
// subtraction per quantity (Section "Estimator": stage quantities are sums over layers).
// ----------------------------------------------------------------------------------
template <typename T> struct SProf {
    T PF[kMaxL + 1], PB[kMaxL + 1];
    long long PA[kMaxL + 1], PS[kMaxL + 1], PP[kMaxL + 1];
    T XT[2][kMaxL];
    long long cap, bw_sync;
    int L, n_dp, n_pp, n_micro;
    int intval, sched;   // sched: order of the computations on a stage (cm_schedule), an option carried along
};

template <typename T>
__device__ __forceinline__ void stage_profile(SProf<T> &s, const Tables &tb) {
    const DevProfile *p = tb.prof;
    const int L = p->L;
    for (int l = threadIdx.x; l <= L; l += blockDim.x) {
        s.PF[l] = Num<T>::PF(p)[l];
        s.PB[l] = Num<T>::PB(p)[l];
        s.PA[l] = p->PA[l];
        s.PS[l] = p->PS[l];
        s.PP[l] = p->PP[l];
        if (l < L) {
            s.XT[0][l] = Num<T>::XT(p, 0)[l];
            s.XT[1][l] = Num<T>::XT(p, 1)[l];
        }
    }
    if (threadIdx.x == 0) {
        s.cap = p->cap;
        s.bw_sync = p->bw_sync;
        s.L = L;
        s.n_dp = p->n_dp;
        s.n_pp = p->n_pp;
        s.n_micro = p->n_micro;
        s.intval = p->intval;
        s.sched = tb.sched;
    }
}

// ----------------------------------------------------------------------------------
// Combinatorial number system (colex): rank = sum_u C(c_u, u).  Greedy unranking from
// the largest element; the scan position only moves down, so it costs O(n + t) lookups.
// ----------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t binom_at(const uint64_t *tab, int n, int k) {
    return tab[n * (kBinomCols + 1) + k];
}

// Calls emit(u-1, v) for u = t..1 with v the u-th smallest element (0-based position u-1).
template <typename Emit>
__device__ __forceinline__ void unrank_subset(const uint64_t *tab, uint64_t rank, int n, int t, Emit emit) {
    int v = n;
    for (int u = t; u >= 1; --u) {
        uint64_t c;
        do {
            --v;
            c = binom_at(tab, v, u);
        } while (c > rank);
        rank -= c;
        emit(u - 1, v);
    }
}

// Layer cuts of composition kappa (Section "Planner", layer distribution).
__device__ __forceinline__ void layer_cuts(const uint64_t *tab, int layer_mode, int L, int S,
                                           uint64_t kappa, uint8_t *cuts /* [S+1] */) {
    cuts[0] = 0;
    if (layer_mode == CM_LAYERS_REMAINDER) {
        const int q = L / S, r = L % S;
        uint64_t extra = 0;
        unrank_subset(tab, kappa, S, r, [&](int, int v) { extra |= 1ull << v; });
        int c = 0;
        for (int i = 0; i < S; ++i) {
            c += q + (int)((extra >> i) & 1ull);
            cuts[i + 1] = (uint8_t)c;
        }
    } else {
        unrank_subset(tab, kappa, L - 1, S - 1, [&](int pos, int v) { cuts[pos + 1] = (uint8_t)(v + 1); });
        cuts[S] = (uint8_t)L;
    }
}

// ----------------------------------------------------------------------------------
// Pipeline time by the start/end recurrence (Section "Estimator", the transition
// equation) under the non-interleaved 1F1B order, thread-sequential with O(S) state.
//
// Evaluation order (any order that respects the dependencies gives the same values):
//   phase 1  warm-up forwards, micro-batch by micro-batch, each running up the stages
//            that still have a warm-up slot for it; the last one of a row is left
//            pending for the stage above, whose first steady forward it feeds;
//   phase 2  round k = 0..m-1, stages from last to first: the stage's next forward (if
//            any is left) fed by the pending forward of the stage below, then its k-th
//            backward fed by the k-th backward of the stage above (by its own forward at
//            the last stage).
// State per stage: clock (end of its latest computation) and pend (end of the forward
// it has not consumed yet, transfer included).  xt[i] is the transfer time of the
// boundary between stages i and i+1.
// ----------------------------------------------------------------------------------
// Under the all-forward-all-backward order (sched = CM_SCHED_GPIPE) the forwards run
// micro-batch by micro-batch up the stages, then the backwards micro-batch by micro-batch
// down the stages; the only state is the per-stage clock.
template <typename T>
__device__ __forceinline__ T sim_pipe(int S, int m, const T *F, const T *B, const T *xt, T *clock, T *pend, int sched) {
    for (int i = 0; i < S; ++i) clock[i] = (T)0;
    if (sched == CM_SCHED_GPIPE) {
        for (int j = 0; j < m; ++j) {
            T chain = (T)0;
            for (int i = 0; i < S; ++i) {
                const T start = i > 0 ? tmax(clock[i], chain) : clock[i];
                const T end = start + F[i];
                clock[i] = end;
                chain = end + xt[i];
            }
        }
        for (int j = 0; j < m; ++j) {
            T chain_b = (T)0;
            for (int i = S - 1; i >= 0; --i) {
                const T start = i < S - 1 ? tmax(clock[i], chain_b + xt[i]) : clock[i];
                const T end = start + B[i];
                clock[i] = end;
                chain_b = end;
            }
        }
        return clock[0];
    }
    const int n_rows = m < S - 1 ? m : S - 1;
    for (int j = 0; j < n_rows; ++j) {
        T chain = (T)0;
        const int i_max = S - 2 - j;
        for (int i = 0; i <= i_max; ++i) {
            T start = i > 0 ? tmax(clock[i], chain) : clock[i];
            T end = start + F[i];
            clock[i] = end;
            chain = end + xt[i];
        }
        pend[i_max + 1] = chain;
    }
    for (int k = 0; k < m; ++k) {
        T chain_b = (T)0;
        for (int i = S - 1; i >= 0; --i) {
            int w = S - 1 - i;
            if (w > m) w = m;
            T c = clock[i];
            T fend = (T)0;
            if (w + k < m) {
                T start = i > 0 ? tmax(c, pend[i]) : c;
                fend = start + F[i];
                c = fend;
                if (i < S - 1) pend[i + 1] = fend + xt[i];
            }
            T dep = i < S - 1 ? chain_b + xt[i] : fend;
            T start = tmax(c, dep);
            T end = start + B[i];
            clock[i] = end;
            chain_b = end;
        }
    }
    return clock[0];
}

// Peak memory of a stage at position i of S with m micro-batches (Section "Estimator",
// memory estimator): static bytes + min(S - i, m) in-flight activations under 1F1B, all m of
// them under the all-forward-all-backward order.
__device__ __forceinline__ bool stage_fits(long long stat, long long act, int i, int S, int m, long long cap, int sched) {
    int inflight = S - i;
    if (m < inflight || sched == CM_SCHED_GPIPE) inflight = m;
    return stat + (long long)inflight * act <= cap;
}

// Cost of one pipeline given by its cuts: memory check, stage sums from the prefix
// arrays, recurrence, gradient-sync lower bound.  Returns false if infeasible.
template <typename T>
__device__ __forceinline__ bool pipe_cost_from_cuts(const SProf<T> &sp, int S, int m, const uint8_t *cuts,
                                                   uint64_t tier_mask, int n_sync, T &cost) {
    if (m < 1) return false;
    for (int i = 0; i < S; ++i) {
        const int lo = cuts[i], hi = cuts[i + 1];
        if (hi <= lo) return false;
        if (!stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched)) return false;
    }
    T F[kMaxS], B[kMaxS], xt[kMaxS], clock[kMaxS], pend[kMaxS];
    long long g_max = 0;
    for (int i = 0; i < S; ++i) {
        const int lo = cuts[i], hi = cuts[i + 1];
        F[i] = sp.PF[hi] - sp.PF[lo];
        B[i] = sp.PB[hi] - sp.PB[lo];
        xt[i] = i < S - 1 ? sp.XT[(tier_mask >> i) & 1ull][hi - 1] : (T)0;
        long long g = sp.PP[hi] - sp.PP[lo];
        g_max = g > g_max ? g : g_max;
    }
    T t = sim_pipe<T>(S, m, F, B, xt, clock, pend, sp.sched);
    // the sync time is monotone in the gradient bytes, so max over stages = sync of the max
    cost = t + Num<T>::sync(g_max, n_sync, sp.bw_sync, sp.intval);
    return true;
}

// ----------------------------------------------------------------------------------
// A segment of one scenario, resolved from the template tables: the template gives the
// shape (stages, micro-batches, peers, compositions), the scenario gives the link tiers
// -- n bits cut out of its node-crossing bit string at the pipeline's survivor offset.
// ----------------------------------------------------------------------------------
struct SegView {
    uint64_t tier, K;
    uint32_t row;          // row of seg_best
    uint32_t feas_first, feas_count;
    int S, m, n_sync;
};

// Candidates a pass walks in a segment, and the layer composition behind position idx of
// that walk: the listed memory-feasible ones in ascending order, or all of them.
__device__ __forceinline__ uint64_t walk_count(const SegView &g) {
    return g.feas_first != kNoFeasList ? (uint64_t)g.feas_count : (g.K ? g.K + 1 : 1);
}
__device__ __forceinline__ uint64_t walk_kappa(const uint32_t *feas, uint32_t feas_first, uint64_t idx) {
    return feas_first != kNoFeasList ? (uint64_t)feas[feas_first + idx] : idx;
}

__device__ __forceinline__ uint64_t cut_bits(const uint64_t *words, int off, int n /* <= 63 */) {
    const int w = off >> 6, sh = off & 63;
    uint64_t v = words[w] >> sh;
    if (sh) v |= words[w + 1] << (64 - sh);
    return v & ((1ull << n) - 1ull);
}

__device__ __forceinline__ SegView seg_view(const BatchDev &bd, uint32_t scen_id, uint32_t tseg_row) {
    const Scen &sc = bd.scen[scen_id];
    const TSeg g = bd.tseg[tseg_row];
    SegView v;
    v.S = g.S;
    v.m = g.m;
    v.n_sync = g.n_sync;
    v.K = g.K;
    v.feas_first = g.feas_first;
    v.feas_count = g.feas_count;
    v.row = sc.seg_base + (tseg_row - bd.tmpl[sc.tmpl].tseg_first);
    v.tier = cut_bits(bd.cross + sc.cross_first, g.off, g.S - 1);
    return v;
}

// Candidate kappa of a segment: an enumerated composition or the min-max partition.
template <typename T>
__device__ __forceinline__ bool segment_candidate_cost(const SProf<T> &sp, const Tables &tb, const SegView &g,
                                                       int layer_mode, uint64_t kappa, T &cost) {
    uint8_t cuts[kMaxS + 1];
    const int S = g.S;
    if (g.m < 1) return false;
    if (kappa < g.K) {
        layer_cuts(tb.binom, layer_mode, sp.L, S, kappa, cuts);
    } else {
        const uint8_t *mm = tb.mm_cuts + (size_t)tb.mm_slot(S, g.m) * (kMaxS + 1);
        if (mm[0] != 0) return false;  // no memory-feasible partition exists
        for (int i = 0; i <= S; ++i) cuts[i] = mm[i];
    }
    return pipe_cost_from_cuts<T>(sp, S, g.m, cuts, g.tier, g.n_sync, cost);
}

// ----------------------------------------------------------------------------------
// Micro-batch split of a strategy from its rank (Section "Planner", batch distribution).
// ----------------------------------------------------------------------------------
__device__ __forceinline__ void split_micro(const uint64_t *tab, int batch_mode, int G, const Strat &s,
                                            uint64_t beta, uint16_t *micro) {
    const int dp = s.dp;
    if (batch_mode == CM_BATCH_REMAINDER) {
        for (int p = 0; p < dp; ++p) micro[p] = s.m_lo[p];
        unrank_subset(tab, beta, dp, s.R, [&](int, int v) { micro[v] = (uint16_t)(micro[v] + 1); });
    } else {
        int cutpos[kMaxP];
        unrank_subset(tab, beta, G - 1, dp - 1, [&](int pos, int v) { cutpos[pos] = v + 1; });
        int prev = 0;
        for (int p = 0; p < dp - 1; ++p) { micro[p] = (uint16_t)(cutpos[p] - prev); prev = cutpos[p]; }
        micro[dp - 1] = (uint16_t)(G - prev);
    }
}

__device__ __forceinline__ bool pair_less(uint64_t c1, uint64_t i1, uint64_t c2, uint64_t i2) {
    return c1 < c2 || (c1 == c2 && i1 < i2);
}

// Step time of one (strategy, split) item of a scenario from its per-segment minima `best`
// (rows in template order): the slowest pipeline's best cost (Section "Estimator": step
// time = max over pipelines).  inf if a pipeline has no feasible plan.
__device__ __forceinline__ uint32_t strat_of_item(const BatchDev &bd, const Tmpl &tp, uint64_t item) {
    uint32_t lo = 0, hi = tp.n_strat - 1;
    while (lo < hi) {
        uint32_t mid = (lo + hi + 1) >> 1;
        if (bd.strat[tp.strat_first + mid].split_first <= item) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ __forceinline__ uint64_t item_step_time(const Tables &tb, const BatchDev &bd, const Tmpl &tp,
                                                   const uint64_t *best, uint64_t item, uint64_t inf) {
    const Strat &s = bd.strat[tp.strat_first + strat_of_item(bd, tp, item)];
    uint16_t micro[kMaxP];
    split_micro(tb.binom, bd.batch_mode, tb.prof->G, s, item - s.split_first, micro);
    uint64_t T = 0;
    for (int p = 0; p < s.dp; ++p) {
        uint64_t c = inf;
        const int off = (int)micro[p] - (int)s.m_lo[p];
        if (micro[p] >= 1 && off >= 0 && off < s.n_m) c = best[s.seg_first - tp.tseg_first + p * s.n_m + off];
        c = c > inf ? inf : c;   // a segment nobody improved still holds its all-ones initial value
        T = c > T ? c : T;
    }
    return T;
}

// The winner record of an item: strategy, micro-batches and segment rows of its pipelines.
__device__ __forceinline__ void decode_winner(const Tables &tb, const BatchDev &bd, const Tmpl &tp, uint32_t scen,
                                              uint64_t cost_bits, uint64_t item, uint64_t inf, Winner &w) {
    w.cost_bits = cost_bits >= inf ? inf : cost_bits;
    w.item = item;
    w.strat = 0;
    w.dp = 0;
    w.scen = scen;
    w.pad = 0;
    for (int p = 0; p < kMaxP; ++p) { w.seg[p] = 0; w.micro[p] = 0; }
    if (cost_bits < inf) {
        const uint32_t si = strat_of_item(bd, tp, item);
        const Strat &s = bd.strat[tp.strat_first + si];
        w.strat = tp.strat_first + si;
        w.dp = s.dp;
        split_micro(tb.binom, bd.batch_mode, tb.prof->G, s, item - s.split_first, w.micro);
        for (int p = 0; p < s.dp; ++p) w.seg[p] = s.seg_first + p * s.n_m + (w.micro[p] - s.m_lo[p]);
    }
}

__device__ __forceinline__ void plan_clear(cm_plan &pl, int policy) {
    pl.policy = policy;
    pl.feasible = 0;
    pl.cost = 0.0;
    pl.cost_ns = 0;
    pl.strategy = 0;
    pl.n_pipes = 0;
    pl.split_rank = 0;
    for (int p = 0; p < kMaxP; ++p) { pl.stages[p] = 0; pl.micro[p] = 0; pl.kappa[p] = 0; }
}

__device__ __forceinline__ void plan_set_cost(cm_plan &pl, uint64_t bits, const BatchDev &bd) {
    if (bd.mode == CM_COST_INT64NS) pl.cost_ns = batch_cost_ns(bd, bits);
    else pl.cost = __longlong_as_double((long long)bits);
}

// Start values of the tie-break pass for one winner record: "not found yet" for every
// pipeline, except that a segment whose only candidate is the min-max partition has nothing
// to search -- that candidate is feasible and within the step time, or the pair would not have
// won -- so its rank is known at once and the tie-break kernels leave it alone.
__device__ __forceinline__ void init_kappa_sel(const BatchDev &bd, const Winner &w, uint64_t *slot /* [kMaxP] */, int p) {
    slot[p] = (p < (int)w.dp && w.cost_bits < batch_inf_bits(bd) && bd.tseg[w.seg[p]].K == 0) ? 0ull : ~0ull;
}

// ----------------------------------------------------------------------------------
// The pipeline-time recurrence of ONE pipeline spread over a warp: PER consecutive stages
// per lane (S <= 32 * PER), walked in lock step over time slots.  With unit durations the
// 1F1B schedule puts forward (i,j) at slot i+j while j <= S-1-i and at slot i+2j afterwards,
// and backward (i,j) at slot 2S-1-i+2j; taking those slots as the evaluation order is a
// valid topological order for arbitrary durations and every m >= 1.  Every stage keeps
// its clock, its latest forward end (transfer added) and its latest backward end; inputs
// of a slot are gathered from the neighbours' state before any stage of the slot updates.
// F, B, xt: the lane's own stages.  Returns the pipeline time in every lane.
// ----------------------------------------------------------------------------------
// Under the all-forward-all-backward order forward (i,j) sits at slot i+j and backward (i,j)
// at slot (S+m-1) + (S-1-i) + j.
// The loop is branch-free inside a slot -- lanes that run a forward, a backward or nothing take
// the same instructions, so the stages of a lane and the two kinds of work interleave -- and
// the slot tests are kept short, because one warp alone issues them: times are non-negative,
// so "no dependency" (forward of stage 0, backward of the last stage) is a dependency on time 0
// (a stage past the end never runs and keeps its zeros), and under 1F1B the parity of s - i
// says which kind of work a steady-state slot can hold.
template <typename T, int PER>
__device__ __forceinline__ T sim_lockstep_n(int S, int m, const T *F, const T *B, const T *xt, int sched) {
    const int lane = threadIdx.x & 31;
    T clock[PER], last_f[PER], last_b[PER];
    int d[PER];          // slot - stage
    unsigned mk[PER];    // micro-batches of the stage (0: past the end)
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        clock[k] = (T)0; last_f[k] = (T)0; last_b[k] = (T)0;
        d[k] = -(lane * PER + k);
        mk[k] = lane * PER + k < S ? (unsigned)m : 0u;
    }
    auto slot = [&](auto only_forward, auto pick) {
        T up = __shfl_up_sync(0xffffffffu, last_f[PER - 1], 1);
        T down = __shfl_down_sync(0xffffffffu, last_b[0], 1);
        up = lane == 0 ? (T)0 : up;       // the end lanes get their own value back from the shuffle
        down = lane == 31 ? (T)0 : down;
        T f_in[PER], b_in[PER];
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            f_in[k] = k == 0 ? up : last_f[k > 0 ? k - 1 : 0];
            b_in[k] = k == PER - 1 ? down : last_b[k < PER - 1 ? k + 1 : 0];
        }
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            bool is_f, is_b;
            pick(k, is_f, is_b);
            if constexpr (decltype(only_forward)::value) {
                const T fin = tmax(clock[k], f_in[k]) + F[k];
                clock[k] = is_f ? fin : clock[k];
                last_f[k] = is_f ? fin + xt[k] : last_f[k];
            } else {
                const T dep = is_f ? f_in[k] : b_in[k] + xt[k];
                const T fin = tmax(clock[k], dep) + (is_f ? F[k] : B[k]);
                clock[k] = (is_f || is_b) ? fin : clock[k];
                last_f[k] = is_f ? fin + xt[k] : last_f[k];
                last_b[k] = is_b ? fin : last_b[k];
            }
            ++d[k];
        }
    };
    using Yes = std::true_type;
    using No = std::false_type;
    if (sched == CM_SCHED_GPIPE) {
        // forward (i,j) at slot i+j; backward (i,j) at slot (S+m-1) + (S-1-i) + j
        for (int s = 0; s < S + m - 1; ++s)
            slot(Yes{}, [&](int k, bool &is_f, bool &is_b) { is_f = (unsigned)d[k] < mk[k]; is_b = false; });
        int e[PER];
#pragma unroll
        for (int k = 0; k < PER; ++k) e[k] = -(S - 1 - (lane * PER + k));
        for (int s = 0; s < S + m - 1; ++s)
            slot(No{}, [&](int k, bool &is_f, bool &is_b) { is_f = false; is_b = (unsigned)e[k] < mk[k]; ++e[k]; });
    } else {
        // slots 0 .. S-1: warm-up forwards only (the first backward sits at slot S)
        for (int s = 0; s < S; ++s)
            slot(Yes{}, [&](int k, bool &is_f, bool &is_b) { is_f = (unsigned)d[k] < mk[k]; is_b = false; });
        // afterwards forward j = (s-i)/2 when s-i is even and j > S-1-i; backward (s-i-(2S-1-2i))/2 when s-i is odd
        int warm[PER], off[PER];
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            warm[k] = S - 1 - (lane * PER + k);
            off[k] = 2 * S - 1 - 2 * (lane * PER + k);
        }
        const int n_slots = 2 * (S + m) - 2;
        for (int s = S; s < n_slots; ++s)
            slot(No{}, [&](int k, bool &is_f, bool &is_b) {
                const bool even = (d[k] & 1) == 0;
                const int j = d[k] >> 1;
                is_f = even && j > warm[k] && (unsigned)j < mk[k];
                is_b = !even && ((unsigned)(d[k] - off[k]) >> 1) < mk[k];
            });
    }
    return __shfl_sync(0xffffffffu, clock[0], 0);
}

// The 1F1B order with TWO consecutive stages per lane (stage 2l and 2l+1; S <= 64).  After the
// warm-up slots a stage alternates forward and backward, even stages run their forwards in even
// slots and odd stages in odd ones, so which kind of work each of a lane's two stages can do in
// a slot is known at compile time once the loop takes an even and an odd slot per iteration:
// no selects between forward and backward operands.  In the odd slot both inputs are the lane's
// own (the forward of stage 2l feeds stage 2l+1, the backward of stage 2l+1 feeds stage 2l), so
// only the even slot shuffles.  With h = slot / 2 and c = h + l + 1 - S the micro-batch tests are
//   even slot: stage 2l   forward  j = h - l     runs iff 0 <= c - 1 < m - S + 2l
//              stage 2l+1 backward j = c         runs iff 0 <= c < m
//   odd slot:  stage 2l   backward j = c         runs iff 0 <= c < m
//              stage 2l+1 forward  j = h - l     runs iff 0 <= c < m - S + 2l + 1
// Same operations on the same operands as sim_lockstep_n: identical bits.
template <typename T>
__device__ __forceinline__ T sim_lockstep_pairs(int S, int m, const T *F, const T *B, const T *xt) {
    const int lane = threadIdx.x & 31;
    const bool valid0 = 2 * lane < S, valid1 = 2 * lane + 1 < S;
    T clock0 = (T)0, clock1 = (T)0, last_f0 = (T)0, last_f1 = (T)0, last_b0 = (T)0, last_b1 = (T)0;
    {   // slots 0 .. S-1: warm-up forwards only, forward (i,j) at slot i+j
        int d0 = -2 * lane, d1 = -2 * lane - 1;
        const unsigned m0 = valid0 ? (unsigned)m : 0u, m1 = valid1 ? (unsigned)m : 0u;
        for (int s = 0; s < S; ++s) {
            T up = __shfl_up_sync(0xffffffffu, last_f1, 1);
            up = lane == 0 ? (T)0 : up;
            const T fin0 = tmax(clock0, up) + F[0];
            const T fin1 = tmax(clock1, last_f0) + F[1];
            if ((unsigned)d0 < m0) { clock0 = fin0; last_f0 = fin0 + xt[0]; }
            if ((unsigned)d1 < m1) { clock1 = fin1; last_f1 = fin1 + xt[1]; }
            ++d0; ++d1;
        }
    }
    const int f0 = m - S + 2 * lane;
    const unsigned lim_f0 = valid0 && f0 > 0 ? (unsigned)f0 : 0u;
    const unsigned lim_f1 = valid1 && f0 + 1 > 0 ? (unsigned)(f0 + 1) : 0u;
    const unsigned lim_b0 = valid0 ? (unsigned)m : 0u, lim_b1 = valid1 ? (unsigned)m : 0u;
    int h = S >> 1;
    int c = h + lane + 1 - S;
    auto odd_slot = [&]() {
        const T fin0 = tmax(clock0, last_b1 + xt[0]) + B[0];
        const T fin1 = tmax(clock1, last_f0) + F[1];
        if ((unsigned)c < lim_b0) { clock0 = fin0; last_b0 = fin0; }
        if ((unsigned)c < lim_f1) { clock1 = fin1; last_f1 = fin1 + xt[1]; }
    };
    if (S & 1) {   // slot S is odd
        odd_slot();
        ++h; ++c;
    }
    for (; h <= S + m - 2; ++h, ++c) {
        T up = __shfl_up_sync(0xffffffffu, last_f1, 1);
        T down = __shfl_down_sync(0xffffffffu, last_b0, 1);
        up = lane == 0 ? (T)0 : up;       // the end lanes get their own value back from the shuffle
        down = lane == 31 ? (T)0 : down;
        const T fin0 = tmax(clock0, up) + F[0];
        const T fin1 = tmax(clock1, down + xt[1]) + B[1];
        if ((unsigned)(c - 1) < lim_f0) { clock0 = fin0; last_f0 = fin0 + xt[0]; }
        if ((unsigned)c < lim_b1) { clock1 = fin1; last_b1 = fin1; }
        odd_slot();
    }
    return __shfl_sync(0xffffffffu, clock0, 0);
}

// Bare time of one pipeline (no synchronisation term), its stages spread over the warp, two per lane.
template <typename T>
__device__ __forceinline__ T warp_pipe_time(const SProf<T> &sp, const uint8_t *cuts, int S, int m, uint64_t tier, int lane) {
    T F[2], B[2], xt[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int i = lane * 2 + k;
        F[k] = (T)0; B[k] = (T)0; xt[k] = (T)0;
        if (i < S) {
            const int lo = cuts[i], hi = cuts[i + 1];
            F[k] = sp.PF[hi] - sp.PF[lo];
            B[k] = sp.PB[hi] - sp.PB[lo];
            if (i < S - 1) xt[k] = sp.XT[(tier >> i) & 1ull][hi - 1];
        }
    }
    return sp.sched == CM_SCHED_GPIPE ? sim_lockstep_n<T, 2>(S, m, F, B, xt, sp.sched) : sim_lockstep_pairs<T>(S, m, F, B, xt);
}

__device__ __forceinline__ uint64_t warp_min_u64(uint64_t v) {
    for (int o = 16; o > 0; o >>= 1) {
        uint64_t w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w < v ? w : v;
    }
    return v;
}

}  // namespace cm
