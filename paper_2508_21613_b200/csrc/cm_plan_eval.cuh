// Per-plan evaluation shared by the search pass (cm_cost.cu) and the tie-break pass
// (cm_kernels.cu): walking a plan's layer cuts from its rank, the recurrence with the
// per-stage state in registers, and the whole cost of one pipeline-plan of S <= 16 stages.
#pragma once

#include "cm_device.cuh"

namespace cm {

// ----------------------------------------------------------------------------------
// Layer cuts of a plan, stage after stage (no array: the caller consumes them in order).
//   kind 0  REMAINDER: n_i = q + bit i of a           (a = subset mask from the rank)
//   kind 1  FULL:      cut positions are the set bits of the 128-bit mask (a, b)
//   kind 2  min-max partition row
// ----------------------------------------------------------------------------------
struct CutWalker {
    uint64_t a, b;
    const uint8_t *row;
    int kind, q, L, S, i, pos;
    __device__ __forceinline__ int next() {   // upper cut of stage i, then advance
        int hi;
        if (kind == 0) {
            hi = pos + q + (int)((a >> i) & 1ull);
        } else if (kind == 1) {
            if (i == S - 1) hi = L;
            else if (a) { hi = __ffsll((long long)a); a &= a - 1; }
            else { hi = 64 + __ffsll((long long)b); b &= b - 1; }
        } else {
            hi = row[i + 1];
        }
        pos = hi;
        ++i;
        return hi;
    }
};

__device__ __forceinline__ bool make_walker(CutWalker &w, const Tables &tb, int layer_mode, int L, int S,
                                            uint64_t kappa, uint64_t K, uint32_t mm_slot) {
    w.a = 0; w.b = 0; w.row = nullptr; w.q = 0; w.L = L; w.S = S; w.i = 0; w.pos = 0;
    if (kappa < K) {
        if (layer_mode == CM_LAYERS_REMAINDER) {
            w.kind = 0;
            w.q = L / S;
            uint64_t mask = 0;
            unrank_subset(tb.binom, kappa, S, L % S, [&](int, int v) { mask |= 1ull << v; });
            w.a = mask;
        } else {
            w.kind = 1;
            uint64_t m0 = 0, m1 = 0;
            unrank_subset(tb.binom, kappa, L - 1, S - 1, [&](int, int v) {
                if (v < 64) m0 |= 1ull << v; else m1 |= 1ull << (v - 64);
            });
            w.a = m0; w.b = m1;
        }
        return true;
    }
    w.kind = 2;
    w.row = tb.mm_cuts + (size_t)mm_slot * (kMaxS + 1);
    return w.row[0] == 0;   // 255 marks "no memory-feasible partition"
}

// ----------------------------------------------------------------------------------
// The recurrence in "rounds", S compile-time, clock and pending forward in registers.
//
// Round t = 0 .. S-2+m; stages are visited from last to first.  In round t stage i runs
//   its forward of micro-batch t-i      if 0 <= t-i < m   (fed by the forward that stage
//                                        i-1 ran in round t-1 and left pending), then
//   its backward of micro-batch t-S+1   if t >= S-1       (fed by the backward stage i+1
//                                        ran just before in the same round; by its own
//                                        forward at the last stage).
// Per stage this is exactly the 1F1B order -- min(S-1-i, m) forwards, forward/backward
// pairs, the remaining backwards -- for every m >= 1, and every dependency is either one
// round or one stage old, so two values per stage are all the state there is.
// Rounds S-1 .. m-1 have every stage fully active and carry no predicate at all; the
// ramp-up and ramp-down rounds skip inactive stages with warp-uniform branches.
//
// stage(i) returns the stage's forward and backward time, xt(i) the transfer time of the
// boundary above stage i; both are called with compile-time i only.
// ----------------------------------------------------------------------------------
template <typename T> struct alignas(16) FB { T f, b; };

// Shared-memory loads the compiler must issue where they stand: the stage times are loop
// invariants, and hoisting ~100 of them into registers would push the per-stage state out.
template <typename T>
__device__ __forceinline__ FB<T> lds_fb(const FB<T> *p) {
    unsigned long long a, b;
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"((unsigned)__cvta_generic_to_shared(p)));
    FB<T> d;
    d.f = Num<T>::from_bits(a);
    d.b = Num<T>::from_bits(b);
    return d;
}
template <typename T>
__device__ __forceinline__ T lds_t(const T *p) {
    unsigned long long a;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(a) : "r"((unsigned)__cvta_generic_to_shared(p)));
    return Num<T>::from_bits(a);
}

template <typename T, int S, typename StageFn, typename XtFn>
__device__ __forceinline__ T sim_rounds(int m, StageFn stage, XtFn xt) {
    T clock[S], pend[S];
#pragma unroll
    for (int i = 0; i < S; ++i) { clock[i] = (T)0; pend[i] = (T)0; }
    // ramp-up: forwards only
    for (int t = 0; t < S - 1; ++t) {
#pragma unroll
        for (int i = S - 2; i >= 0; --i) {
            if (i <= t && t < i + m) {
                const T fstart = i > 0 ? tmax(clock[i], pend[i]) : clock[i];
                const T fend = fstart + stage(i).f;
                clock[i] = fend;
                pend[i + 1] = fend + xt(i);
            }
        }
    }
    // steady rounds: every stage does one forward and one backward
    // four rounds per trip: the backward chain of one round overlaps the forwards of the
    // next ones in the instruction stream, which hides its fixed latencies
#pragma unroll 4
    for (int t = S - 1; t < m; ++t) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            const FB<T> d = stage(i);
            const T x = i < S - 1 ? xt(i) : (T)0;
            const T fstart = i > 0 ? tmax(clock[i], pend[i]) : clock[i];
            const T fend = fstart + d.f;
            if (i < S - 1) pend[i + 1] = fend + x;
            const T dep = i < S - 1 ? chain_b + x : fend;
            const T bstart = tmax(fend, dep);
            const T bend = bstart + d.b;
            clock[i] = bend;
            chain_b = bend;
        }
    }
    // ramp-down: every stage still has a backward, the upper ones a forward too
    for (int t = (m > S - 1 ? m : S - 1); t < S - 1 + m; ++t) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            const FB<T> d = stage(i);
            const T x = i < S - 1 ? xt(i) : (T)0;
            T c = clock[i];
            if (t < i + m) {
                const T fstart = i > 0 ? tmax(c, pend[i]) : c;
                c = fstart + d.f;
                if (i < S - 1) pend[i + 1] = c + x;
            }
            const T dep = i < S - 1 ? chain_b + x : c;
            const T bstart = tmax(c, dep);
            const T bend = bstart + d.b;
            clock[i] = bend;
            chain_b = bend;
        }
    }
    return clock[0];
}

// ----------------------------------------------------------------------------------
// The same recurrence for shallow pipelines (S <= 16) with m >= S-1, where every stage
// has its full warm-up: warm-up and cool-down are unrolled triangles without a single
// branch (S^2 cells of code, affordable at this depth), the steady rounds as above.
// Order: warm-up forwards micro-batch by micro-batch up the stages, the last forward of
// a row left pending for the stage above; then rounds k = 0..m-1 from the last stage to
// the first, forward (while one is left) then backward.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__device__ __forceinline__ T sim_regs(int m, const FB<T> (&st)[S], const T (&xt)[S]) {
    T clock[S], pend[S];
#pragma unroll
    for (int i = 0; i < S; ++i) { clock[i] = (T)0; pend[i] = (T)0; }
#pragma unroll
    for (int j = 0; j < S - 1; ++j) {
        T chain = (T)0;
#pragma unroll
        for (int i = 0; i <= S - 2 - j; ++i) {
            const T start = i > 0 ? tmax(clock[i], chain) : clock[i];
            const T end = start + st[i].f;
            clock[i] = end;
            chain = end + xt[i];
        }
        pend[S - 1 - j] = chain;
    }
#pragma unroll 4
    for (int k = 0; k <= m - S; ++k) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            const T fstart = i > 0 ? tmax(clock[i], pend[i]) : clock[i];
            const T fend = fstart + st[i].f;
            if (i < S - 1) pend[i + 1] = fend + xt[i];
            const T dep = i < S - 1 ? chain_b + xt[i] : fend;
            const T bstart = tmax(fend, dep);
            const T bend = bstart + st[i].b;
            clock[i] = bend;
            chain_b = bend;
        }
    }
#pragma unroll
    for (int r = 0; r < S - 1; ++r) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            T c = clock[i];
            if (i > r) {
                const T fstart = i > 0 ? tmax(c, pend[i]) : c;
                c = fstart + st[i].f;
                if (i < S - 1) pend[i + 1] = c + xt[i];
            }
            const T dep = i < S - 1 ? chain_b + xt[i] : c;
            const T bstart = tmax(c, dep);
            const T bend = bstart + st[i].b;
            clock[i] = bend;
            chain_b = bend;
        }
    }
    return clock[0];
}

// ----------------------------------------------------------------------------------
// Cost of pipeline-plan kappa of a segment with S <= kRegStagesMax stages and m >= S-1
// micro-batches, everything in registers.  Returns false if the plan is infeasible.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__device__ __forceinline__ bool plan_cost_regs(const SProf<T> &sp, const Tables &tb, int layer_mode,
                                               const SegView &g, uint64_t kappa, T &cost) {
    const int m = g.m;
    CutWalker cw;
    bool ok = make_walker(cw, tb, layer_mode, sp.L, S, kappa, g.K, tb.mm_slot(S, m));
    FB<T> st[S];
    T xts[S];
    long long g_max = 0;
    int lo = 0;
#pragma unroll
    for (int i = 0; i < S; ++i) {
        const int hi = ok ? cw.next() : lo + 1;
        ok = ok && hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap);
        st[i].f = sp.PF[hi] - sp.PF[lo];
        st[i].b = sp.PB[hi] - sp.PB[lo];
        xts[i] = i < S - 1 ? sp.XT[(g.tier >> i) & 1ull][hi - 1] : (T)0;
        const long long gb = sp.PP[hi] - sp.PP[lo];
        g_max = gb > g_max ? gb : g_max;
        lo = hi;
    }
    if (!ok) return false;
    cost = sim_regs<T, S>(m, st, xts) + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    return true;
}

// ----------------------------------------------------------------------------------
// Cost of one pipeline-plan of a deep pipeline (S compile-time, any m >= 1): clock and
// pending forward in registers, the stage times in this lane's shared-memory columns
// fcol / xcol (element i at index i * kChunk).  Returns false if the plan is infeasible.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__device__ __forceinline__ bool plan_cost_wide_lane(const SProf<T> &sp, const Tables &tb, int layer_mode,
                                                    const SegView &g, uint64_t kappa, FB<T> *fcol, T *xcol, T &cost) {
    const int m = g.m;
    if (m < 1) return false;
    CutWalker cw;
    bool ok = make_walker(cw, tb, layer_mode, sp.L, S, kappa, g.K, tb.mm_slot(S, m));
    long long g_max = 0;
    int lo = 0;
    for (int i = 0; i < S && ok; ++i) {
        const int hi = cw.next();
        ok = hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap);
        FB<T> d;
        d.f = sp.PF[hi] - sp.PF[lo];
        d.b = sp.PB[hi] - sp.PB[lo];
        fcol[i * kChunk] = d;
        xcol[i * kChunk] = i < S - 1 ? sp.XT[(g.tier >> i) & 1ull][hi - 1] : (T)0;
        const long long gb = sp.PP[hi] - sp.PP[lo];
        g_max = gb > g_max ? gb : g_max;
        lo = hi;
    }
    if (!ok) return false;
    const T t = sim_rounds<T, S>(m, [&](int i) { return lds_fb<T>(fcol + i * kChunk); },
                                 [&](int i) { return lds_t<T>(xcol + i * kChunk); });
    cost = t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    return true;
}

// The same with S chosen at run time (one kernel for every shallow depth; used where the
// work is too small to be worth one launch per depth).  Caller guarantees 1 <= S <= 16, m >= S-1.
template <typename T>
__device__ __forceinline__ bool plan_cost_regs_any(const SProf<T> &sp, const Tables &tb, int layer_mode,
                                                   const SegView &g, uint64_t kappa, T &cost) {
    switch (g.S) {
#define CM_CASE(S) case S: return plan_cost_regs<T, S>(sp, tb, layer_mode, g, kappa, cost);
        CM_CASE(1) CM_CASE(2) CM_CASE(3) CM_CASE(4) CM_CASE(5) CM_CASE(6) CM_CASE(7) CM_CASE(8)
        CM_CASE(9) CM_CASE(10) CM_CASE(11) CM_CASE(12) CM_CASE(13) CM_CASE(14) CM_CASE(15) CM_CASE(16)
#undef CM_CASE
    default: return false;
    }
}

}  // namespace cm
