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
// Rounds S-1 .. m-1 have every stage fully active and carry no predicate at all.
// ----------------------------------------------------------------------------------
template <typename T> struct alignas(16) FB { T f, b; };

// Where the recurrence finds its stage times.  Both sources are addressed with compile-time
// stage indices only, so a register source stays in registers and a shared-memory source is
// read with "base register + immediate" addresses: no address arithmetic per load.
//
// SmemStages: stage i's (f, b) pair at byte offset i * FB_STRIDE from `fb`, the transfer time
// of the boundary above it at i * XT_STRIDE from `xt` (32-bit shared-window addresses).  The
// loads are written where they are needed; the assembler keeps as many of these loop
// invariants in registers as the per-stage state leaves room for and reloads the rest
// (measured: 0.6-0.7 shared loads per cell where one per cell is written).
template <typename T, int FB_STRIDE, int XT_STRIDE> struct SmemStages {
    unsigned fb, xt;
    template <int I> __device__ __forceinline__ FB<T> stage() const {
        unsigned long long a, b;
        asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(a), "=l"(b) : "r"(fb), "n"(I * FB_STRIDE));
        FB<T> d;
        d.f = Num<T>::from_bits(a);
        d.b = Num<T>::from_bits(b);
        return d;
    }
    template <int I> __device__ __forceinline__ T f() const {
        unsigned long long a;
        asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(a) : "r"(fb), "n"(I * FB_STRIDE));
        return Num<T>::from_bits(a);
    }
    template <int I> __device__ __forceinline__ T b() const {
        unsigned long long a;
        asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(a) : "r"(fb), "n"(I * FB_STRIDE + 8));
        return Num<T>::from_bits(a);
    }
    template <int I> __device__ __forceinline__ T x() const {
        unsigned long long a;
        asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(a) : "r"(xt), "n"(I * XT_STRIDE));
        return Num<T>::from_bits(a);
    }
};
template <typename P> __device__ __forceinline__ unsigned smem_addr(const P *p) { return (unsigned)__cvta_generic_to_shared(p); }

// RegStages: the stage times of a shallow pipeline, held by the caller in registers.
template <typename T, int S> struct RegStages {
    const FB<T> (&st)[S];
    const T (&xt)[S];
    template <int I> __device__ __forceinline__ FB<T> stage() const { return st[I]; }
    template <int I> __device__ __forceinline__ T f() const { return st[I].f; }
    template <int I> __device__ __forceinline__ T b() const { return st[I].b; }
    template <int I> __device__ __forceinline__ T x() const { return xt[I]; }
};

// Where a pipeline's pending forwards live (one value per stage, written by the stage below,
// read one round later): in registers up to kWideStagesMax stages, beyond that in a per-lane
// shared-memory column (element i at byte offset i * STRIDE), because clock and pend of 64
// stages do not fit the register file of a thread.  Entries are written before they are read.
template <typename T, int S> struct RegPend {
    T v[S];
    template <int I> __device__ __forceinline__ T get() const { return v[I]; }
    template <int I> __device__ __forceinline__ void set(T x) { v[I] = x; }
};
template <typename T, int STRIDE> struct SmemPend {
    unsigned base;
    template <int I> __device__ __forceinline__ T get() const {
        unsigned long long a;
        asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(a) : "r"(base), "n"(I * STRIDE) : "memory");
        return Num<T>::from_bits(a);
    }
    template <int I> __device__ __forceinline__ void set(T x) const {
        asm volatile("st.shared.b64 [%0+%1], %2;" : : "r"(base), "n"(I * STRIDE), "l"(Num<T>::bits(x)) : "memory");
    }
};

// State and cells of one pipeline of S stages (S compile-time): clock = end of the stage's
// latest computation, pend = end of the forward the stage has not consumed yet (transfer
// included).  Every method takes its stage as a template argument.
template <typename T, int S, typename Src, typename Pend = RegPend<T, S>> struct Rounds {
    T clock[S];
    Pend pend;
    const Src &src;
    __device__ __forceinline__ explicit Rounds(const Src &s, Pend p = Pend()) : pend(p), src(s) {
#pragma unroll
        for (int i = 0; i < S; ++i) clock[i] = (T)0;
    }
    // forward of stage I: fed by the forward stage I-1 ran one round earlier
    template <int I> __device__ __forceinline__ void fwd() {
        T fstart = clock[I];
        if constexpr (I > 0) fstart = tmax(fstart, pend.template get<I>());
        const T fend = fstart + src.template f<I>();
        clock[I] = fend;
        if constexpr (I < S - 1) pend.template set<I + 1>(fend + src.template x<I>());
    }
    // backward of stage I: fed by the backward stage I+1 ran just before in the same round
    // (chain_b), at the last stage by its own forward, which is what clock holds there
    template <int I> __device__ __forceinline__ void bwd(T &chain_b) {
        const T c = clock[I];
        T bstart = c;
        if constexpr (I < S - 1) bstart = tmax(c, chain_b + src.template x<I>());
        const T bend = bstart + src.template b<I>();
        clock[I] = bend;
        chain_b = bend;
    }
    // forward then backward of stage I (a steady round)
    template <int I> __device__ __forceinline__ void both(T &chain_b) {
        const FB<T> d = src.template stage<I>();
        T fstart = clock[I];
        if constexpr (I > 0) fstart = tmax(fstart, pend.template get<I>());
        const T fend = fstart + d.f;
        T bstart = fend;
        if constexpr (I < S - 1) {
            const T x = src.template x<I>();
            pend.template set<I + 1>(fend + x);
            bstart = tmax(fend, chain_b + x);
        }
        const T bend = bstart + d.b;
        clock[I] = bend;
        chain_b = bend;
    }
    // forward of stage I fed through `chain` by the forward stage I-1 ran just before (the
    // all-forward-all-backward order walks a micro-batch up the stages); stages I .. S-1
    template <int I> __device__ __forceinline__ void fwd_up(T &chain) {
        const T fstart = I > 0 ? tmax(clock[I], chain) : clock[I];
        const T fend = fstart + src.template f<I>();
        clock[I] = fend;
        if constexpr (I < S - 1) {
            chain = fend + src.template x<I>();
            fwd_up<I + 1>(chain);
        }
    }
    // stages I, I-1, .., 0
    template <int I> __device__ __forceinline__ void fwd_down() { fwd<I>(); if constexpr (I > 0) fwd_down<I - 1>(); }
    template <int I> __device__ __forceinline__ void bwd_down(T &chain_b) { bwd<I>(chain_b); if constexpr (I > 0) bwd_down<I - 1>(chain_b); }
    template <int I> __device__ __forceinline__ void both_down(T &chain_b) { both<I>(chain_b); if constexpr (I > 0) both_down<I - 1>(chain_b); }
    // forwards of stages I, I-1, .., last (last >= 1, warp-uniform)
    template <int I> __device__ __forceinline__ void fwd_down_to(int last) {
        fwd<I>();
        if constexpr (I > 1) { if (I != last) fwd_down_to<I - 1>(last); }
    }
    // stages I .. 0, each only if `active(i)`: the general ramp rounds
    template <int I, typename Pred> __device__ __forceinline__ void fwd_down_if(Pred active) {
        if (active(I)) fwd<I>();
        if constexpr (I > 0) fwd_down_if<I - 1>(active);
    }
    template <int I, typename Pred> __device__ __forceinline__ void fwd_if_bwd_down(Pred active, T &chain_b) {
        if (active(I)) fwd<I>();
        bwd<I>(chain_b);
        if constexpr (I > 0) fwd_if_bwd_down<I - 1>(active, chain_b);
    }
    // park the state (clocks, and the pending forwards of stages 1 .. S-1) in memory / bring it back
    template <int I> __device__ __forceinline__ void park(volatile T *mem) const {
        mem[I] = clock[I];
        if constexpr (I > 0) { mem[S + I] = pend.template get<I>(); park<I - 1>(mem); }
    }
    template <int I> __device__ __forceinline__ void unpark(const volatile T *mem) {
        clock[I] = mem[I];
        if constexpr (I > 0) { pend.template set<I>(mem[S + I]); unpark<I - 1>(mem); }
    }
    // forwards of stages `top`, top-1, .., 0 with top chosen at run time (top <= S-2): a jump
    // into the unrolled sequence, so that a ramp-up round costs its active stages and nothing more
    __device__ __forceinline__ void fwd_down_from(int top) {
        switch (top) {
#define CM_RAMP(K) case K: if constexpr (K <= S - 2) fwd<(K <= S - 2 ? K : 0)>(); [[fallthrough]];
            CM_RAMP(62) CM_RAMP(61) CM_RAMP(60) CM_RAMP(59) CM_RAMP(58) CM_RAMP(57) CM_RAMP(56) CM_RAMP(55)
            CM_RAMP(54) CM_RAMP(53) CM_RAMP(52) CM_RAMP(51) CM_RAMP(50) CM_RAMP(49) CM_RAMP(48) CM_RAMP(47)
            CM_RAMP(46) CM_RAMP(45) CM_RAMP(44) CM_RAMP(43) CM_RAMP(42) CM_RAMP(41) CM_RAMP(40) CM_RAMP(39)
            CM_RAMP(38) CM_RAMP(37) CM_RAMP(36) CM_RAMP(35) CM_RAMP(34) CM_RAMP(33) CM_RAMP(32) CM_RAMP(31)
            CM_RAMP(30) CM_RAMP(29) CM_RAMP(28) CM_RAMP(27) CM_RAMP(26) CM_RAMP(25) CM_RAMP(24) CM_RAMP(23)
            CM_RAMP(22) CM_RAMP(21) CM_RAMP(20) CM_RAMP(19) CM_RAMP(18) CM_RAMP(17) CM_RAMP(16) CM_RAMP(15)
            CM_RAMP(14) CM_RAMP(13) CM_RAMP(12) CM_RAMP(11) CM_RAMP(10) CM_RAMP(9) CM_RAMP(8) CM_RAMP(7)
            CM_RAMP(6) CM_RAMP(5) CM_RAMP(4) CM_RAMP(3) CM_RAMP(2) CM_RAMP(1) CM_RAMP(0)
#undef CM_RAMP
        default: break;
        }
    }
};

// ----------------------------------------------------------------------------------
// The recurrence in "rounds" (see above), any m >= 1.
//   ramp-up    rounds 0 .. S-2        forwards only: stages max(0, t-m+1) .. t
//   steady     rounds S-1 .. m-1      every stage one forward and one backward, no predicate
//   ramp-down  rounds max(m,S-1) .. S-2+m   every stage a backward, stages above t-m a forward first
// With m >= S-1 (every stage gets its full warm-up: the common case) the ramp rounds touch
// exactly their active stages: ramp-up jumps into the unrolled forward sequence at stage t,
// ramp-down runs the forwards from the last stage down to stage t-m+1 and then all
// backwards (within a round the forwards depend only on the round before, so they may all
// precede the backwards).  With fewer micro-batches the ramp rounds test every stage.
// ----------------------------------------------------------------------------------
template <typename T, int S, typename Src, typename Pend = RegPend<T, S>>
__device__ __forceinline__ T sim_rounds(int m, const Src &src, Pend pend = Pend()) {
    Rounds<T, S, Src, Pend> r(src, pend);
    if constexpr (S == 1) {
        for (int t = 0; t < m; ++t) { T chain_b = (T)0; r.template both<0>(chain_b); }
        return r.clock[0];
    } else {
        if (m >= S - 1) {
            for (int t = 0; t < S - 1; ++t) r.fwd_down_from(t);
        } else {
            for (int t = 0; t < S - 1; ++t) r.template fwd_down_if<S - 2>([&](int i) { return i <= t && t < i + m; });
        }
        // four rounds per trip: the backward chain of one round overlaps the forwards of the
        // next ones in the instruction stream, which hides its fixed latencies
#pragma unroll 4
        for (int t = S - 1; t < m; ++t) {
            T chain_b = (T)0;
            r.template both_down<S - 1>(chain_b);
        }
        if (m >= S - 1) {
            for (int q = 0; q < S - 1; ++q) {      // round m + q: forwards of stages S-1 .. q+1
                r.template fwd_down_to<S - 1>(q + 1);
                T chain_b = (T)0;
                r.template bwd_down<S - 1>(chain_b);
            }
        } else {
            for (int t = S - 1; t < S - 1 + m; ++t) {
                T chain_b = (T)0;
                r.template fwd_if_bwd_down<S - 1>([&](int i) { return t < i + m; }, chain_b);
            }
        }
        return r.clock[0];
    }
}

// Pipeline times for m AND m+1 micro-batches from one recurrence (1F1B, m >= S-1, S >= 2).
// Round t runs forward t-i and backward t-S+1: whether a micro-batch m exists shows first in
// round m, so rounds 0 .. m-1 of the two recurrences are the same operations on the same values
// and are run once.  The state (2S-1 values) is then parked in local memory, the ramp-down of
// the m-recurrence runs, the state comes back, and one more steady round plus the ramp-down
// finish the (m+1)-recurrence.  The two tails share their code (a loop of two trips); each
// hands its pipeline time to emit(v, t), v = 0 for m and 1 for m+1, so that nothing has to
// stay in registers across the second tail.
template <typename T, int S, typename Src, typename Emit>
__device__ __forceinline__ void sim_rounds_pair(int m, const Src &src, Emit emit) {
    static_assert(S >= 2, "a one-stage pipeline has no ramp");
    Rounds<T, S, Src, RegPend<T, S>> r(src);
    for (int t = 0; t < S - 1; ++t) r.fwd_down_from(t);
#pragma unroll 4
    for (int t = S - 1; t < m; ++t) {
        T chain_b = (T)0;
        r.template both_down<S - 1>(chain_b);
    }
    T parked[2 * S];
    volatile T *mem = parked;   // volatile: real local-memory stores and loads, not 2S more registers
    r.template park<S - 1>(mem);
#pragma unroll 1
    for (int v = 0; v < 2; ++v) {
        if (v) {
            r.template unpark<S - 1>(mem);
            T chain_b = (T)0;
            r.template both_down<S - 1>(chain_b);
        }
        for (int q = 0; q < S - 1; ++q) {
            r.template fwd_down_to<S - 1>(q + 1);
            T chain_b = (T)0;
            r.template bwd_down<S - 1>(chain_b);
        }
        emit(v, r.clock[0]);
    }
}

// The all-forward-all-backward order (CM_SCHED_GPIPE): every micro-batch's forward runs up the
// stages, then every micro-batch's backward runs down; the per-stage clock is all the state.
template <typename T, int S, typename Src>
__device__ __forceinline__ T sim_afab(int m, const Src &src) {
    Rounds<T, S, Src> r(src);
#pragma unroll 4
    for (int j = 0; j < m; ++j) {
        T chain = (T)0;
        r.template fwd_up<0>(chain);
    }
#pragma unroll 4
    for (int j = 0; j < m; ++j) {
        T chain_b = (T)0;
        r.template bwd_down<S - 1>(chain_b);
    }
    return r.clock[0];
}

// Pipeline time of S stages under the order `sched`, stage times from `src`.
template <typename T, int S, typename Src, typename Pend = RegPend<T, S>>
__device__ __forceinline__ T sim_stages(int sched, int m, const Src &src, Pend pend = Pend()) {
    return sched == CM_SCHED_GPIPE ? sim_afab<T, S>(m, src) : sim_rounds<T, S, Src, Pend>(m, src, pend);
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

// sim_regs for m AND m+1 micro-batches (m >= S-1): warm-up and the m-S+1 steady rounds of the
// two recurrences coincide (see sim_rounds_pair) and run once; the state is parked in local
// memory, the cool-down of m runs and hands its time to emit(0, t); the state comes back, one
// more steady round and the cool-down give emit(1, t) for m+1.  The tails are one loop of two trips.
template <typename T, int S, typename Emit>
__device__ __forceinline__ void sim_regs_pair(int m, const FB<T> (&st)[S], const T (&xt)[S], Emit emit) {
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
    auto steady = [&]() {
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
    };
#pragma unroll 4
    for (int k = 0; k <= m - S; ++k) steady();
    T parked[2 * S];
    volatile T *mem = parked;   // volatile: real local-memory stores and loads, not 2S more registers
#pragma unroll
    for (int i = 0; i < S; ++i) { mem[i] = clock[i]; if (i > 0) mem[S + i] = pend[i]; }
#pragma unroll 1
    for (int v = 0; v < 2; ++v) {
        if (v) {
#pragma unroll
            for (int i = 0; i < S; ++i) { clock[i] = mem[i]; if (i > 0) pend[i] = mem[S + i]; }
            steady();
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
        emit(v, clock[0]);
    }
}

// ----------------------------------------------------------------------------------
// Cost of pipeline-plan kappa of a segment with S <= kRegStagesMax stages and m >= S-1
// micro-batches, everything in registers.  Returns false if the plan is infeasible.
// ----------------------------------------------------------------------------------
// ANY_M = true lifts the condition on m: the rounds form of the recurrence (any m >= 1) instead
// of the unrolled triangles -- for the few segments with fewer micro-batches than warm-up slots.
template <typename T, int S, bool ANY_M = false>
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
        ok = ok && hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
        st[i].f = sp.PF[hi] - sp.PF[lo];
        st[i].b = sp.PB[hi] - sp.PB[lo];
        xts[i] = i < S - 1 ? sp.XT[(g.tier >> i) & 1ull][hi - 1] : (T)0;
        const long long gb = sp.PP[hi] - sp.PP[lo];
        g_max = gb > g_max ? gb : g_max;
        lo = hi;
    }
    if (!ok) return false;
    T t;
    if constexpr (ANY_M) {
        if (m < 1) return false;
        const RegStages<T, S> src{st, xts};
        t = sim_stages<T, S>(sp.sched, m, src);
    } else if (sp.sched == CM_SCHED_GPIPE) {
        const RegStages<T, S> src{st, xts};
        t = sim_afab<T, S>(m, src);
    } else {
        t = sim_regs<T, S>(m, st, xts);
    }
    cost = t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    return true;
}

// The same for a micro-batch pair (Bucket::pair; 1F1B, m >= S): cost of the plan with m
// micro-batches and with m + 1, one composition, one recurrence.
template <typename T, int S>
__device__ __forceinline__ bool plan_cost_regs_pair(const SProf<T> &sp, const Tables &tb, int layer_mode,
                                                    const SegView &g, uint64_t kappa, T &cost_m, T &cost_m1) {
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
        ok = ok && hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
        st[i].f = sp.PF[hi] - sp.PF[lo];
        st[i].b = sp.PB[hi] - sp.PB[lo];
        xts[i] = i < S - 1 ? sp.XT[(g.tier >> i) & 1ull][hi - 1] : (T)0;
        const long long gb = sp.PP[hi] - sp.PP[lo];
        g_max = gb > g_max ? gb : g_max;
        lo = hi;
    }
    if (!ok) return false;
    const T sync = Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    sim_regs_pair<T, S>(m, st, xts, [&](int v, T t) { if (v) cost_m1 = t + sync; else cost_m = t + sync; });
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
        ok = hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
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
    const SmemStages<T, (int)sizeof(FB<T>) * kChunk, (int)sizeof(T) * kChunk> src{smem_addr(fcol), smem_addr(xcol)};
    const T t = sim_stages<T, S>(sp.sched, m, src);
    cost = t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    return true;
}

// The same for a micro-batch pair (Bucket::pair; 1F1B, m >= S): the plan with m micro-batches
// and with m + 1, one composition, one recurrence.
template <typename T, int S>
__device__ __forceinline__ bool plan_cost_wide_lane_pair(const SProf<T> &sp, const Tables &tb, int layer_mode, const SegView &g,
                                                         uint64_t kappa, FB<T> *fcol, T *xcol, T &cost_m, T &cost_m1) {
    const int m = g.m;
    CutWalker cw;
    bool ok = make_walker(cw, tb, layer_mode, sp.L, S, kappa, g.K, tb.mm_slot(S, m));
    long long g_max = 0;
    int lo = 0;
    for (int i = 0; i < S && ok; ++i) {
        const int hi = cw.next();
        ok = hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
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
    const SmemStages<T, (int)sizeof(FB<T>) * kChunk, (int)sizeof(T) * kChunk> src{smem_addr(fcol), smem_addr(xcol)};
    const T sync = Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval);
    sim_rounds_pair<T, S>(m, src, [&](int v, T t) { if (v) cost_m1 = t + sync; else cost_m = t + sync; });
    return true;
}

// The same with S chosen at run time (one kernel for every shallow depth; used where the
// work is too small to be worth one launch per depth).  Caller guarantees 1 <= S <= 16, and
// m >= S-1 unless ANY_M.
template <typename T, bool ANY_M = false>
__device__ __forceinline__ bool plan_cost_regs_any(const SProf<T> &sp, const Tables &tb, int layer_mode,
                                                   const SegView &g, uint64_t kappa, T &cost) {
    switch (g.S) {
#define CM_CASE(S) case S: return plan_cost_regs<T, S, ANY_M>(sp, tb, layer_mode, g, kappa, cost);
        CM_CASE(1) CM_CASE(2) CM_CASE(3) CM_CASE(4) CM_CASE(5) CM_CASE(6) CM_CASE(7) CM_CASE(8)
        CM_CASE(9) CM_CASE(10) CM_CASE(11) CM_CASE(12) CM_CASE(13) CM_CASE(14) CM_CASE(15) CM_CASE(16)
#undef CM_CASE
    default: return false;
    }
}

}  // namespace cm
