// Search pass of the plan search (sm_100a): every pipeline-plan of every segment ->
// least cost per segment.  This is the hot kernel: 2 * stages * micro-batches
// recurrence cells per plan (Section "Estimator", the start/end transition equation;
// the paper puts the estimator at O(N_pp x N_m) per asymmetric pipeline).
//
// Work layout: segments with the same (stages S, micro-batches m) are bucketed, so all
// lanes of a warp run recurrences of the same shape.  Three kernels share one evaluation
// order (sim_rounds below):
//
//   cm_cost_regs_kernel<T, S>       S = 1..16, m >= S-1.  One thread per plan, everything in
//       registers: stage forward/backward/transfer times, per-stage clock and pending
//       forward; every loop over stages is unrolled, so a cell costs its two adds and one
//       max and nothing else.
//   cm_cost_wide_kernel<T, S, UNI>  S = 17..64.  Up to 48 stages clock and pending forward stay in
//       registers (4 S of them), the stage times move to shared memory.
//       UNI = true ("transposed"): the 32 lanes of a warp take the SAME layer composition
//       in 32 DIFFERENT segments of the bucket (they differ in link tiers and sync
//       peers only), so stage times are warp-uniform -- one broadcast 16-byte load per
//       stage and round -- and memory feasibility is decided once per warp.
//       UNI = false: one plan per lane as in the register kernel, stage times in a
//       per-lane shared-memory column; for buckets with too few segments to transpose.
//       S = 49..64 (transposed only): the pending forwards move to a per-lane shared-memory
//       column as well; one CTA per SM.
//   cm_cost_short_kernel<T>         S <= 16 with m < S-1: the rounds form, all in registers.
#pragma once

#include <atomic>

#include "cm_plan_eval.cuh"

namespace cm {

// Bucket that owns a chunk: the last bucket of the class whose first chunk is not above it.
__device__ __forceinline__ uint32_t find_bucket(const Bucket *bk, uint32_t b0, uint32_t b1, uint64_t chunk) {
    uint32_t lo = b0, hi = b1 - 1;
    while (lo < hi) {
        uint32_t mid = (lo + hi + 1) >> 1;
        if (bk[mid].chunk_first <= chunk) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// (segment-in-bucket, kappa) of plan `tid` of a chunk whose first plan is `base`
// (plan-major buckets: index = segment-in-bucket * count + kappa).
__device__ __forceinline__ void plan_of_thread(uint64_t base, uint64_t count, uint32_t tid,
                                               uint64_t &seg_local, uint64_t &kappa) {
    const uint64_t seg0 = base / count, rem0 = base - seg0 * count;
    if (count > (uint64_t)kChunk) {
        const uint64_t x = rem0 + tid;
        const bool wrap = x >= count;
        seg_local = seg0 + (wrap ? 1 : 0);
        kappa = wrap ? x - count : x;
    } else {
        const uint32_t x = (uint32_t)rem0 + tid, c = (uint32_t)count;
        const uint32_t q = x / c;
        seg_local = seg0 + q;
        kappa = x - q * c;
    }
}

// Segment number `seg_local` of a bucket = (template segment of the bucket, scenario of the
// template), scenario minor.
__device__ __forceinline__ SegView bucket_segment(const BatchDev &bd, const Bucket &bk, uint32_t seg_local) {
    if (bk.tmpl == kSharedBucket) {   // a range of the list of distinct segments
        const uint2 p = bd.useg[bk.list_first + seg_local];
        return seg_view(bd, p.x, p.y + (bk.pair == 2 ? 1u : 0u));   // pair == 2: the second rows of a list of pair heads
    }
    const Tmpl &tp = bd.tmpl[bk.tmpl];
    const uint32_t ti = seg_local / tp.n_scen, si = seg_local - ti * tp.n_scen;
    return seg_view(bd, bd.tmpl_scen[tp.scen_first + si], bd.bucket_tseg[bk.list_first + ti]);
}

// Least cost per segment from per-lane (segment row, cost bits): lanes of one segment
// are contiguous, so a segmented shuffle scan leaves each run's minimum in its last lane,
// which issues the one atomicMin.
__device__ __forceinline__ void segmented_min_commit(uint64_t *seg_best, uint32_t row, uint64_t bits, uint64_t inf) {
    const uint32_t lane = threadIdx.x & 31;
    for (int o = 1; o < 32; o <<= 1) {
        const uint64_t ov = __shfl_up_sync(0xffffffffu, bits, o);
        const uint32_t orow = __shfl_up_sync(0xffffffffu, row, o);
        if (lane >= (uint32_t)o && orow == row && ov < bits) bits = ov;
    }
    const uint32_t next_row = __shfl_down_sync(0xffffffffu, row, 1);
    const bool last = lane == 31 || next_row != row;
    if (last && row != 0xffffffffu && bits < inf) atomicMin((unsigned long long *)&seg_best[row], (unsigned long long)bits);
}

// Work counters of the search pass: recurrence cells simulated and plans whose recurrence ran
// (the memory-feasible ones).  A thread reports both in one word -- cells in the low 40 bits,
// plans above -- so that one shuffle reduction serves both; counters[0] takes the cells,
// counters[2] the plans.
constexpr int kWorkPlanShift = 40;
__device__ __forceinline__ unsigned long long one_plan(unsigned long long cells) { return cells + (1ull << kWorkPlanShift); }
// a pair (m and m + 1 micro-batches in one recurrence, sim_rounds_pair): the cells of the longer
// recurrence plus the ramp-down of the shorter one (S-1 rounds of S backwards and S-1-q forwards)
template <int S> __device__ __forceinline__ unsigned long long pair_plans(int m) {
    return 2ull * S * (m + 1) + 3ull * S * (S - 1) / 2 + (2ull << kWorkPlanShift);
}
__device__ __forceinline__ void add_work(unsigned long long *counters, unsigned long long packed) {
    if (!packed) return;
    atomicAdd(&counters[0], packed & ((1ull << kWorkPlanShift) - 1ull));
    atomicAdd(&counters[2], packed >> kWorkPlanShift);
}
__device__ __forceinline__ void count_cells(unsigned long long *counters, unsigned long long my_work,
                                            unsigned long long *smem /* [kChunk/32] */) {
    for (int o = 16; o > 0; o >>= 1) my_work += __shfl_xor_sync(0xffffffffu, my_work, o);
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = my_work;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long c = 0;
        for (int w = 0; w < kChunk / 32; ++w) c += smem[w];
        add_work(counters, c);
    }
}

// ----------------------------------------------------------------------------------
// S <= 16: one thread per plan, all in registers.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__global__ void __launch_bounds__(kChunk) cm_cost_regs_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1,
                                                              uint64_t chunk_offset) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        row = g.row;
        T cost;
        if (plan_cost_regs<T, S>(sp, tb, bd.layer_mode, g, kappa, cost)) {
            bits = Num<T>::bits(cost);
            my_cells = one_plan(2ull * S * g.m);
        }
    }
    segmented_min_commit(bd.seg_best, row, bits, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

// The same over micro-batch pairs (Bucket::pair): a thread evaluates its plan for the segment
// (m micro-batches) and for the next row (the same pipeline with m + 1) in one recurrence.
template <typename T, int S>
__global__ void __launch_bounds__(kChunk) cm_cost_regs_pair_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1,
                                                                   uint64_t chunk_offset) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits0 = inf_bits<T>(), bits1 = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        row = g.row;
        T c0, c1;
        if (plan_cost_regs_pair<T, S>(sp, tb, bd.layer_mode, g, kappa, c0, c1)) {
            bits0 = Num<T>::bits(c0);
            bits1 = Num<T>::bits(c1);
            my_cells = pair_plans<S>(g.m);
        }
    }
    segmented_min_commit(bd.seg_best, row, bits0, inf_bits<T>());
    segmented_min_commit(bd.seg_best, row == 0xffffffffu ? row : row + 1, bits1, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

// Every shallow depth in one launch: for batches so small that a launch per depth would
// cost more than the work (a single failure scenario of a 32-device job is ~250 CTAs).
template <typename T>
__global__ void __launch_bounds__(kChunk) cm_cost_regs_any_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = (uint64_t)blockIdx.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        row = g.row;
        T cost;
        if (plan_cost_regs_any<T>(sp, tb, bd.layer_mode, g, kappa, cost)) {
            bits = Num<T>::bits(cost);
            my_cells = one_plan(2ull * g.S * g.m);
        }
    }
    segmented_min_commit(bd.seg_best, row, bits, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

// ----------------------------------------------------------------------------------
// 16 < S <= 48: stage times in shared memory.
// Dynamic shared memory:  UNI:  FB<T> fb[4 warps][S] | T xt[S][128] | uint8 cuts[4][S+1]
//                         !UNI: FB<T> fb[S][128]     | T xt[S][128]
// ----------------------------------------------------------------------------------
#ifndef CM_WIDE3
#define CM_WIDE3 34   // deepest pipeline compiled for three resident CTAs per SM (<= 168 registers)
#endif
// Transposed kernel: up to this depth a warp takes several items per CTA (see the kernel);
// deeper pipelines keep one item per warp -- their items are long enough to hide the CTA's
// fixed cost, and their recurrence leaves no register for anything carried across it.
#define CM_UNI_BATCH_STAGES kUniBatchStagesMax
// Beyond kWideStagesMax stages the pending forwards move to a second per-lane column behind the
// cuts (transposed layout only: a per-lane column of stage times as well would not fit).
template <int S, bool UNI, typename T> constexpr size_t wide_smem_bytes() {
    return UNI ? sizeof(FB<T>) * 4 * S + sizeof(T) * S * kChunk + 4 * (((S + 1) + 7) / 8 * 8) +
                     (S > kWideStagesMax ? sizeof(T) * S * kChunk : 0)
               : sizeof(FB<T>) * S * kChunk + sizeof(T) * S * kChunk;
}
template <int S> constexpr int wide_ctas_per_sm() { return S <= CM_WIDE3 ? 3 : (S <= kWideStagesMax ? 2 : 1); }

// Transposed kernel, per warp item: the layer composition kappa of an (S, m) bucket is the same
// in all 32 segments the warp evaluates, so its cuts, stage times and memory check are worked
// out once per warp -- every lane walks the cuts (lane 0 keeps them in `cuts`), then the stages
// are shared out over the lanes for the sums and the check.  Returns, warp-uniform, whether
// the composition is feasible; g_max = largest gradient bytes of a stage (in every lane).
template <typename T, int S>
__device__ __forceinline__ bool uni_composition(const SProf<T> &sp, const Tables &tb, int layer_mode, int m, uint64_t kappa,
                                                uint64_t K, FB<T> *fb, uint8_t *cuts, uint32_t lane, long long &g_max) {
    CutWalker cw;
    bool ok = make_walker(cw, tb, layer_mode, sp.L, S, kappa, K, tb.mm_slot(S, m));
    if (ok) {
        int lo = 0;
        for (int i = 0; i < S; ++i) {
            const int hi = cw.next();
            ok = ok && hi > lo;
            if (lane == 0) cuts[i + 1] = (uint8_t)hi;
            lo = hi;
        }
        if (lane == 0) cuts[0] = 0;
    }
    __syncwarp();
    g_max = 0;
    if (ok) {
        for (int i = lane; i < S; i += 32) {
            const int lo = cuts[i], hi = cuts[i + 1];
            ok = ok && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
            FB<T> d;
            d.f = sp.PF[hi] - sp.PF[lo];
            d.b = sp.PB[hi] - sp.PB[lo];
            fb[i] = d;
            const long long gb = sp.PP[hi] - sp.PP[lo];
            g_max = gb > g_max ? gb : g_max;
        }
        for (int o = 16; o > 0; o >>= 1) {
            const long long og = __shfl_xor_sync(0xffffffffu, g_max, o);
            g_max = og > g_max ? og : g_max;
        }
    }
    return __all_sync(0xffffffffu, ok);
}

template <typename T, int S, bool UNI>
__global__ void __launch_bounds__(kChunk, wide_ctas_per_sm<S>()) cm_cost_wide_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset, int uni_items) {
    static_assert(UNI || S <= kWideStagesMax, "pipelines deeper than kWideStagesMax exist in the transposed layout only");
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    extern __shared__ __align__(16) unsigned char dyn[];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const int m = bk.m;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    unsigned long long my_cells = 0;

    if (UNI) {
        // warp item = (kappa, group of 32 segments), group minor.  Up to CM_UNI_BATCH_STAGES a warp
        // takes uni_items consecutive items, so that the CTA's fixed cost (staging the profile) is
        // spread over more work and a composition shared by consecutive groups is set up only
        // once; everything an item needs from the previous one lives in shared memory -- nothing
        // but the loop counter stays in registers across the recurrence, whose per-stage state
        // needs nearly all of them.  Deeper pipelines keep one item per warp.
        constexpr bool kBatch = S <= CM_UNI_BATCH_STAGES;
        __shared__ Bucket bks;
        __shared__ unsigned long long st_kappa[kChunk / 32];
        __shared__ long long st_gmax[kChunk / 32];
        __shared__ int st_ok[kChunk / 32];
        if (tid == 0) bks = bk;
        if (lane == 0) { st_kappa[warp] = ~0ull; st_ok[warp] = 0; st_gmax[warp] = 0; cells_w[warp] = 0; }
        __syncthreads();
        FB<T> *fb = reinterpret_cast<FB<T> *>(dyn) + warp * S;
        T *xcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * 4 * S) + tid;           // [i * kChunk]
        uint8_t *cuts = dyn + sizeof(FB<T>) * 4 * S + sizeof(T) * S * kChunk + warp * (((S + 1) + 7) / 8 * 8);
        const int n_items = kBatch ? uni_items : 1;
        for (int r = 0; r < n_items; ++r) {
            const uint64_t item = ((chunk - bks.chunk_first) * (kChunk / 32) + warp) * (uint64_t)n_items + r;
            const uint32_t n_groups = (bks.n_seg + 31) / 32;
            const uint64_t pos = item / n_groups;              // position in the bucket's walk
            if (pos >= bks.count || m < 1) break;              // warp-uniform; items ascend
            const uint64_t kappa = walk_kappa(bd.feas, bks.feas_first, pos);
            const uint32_t seg_local = (uint32_t)(item - pos * n_groups) * 32 + lane;
            const bool active = seg_local < bks.n_seg;
            const SegView g = bucket_segment(bd, bks, active ? seg_local : 0);
            if (kappa != st_kappa[warp]) {
                long long g_max;
                const bool ok = uni_composition<T, S>(sp, tb, bd.layer_mode, m, kappa, g.K, fb, cuts, lane, g_max);
                if (lane == 0) { st_kappa[warp] = kappa; st_ok[warp] = ok ? 1 : 0; st_gmax[warp] = g_max; }
                __syncwarp();
            }
            if (st_ok[warp]) {
                // transfer times of this lane's segment (its own link tiers)
                for (int i = 0; i < S - 1; ++i) xcol[i * kChunk] = sp.XT[(g.tier >> i) & 1ull][cuts[i + 1] - 1];
                const uint32_t row = g.row;
                const int n_sync = g.n_sync;
                __syncwarp();
                const SmemStages<T, (int)sizeof(FB<T>), (int)sizeof(T) * kChunk> src{smem_addr(fb), smem_addr(xcol)};
                T t;
                if constexpr (S <= kWideStagesMax) {
                    t = sim_stages<T, S>(sp.sched, m, src);
                } else {
                    // 8-byte aligned column behind the four cut rows
                    T *pcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * 4 * S + sizeof(T) * S * kChunk + 4 * (((S + 1) + 7) / 8 * 8)) + tid;
                    using ColPend = SmemPend<T, (int)sizeof(T) * kChunk>;
                    t = sim_stages<T, S, SmemStages<T, (int)sizeof(FB<T>), (int)sizeof(T) * kChunk>, ColPend>(sp.sched, m, src, ColPend{smem_addr(pcol)});
                }
                if (active) {
                    const uint64_t bits = Num<T>::bits(t + Num<T>::sync(st_gmax[warp], n_sync, sp.bw_sync, sp.intval));
                    if (bits < bd.seg_best[row]) atomicMin((unsigned long long *)&bd.seg_best[row], (unsigned long long)bits);
                }
                const uint32_t n_active = __popc(__ballot_sync(0xffffffffu, active));
                if (lane == 0) cells_w[warp] += one_plan(2ull * S * m) * n_active;
                __syncwarp();   // the next item overwrites the stage times and cuts
            }
        }
        __syncthreads();
        if (tid == 0) {
            unsigned long long c = 0;
            for (int w = 0; w < kChunk / 32; ++w) c += cells_w[w];
            add_work(bd.counters, c);
        }
        return;
    } else {
        FB<T> *fcol = reinterpret_cast<FB<T> *>(dyn) + tid;                               // [i * kChunk]
        T *xcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * S * kChunk) + tid;           // [i * kChunk]
        const uint64_t base = (chunk - bk.chunk_first) * kChunk;
        uint64_t seg_local, kappa;
        plan_of_thread(base, bk.count, tid, seg_local, kappa);
        if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
        uint32_t row = 0xffffffffu;
        uint64_t bits = inf_bits<T>();
        if (seg_local < bk.n_seg && m >= 1) {
            const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
            row = g.row;
            T cost;
            if (plan_cost_wide_lane<T, S>(sp, tb, bd.layer_mode, g, kappa, fcol, xcol, cost)) {
                bits = Num<T>::bits(cost);
                my_cells = one_plan(2ull * S * m);
            }
        }
        segmented_min_commit(bd.seg_best, row, bits, inf_bits<T>());
    }
    count_cells(&bd.counters[0], my_cells, cells_w);
}

// ----------------------------------------------------------------------------------
// Micro-batch pairs, 17 <= S <= 48, transposed layout: every segment of the bucket stands for
// itself (m micro-batches) and its next row (the same pipeline with m + 1); one recurrence
// serves both (sim_rounds_pair).  Built only for 1F1B with m >= S, where the two walk the same
// feasible compositions and have the same min-max partition (a stage holds S - i micro-batches
// in flight either way), so the composition is set up once, with m.  What the two commits need
// (row, peers) waits in the free last entry of the lane's transfer-time column, not in registers.
// Dynamic shared memory as the transposed cm_cost_wide_kernel.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__global__ void __launch_bounds__(kChunk, wide_ctas_per_sm<S>()) cm_cost_pair_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset, int uni_items) {
    static_assert(S >= kPairStagesMin && S <= kPairStagesMax, "pairs exist for the register-resident deep kernels only");
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    __shared__ Bucket bks;
    __shared__ unsigned long long st_kappa[kChunk / 32];
    __shared__ long long st_gmax[kChunk / 32];
    __shared__ int st_ok[kChunk / 32];
    extern __shared__ __align__(16) unsigned char dyn[];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    if (tid == 0) bks = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    if (lane == 0) { st_kappa[warp] = ~0ull; st_ok[warp] = 0; st_gmax[warp] = 0; cells_w[warp] = 0; }
    __syncthreads();
    constexpr bool kBatch = S <= CM_UNI_BATCH_STAGES;
    FB<T> *fb = reinterpret_cast<FB<T> *>(dyn) + warp * S;
    T *xcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * 4 * S) + tid;           // [i * kChunk]
    uint8_t *cuts = dyn + sizeof(FB<T>) * 4 * S + sizeof(T) * S * kChunk + warp * (((S + 1) + 7) / 8 * 8);
    unsigned long long *note = reinterpret_cast<unsigned long long *>(xcol + (S - 1) * kChunk);   // entry S-1 holds no transfer time
    const int n_items = kBatch ? uni_items : 1;
    for (int r = 0; r < n_items; ++r) {
        const int m = bks.m;
        const uint64_t item = ((chunk - bks.chunk_first) * (kChunk / 32) + warp) * (uint64_t)n_items + r;
        const uint32_t n_groups = (bks.n_seg + 31) / 32;
        const uint64_t pos = item / n_groups;
        if (pos >= bks.count) break;                       // warp-uniform; items ascend
        const uint64_t kappa = walk_kappa(bd.feas, bks.feas_first, pos);
        const uint32_t seg_local = (uint32_t)(item - pos * n_groups) * 32 + lane;
        const bool active = seg_local < bks.n_seg;
        const SegView g = bucket_segment(bd, bks, active ? seg_local : 0);
        if (kappa != st_kappa[warp]) {
            long long g_max;
            const bool ok = uni_composition<T, S>(sp, tb, bd.layer_mode, m, kappa, g.K, fb, cuts, lane, g_max);
            if (lane == 0) { st_kappa[warp] = kappa; st_ok[warp] = ok ? 1 : 0; st_gmax[warp] = g_max; }
            __syncwarp();
        }
        if (st_ok[warp]) {
            for (int i = 0; i < S - 1; ++i) xcol[i * kChunk] = sp.XT[(g.tier >> i) & 1ull][cuts[i + 1] - 1];
            *note = active ? ((unsigned long long)g.n_sync << 32) | g.row : ~0ull;
            __syncwarp();
            const SmemStages<T, (int)sizeof(FB<T>), (int)sizeof(T) * kChunk> src{smem_addr(fb), smem_addr(xcol)};
            // (the commit works from the thread index and shared memory alone: it keeps no register
            // alive across the recurrence)
            sim_rounds_pair<T, S>(m, src, [&bd](int v, T t) {
                const unsigned long long nt =
                    reinterpret_cast<const unsigned long long *>(dyn + sizeof(FB<T>) * 4 * S + sizeof(T) * (S - 1) * kChunk)[threadIdx.x];
                if (nt == ~0ull) return;
                const uint32_t row = (uint32_t)nt + (uint32_t)v;
                const uint64_t bits = Num<T>::bits(t + Num<T>::sync(st_gmax[threadIdx.x >> 5], (int)(nt >> 32), sp.bw_sync, sp.intval));
                if (bits < bd.seg_best[row]) atomicMin((unsigned long long *)&bd.seg_best[row], (unsigned long long)bits);
            });
            const uint32_t n_active = __popc(__ballot_sync(0xffffffffu, *note != ~0ull));
            if (lane == 0) cells_w[warp] += pair_plans<S>(bks.m) * n_active;
            __syncwarp();   // the next item overwrites the stage times and cuts
        }
    }
    __syncthreads();
    if (tid == 0) {
        unsigned long long c = 0;
        for (int w = 0; w < kChunk / 32; ++w) c += cells_w[w];
        add_work(bd.counters, c);
    }
}

// Micro-batch pairs in the per-lane layout (buckets with too few pairs for a transposed warp:
// a failure handled on its own): one plan per lane, evaluated for the segment and for its next
// row.  Dynamic shared memory as the per-lane cm_cost_wide_kernel.
template <typename T, int S>
__global__ void __launch_bounds__(kChunk, wide_ctas_per_sm<S>()) cm_cost_lane_pair_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset) {
    static_assert(S >= kPairStagesMin && S <= kPairStagesMax, "pairs exist for the register-resident deep kernels only");
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    extern __shared__ __align__(16) unsigned char dyn[];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint32_t tid = threadIdx.x;
    FB<T> *fcol = reinterpret_cast<FB<T> *>(dyn) + tid;                               // [i * kChunk]
    T *xcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * S * kChunk) + tid;           // [i * kChunk]
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, tid, seg_local, kappa);
    if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits0 = inf_bits<T>(), bits1 = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        row = g.row;
        T c0, c1;
        if (plan_cost_wide_lane_pair<T, S>(sp, tb, bd.layer_mode, g, kappa, fcol, xcol, c0, c1)) {
            bits0 = Num<T>::bits(c0);
            bits1 = Num<T>::bits(c1);
            my_cells = pair_plans<S>(bk.m);
        }
    }
    segmented_min_commit(bd.seg_best, row, bits0, inf_bits<T>());
    segmented_min_commit(bd.seg_best, row == 0xffffffffu ? row : row + 1, bits1, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

// Shallow pipelines (<= 16 stages) with fewer micro-batches than warm-up slots (m < S-1): the
// rounds form of the recurrence, state and stage times in registers, every such depth in one launch.
template <typename T>
__global__ void __launch_bounds__(kChunk) cm_cost_short_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    if (seg_local < bk.n_seg) kappa = walk_kappa(bd.feas, bk.feas_first, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        row = g.row;
        T cost;
        if (plan_cost_regs_any<T, true>(sp, tb, bd.layer_mode, g, kappa, cost)) {
            bits = Num<T>::bits(cost);
            my_cells = one_plan(2ull * g.S * g.m);
        }
    }
    segmented_min_commit(bd.seg_best, row, bits, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

static dim3 chunk_grid(uint64_t n) {
    const uint64_t maxx = 1u << 30;
    if (n <= maxx) return dim3((unsigned)n, 1, 1);
    return dim3((unsigned)maxx, (unsigned)((n + maxx - 1) / maxx), 1);
}

template <typename T, int S>
static cudaError_t launch_regs(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_regs_kernel<T, S><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

template <typename T, int S, bool UNI>
static cudaError_t launch_wide_one(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    constexpr size_t smem = wide_smem_bytes<S, UNI, T>();
    // One bit per device: the attribute sticks to the function on that device.  Setting it is
    // idempotent, so two host threads (distinct contexts) that both find the bit clear both set
    // it; the bit itself is atomic.
    static std::atomic<uint64_t> configured{0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 64 || !((configured.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(cm_cost_wide_kernel<T, S, UNI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    cm_cost_wide_kernel<T, S, UNI><<<chunk_grid(c.n_chunks), kChunk, smem, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin, (int)c.uni_items);
    return cudaGetLastError();
}

template <typename T, int S>
static cudaError_t launch_pair_one(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    constexpr size_t smem = wide_smem_bytes<S, true, T>();
    static std::atomic<uint64_t> configured{0};   // as in launch_wide_one
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 64 || !((configured.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(cm_cost_pair_kernel<T, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    cm_cost_pair_kernel<T, S><<<chunk_grid(c.n_chunks), kChunk, smem, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin, (int)c.uni_items);
    return cudaGetLastError();
}

template <typename T, int S>
static cudaError_t launch_lane_pair_one(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    constexpr size_t smem = wide_smem_bytes<S, false, T>();
    static std::atomic<uint64_t> configured{0};   // as in launch_wide_one
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 64 || !((configured.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(cm_cost_lane_pair_kernel<T, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    cm_cost_lane_pair_kernel<T, S><<<chunk_grid(c.n_chunks), kChunk, smem, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

template <typename T, int S>
static cudaError_t launch_wide(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    if (c.kind == CM_CLASS_WIDE_PAIR || c.kind == CM_CLASS_WIDE_LANE_PAIR) {
        if constexpr (S >= kPairStagesMin && S <= kPairStagesMax)
            return c.kind == CM_CLASS_WIDE_PAIR ? launch_pair_one<T, S>(t, b, c, st) : launch_lane_pair_one<T, S>(t, b, c, st);
        else return cudaErrorInvalidValue;
    }
    if constexpr (S > kWideStagesMax) return c.kind == CM_CLASS_WIDE_UNI ? launch_wide_one<T, S, true>(t, b, c, st) : cudaErrorInvalidValue;
    else return c.kind == CM_CLASS_WIDE_UNI ? launch_wide_one<T, S, true>(t, b, c, st) : launch_wide_one<T, S, false>(t, b, c, st);
}


// ---------------------------------------------------------------------------------
// Launchers per cost type.  They are explicitly instantiated in four translation units
// (shallow / deep x fp64 / int64) so that the hundred-odd kernel instantiations compile
// side by side; cm_cost.cu only dispatches.
// ---------------------------------------------------------------------------------
template <typename T>
cudaError_t launch_shallow_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    switch (c.stages) {
#define CM_CASE(S) case S: return launch_regs<T, S>(t, b, c, st);
        CM_CASE(1) CM_CASE(2) CM_CASE(3) CM_CASE(4) CM_CASE(5) CM_CASE(6) CM_CASE(7) CM_CASE(8)
        CM_CASE(9) CM_CASE(10) CM_CASE(11) CM_CASE(12) CM_CASE(13) CM_CASE(14) CM_CASE(15) CM_CASE(16)
#undef CM_CASE
    default: return cudaErrorInvalidValue;
    }
}

template <typename T, int S>
static cudaError_t launch_regs_pair(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_regs_pair_kernel<T, S><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_shallow_pair_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    switch (c.stages) {
#define CM_CASE(S) case S: return launch_regs_pair<T, S>(t, b, c, st);
        CM_CASE(1) CM_CASE(2) CM_CASE(3) CM_CASE(4) CM_CASE(5) CM_CASE(6) CM_CASE(7) CM_CASE(8)
        CM_CASE(9) CM_CASE(10) CM_CASE(11) CM_CASE(12) CM_CASE(13) CM_CASE(14) CM_CASE(15) CM_CASE(16)
#undef CM_CASE
    default: return cudaErrorInvalidValue;
    }
}

template <typename T>
cudaError_t launch_shallow_any(const Tables &t, const BatchDev &b, uint32_t b0, uint32_t b1, uint64_t chunks, cudaStream_t st) {
    cm_cost_regs_any_kernel<T><<<(unsigned)chunks, kChunk, 0, st>>>(t, b, b0, b1);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_short_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_short_kernel<T><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

// Deep pipelines are instantiated per stage count; the stage counts LO .. HI of one cost type
// form one translation unit (cm_cost_deep.cu, compiled once per range), so that the kernel
// instantiations compile side by side.
template <typename T, int S, int HI>
static cudaError_t deep_dispatch(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    if (c.stages == S) return launch_wide<T, S>(t, b, c, st);
    if constexpr (S < HI) return deep_dispatch<T, S + 1, HI>(t, b, c, st);
    else return cudaErrorInvalidValue;
}
template <typename T, int LO, int HI>
cudaError_t launch_deep_range(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    return deep_dispatch<T, LO, HI>(t, b, c, st);
}

// ----------------------------------------------------------------------------------
// Tie-break pass for the winners' deep pipelines (17..48 stages): the lowest layer
// composition that is feasible with cost <= T*.  Same grid as the generic tie-break
// kernel -- x = (scenario, pipeline), y = tiles of kChunk compositions -- one launch per
// stage count; CTAs whose winner segment has another depth leave at once.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__global__ void __launch_bounds__(kChunk, wide_ctas_per_sm<S>()) cm_tiebreak_wide_kernel(Tables tb, BatchDev bd) {
    __shared__ SProf<T> sp;
    __shared__ uint64_t red[kChunk / 32];
    __shared__ SegView g;
    __shared__ uint64_t found_so_far;
    extern __shared__ __align__(16) unsigned char dyn[];
    const uint32_t b = blockIdx.x / bd.dp_max, p = blockIdx.x % bd.dp_max;
    const Winner &w = bd.winner[b];
    if (w.cost_bits >= inf_bits<T>() || p >= w.dp) return;            // uniform over the CTA
    if (bd.tseg[w.seg[p]].S != S) return;
    stage_profile(sp, tb);
    FB<T> *fcol = reinterpret_cast<FB<T> *>(dyn) + threadIdx.x;
    T *xcol = reinterpret_cast<T *>(dyn + sizeof(FB<T>) * S * kChunk) + threadIdx.x;
    uint64_t *slot = &bd.kappa_sel[b * kMaxP + p];
    for (uint64_t tile = blockIdx.y; tile < bd.max_tiles_per_seg; tile += gridDim.y) {
        __syncthreads();
        if (threadIdx.x == 0) {
            g = seg_view(bd, w.scen, w.seg[p]);
            found_so_far = *(volatile uint64_t *)slot;
        }
        __syncthreads();
        const uint64_t count = walk_count(g);
        const uint64_t first = tile * kChunk;
        // uniform: later tiles hold higher compositions than one already found
        if (first >= count || found_so_far <= walk_kappa(bd.feas, g.feas_first, first)) break;
        uint64_t hit = ~0ull;
        if (first + threadIdx.x < count) {
            const uint64_t kappa = walk_kappa(bd.feas, g.feas_first, first + threadIdx.x);
            T cost;
            if (plan_cost_wide_lane<T, S>(sp, tb, bd.layer_mode, g, kappa, fcol, xcol, cost) &&
                Num<T>::bits(cost) <= w.cost_bits)
                hit = kappa;
        }
        hit = warp_min_u64(hit);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = hit;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int q = 0; q < kChunk / 32; ++q) hit = red[q] < hit ? red[q] : hit;
            if (hit != ~0ull) atomicMin((unsigned long long *)slot, (unsigned long long)hit);
            const uint64_t n = count - first < (uint64_t)kChunk ? count - first : (uint64_t)kChunk;
            atomicAdd(&bd.counters[1], (unsigned long long)n);
        }
    }
}

template <typename T, int S>
static cudaError_t launch_tiebreak_wide_one(const Tables &t, const BatchDev &b, cudaStream_t st) {
    constexpr size_t smem = wide_smem_bytes<S, false, T>();
    static std::atomic<uint64_t> configured{0};   // as in launch_wide_one
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 64 || !((configured.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(cm_tiebreak_wide_kernel<T, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    const uint64_t nx = (uint64_t)b.B * b.dp_max;
    if (nx >= (1ull << 31)) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)nx, tiebreak_grid_y(nx, b.max_tiles_per_seg), 1);
    cm_tiebreak_wide_kernel<T, S><<<grid, kChunk, smem, st>>>(t, b);
    return cudaGetLastError();
}

template <typename T, int S, int HI>
static cudaError_t tiebreak_dispatch(const Tables &t, const BatchDev &b, int stages, cudaStream_t st) {
    if constexpr (S <= kWideStagesMax) {   // deeper winners are completed by the generic tie-break kernel
        if (stages == S) return launch_tiebreak_wide_one<T, S>(t, b, st);
    }
    if constexpr (S < HI) return tiebreak_dispatch<T, S + 1, HI>(t, b, stages, st);
    else return cudaSuccess;
}
template <typename T, int LO, int HI>
cudaError_t launch_tiebreak_range(const Tables &t, const BatchDev &b, int S, cudaStream_t st) {
    return tiebreak_dispatch<T, LO, HI>(t, b, S, st);
}

}  // namespace cm
