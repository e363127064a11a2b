// Search pass of the plan search (sm_100a): every pipeline-plan of every segment ->
// least cost per segment.  This is the hot kernel: 2 * stages * micro-batches
// recurrence cells per plan (Section "Estimator", the start/end transition equation;
// the paper puts the estimator at O(N_pp x N_m) per asymmetric pipeline).
//
// Work layout: segments with the same (stages S, micro-batches m) are bucketed, a CTA
// takes kChunk consecutive pipeline-plans of one bucket, one thread per plan, so all
// lanes of a warp run recurrences of the same shape.
//
//   cm_cost_regs_kernel<T, S>   S compile-time (1..kRegStagesMax), m >= S-1: the whole
//       per-plan state -- stage forward/backward/transfer times, per-stage clock and
//       pending forward -- lives in registers and every loop over stages is unrolled,
//       so a cell costs its two adds and one max and nothing else.
//   cm_cost_generic_kernel<T>   any S <= CM_MAX_STAGES and any m: same arithmetic with
//       the per-stage state in local memory.
//
// The recurrence is latency-bound along the backward chain of one plan (each cell needs
// the previous cell's end) but the forwards of a round are independent of it, and warps
// of other plans fill the remaining issue slots.
#include "cm_device.cuh"

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

// (segment-in-bucket, kappa) of plan `tid` of a chunk whose first plan is `base`.
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

__device__ __forceinline__ void count_cells(unsigned long long *counter, unsigned long long my_cells,
                                            unsigned long long *smem /* [kChunk/32] */) {
    for (int o = 16; o > 0; o >>= 1) my_cells += __shfl_xor_sync(0xffffffffu, my_cells, o);
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = my_cells;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long c = 0;
        for (int w = 0; w < kChunk / 32; ++w) c += smem[w];
        if (c) atomicAdd(counter, c);
    }
}

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
// Register-resident recurrence, S compile-time, m >= S-1 (every stage has its full
// warm-up).  Same dependency order as sim_pipe; the steady rounds k = 0..m-S need no
// predicate at all, warm-up and cool-down are unrolled triangles.
// ----------------------------------------------------------------------------------
template <typename T, int S>
__device__ __forceinline__ T sim_regs(int m, const T (&F)[S], const T (&B)[S], const T (&xt)[S]) {
    T clock[S], pend[S];
#pragma unroll
    for (int i = 0; i < S; ++i) { clock[i] = (T)0; pend[i] = (T)0; }
    // warm-up forwards: micro-batch j runs up stages 0 .. S-2-j
#pragma unroll
    for (int j = 0; j < S - 1; ++j) {
        T chain = (T)0;
#pragma unroll
        for (int i = 0; i <= S - 2 - j; ++i) {
            const T start = i > 0 ? tmax(clock[i], chain) : clock[i];
            const T end = start + F[i];
            clock[i] = end;
            chain = end + xt[i];
        }
        pend[S - 1 - j] = chain;
    }
    // steady rounds: every stage does one forward and one backward
    for (int k = 0; k <= m - S; ++k) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            const T fstart = i > 0 ? tmax(clock[i], pend[i]) : clock[i];
            const T fend = fstart + F[i];
            if (i < S - 1) pend[i + 1] = fend + xt[i];
            const T dep = i < S - 1 ? chain_b + xt[i] : fend;
            const T bstart = tmax(fend, dep);
            const T bend = bstart + B[i];
            clock[i] = bend;
            chain_b = bend;
        }
    }
    // cool-down rounds r = 0..S-2: only stages above r still have a forward left
#pragma unroll
    for (int r = 0; r < S - 1; ++r) {
        T chain_b = (T)0;
#pragma unroll
        for (int i = S - 1; i >= 0; --i) {
            T c = clock[i];
            T fend = (T)0;
            if (i > r) {
                const T fstart = i > 0 ? tmax(c, pend[i]) : c;
                fend = fstart + F[i];
                c = fend;
                if (i < S - 1) pend[i + 1] = fend + xt[i];
            }
            const T dep = i < S - 1 ? chain_b + xt[i] : fend;
            const T bstart = tmax(c, dep);
            const T bend = bstart + B[i];
            clock[i] = bend;
            chain_b = bend;
        }
    }
    return clock[0];
}

template <typename T, int S>
__global__ void __launch_bounds__(kChunk) cm_cost_regs_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb.prof);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const int m = bk.m, L = sp.L;
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        row = bd.order[bk.seg_begin + seg_local];
        const Seg *g = bd.seg + row;
        const uint64_t tier = g->tier_mask, K = g->K;
        const int n_sync = g->n_sync;
        CutWalker cw;
        bool ok = make_walker(cw, tb, bd.layer_mode, L, S, kappa, K, g->mm_slot);
        T F[S], B[S], xt[S];
        long long g_max = 0;
        int lo = 0;
#pragma unroll
        for (int i = 0; i < S; ++i) {
            const int hi = ok ? cw.next() : lo + 1;
            ok = ok && hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap);
            F[i] = sp.PF[hi] - sp.PF[lo];
            B[i] = sp.PB[hi] - sp.PB[lo];
            xt[i] = i < S - 1 ? sp.XT[(tier >> i) & 1ull][hi - 1] : (T)0;
            const long long gb = sp.PP[hi] - sp.PP[lo];
            g_max = gb > g_max ? gb : g_max;
            lo = hi;
        }
        if (ok) {
            const T t = sim_regs<T, S>(m, F, B, xt);
            bits = Num<T>::bits(t + Num<T>::sync(g_max, n_sync, sp.bw_sync));
            my_cells = 2ull * S * m;
        }
    }
    segmented_min_commit(bd.seg_best, row, bits, inf_bits<T>());
    count_cells(&bd.counters[0], my_cells, cells_w);
}

template <typename T>
__global__ void __launch_bounds__(kChunk) cm_cost_generic_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb.prof);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const uint64_t base = (chunk - bk.chunk_first) * kChunk;
    uint64_t seg_local, kappa;
    plan_of_thread(base, bk.count, threadIdx.x, seg_local, kappa);
    uint32_t row = 0xffffffffu;
    uint64_t bits = inf_bits<T>();
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg) {
        row = bd.order[bk.seg_begin + seg_local];
        const Seg g = bd.seg[row];
        T cost;
        if (segment_candidate_cost<T>(sp, tb, g, bd.layer_mode, kappa, cost)) {
            bits = Num<T>::bits(cost);
            my_cells = 2ull * g.S * g.m;
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
static void launch_regs(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_regs_kernel<T, S><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end);
}

template <typename T>
static void launch_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    switch (c.stages) {
    case 1: launch_regs<T, 1>(t, b, c, st); break;
    case 2: launch_regs<T, 2>(t, b, c, st); break;
    case 3: launch_regs<T, 3>(t, b, c, st); break;
    case 4: launch_regs<T, 4>(t, b, c, st); break;
    case 5: launch_regs<T, 5>(t, b, c, st); break;
    case 6: launch_regs<T, 6>(t, b, c, st); break;
    case 7: launch_regs<T, 7>(t, b, c, st); break;
    case 8: launch_regs<T, 8>(t, b, c, st); break;
    case 9: launch_regs<T, 9>(t, b, c, st); break;
    case 10: launch_regs<T, 10>(t, b, c, st); break;
    case 11: launch_regs<T, 11>(t, b, c, st); break;
    case 12: launch_regs<T, 12>(t, b, c, st); break;
    case 13: launch_regs<T, 13>(t, b, c, st); break;
    case 14: launch_regs<T, 14>(t, b, c, st); break;
    case 15: launch_regs<T, 15>(t, b, c, st); break;
    case 16: launch_regs<T, 16>(t, b, c, st); break;
    default:
        cm_cost_generic_kernel<T><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end);
        break;
    }
}

// The chunks of a class beyond its last bucket's plans are empty lanes; a chunk index
// past n_chunks cannot occur because the grid is exactly n_chunks (x * y may overshoot
// only in the 2-D case, where the surplus CTAs find the last bucket and idle).
cudaError_t launch_cost_pass1(const Tables &t, const BatchDev &b, const LaunchClass *classes, int n_classes,
                              cudaStream_t st, int *launches) {
    for (int i = 0; i < n_classes; ++i) {
        if (classes[i].n_chunks == 0) continue;
        if (b.mode == CM_COST_INT64NS) launch_class<long long>(t, b, classes[i], st);
        else launch_class<double>(t, b, classes[i], st);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (launches) ++*launches;
    }
    return cudaSuccess;
}

}  // namespace cm
