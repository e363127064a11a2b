// Search pass for segments deeper than the register-resident kernels whose only candidate is
// the min-max partition (layer mode MINMAX, or more compositions than kappa_cap).  One such
// plan is a single dependent chain of 2*S*m recurrence cells, about 100 us when one thread
// walks it; here a warp walks it in lock step with the stages spread over its lanes (two per
// lane above 32 stages), which takes 2*(S+m) slots of a few dozen cycles.  Four segments per
// CTA, every depth in the same launch.  Section "Estimator": the values are the same in any
// evaluation order that respects the dependencies.
#include "cm_cost_impl.cuh"

namespace cm {

template <typename T>
__global__ void __launch_bounds__(kChunk) cm_cost_solo_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = bk.S, m = bk.m;
    const uint64_t seg_local = (chunk - bk.chunk_first) * (kChunk / 32) + warp;
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg && m >= 1) {                       // warp-uniform
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        const uint8_t *cuts = tb.mm_cuts + (size_t)tb.mm_slot(S, m) * (kMaxS + 1);
        bool ok = cuts[0] == 0;                                 // 255: no memory-feasible partition exists
        long long g_max = 0;
        if (ok)
            for (int i = lane; i < S; i += 32) {
                const int lo = cuts[i], hi = cuts[i + 1];
                ok = ok && hi > lo && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
                const long long gb = sp.PP[hi] - sp.PP[lo];
                g_max = gb > g_max ? gb : g_max;
            }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            for (int o = 16; o > 0; o >>= 1) {
                const long long og = __shfl_xor_sync(0xffffffffu, g_max, o);
                g_max = og > g_max ? og : g_max;
            }
            const T t = warp_pipe_time<T>(sp, cuts, S, m, g.tier, lane);
            if (lane == 0) {
                const uint64_t bits = Num<T>::bits(t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval));
                if (bits < bd.seg_best[g.row]) atomicMin((unsigned long long *)&bd.seg_best[g.row], (unsigned long long)bits);
                my_cells = one_plan(2ull * S * m);
            }
        }
    }
    count_cells(&bd.counters[0], my_cells, cells_w);
}

template <typename T>
cudaError_t launch_solo_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_solo_kernel<T><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

// A warp per plan for buckets of few plans (what the memory screen leaves of a workload that
// memory decides): the plan's cuts are walked by every lane, kept by lane 0, then checked and
// timed with the stages spread over the lanes.  Plans are numbered segment-major within the
// bucket; four per CTA; every depth above kRegStagesMax in the same launch.
template <typename T>
__global__ void __launch_bounds__(kChunk) cm_cost_warp_kernel(Tables tb, BatchDev bd, uint32_t b0, uint32_t b1, uint64_t chunk_offset) {
    __shared__ SProf<T> sp;
    __shared__ unsigned long long cells_w[kChunk / 32];
    __shared__ uint8_t cuts_s[kChunk / 32][kMaxS + 8];
    const uint64_t chunk = chunk_offset + (uint64_t)blockIdx.x + (uint64_t)blockIdx.y * gridDim.x;
    stage_profile(sp, tb);
    const Bucket bk = bd.bucket[find_bucket(bd.bucket, b0, b1, chunk)];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = bk.S, m = bk.m;
    const uint64_t plan = (chunk - bk.chunk_first) * (kChunk / 32) + warp;
    const uint64_t seg_local = plan / bk.count;
    unsigned long long my_cells = 0;
    if (seg_local < bk.n_seg && m >= 1) {                       // warp-uniform
        const uint64_t kappa = walk_kappa(bd.feas, bk.feas_first, plan - seg_local * bk.count);
        const SegView g = bucket_segment(bd, bk, (uint32_t)seg_local);
        uint8_t *cuts = cuts_s[warp];
        CutWalker cw;
        bool ok = make_walker(cw, tb, bd.layer_mode, sp.L, S, kappa, g.K, tb.mm_slot(S, m));
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
        long long g_max = 0;
        if (ok)
            for (int i = lane; i < S; i += 32) {
                const int lo = cuts[i], hi = cuts[i + 1];
                ok = ok && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S, m, sp.cap, sp.sched);
                const long long gb = sp.PP[hi] - sp.PP[lo];
                g_max = gb > g_max ? gb : g_max;
            }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            for (int o = 16; o > 0; o >>= 1) {
                const long long og = __shfl_xor_sync(0xffffffffu, g_max, o);
                g_max = og > g_max ? og : g_max;
            }
            const T t = warp_pipe_time<T>(sp, cuts, S, m, g.tier, lane);
            if (lane == 0) {
                const uint64_t bits = Num<T>::bits(t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval));
                if (bits < bd.seg_best[g.row]) atomicMin((unsigned long long *)&bd.seg_best[g.row], (unsigned long long)bits);
                my_cells = one_plan(2ull * S * m);
            }
        }
    }
    count_cells(&bd.counters[0], my_cells, cells_w);
}

template <typename T>
cudaError_t launch_warp_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    cm_cost_warp_kernel<T><<<chunk_grid(c.n_chunks), kChunk, 0, st>>>(t, b, c.bucket_begin, c.bucket_end, c.chunk_begin);
    return cudaGetLastError();
}

template cudaError_t launch_warp_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_warp_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_solo_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_solo_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);

}  // namespace cm
