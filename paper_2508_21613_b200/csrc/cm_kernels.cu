// Kernels of the plan search (sm_100a) and their launchers.
//
//   cm_prefix_kernel      per-layer prefix sums and per-boundary transfer times
//   cm_minmax_kernel      min-max contiguous layer partition per (stages, micro-batches)
//   cm_feasible_kernel    memory-feasible layer compositions per (stages, micro-batches), listed once
//   (data rerouting / redundant computation: cm_policy.cu)
//   (the search pass over every pipeline-plan lives in cm_cost.cu)
//   cm_split_kernel       (cost, index) argmin over (strategy, micro-batch split) per scenario
//   cm_winner_kernel      finishes that argmin and decodes the winner
//   cm_tiebreak_kernel    pass 2: lowest layer composition that meets the winning cost
//   cm_finalize_kernel    assembles the plans and picks the best policy
//   cm_evaluate_kernel    per-candidate cost / feasibility for cm_evaluate
//   cm_pick_kernel        best of several spaces for cm_select
#include <algorithm>
#include <atomic>

#include "cm_plan_eval.cuh"

namespace cm {

// ----------------------------------------------------------------------------------
// Prefix sums, accumulated left to right so that every consumer of a stage quantity
// performs the same single subtraction (Section "Estimator": stage time / memory are
// sums over the stage's layers).  One thread per array; the arrays are <= 129 long.
// ----------------------------------------------------------------------------------
__global__ void cm_prefix_kernel(DevProfile *p) {
    const int L = p->L;
    switch (threadIdx.x) {
    // intval: the double arrays carry the integer-nanosecond inputs (sums exact below 2^53)
    case 0: { double a = 0.0; p->PFd[0] = a; for (int l = 0; l < L; ++l) { a = a + (p->intval ? (double)p->fwd_i[l] : p->fwd[l]); p->PFd[l + 1] = a; } break; }
    case 1: { double a = 0.0; p->PBd[0] = a; for (int l = 0; l < L; ++l) { a = a + (p->intval ? (double)p->bwd_i[l] : p->bwd[l]); p->PBd[l + 1] = a; } break; }
    case 2: { int64_t a = 0; p->PFi[0] = a; for (int l = 0; l < L; ++l) { a += p->fwd_i[l]; p->PFi[l + 1] = a; } break; }
    case 3: { int64_t a = 0; p->PBi[0] = a; for (int l = 0; l < L; ++l) { a += p->bwd_i[l]; p->PBi[l + 1] = a; } break; }
    case 4: { int64_t a = 0; p->PA[0] = a; for (int l = 0; l < L; ++l) { a += p->act[l]; p->PA[l + 1] = a; } break; }
    case 5: { int64_t a = 0; p->PS[0] = a; for (int l = 0; l < L; ++l) { a += 2 * p->par[l] + p->opt[l]; p->PS[l + 1] = a; } break; }
    case 6: { int64_t a = 0; p->PP[0] = a; for (int l = 0; l < L; ++l) { a += p->par[l]; p->PP[l + 1] = a; } break; }
    case 7: { int64_t a = 0; p->PW[0] = a; for (int l = 0; l < L; ++l) { a += p->par[l] + p->opt[l]; p->PW[l + 1] = a; } break; }
    default: break;
    }
    for (int l = threadIdx.x; l < L; l += blockDim.x) {
        p->XTd[0][l] = p->intval ? (double)(p->p2p[l] / p->bw_intra) : (double)p->p2p[l] / (double)p->bw_intra;
        p->XTd[1][l] = p->intval ? (double)(p->p2p[l] / p->bw_inter) : (double)p->p2p[l] / (double)p->bw_inter;
        p->XTi[0][l] = p->p2p[l] / p->bw_intra;
        p->XTi[1][l] = p->p2p[l] / p->bw_inter;
    }
}

cudaError_t launch_prefix(DevProfile *prof, cudaStream_t st) {
    cm_prefix_kernel<<<1, 128, 0, st>>>(prof);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Min-max layer partition: D[l][s] = min_k max(D[k][s-1], W(k,l)), W = forward+backward
// time of layers [k,l), only over stages that fit in memory at position s-1.  One CTA
// per (S, m) key; stage columns are swept one after the other, the layers of a column
// go to the warps, the split points k to the lanes, and a warp-shuffle argmin carrying
// (value, k) with the lowest k on ties closes each cell.  Backtracking follows the
// stored argmin, which is the smallest k that attains D[l][s].
// ----------------------------------------------------------------------------------
// a warp per layer of a DP column: 32 warps take the column of a 96-layer model in three sweeps
// (the kernel sits on the path of the first search of a survivor count)
constexpr int kMinmaxThreads = 1024;
template <typename T>
__global__ void __launch_bounds__(kMinmaxThreads) cm_minmax_kernel(Tables tb, const uint32_t *keys, int n_keys) {
    __shared__ T PF[kMaxL + 1], PB[kMaxL + 1];
    __shared__ long long PA[kMaxL + 1], PS[kMaxL + 1];
    __shared__ T D[2][kMaxL + 1];
    __shared__ uint8_t argk[kMaxS + 1][kMaxL + 1];
    const DevProfile *p = tb.prof;
    const int L = p->L;
    const uint32_t key = keys[blockIdx.x];
    const int S = (int)(key >> 16), m = (int)(key & 0xffffu);
    const long long cap = p->cap;
    for (int l = threadIdx.x; l <= L; l += blockDim.x) {
        PF[l] = Num<T>::PF(p)[l];
        PB[l] = Num<T>::PB(p)[l];
        PA[l] = p->PA[l];
        PS[l] = p->PS[l];
        D[0][l] = Num<T>::inf();
        D[1][l] = Num<T>::inf();
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const T INF = Num<T>::inf();
    for (int s = 1; s <= S; ++s) {
        T *cur = D[s & 1];
        const T *prev = D[(s - 1) & 1];
        for (int l = s + warp; l <= L; l += n_warps) {
            T best = INF;
            int best_k = 0;
            if (s == 1) {
                if (lane == 0 && stage_fits(PS[l] - PS[0], PA[l] - PA[0], 0, S, m, cap, tb.sched))
                    best = (PF[l] - PF[0]) + (PB[l] - PB[0]);
            } else {
                for (int k = s - 1 + lane; k <= l - 1; k += 32) {
                    if (prev[k] == INF) continue;
                    if (!stage_fits(PS[l] - PS[k], PA[l] - PA[k], s - 1, S, m, cap, tb.sched)) continue;
                    T w = (PF[l] - PF[k]) + (PB[l] - PB[k]);
                    T v = tmax(prev[k], w);
                    if (v < best) { best = v; best_k = k; }
                }
            }
            for (int o = 16; o > 0; o >>= 1) {
                T ov = __shfl_xor_sync(0xffffffffu, best, o);
                int ok = __shfl_xor_sync(0xffffffffu, best_k, o);
                if (ov < best || (ov == best && ov != INF && ok < best_k)) { best = ov; best_k = ok; }
            }
            if (lane == 0) {
                cur[l] = best;
                argk[s][l] = (uint8_t)best_k;
            }
        }
        // cells of this column below the first reachable layer stay infinite
        for (int l = threadIdx.x; l < s; l += blockDim.x) cur[l] = INF;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint8_t *out = tb.mm_cuts + ((size_t)(S - 1) * tb.mm_stride_m + m) * (kMaxS + 1);
        if (D[S & 1][L] == INF) {
            out[0] = 255;
        } else {
            int l = L;
            out[S] = (uint8_t)L;
            for (int s = S; s >= 2; --s) {
                l = argk[s][l];
                out[s - 1] = (uint8_t)l;
            }
            out[0] = 0;
        }
    }
}

cudaError_t launch_minmax(const Tables &t, const uint32_t *keys_dev, int n_keys, int mode, cudaStream_t st) {
    if (n_keys <= 0) return cudaSuccess;
    if (mode == CM_COST_INT64NS) cm_minmax_kernel<long long><<<n_keys, kMinmaxThreads, 0, st>>>(t, keys_dev, n_keys);
    else cm_minmax_kernel<double><<<n_keys, kMinmaxThreads, 0, st>>>(t, keys_dev, n_keys);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Memory-feasible layer compositions of an (S, m) key, in ascending order (Section
// "Estimator", memory estimator: a stage's peak depends on its layers, its position and the
// micro-batches in flight -- not on the failure scenario, so this is done once per key and
// profile).  One CTA per key walks kappa = 0 .. K-1 in chunks of its size and compacts the
// feasible ranks in order (ballot + prefix over the warps); the min-max partition, candidate
// K, closes the list if a memory-feasible partition exists.
// ----------------------------------------------------------------------------------
constexpr int kFeasThreads = 1024;
__global__ void __launch_bounds__(kFeasThreads) cm_feasible_kernel(Tables tb, int layer_mode, const uint32_t *keys,
                                                                   const uint64_t *Ks, const uint32_t *first,
                                                                   uint32_t *pool, uint32_t *count_out, int binom_rows_staged) {
    __shared__ long long PA[kMaxL + 1], PS[kMaxL + 1];
    __shared__ uint32_t warp_cnt[kFeasThreads / 32];
    __shared__ uint32_t running;
    // the rows of the binomial table that unranking reads (n <= stages under the remainder rule,
    // n < layers under the full enumeration), staged once: a rank is unranked through ~S dependent
    // look-ups, and this kernel sits on the path of the first search of a survivor count
    extern __shared__ uint64_t binom_s[];
    const DevProfile *p = tb.prof;
    const int L = p->L;
    for (int q = threadIdx.x; q < binom_rows_staged * (kBinomCols + 1); q += blockDim.x) binom_s[q] = tb.binom[q];
    tb.binom = binom_s;
    const uint32_t key = keys[blockIdx.x];
    const int S = (int)(key >> 16), m = (int)(key & 0xffffu);
    const uint64_t K = Ks[blockIdx.x];
    uint32_t *out = pool + first[blockIdx.x];
    const long long cap = p->cap;
    for (int l = threadIdx.x; l <= L; l += blockDim.x) { PA[l] = p->PA[l]; PS[l] = p->PS[l]; }
    if (threadIdx.x == 0) running = 0;
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint64_t base = 0; base < K; base += kFeasThreads) {
        const uint64_t kappa = base + threadIdx.x;
        bool ok = kappa < K;
        if (ok) {
            CutWalker cw;
            make_walker(cw, tb, layer_mode, L, S, kappa, K, 0);
            int lo = 0;
            for (int i = 0; i < S && ok; ++i) {
                const int hi = cw.next();
                ok = hi > lo && stage_fits(PS[hi] - PS[lo], PA[hi] - PA[lo], i, S, m, cap, tb.sched);
                lo = hi;
            }
        }
        const uint32_t vote = __ballot_sync(0xffffffffu, ok);
        if (lane == 0) warp_cnt[warp] = __popc(vote);
        __syncthreads();
        uint32_t before = running, total = 0;
        for (uint32_t w = 0; w < kFeasThreads / 32; ++w) {
            const uint32_t c = warp_cnt[w];
            if (w < warp) before += c;
            total += c;
        }
        if (ok) out[before + __popc(vote & ((1u << lane) - 1u))] = (uint32_t)kappa;
        __syncthreads();
        if (threadIdx.x == 0) running += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint32_t n = running;
        if (tb.mm_cuts[(size_t)tb.mm_slot(S, m) * (kMaxS + 1)] == 0) out[n++] = (uint32_t)K;
        count_out[blockIdx.x] = n;
    }
}

cudaError_t launch_feasible(const Tables &t, int layer_mode, const uint32_t *keys_dev, const uint64_t *K_dev,
                            const uint32_t *first_dev, int n_keys, uint32_t *pool, uint32_t *count_dev, cudaStream_t st) {
    if (n_keys <= 0) return cudaSuccess;
    // rows 0 .. 64 (remainder rule: n <= CM_MAX_STAGES) or 0 .. 127 (full enumeration: n < CM_MAX_LAYERS)
    const int rows = std::min(t.binom_rows, layer_mode == CM_LAYERS_REMAINDER ? kMaxS + 1 : kMaxL);
    const size_t smem = (size_t)rows * (kBinomCols + 1) * sizeof(uint64_t);
    static std::atomic<uint64_t> configured{0};   // one bit per device, as for the deep cost kernels
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 64 || !((configured.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(cm_feasible_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)((size_t)kMaxL * (kBinomCols + 1) * sizeof(uint64_t)));
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    cm_feasible_kernel<<<n_keys, kFeasThreads, smem, st>>>(t, layer_mode, keys_dev, K_dev, first_dev, pool, count_dev, rows);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Segments shared between scenarios (USegDev): one CTA per searched scenario, a thread per
// template segment.  cm_useg_key_kernel finds or claims the slot of the row's tier word in its
// class's table (linear probing, at most as many probes as the table has slots; a table holds
// at least twice the rows of its class) and leaves the lowest row per slot as its
// representative; cm_useg_list_kernel appends every representative to its class's list (the
// order within a class is whatever the atomics give: results do not depend on it);
// cm_useg_copy_kernel, after the search pass, gives every other row its representative's minimum.
// ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
    x ^= x >> 27; x *= 0x94d049bb133111ebull;
    x ^= x >> 31;
    return (uint32_t)x;
}

// phase 0: the heads of the pair classes; phase 1 (a launch of its own, after phase 0 is complete):
// every other row, which joins a pair it finds in the tables of phase 0 before it is keyed itself
__device__ __forceinline__ uint32_t useg_find(const USegDev &ud, const USegClass &c, unsigned long long tier) {
    uint32_t h = mix64(tier) & c.tab_mask;
    for (uint32_t probe = 0; probe <= c.tab_mask; ++probe) {
        const unsigned long long v = ud.tab[c.tab_first + h];
        if (v == tier) return c.tab_first + h;
        if (v == ~0ull) break;
        h = (h + 1) & c.tab_mask;
    }
    return kNoSegClass;
}

__global__ void __launch_bounds__(128) cm_useg_key_kernel(BatchDev bd, USegDev ud, int phase) {
    const uint32_t scen_id = bd.tmpl_scen[blockIdx.x];
    const Scen sc = bd.scen[scen_id];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    for (uint32_t i = threadIdx.x; i < tp.n_tseg; i += blockDim.x) {
        const uint32_t trow = tp.tseg_first + i, row = sc.seg_base + i;
        const uint32_t ci = ud.tseg_cls[trow];
        if (ci == kNoSegClass || ci == kPartnerSeg) {
            if (phase == 0) ud.slot_of[row] = ci;
            continue;
        }
        if ((ci < ud.n_pair_cls) != (phase == 0)) continue;
        const TSeg g = bd.tseg[trow];
        const unsigned long long tier = cut_bits(bd.cross + sc.cross_first, g.off, g.S - 1);   // < 2^63: never all-ones
        if (phase == 1) {
            uint32_t found = kNoSegClass;
            const uint32_t lh = ud.look_head[trow], lp = ud.look_part[trow];
            if (lh != kNoSegClass) found = useg_find(ud, ud.cls[lh], tier);
            if (found == kNoSegClass && lp != kNoSegClass) {
                found = useg_find(ud, ud.cls[lp], tier);
                if (found != kNoSegClass) found |= kSecondRowFlag;
            }
            if (found != kNoSegClass) { ud.slot_of[row] = found; continue; }
        }
        const USegClass c = ud.cls[ci];
        uint32_t slot = kNoSegClass;
        uint32_t h = mix64(tier) & c.tab_mask;
        for (uint32_t probe = 0; probe <= c.tab_mask; ++probe) {
            const unsigned long long old = atomicCAS(&ud.tab[c.tab_first + h], ~0ull, tier);
            if (old == ~0ull || old == tier) { slot = c.tab_first + h; break; }
            h = (h + 1) & c.tab_mask;
        }
        if (slot == kNoSegClass) atomicAdd(&ud.count[ud.n_cls], 1u);   // (no free slot: cannot happen)
        else atomicMin(&ud.rep[slot], row);
        ud.slot_of[row] = slot;
    }
}

__global__ void __launch_bounds__(128) cm_useg_list_kernel(BatchDev bd, USegDev ud) {
    const uint32_t scen_id = bd.tmpl_scen[blockIdx.x];
    const Scen sc = bd.scen[scen_id];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    for (uint32_t i = threadIdx.x; i < tp.n_tseg; i += blockDim.x) {
        const uint32_t trow = tp.tseg_first + i, row = sc.seg_base + i;
        const uint32_t slot = ud.slot_of[row];
        if (slot == kNoSegClass || slot == kPartnerSeg || (slot & kSecondRowFlag) || ud.rep[slot] != row) continue;
        const uint32_t ci = ud.tseg_cls[trow];   // a representative was keyed in its own class
        const uint32_t pos = atomicAdd(&ud.count[ci], 1u);
        ud.list[ud.cls[ci].list_first + pos] = make_uint2(scen_id, trow);
    }
}

__global__ void __launch_bounds__(256) cm_useg_copy_kernel(BatchDev bd, USegDev ud) {
    const uint32_t row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= bd.n_rows) return;
    uint32_t slot = ud.slot_of[row];
    if (slot == kNoSegClass) return;
    uint32_t second = 0;
    if (slot == kPartnerSeg) {   // second row of a keyed pair head
        slot = ud.slot_of[row - 1];
        second = 1;
    } else if (slot & kSecondRowFlag) {
        slot &= ~kSecondRowFlag;
        second = 1;
    }
    const uint32_t r = ud.rep[slot] + second;
    if (r != row) bd.seg_best[row] = bd.seg_best[r];   // representatives and their second rows are only read here
}

__global__ void __launch_bounds__(128) cm_dup_copy_kernel(BatchDev bd) {
    const Scen sc = bd.scen[bd.tmpl_scen[blockIdx.x]];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    for (uint32_t i = threadIdx.x; i < tp.n_tseg; i += blockDim.x) {
        const uint32_t c = bd.tseg_canon[tp.tseg_first + i];
        if (c != tp.tseg_first + i) bd.seg_best[sc.seg_base + i] = bd.seg_best[sc.seg_base + (c - tp.tseg_first)];
    }
}

cudaError_t launch_dup_copy(const BatchDev &b, cudaStream_t st) {
    if (!b.tseg_canon || b.n_rep_scen == 0) return cudaSuccess;
    cm_dup_copy_kernel<<<b.n_rep_scen, 128, 0, st>>>(b);
    return cudaGetLastError();
}

cudaError_t launch_useg_keys(const BatchDev &b, const USegDev &u, cudaStream_t st) {
    if (u.n_rep_scen == 0) return cudaSuccess;
    cm_useg_key_kernel<<<u.n_rep_scen, 128, 0, st>>>(b, u, 0);
    cm_useg_key_kernel<<<u.n_rep_scen, 128, 0, st>>>(b, u, 1);
    cm_useg_list_kernel<<<u.n_rep_scen, 128, 0, st>>>(b, u);
    return cudaGetLastError();
}

cudaError_t launch_useg_copy(const BatchDev &b, const USegDev &u, cudaStream_t st) {
    if (b.n_rows == 0) return cudaSuccess;
    cm_useg_copy_kernel<<<(b.n_rows + 255) / 256, 256, 0, st>>>(b, u);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Locate the segment that owns a tile / a candidate: the last row whose first index is
// not above the query (rows are sorted and every segment owns at least one).
// ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t find_row(const TSeg *seg, uint32_t n, uint64_t q) {
    uint32_t lo = 0, hi = n - 1;
    while (lo < hi) {
        uint32_t mid = (lo + hi + 1) >> 1;
        if (seg[mid].cand_first <= q) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ----------------------------------------------------------------------------------
// Split reduction: item = (strategy, split rank) of one scenario; its step time is the
// slowest pipeline's best cost (Section "Estimator": step time = max over pipelines).
// Hierarchical argmin carrying (cost, item) with the lowest item on ties:
// thread-serial over a strided range -> warp shuffle -> shared memory -> one partial
// per block -> cm_winner_kernel over the scenario's partials.
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) cm_split_kernel(Tables tb, BatchDev bd, uint64_t inf) {
    __shared__ uint64_t rc[8], ri[8];
    const uint32_t b = bd.red_scen[blockIdx.x];
    const Scen sc = bd.scen[b];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    const uint32_t local = blockIdx.x - sc.red_first;
    const uint64_t *best = bd.seg_best + sc.seg_base;   // this scenario's rows, in template order
    uint64_t best_c = inf, best_i = ~0ull;
    for (uint64_t item = (uint64_t)local * blockDim.x + threadIdx.x; item < tp.n_split_total;
         item += (uint64_t)tp.n_red * blockDim.x) {
        const uint64_t T = item_step_time(tb, bd, tp, best, item, inf);
        if (pair_less(T, item, best_c, best_i)) { best_c = T; best_i = item; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        uint64_t oc = __shfl_xor_sync(0xffffffffu, best_c, o);
        uint64_t oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (pair_less(oc, oi, best_c, best_i)) { best_c = oc; best_i = oi; }
    }
    if ((threadIdx.x & 31) == 0) { rc[threadIdx.x >> 5] = best_c; ri[threadIdx.x >> 5] = best_i; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (pair_less(rc[w], ri[w], best_c, best_i)) { best_c = rc[w]; best_i = ri[w]; }
        bd.partial[blockIdx.x].cost_bits = best_c;
        bd.partial[blockIdx.x].item = best_i;
    }
}

// Grid level of the argmin: one warp per scenario over its block partials, then decode
// the winner (strategy, split -> micro-batches, segment rows) for the tie-break pass.
__global__ void __launch_bounds__(32) cm_winner_kernel(Tables tb, BatchDev bd, uint64_t inf) {
    const uint32_t b = blockIdx.x;
    const Scen sc = bd.scen[b];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    uint64_t best_c = inf, best_i = ~0ull;
    for (uint32_t r = threadIdx.x; r < (sc.rep == b ? tp.n_red : 0u); r += 32) {
        const Partial q = bd.partial[sc.red_first + r];
        if (pair_less(q.cost_bits, q.item, best_c, best_i)) { best_c = q.cost_bits; best_i = q.item; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        uint64_t oc = __shfl_xor_sync(0xffffffffu, best_c, o);
        uint64_t oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (pair_less(oc, oi, best_c, best_i)) { best_c = oc; best_i = oi; }
    }
    if (threadIdx.x == 0) {
        Winner w;
        if (sc.rep != b) { best_c = inf; best_i = ~0ull; }   // shares another scenario's search: nothing to tie-break here
        decode_winner(tb, bd, tp, b, best_c, best_i, inf, w);
        bd.winner[b] = w;
    }
    __syncthreads();   // the record is written: one thread per pipeline sets its start value
    if (threadIdx.x < kMaxP) init_kappa_sel(bd, bd.winner[b], bd.kappa_sel + (size_t)b * kMaxP, (int)threadIdx.x);
}

// Both levels in one launch, for batches in which no scenario needs more than one block of the
// split reduction (up to 1024 (strategy, split) pairs each): one CTA per scenario.
__global__ void __launch_bounds__(256) cm_split_winner_kernel(Tables tb, BatchDev bd, uint64_t inf) {
    __shared__ uint64_t rc[8], ri[8];
    const uint32_t b = blockIdx.x;
    const Scen sc = bd.scen[b];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    const uint64_t *best = bd.seg_best + sc.seg_base;
    uint64_t best_c = inf, best_i = ~0ull;
    if (sc.rep == b)
        for (uint64_t item = threadIdx.x; item < tp.n_split_total; item += blockDim.x) {
            const uint64_t T = item_step_time(tb, bd, tp, best, item, inf);
            if (pair_less(T, item, best_c, best_i)) { best_c = T; best_i = item; }
        }
    for (int o = 16; o > 0; o >>= 1) {
        uint64_t oc = __shfl_xor_sync(0xffffffffu, best_c, o);
        uint64_t oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (pair_less(oc, oi, best_c, best_i)) { best_c = oc; best_i = oi; }
    }
    if ((threadIdx.x & 31) == 0) { rc[threadIdx.x >> 5] = best_c; ri[threadIdx.x >> 5] = best_i; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (pair_less(rc[w], ri[w], best_c, best_i)) { best_c = rc[w]; best_i = ri[w]; }
        Winner w;
        decode_winner(tb, bd, tp, b, best_c, best_i, inf, w);
        bd.winner[b] = w;
    }
    __syncthreads();   // the record is written: one thread per pipeline sets its start value
    if (threadIdx.x < kMaxP) init_kappa_sel(bd, bd.winner[b], bd.kappa_sel + (size_t)b * kMaxP, (int)threadIdx.x);
}

cudaError_t launch_split_reduce(const Tables &t, const BatchDev &b, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const uint64_t inf = batch_inf_bits(b);
    if (b.n_red_blocks <= (uint32_t)b.B && b.max_red_per_scen <= 1) {
        cm_split_winner_kernel<<<b.B, 256, 0, st>>>(t, b, inf);
        return cudaGetLastError();
    }
    if (b.n_red_blocks) {
        cm_split_kernel<<<b.n_red_blocks, 256, 0, st>>>(t, b, inf);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    cm_winner_kernel<<<b.B, 32, 0, st>>>(t, b, inf);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Pass 2 (tie-break): among optimal plans the lexicographically smallest tuple wins, so
// each pipeline of the winning (strategy, split) takes the LOWEST layer composition
// that is feasible with cost <= T* (not its own argmin).  grid.x = (scenario, pipeline),
// grid.y = tiles of a segment.  Tiles above an already found index return at once.
// ----------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kTile) cm_tiebreak_kernel(Tables tb, BatchDev bd, int deep_elsewhere_all) {
    __shared__ SProf<T> sp;
    __shared__ uint64_t red[kTile / 32];
    __shared__ SegView g;
    __shared__ uint64_t found_so_far;
    stage_profile(sp, tb);
    // grid.x runs over (scenario, pipeline), grid.y over tiles: CTAs are dispatched x-fastest,
    // so every segment's first tile is evaluated before anybody's second one and most later
    // tiles find their answer already there.
    const uint32_t y = blockIdx.x;
    const uint32_t b = y / bd.dp_max, p = y % bd.dp_max;
    const Winner &w = bd.winner[b];
    if (w.cost_bits >= inf_bits<T>() || p >= w.dp) return;          // uniform over the CTA
    {
        const int S = bd.tseg[w.seg[p]].S;   // 17..48 stages: cm_tiebreak_wide_kernel's job
        if (S > kRegStagesMax && (S <= kWideStagesMax || deep_elsewhere_all)) return;
    }
    for (uint64_t tile = blockIdx.y; tile < bd.max_tiles_per_seg; tile += gridDim.y) {
        uint64_t *slot = &bd.kappa_sel[b * kMaxP + p];
        __syncthreads();
        if (threadIdx.x == 0) {
            g = seg_view(bd, w.scen, w.seg[p]);
            found_so_far = *(volatile uint64_t *)slot;
        }
        __syncthreads();
        const uint64_t count = walk_count(g);
        const uint64_t first = tile * kTile;
        // uniform: later tiles hold higher compositions than one already found
        if (first >= count || found_so_far <= walk_kappa(bd.feas, g.feas_first, first)) break;
        uint64_t hit = ~0ull;
        if (first + threadIdx.x < count) {
            const uint64_t kappa = walk_kappa(bd.feas, g.feas_first, first + threadIdx.x);
            T cost;
            // shallow pipelines take the register-resident evaluations, pipelines deeper than
            // kWideStagesMax the local-memory one (the depths between: cm_tiebreak_wide_kernel)
            bool ok;
            if (g.S > kRegStagesMax) ok = segment_candidate_cost<T>(sp, tb, g, bd.layer_mode, kappa, cost);
            else if (g.m >= g.S - 1) ok = plan_cost_regs_any<T>(sp, tb, bd.layer_mode, g, kappa, cost);
            else ok = plan_cost_regs_any<T, true>(sp, tb, bd.layer_mode, g, kappa, cost);
            if (ok && Num<T>::bits(cost) <= w.cost_bits) hit = kappa;
        }
        hit = warp_min_u64(hit);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = hit;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int q = 0; q < kTile / 32; ++q) hit = red[q] < hit ? red[q] : hit;
            if (hit != ~0ull) atomicMin((unsigned long long *)slot, (unsigned long long)hit);
            uint64_t n = count - first < kTile ? count - first : kTile;
            atomicAdd(&bd.counters[1], (unsigned long long)n);
        }
    }
}

cudaError_t launch_cost_pass2(const Tables &t, const BatchDev &b, cudaStream_t st, bool deep_elsewhere_all) {
    if (b.B <= 0 || b.max_tiles_per_seg == 0 || b.dp_max == 0) return cudaSuccess;
    const uint64_t nx = (uint64_t)b.B * b.dp_max;
    if (nx >= (1ull << 31)) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)nx, tiebreak_grid_y(nx, b.max_tiles_per_seg), 1);
    if (native_i64(b)) cm_tiebreak_kernel<long long><<<grid, kTile, 0, st>>>(t, b, deep_elsewhere_all ? 1 : 0);
    else cm_tiebreak_kernel<double><<<grid, kTile, 0, st>>>(t, b, deep_elsewhere_all ? 1 : 0);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// The same pass when there are only a few winners (a single failure being handled): with one
// plan per lane the first tile alone is a dependent chain of 2*S*m cells in every thread (0.1-0.2
// ms at 30+ stages), whatever the number of compositions that are really needed.  Here a WARP
// takes one composition and walks the pipeline in lock step, stages over its lanes (two per lane
// above 32 stages): 2(S+m) slots of a few dozen cycles.  grid.x = (scenario, pipeline), grid.y
// strides over the walk in groups of four compositions (one per warp), lowest first; a warp
// stops as soon as a composition at or below its own has been found.  Every depth above
// kRegStagesMax in one launch.
// ----------------------------------------------------------------------------------
constexpr int kWarpTieWarps = 4;
template <typename T>
__global__ void __launch_bounds__(kWarpTieWarps * 32) cm_tiebreak_warp_kernel(Tables tb, BatchDev bd) {
    __shared__ SProf<T> sp;
    __shared__ uint8_t cuts_s[kWarpTieWarps][kMaxS + 8];
    const uint32_t b = blockIdx.x / bd.dp_max, p = blockIdx.x % bd.dp_max;
    const Winner &w = bd.winner[b];
    if (w.cost_bits >= inf_bits<T>() || p >= w.dp) return;          // uniform over the CTA
    const SegView g = seg_view(bd, w.scen, w.seg[p]);
    if (g.S <= kRegStagesMax || g.K == 0) return;                   // shallow: cm_tiebreak_kernel; one candidate: known already
    stage_profile(sp, tb);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = g.S, m = g.m;
    uint8_t *cuts = cuts_s[warp];
    uint64_t *slot = &bd.kappa_sel[b * kMaxP + p];
    const uint64_t count = walk_count(g);
    unsigned long long evaluated = 0;
    for (uint64_t pos = (uint64_t)blockIdx.y * kWarpTieWarps + warp; pos < count; pos += (uint64_t)gridDim.y * kWarpTieWarps) {
        const uint64_t kappa = walk_kappa(bd.feas, g.feas_first, pos);
        uint64_t found = 0;
        if (lane == 0) found = *(volatile uint64_t *)slot;
        found = __shfl_sync(0xffffffffu, found, 0);
        if (found <= kappa) break;                                  // later compositions of this warp are higher still
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
            const uint64_t bits = Num<T>::bits(t + Num<T>::sync(g_max, g.n_sync, sp.bw_sync, sp.intval));
            if (lane == 0 && bits <= w.cost_bits) atomicMin((unsigned long long *)slot, (unsigned long long)kappa);
        }
        ++evaluated;
        __syncwarp();                                               // the next composition overwrites the cuts
    }
    if (lane == 0 && evaluated) atomicAdd(&bd.counters[1], evaluated);
}

cudaError_t launch_tiebreak_warp(const Tables &t, const BatchDev &b, cudaStream_t st) {
    if (b.B <= 0 || b.max_tiles_per_seg == 0 || b.dp_max == 0) return cudaSuccess;
    const uint64_t nx = (uint64_t)b.B * b.dp_max;
    if (nx >= (1ull << 31)) return cudaErrorInvalidConfiguration;
    // as many groups of four compositions side by side as fill the GPU a few times over
    uint64_t y = (4096 + nx - 1) / nx;
    const uint64_t groups = (uint64_t)b.max_tiles_per_seg * (kTile / kWarpTieWarps);
    if (y > groups) y = groups;
    if (y > 65535) y = 65535;
    if (y < 1) y = 1;
    dim3 grid((unsigned)nx, (unsigned)y, 1);
    if (native_i64(b)) cm_tiebreak_warp_kernel<long long><<<grid, kWarpTieWarps * 32, 0, st>>>(t, b);
    else cm_tiebreak_warp_kernel<double><<<grid, kWarpTieWarps * 32, 0, st>>>(t, b);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Assemble the per-policy plans and the overall best: least cost, ties to the lowest
// policy id (Algorithm 1 keeps the plan with the least estimated time).
// ----------------------------------------------------------------------------------
__global__ void cm_finalize_kernel(Tables tb, BatchDev bd, uint64_t inf) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) {
        // work counters ride home behind the plans (they start at all-ones, i.e. -1)
        unsigned long long *tail = reinterpret_cast<unsigned long long *>(bd.plans + (size_t)bd.B * 4);
        for (int i = 0; i < 4; ++i) tail[i] = bd.counters[i] + 1ull;
    }
    if (b >= bd.B) return;
    const DevProfile *p = tb.prof;
    const Scen sc = bd.scen[b];
    cm_plan *out = bd.plans + (size_t)b * 4;
    uint64_t cost[3] = {inf, inf, inf};
    for (int pol = 0; pol < 2; ++pol) {
        cm_plan pl;
        plan_clear(pl, pol);
        pl.n_pipes = (uint32_t)p->n_dp;
        for (int k = 0; k < p->n_dp && k < kMaxP; ++k) {
            pl.stages[k] = (uint16_t)p->n_pp;
            pl.micro[k] = (uint16_t)p->n_micro;
        }
        uint64_t c = (sc.policy_mask & (1u << pol)) ? bd.pol_cost[2 * b + pol] : inf;
        if (c < inf) {
            pl.feasible = 1;
            plan_set_cost(pl, c, bd);
            if (pol == CM_REDUNDANT)
                for (int k = 0; k < p->n_dp && k < kMaxP; ++k) pl.stages[k] = bd.rc_stages[b * kMaxP + k];
            cost[pol] = c;
        }
        out[pol] = pl;
    }
    {
        cm_plan pl;
        plan_clear(pl, CM_DYNPAR);
        const Winner &w = bd.winner[sc.rep];   // its own search, or the one it shares
        if ((sc.policy_mask & (1u << CM_DYNPAR)) && w.cost_bits < inf) {
            const Strat &s = bd.strat[w.strat];
            pl.feasible = 1;
            plan_set_cost(pl, w.cost_bits, bd);
            pl.strategy = w.strat - bd.tmpl[sc.tmpl].strat_first;
            pl.n_pipes = w.dp;
            pl.split_rank = w.item - s.split_first;
            for (uint32_t q = 0; q < w.dp; ++q) {
                pl.stages[q] = s.S[q];
                pl.micro[q] = w.micro[q];
                pl.kappa[q] = bd.kappa_sel[sc.rep * kMaxP + q];
            }
            cost[2] = w.cost_bits;
        }
        out[2] = pl;
    }
    int win = -1;
    for (int pol = 0; pol < 3; ++pol)
        if (cost[pol] < inf && (win < 0 || cost[pol] < cost[win])) win = pol;
    if (win >= 0) out[3] = out[win];
    else { cm_plan pl; plan_clear(pl, 0); out[3] = pl; }
}

cudaError_t launch_finalize(const Tables &t, const BatchDev &b, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const uint64_t inf = batch_inf_bits(b);
    cm_finalize_kernel<<<(b.B + 127) / 128, 128, 0, st>>>(t, b, inf);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// cm_evaluate: one thread per requested candidate.
// ----------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) cm_evaluate_kernel(Tables tb, BatchDev bd, uint64_t first, uint64_t count,
                                                          const uint64_t *idx, uint64_t n_cand, double *cost,
                                                          int64_t *cost_ns, uint8_t *feas) {
    __shared__ SProf<T> sp;
    stage_profile(sp, tb);
    __syncthreads();
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count) return;
    const uint64_t e = idx ? idx[t] : first + t;
    T c = Num<T>::inf();
    bool ok = false;
    if (e < n_cand) {
        // spaces hold one scenario: its template's segments are sorted by first candidate
        const Tmpl tp = bd.tmpl[bd.scen[0].tmpl];
        const uint32_t s = tp.tseg_first + find_row(bd.tseg + tp.tseg_first, tp.n_tseg, e);
        const SegView g = seg_view(bd, 0, s);
        T v;
        if (segment_candidate_cost<T>(sp, tb, g, bd.layer_mode, e - bd.tseg[s].cand_first, v)) { c = v; ok = true; }
    }
    if (cost && bd.mode == CM_COST_FP64) cost[t] = __longlong_as_double((long long)Num<T>::bits(c));
    if (cost_ns && bd.mode == CM_COST_INT64NS) cost_ns[t] = batch_cost_ns(bd, Num<T>::bits(c));
    if (feas) feas[t] = ok ? 1 : 0;
}

// One-candidate policies through cm_evaluate: the cost cm_policy_kernel left behind.
__global__ void cm_evaluate_single_kernel(BatchDev bd, int policy, uint64_t inf, uint64_t first, uint64_t count,
                                          const uint64_t *idx, double *cost, int64_t *cost_ns, uint8_t *feas) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count) return;
    const uint64_t e = idx ? idx[t] : first + t;
    uint64_t c = e == 0 ? bd.pol_cost[policy] : inf;
    if (cost && bd.mode == CM_COST_FP64) cost[t] = __longlong_as_double((long long)c);
    if (cost_ns && bd.mode == CM_COST_INT64NS) cost_ns[t] = batch_cost_ns(bd, c);
    if (feas) feas[t] = c < inf ? 1 : 0;
}

cudaError_t launch_evaluate(const Tables &t, const BatchDev &b, uint64_t n_cand, int single_policy,
                            uint64_t first, uint64_t count, const uint64_t *idx, double *cost,
                            int64_t *cost_ns, uint8_t *feas, cudaStream_t st) {
    if (count == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((count + 127) / 128);
    const uint64_t inf = batch_inf_bits(b);
    if (single_policy >= 0)
        cm_evaluate_single_kernel<<<blocks, 128, 0, st>>>(b, single_policy, inf, first, count, idx, cost, cost_ns, feas);
    else if (native_i64(b))
        cm_evaluate_kernel<long long><<<blocks, 128, 0, st>>>(t, b, first, count, idx, n_cand, cost, cost_ns, feas);
    else
        cm_evaluate_kernel<double><<<blocks, 128, 0, st>>>(t, b, first, count, idx, n_cand, cost, cost_ns, feas);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// cm_select over several spaces: least cost, ties to the lowest policy id, then to the
// earlier space.
// ----------------------------------------------------------------------------------
__global__ void cm_pick_kernel(const cm_plan *const *plans, int n, cm_plan *out, int mode) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int win = -1;
    for (int i = 0; i < n; ++i) {
        const cm_plan &q = *plans[i];
        if (!q.feasible) continue;
        if (win < 0) { win = i; continue; }
        const cm_plan &w = *plans[win];
        bool less, equal;
        if (mode == CM_COST_INT64NS) { less = q.cost_ns < w.cost_ns; equal = q.cost_ns == w.cost_ns; }
        else { less = q.cost < w.cost; equal = q.cost == w.cost; }
        if (less || (equal && q.policy < w.policy)) win = i;
    }
    if (win >= 0) *out = *plans[win];
    else { cm_plan pl; plan_clear(pl, 0); *out = pl; }
}

cudaError_t launch_pick(const cm_plan *const *plans_dev, int n, cm_plan *out_dev, int mode, cudaStream_t st) {
    cm_pick_kernel<<<1, 32, 0, st>>>(plans_dev, n, out_dev, mode);
    return cudaGetLastError();
}

}  // namespace cm
