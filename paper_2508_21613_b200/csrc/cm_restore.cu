// Transition time and the full objective (sm_100a).
//
//   cm_shortlist_kernel       per scenario: the topk (strategy, split) pairs of least step time
//   (the tie-break kernels then complete every shortlisted pair to a plan)
//   cm_plan_matching_kernel   one warp per shortlisted plan: layer ranges of the survivors
//                             before and after, minimum-cost perfect matching
//   cm_range_matching_kernel  the same matching over caller-given layer ranges
//   cm_plan_rounds_kernel     one warp per shortlisted plan: communication rounds of the
//                             asymmetric synchronisation and the step time they give
//   cm_objective_kernel       per scenario: steps before the next fault of every candidate,
//                             the best one, its plan and its migration scheme
//
// Section "Restorer", Weight Transfer: the N x N cost matrix is never stored.  Old and new
// holdings are contiguous layer ranges, so Cost[i][j] = W(new_j) - W(new_j ∩ old_i) is two
// prefix differences; a warp keeps the potentials of the Kuhn-Munkres iteration in shared
// memory, its lanes share the columns (their potentials and slacks stay in registers), and
// the argmin over the columns is a shuffle reduction carrying (slack, column) with the
// lowest column on ties.
#include <climits>

#include "cm_device.cuh"

namespace cm {

// ----------------------------------------------------------------------------------
// Shortlist: topk rounds of a block-wide argmin over the scenario's (strategy, split)
// items; round r takes the least (step time, item) pair that comes after round r-1's.
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) cm_shortlist_kernel(Tables tb, BatchDev bd, ObjDev od, uint64_t inf) {
    __shared__ uint64_t rc[8], ri[8];
    __shared__ uint64_t last_c, last_i;
    const uint32_t b = blockIdx.x;
    const Scen sc = bd.scen[b];
    const Tmpl tp = bd.tmpl[sc.tmpl];
    const uint64_t *best = bd.seg_best + sc.seg_base;
    const bool searched = (sc.policy_mask & (1u << CM_DYNPAR)) != 0;
    bool exhausted = !searched || tp.n_split_total == 0;
    for (int r = 0; r < od.topk; ++r) {
        uint64_t best_c = inf, best_i = ~0ull;
        if (!exhausted) {
            const uint64_t lc = r ? last_c : 0, li = r ? last_i : 0;
            for (uint64_t item = threadIdx.x; item < tp.n_split_total; item += blockDim.x) {
                const uint64_t T = item_step_time(tb, bd, tp, best, item, inf);
                if (T >= inf) continue;
                if (r && !pair_less(lc, li, T, item)) continue;     // taken by an earlier round
                if (pair_less(T, item, best_c, best_i)) { best_c = T; best_i = item; }
            }
        }
        for (int o = 16; o > 0; o >>= 1) {
            uint64_t oc = __shfl_xor_sync(0xffffffffu, best_c, o);
            uint64_t oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (pair_less(oc, oi, best_c, best_i)) { best_c = oc; best_i = oi; }
        }
        __syncthreads();   // everybody has read last_c / last_i of the previous round
        if ((threadIdx.x & 31) == 0) { rc[threadIdx.x >> 5] = best_c; ri[threadIdx.x >> 5] = best_i; }
        __syncthreads();
        const size_t slot = (size_t)b * od.topk + r;
        if (threadIdx.x == 0) {
            for (int w = 1; w < 8; ++w)
                if (pair_less(rc[w], ri[w], best_c, best_i)) { best_c = rc[w]; best_i = ri[w]; }
            last_c = best_c;
            last_i = best_i;
            Winner w;
            decode_winner(tb, bd, tp, b, best_c, best_i, inf, w);
            od.short_win[slot] = w;
            od.short_bytes[slot] = -1;
        }
        __syncthreads();   // last_c / last_i and the record are written
        if (threadIdx.x < kMaxP) init_kappa_sel(bd, od.short_win[slot], od.short_kappa + slot * kMaxP, (int)threadIdx.x);
        __syncthreads();
        if (last_c >= inf) exhausted = true;   // uniform: nothing is left for later rounds either
    }
}

cudaError_t launch_shortlist(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const uint64_t inf = batch_inf_bits(b);
    cm_shortlist_kernel<<<b.B, 256, 0, st>>>(t, b, o, inf);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Minimum-cost perfect matching, one warp per problem.  Rows = devices with their old layer
// range, columns = positions with their new range, Cost[i][j] = range_cost below.
//
// Devices that hold the same old range are interchangeable (the survivors of one old stage: up
// to N_dp of them), so the rows are first folded into CLASSES with a capacity, and the problem
// is solved as a transportation problem by successive shortest augmenting paths with
// potentials (Kuhn-Munkres, columns entering one at a time): u per class, v per column, reduced
// cost Cost - u - v >= 0.  For an entering column an alternating tree grows over classes;
// scanning a tree column is ONE cost evaluation per lane (lane = class), a class whose slack
// reaches zero joins the tree in the same pass as every other such class, and with it the
// columns it currently serves; only when nothing is tight do the potentials move by the least
// slack, which costs the warp-wide reduction.  The first class with spare capacity ends the
// search and the matching is flipped along the path.  Every loop is bounded by the problem
// size.  Lane `lane` owns classes c*32+lane, c < NC.
// ----------------------------------------------------------------------------------
constexpr int kMatchWarps = 4;

struct MatchWork {
    long long v[kMaxMatch];                       // column potentials
    long long tbase[kMaxMatch];                   // tree columns: potential shift already applied when they joined
    int cnt[kMaxMatch];                           // class: columns it serves now
    int head[kMaxMatch];                          // class: first column of its list (-1 = none)
    short cap[kMaxMatch];                         // class: rows folded into it
    short way[kMaxMatch];                         // class: tree column that gave its least slack
    short next_col[kMaxMatch];                    // column: next column served by the same class
    short tcol[kMaxMatch];                        // tree columns in the order they joined
    short row_class[kMaxMatch];                   // row -> class
    short match[kMaxMatch];                       // column -> class while solving; column -> row on return
    uint8_t olo[kMaxMatch], ohi[kMaxMatch], nlo[kMaxMatch], nhi[kMaxMatch];   // inputs
    uint8_t clo[kMaxMatch], chi[kMaxMatch];       // class ranges
};

__device__ __forceinline__ long long range_cost(const long long *PW, long long need, int a, int b, int x, int y) {
    const int lo = max(a, x), hi = min(b, y);
    return need - (hi > lo ? PW[hi] - PW[lo] : 0ll);
}

// warp minimum of a non-negative 64-bit value: two hardware min-reductions
__device__ __forceinline__ long long warp_min_nonneg(long long x) {
    const uint32_t hi = (uint32_t)((unsigned long long)x >> 32), lo = (uint32_t)x;
    const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
    const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
    return (long long)(((unsigned long long)mhi << 32) | mlo);
}

// Returns the total of the matching (same value in every lane), -1 if the iteration broke
// down (cannot happen for n >= 1; guards the loops).  On return w.match[j] = row of column j.
template <int NC>
__device__ long long warp_match(MatchWork &w, const long long *PW, int n, int lane) {
    const long long INF = LLONG_MAX / 4;
    // ---- fold equal rows into classes, numbered by their first row
    for (int i = lane; i < n; i += 32) {
        int first = i;
        for (int k = 0; k < i; ++k)
            if (w.olo[k] == w.olo[i] && w.ohi[k] == w.ohi[i]) { first = k; break; }
        w.tcol[i] = (short)first;                 // scratch: first row of i's class
        w.cap[i] = 0; w.cnt[i] = 0; w.head[i] = -1; w.match[i] = -1; w.next_col[i] = -1;
    }
    __syncwarp();
    int R = 0;
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const bool is_first = i < n && w.tcol[i] == i;
        const uint32_t mask = __ballot_sync(0xffffffffu, is_first);
        if (is_first) {
            const int r = R + __popc(mask & ((1u << lane) - 1u));
            w.row_class[i] = (short)r;
            w.clo[r] = w.olo[i];
            w.chi[r] = w.ohi[i];
        }
        R += __popc(mask);
    }
    __syncwarp();
    for (int i = lane; i < n; i += 32) {
        const int r = w.row_class[w.tcol[i]];
        if (w.tcol[i] != i) w.row_class[i] = (short)r;
        atomicAdd(&w.cnt[r], 1);                  // counted in cnt, moved to cap below
    }
    __syncwarp();
    for (int r = lane; r < R; r += 32) { w.cap[r] = (short)w.cnt[r]; w.cnt[r] = 0; }
    __syncwarp();
    // ---- start: v[j] = cheapest class of column j (u = 0), then every column claims a class that
    // attains it and still has room, lowest class first.  Most positions find a device that
    // already holds most of their layers, so few columns are left for the augmenting phase.
    for (int j = lane; j < n; j += 32) {
        const int x = w.nlo[j], y = w.nhi[j];
        const long long need = y > x ? PW[y] - PW[x] : 0ll;
        long long best = INF;
        for (int r = 0; r < R; ++r) {
            const long long c = range_cost(PW, need, w.clo[r], w.chi[r], x, y);
            best = c < best ? c : best;
        }
        w.v[j] = best;
        for (int r = 0; r < R; ++r) {
            if (range_cost(PW, need, w.clo[r], w.chi[r], x, y) != best) continue;
            if (atomicAdd(&w.cnt[r], 1) < (int)w.cap[r]) {
                w.match[j] = (short)r;
                w.next_col[j] = (short)atomicExch(&w.head[r], j);
                break;
            }
            atomicSub(&w.cnt[r], 1);
        }
    }
    __syncwarp();
    // ---- augmenting phase: class potentials and slacks in registers of the owning lane
    long long u[NC], slack[NC], ubase[NC];
    int clo[NC], chi[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int r = c * 32 + lane;
        u[c] = 0;
        clo[c] = r < R ? (int)w.clo[r] : 0;
        chi[c] = r < R ? (int)w.chi[r] : 0;
    }
    bool broken = false;
    for (int j0 = 0; j0 < n && !broken; ++j0) {
        if (w.match[j0] >= 0) continue;             // uniform: served since the start or an earlier flip
        uint32_t tree = 0;                          // bit c: class c*32+lane belongs to the tree
        long long D = 0;                            // potential shift so far
        int nt = 1, scanned = 0, found = -1;
#pragma unroll
        for (int c = 0; c < NC; ++c) slack[c] = INF;
        if (lane == 0) { w.tcol[0] = (short)j0; w.tbase[0] = 0; }
        __syncwarp();
        for (int iter = 0; iter <= 2 * (n + R) + 4 && found < 0; ++iter) {
            // 1. scan the tree columns that have not been scanned yet
            for (; scanned < nt; ++scanned) {
                const int j = w.tcol[scanned];
                const int x = w.nlo[j], y = w.nhi[j];
                const long long need = y > x ? PW[y] - PW[x] : 0ll;
                const long long vj = w.v[j];
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const int r = c * 32 + lane;
                    if (r >= R || ((tree >> c) & 1u)) continue;
                    const long long red = range_cost(PW, need, clo[c], chi[c], x, y) - u[c] - vj;
                    if (red < slack[c]) { slack[c] = red; w.way[r] = (short)j; }
                }
            }
            // 2. classes at zero slack join the tree; one with room ends the search, a full one
            // brings the columns it serves
            bool any_tight = false;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int r = c * 32 + lane;
                const bool tight = r < R && !((tree >> c) & 1u) && slack[c] == 0;
                uint32_t mask = __ballot_sync(0xffffffffu, tight);
                if (tight) { tree |= 1u << c; ubase[c] = D; }
                any_tight = any_tight || mask != 0;
                while (mask && found < 0) {
                    const int rr = c * 32 + (__ffs((int)mask) - 1);
                    mask &= mask - 1;
                    if (w.cnt[rr] < (int)w.cap[rr]) { found = rr; break; }      // uniform
                    int j = w.head[rr];
                    for (int k = 0; k <= n && j >= 0; ++k) {
                        if (nt >= kMaxMatch) { broken = true; break; }
                        if (lane == 0) { w.tcol[nt] = (short)j; w.tbase[nt] = D; }
                        ++nt;
                        j = w.next_col[j];
                    }
                }
            }
            __syncwarp();
            if (found >= 0 || broken) break;
            if (any_tight) continue;
            // 3. nothing tight: shift the potentials by the least slack outside the tree
            long long delta = INF;
#pragma unroll
            for (int c = 0; c < NC; ++c)
                if (c * 32 + lane < R && !((tree >> c) & 1u) && slack[c] < delta) delta = slack[c];
            delta = warp_min_nonneg(delta);
            if (delta >= INF) { broken = true; break; }   // every class is in the tree and full: cannot happen
            D += delta;
#pragma unroll
            for (int c = 0; c < NC; ++c)
                if (!((tree >> c) & 1u)) slack[c] -= delta;
        }
        if (found < 0) broken = true;
        if (broken) break;
        // potentials: tree columns rose, tree classes fell, each by the shift since it joined
        for (int k = lane; k < nt; k += 32) w.v[w.tcol[k]] += D - w.tbase[k];
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if ((tree >> c) & 1u) u[c] -= D - ubase[c];
        __syncwarp();
        // flip along the path: class `found` takes the column that reached it, the class that
        // served this column before takes the one that reached it, ... down to the new column
        if (lane == 0) {
            int r = found;
            for (int step = 0; step <= n; ++step) {
                const int j = w.way[r];
                const int old = w.match[j];
                if (old >= 0) {     // unlink j from the class that served it
                    int q = w.head[old];
                    if (q == j) w.head[old] = w.next_col[j];
                    else
                        for (int k = 0; k <= n && q >= 0; ++k) {
                            const int nx = w.next_col[q];
                            if (nx == j) { w.next_col[q] = w.next_col[j]; break; }
                            q = nx;
                        }
                    --w.cnt[old];
                }
                w.match[j] = (short)r;
                w.next_col[j] = (short)w.head[r];
                w.head[r] = j;
                ++w.cnt[r];
                if (old < 0) break;
                r = old;
            }
        }
        __syncwarp();
    }
    if (broken) return -1;
    long long total = 0;
    for (int j = lane; j < n; j += 32) {
        const int r = w.match[j], x = w.nlo[j], y = w.nhi[j];
        total += range_cost(PW, y > x ? PW[y] - PW[x] : 0ll, w.clo[r], w.chi[r], x, y);
    }
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    __syncwarp();
    // hand the rows of every class to the columns it serves (rows ascending, list order)
    for (int r = lane; r < R; r += 32) {
        int j = w.head[r];
        for (int i = 0; i < n && j >= 0; ++i) {
            if (w.row_class[i] != r) continue;
            const int nx = w.next_col[j];
            w.tcol[j] = (short)i;                 // scratch: row of column j
            j = nx;
        }
    }
    __syncwarp();
    for (int j = lane; j < n; j += 32) w.match[j] = w.tcol[j];
    __syncwarp();
    return total;
}

__device__ __forceinline__ long long warp_match_any(MatchWork &w, const long long *PW, int n, int lane) {
    // the class count is known only inside; NC is chosen for the row count, which bounds it
    if (n <= 32) return warp_match<1>(w, PW, n, lane);
    if (n <= 64) return warp_match<2>(w, PW, n, lane);
    if (n <= 128) return warp_match<4>(w, PW, n, lane);
    return warp_match<8>(w, PW, n, lane);
}

__device__ __forceinline__ void stage_state_bytes(long long *PW, const DevProfile *p) {
    for (int l = threadIdx.x; l <= p->L; l += blockDim.x) PW[l] = p->PW[l];
    __syncthreads();
}

// Layer cuts of pipeline q of a shortlisted plan: its completed layer composition, or the
// min-max partition; false if the completion found no composition (cannot happen for a
// feasible pair) or the partition does not exist.
__device__ __forceinline__ bool pipeline_cuts(const Tables &tb, const BatchDev &bd, const ObjDev &od, size_t slot,
                                              const Winner &w, int q, uint8_t *cuts /* [S+1] */) {
    const TSeg g = bd.tseg[w.seg[q]];
    const uint64_t kappa = od.short_kappa[slot * kMaxP + q];
    const int S = g.S;
    if (kappa < g.K) {
        layer_cuts(tb.binom, bd.layer_mode, tb.prof->L, S, kappa, cuts);
        return true;
    }
    if (kappa != g.K) return false;
    const uint8_t *mm = tb.mm_cuts + (size_t)tb.mm_slot(S, g.m) * (kMaxS + 1);
    if (mm[0] != 0) return false;
    for (int i = 0; i <= S; ++i) cuts[i] = mm[i];
    return true;
}

// One warp per shortlist slot: survivors keep the layers of their old stage (device =
// pipeline * n_pp + stage); position off_p + i of the plan holds stage i of pipeline p.
__global__ void __launch_bounds__(kMatchWarps * 32) cm_plan_matching_kernel(Tables tb, BatchDev bd, ObjDev od, uint64_t inf) {
    __shared__ MatchWork work[kMatchWarps];
    __shared__ long long PW[kMaxL + 1];
    const DevProfile *p = tb.prof;
    stage_state_bytes(PW, p);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t slot = (size_t)blockIdx.x * kMatchWarps + warp;
    if (slot >= (size_t)bd.B * od.topk) return;
    const Winner &w = od.short_win[slot];
    if (w.cost_bits >= inf || w.dp == 0) return;            // empty slot: bytes stay -1
    MatchWork &mw = work[warp];
    const Scen sc = bd.scen[w.scen];
    const int N = p->n_dp * p->n_pp, n_pp = p->n_pp;
    int n = 0;
    for (int base = 0; base < N; base += 32) {
        const int d = base + lane;
        bool alive = d < N;
        for (uint32_t f = 0; f < sc.n_failed; ++f) alive = alive && bd.failed[sc.failed_first + f] != (uint32_t)d;
        const uint32_t mask = __ballot_sync(0xffffffffu, alive);
        const int idx = n + __popc(mask & ((1u << lane) - 1u));
        if (alive && idx < kMaxMatch) {
            mw.olo[idx] = (uint8_t)p->base_cuts[d % n_pp];
            mw.ohi[idx] = (uint8_t)p->base_cuts[d % n_pp + 1];
        }
        n += __popc(mask);
    }
    bool ok = n >= 1 && n <= kMaxMatch;
    int covered = 0;
    if (ok && lane < (int)w.dp) {
        const Strat &s = bd.strat[w.strat];
        int off = 0;
        for (int q = 0; q < lane; ++q) off += s.S[q];
        const int S = s.S[lane];
        uint8_t cuts[kMaxS + 1];
        if (off + S > n) ok = false;
        else ok = pipeline_cuts(tb, bd, od, slot, w, lane, cuts);
        if (ok) {
            for (int i = 0; i < S; ++i) { mw.nlo[off + i] = cuts[i]; mw.nhi[off + i] = cuts[i + 1]; }
            covered = S;
        }
    }
    for (int o = 16; o > 0; o >>= 1) covered += __shfl_xor_sync(0xffffffffu, covered, o);
    ok = __all_sync(0xffffffffu, ok) && covered == n;       // a strategy uses every survivor
    __syncwarp();
    if (!ok) return;
    const long long total = warp_match_any(mw, PW, n, lane);
    if (total < 0) return;
    uint16_t *asg = od.short_assign + slot * kMaxMatch;
    for (int j = lane; j < kMaxMatch; j += 32) asg[j] = j < n ? (uint16_t)mw.match[j] : (uint16_t)0;
    if (lane == 0) od.short_bytes[slot] = total;
}

cudaError_t launch_plan_matching(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const uint64_t inf = batch_inf_bits(b);
    const size_t slots = (size_t)b.B * o.topk;
    cm_plan_matching_kernel<<<(unsigned)((slots + kMatchWarps - 1) / kMatchWarps), kMatchWarps * 32, 0, st>>>(t, b, o, inf);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(kMatchWarps * 32) cm_range_matching_kernel(Tables tb, int n_problems, const int32_t *sizes,
                                                                             const uint8_t *old_lo, const uint8_t *old_hi,
                                                                             const uint8_t *new_lo, const uint8_t *new_hi,
                                                                             int64_t *total, uint16_t *assign) {
    __shared__ MatchWork work[kMatchWarps];
    __shared__ long long PW[kMaxL + 1];
    stage_state_bytes(PW, tb.prof);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = blockIdx.x * kMatchWarps + warp;
    if (q >= n_problems) return;
    MatchWork &mw = work[warp];
    const int n = sizes[q], L = tb.prof->L;
    const size_t base = (size_t)q * kMaxMatch;
    for (int j = lane; j < n; j += 32) {
        mw.olo[j] = (uint8_t)min((int)old_lo[base + j], L); mw.ohi[j] = (uint8_t)min((int)old_hi[base + j], L);
        mw.nlo[j] = (uint8_t)min((int)new_lo[base + j], L); mw.nhi[j] = (uint8_t)min((int)new_hi[base + j], L);
    }
    __syncwarp();
    const long long t = warp_match_any(mw, PW, n, lane);
    if (lane == 0) total[q] = t;
    if (assign)
        for (int j = lane; j < kMaxMatch; j += 32) assign[base + j] = (j < n && t >= 0) ? (uint16_t)mw.match[j] : (uint16_t)0;
}

cudaError_t launch_range_matching(const Tables &t, int n_problems, const int32_t *sizes, const uint8_t *old_lo,
                                  const uint8_t *old_hi, const uint8_t *new_lo, const uint8_t *new_hi,
                                  int64_t *total, uint16_t *assign, cudaStream_t st) {
    if (n_problems <= 0) return cudaSuccess;
    cm_range_matching_kernel<<<(n_problems + kMatchWarps - 1) / kMatchWarps, kMatchWarps * 32, 0, st>>>(
        t, n_problems, sizes, old_lo, old_hi, new_lo, new_hi, total, assign);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Asymmetric synchronisation (Section "Restorer", Asymmetric Communication).  One warp per
// shortlisted plan: lane q evaluates the bare time of pipeline q (one participant: no
// synchronisation term) and writes the stage of every layer; the layer graph (edge = some
// pipeline keeps both layers on one device) is coloured greedily in layer order, lanes
// sharing the earlier layers and OR-reducing the colours their neighbours took; a round
// lasts as long as its largest all-reduce, rounds add up in colour order.
// ----------------------------------------------------------------------------------
struct RoundsWork {
    uint8_t stage_of[kMaxP][kMaxL];
    uint8_t cuts[kMaxP][kMaxS + 4];
    uint8_t colour[kMaxL];
};

template <typename T>
__global__ void __launch_bounds__(kMatchWarps * 32) cm_plan_rounds_kernel(Tables tb, BatchDev bd, ObjDev od) {
    __shared__ SProf<T> sp;
    __shared__ RoundsWork work[kMatchWarps];
    stage_profile(sp, tb);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t slot = (size_t)blockIdx.x * kMatchWarps + warp;
    if (slot >= (size_t)bd.B * od.topk) return;
    if (lane < 2) { od.short_step[slot * 2 + lane] = inf_bits<T>(); od.short_rounds[slot * 2 + lane] = 0; }
    const Winner &w = od.short_win[slot];
    if (w.cost_bits >= inf_bits<T>() || w.dp == 0) return;
    RoundsWork &rw = work[warp];
    const int L = sp.L, dp = (int)w.dp;
    bool ok = true;
    if (lane < dp) {
        uint8_t cuts[kMaxS + 1];
        ok = pipeline_cuts(tb, bd, od, slot, w, lane, cuts);
        if (ok) {
            const int S = bd.tseg[w.seg[lane]].S;
            for (int i = 0; i <= S; ++i) rw.cuts[lane][i] = cuts[i];
            for (int i = 0; i < S; ++i)
                for (int l = cuts[i]; l < cuts[i + 1]; ++l) rw.stage_of[lane][l] = (uint8_t)i;
        }
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;
    __syncwarp();
    T t_pipe = (T)0;
    for (int q = 0; q < dp; ++q) {            // one pipeline after the other, each over the whole warp
        const SegView g = seg_view(bd, w.scen, w.seg[q]);
        t_pipe = tmax(t_pipe, warp_pipe_time<T>(sp, rw.cuts[q], g.S, g.m, g.tier, lane));
    }
    int rounds = 0;
    for (int l = 0; l < L; ++l) {
        uint32_t used[4] = {0u, 0u, 0u, 0u};
        for (int k = lane; k < l; k += 32) {
            bool adjacent = false;
            for (int q = 0; q < dp; ++q) adjacent = adjacent || rw.stage_of[q][l] == rw.stage_of[q][k];
            if (adjacent) { const int c = rw.colour[k]; used[c >> 5] |= 1u << (c & 31); }
        }
        int c = -1;
#pragma unroll
        for (int word = 0; word < 4; ++word) {
            const uint32_t all = __reduce_or_sync(0xffffffffu, used[word]);
            if (c < 0 && all != 0xffffffffu) c = word * 32 + __ffs((int)~all) - 1;
        }
        if (lane == 0) rw.colour[l] = (uint8_t)c;
        rounds = c + 1 > rounds ? c + 1 : rounds;
        __syncwarp();
    }
    T t_sync = (T)0;
    for (int c = 0; c < rounds; ++c) {
        T longest = (T)0;
        for (int l = lane; l < L; l += 32)
            if (rw.colour[l] == c) longest = tmax(longest, Num<T>::sync(sp.PP[l + 1] - sp.PP[l], dp, sp.bw_sync, sp.intval));
        for (int o = 16; o > 0; o >>= 1) {
            const uint64_t other = __shfl_xor_sync(0xffffffffu, Num<T>::bits(longest), o);
            longest = tmax(longest, Num<T>::from_bits(other));
        }
        t_sync = t_sync + longest;
    }
    int domains = 0;
    for (int base = 0; base < L; base += 32) {
        const int l = base + lane;
        bool fresh = l == 0;
        if (l > 0 && l < L)
            for (int q = 0; q < dp; ++q) fresh = fresh || rw.stage_of[q][l] != rw.stage_of[q][l - 1];
        domains += __popc(__ballot_sync(0xffffffffu, fresh && l < L));
    }
    if (lane == 0) {
        od.short_step[slot * 2] = Num<T>::bits(t_pipe + t_sync);
        od.short_step[slot * 2 + 1] = Num<T>::bits(t_sync);
        od.short_rounds[slot * 2] = rounds;
        od.short_rounds[slot * 2 + 1] = domains;
    }
}

cudaError_t launch_plan_rounds(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const size_t slots = (size_t)b.B * o.topk;
    const unsigned grid = (unsigned)((slots + kMatchWarps - 1) / kMatchWarps);
    if (native_i64(b)) cm_plan_rounds_kernel<long long><<<grid, kMatchWarps * 32, 0, st>>>(t, b, o);
    else cm_plan_rounds_kernel<double><<<grid, kMatchWarps * 32, 0, st>>>(t, b, o);
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------
// Objective (Section "Problem Formulation"): steps before the next fault,
// (t_gap - t_trans) / t_step, of rerouting, redundant computation (t_trans = 0) and every
// shortlisted plan (t_trans = restart + matched bytes / bandwidth).  The greatest wins,
// ties to the lower policy id, then to the earlier rank.  fp64: the quotients are compared
// as rounded; int64: fractions are compared exactly by cross-multiplication.
// ----------------------------------------------------------------------------------
struct Frac {
    double nd, dd;          // fp64 mode
    long long ni, di;       // int64 mode
};

__device__ __forceinline__ bool frac_greater(const Frac &a, const Frac &b, int mode) {
    if (mode == CM_COST_INT64NS) return (__int128)a.ni * (__int128)b.di > (__int128)b.ni * (__int128)a.di;
    return a.nd / a.dd > b.nd / b.dd;
}

__device__ __forceinline__ void plan_from_winner(const BatchDev &bd, const Winner &w, const uint64_t *kappa,
                                                 uint64_t step_bits, cm_plan &pl) {
    plan_clear(pl, CM_DYNPAR);
    const Strat &s = bd.strat[w.strat];
    pl.feasible = 1;
    plan_set_cost(pl, step_bits, bd);
    pl.strategy = w.strat - bd.tmpl[bd.scen[w.scen].tmpl].strat_first;
    pl.n_pipes = w.dp;
    pl.split_rank = w.item - s.split_first;
    for (uint32_t q = 0; q < w.dp; ++q) {
        pl.stages[q] = s.S[q];
        pl.micro[q] = w.micro[q];
        pl.kappa[q] = kappa[q];
    }
}

__global__ void __launch_bounds__(32) cm_objective_kernel(Tables tb, BatchDev bd, ObjDev od, uint64_t inf) {
    __shared__ int win_slot;
    const uint32_t b = blockIdx.x;
    const int mode = bd.mode;
    const cm_plan *pol = bd.plans + (size_t)b * 4;
    if (threadIdx.x == 0) {
        cm_transition tr;
        tr.rounds = 0; tr.domains = 0; tr.t_sync = 0.0; tr.t_sync_ns = 0;
        tr.policy = 0; tr.feasible = 0; tr.rank = -1;
        tr.n_survivors = tb.prof->n_dp * tb.prof->n_pp - (int)bd.scen[b].n_failed;
        tr.xfer_bytes = 0; tr.t_trans = 0.0; tr.t_trans_ns = 0; tr.objective = 0.0;
        Frac best{0.0, 1.0, 0, 1};
        bool have = false;
        int slot_sel = -1;
        for (int q = 0; q < 2; ++q) {
            if (!pol[q].feasible) continue;
            Frac j{od.t_gap, pol[q].cost, od.t_gap_i, pol[q].cost_ns};
            if (!have || frac_greater(j, best, mode)) { have = true; best = j; tr.policy = q; }
        }
        for (int r = 0; r < od.topk; ++r) {
            const size_t slot = (size_t)b * od.topk + r;
            const long long bytes = od.short_bytes[slot];
            if (bytes < 0) continue;
            const uint64_t step = od.sync_rounds ? od.short_step[slot * 2] : od.short_win[slot].cost_bits;
            if (step >= inf) continue;
            Frac j{0.0, 1.0, 0, 1};
            double tt = 0.0;
            long long tti = 0;
            if (mode == CM_COST_INT64NS) {
                tti = transition_time_i64(od.t_restart_i, bytes, od.bw_xfer);
                j.ni = od.t_gap_i - tti;
                j.di = batch_cost_ns(bd, step);
            } else {
                tt = transition_time_f64(od.t_restart, bytes, od.bw_xfer);
                j.nd = od.t_gap - tt;
                j.dd = __longlong_as_double((long long)step);
            }
            if (!have || frac_greater(j, best, mode)) {
                have = true; best = j; slot_sel = (int)r;
                tr.policy = CM_DYNPAR; tr.rank = r; tr.xfer_bytes = bytes; tr.t_trans = tt; tr.t_trans_ns = tti;
            }
        }
        cm_plan pl;
        if (!have) plan_clear(pl, 0);
        else if (tr.policy != CM_DYNPAR) {
            pl = pol[tr.policy];
            tr.rank = -1; tr.xfer_bytes = 0; tr.t_trans = 0.0; tr.t_trans_ns = 0;
        } else {
            const size_t slot = (size_t)b * od.topk + slot_sel;
            plan_from_winner(bd, od.short_win[slot], od.short_kappa + slot * kMaxP,
                             od.sync_rounds ? od.short_step[slot * 2] : od.short_win[slot].cost_bits, pl);
            if (od.sync_rounds) {
                tr.rounds = od.short_rounds[slot * 2];
                tr.domains = od.short_rounds[slot * 2 + 1];
                if (mode == CM_COST_INT64NS) tr.t_sync_ns = batch_cost_ns(bd, od.short_step[slot * 2 + 1]);
                else tr.t_sync = __longlong_as_double((long long)od.short_step[slot * 2 + 1]);
            }
        }
        if (have) {
            tr.feasible = 1;
            tr.objective = mode == CM_COST_INT64NS ? (double)best.ni / (double)best.di : best.nd / best.dd;
        }
        od.best[b] = pl;
        // header of the transition record; the matching follows from all lanes
        cm_transition *out = od.trans + b;
        out->policy = tr.policy; out->feasible = tr.feasible; out->rank = tr.rank; out->n_survivors = tr.n_survivors;
        out->xfer_bytes = tr.xfer_bytes; out->t_trans = tr.t_trans; out->t_trans_ns = tr.t_trans_ns;
        out->objective = tr.objective;
        out->rounds = tr.rounds; out->domains = tr.domains; out->t_sync = tr.t_sync; out->t_sync_ns = tr.t_sync_ns;
        win_slot = (have && tr.policy == CM_DYNPAR) ? slot_sel : -1;
    }
    __syncthreads();
    const uint16_t *src = win_slot >= 0 ? od.short_assign + ((size_t)b * od.topk + win_slot) * kMaxMatch : nullptr;
    for (int j = threadIdx.x; j < kMaxMatch; j += 32) od.trans[b].assign[j] = src ? src[j] : (uint16_t)0;
    if (od.short_plans && (int)threadIdx.x < od.topk) {
        const size_t slot = (size_t)b * od.topk + threadIdx.x;
        cm_plan pl;
        const uint64_t step = od.sync_rounds ? od.short_step[slot * 2] : od.short_win[slot].cost_bits;
        if (od.short_bytes[slot] >= 0 && step < inf) plan_from_winner(bd, od.short_win[slot], od.short_kappa + slot * kMaxP, step, pl);
        else plan_clear(pl, CM_DYNPAR);
        od.short_plans[slot] = pl;
    }
}

cudaError_t launch_objective(const Tables &t, const BatchDev &b, const ObjDev &o, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const uint64_t inf = batch_inf_bits(b);
    cm_objective_kernel<<<b.B, 32, 0, st>>>(t, b, o, inf);
    return cudaGetLastError();
}

}  // namespace cm
