// Data rerouting and redundant computation: one plan per scenario each (sm_100a).
//
// Rerouting (Section "Estimator", single- and multi-failure step time): the failed
// devices' micro-batches go to the data-parallel peers of the same stage; with F_i
// failed devices in stage i the step grows by N_m F_i (F_i^st + B_i^st) / (N_dp - F_i) per
// affected stage on top of the unchanged base pipeline; unrecoverable if F_i >= N_dp.
//
// Redundant computation (Section "Limitations of Backup-free Methods", prose): a failed
// stage is taken over by its predecessor; every stage but the last also carries its
// successor's work and state.  Infeasible if stage 0 failed or two neighbours failed.
//
// One CTA per scenario, one warp per pipeline to simulate: warp 0 the base pipeline of
// the rerouting plan, warp 1+k pipeline k of the redundant plan.  Each of these is a
// single recurrence, so there is no plan-level parallelism to hide its dependency chain
// behind; instead the warp spreads the STAGES over its lanes and walks the pipeline in
// lock step, slot by slot.
#include "cm_device.cuh"

namespace cm {

// (the lock-step recurrence with one stage per lane is sim_lockstep_n<T, 1> of cm_device.cuh)

template <typename T> __device__ __forceinline__ T warp_max(T v) {
    for (int o = 16; o > 0; o >>= 1) {
        const T w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w > v ? w : v;
    }
    return v;
}

template <typename T>
__global__ void __launch_bounds__(32 * (kMaxP + 1)) cm_policy_kernel(Tables tb, BatchDev bd) {
    __shared__ SProf<T> sp;
    __shared__ int base_cuts[kMaxS + 1];
    __shared__ uint64_t rc_bits[kMaxP];
    __shared__ uint16_t rc_S[kMaxP];
    const DevProfile *p = tb.prof;
    stage_profile(sp, tb);
    for (int i = threadIdx.x; i <= p->n_pp; i += blockDim.x) base_cuts[i] = p->base_cuts[i];
    __syncthreads();
    const int b = blockIdx.x;
    const Scen sc = bd.scen[b];
    const uint32_t *failed = bd.failed + sc.failed_first;
    const int S0 = sp.n_pp, m = sp.n_micro, n_dp = sp.n_dp;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int dpn = p->devices_per_node;
    const bool wide = S0 > 32;   // deeper than a warp: lane 0 walks the stages serially
    T Fs[kMaxS], Bs[kMaxS], xts[kMaxS], clk[kMaxS], pnd[kMaxS];   // serial path only

    if (warp == 0) {
        // ------------------------------------------------------------ data rerouting
        uint64_t out = inf_bits<T>();
        if (sc.policy_mask & (1u << CM_REROUTE)) {
            if (!wide) {
                const int i = lane;
                int fcnt = 0;
                for (uint32_t f = 0; f < sc.n_failed; ++f) fcnt += ((int)(failed[f] % S0) == i) ? 1 : 0;
                bool ok = m >= 1;
                T F = (T)0, B = (T)0, xt = (T)0, extra_i = (T)0, sync_i = (T)0;
                if (i < S0) {
                    const int lo = base_cuts[i], hi = base_cuts[i + 1];
                    ok = ok && fcnt < n_dp && stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S0, m, sp.cap, sp.sched);
                    F = sp.PF[hi] - sp.PF[lo];
                    B = sp.PB[hi] - sp.PB[lo];
                    const int tier = (i / dpn == (i + 1) / dpn) ? 0 : 1;   // pipeline 0 sits on devices 0 .. S0-1
                    xt = i < S0 - 1 ? sp.XT[tier][hi - 1] : (T)0;
                    if (ok && fcnt > 0) extra_i = Num<T>::reroute_extra(m * fcnt, F + B, n_dp - fcnt, sp.intval);
                    if (ok) sync_i = Num<T>::sync(sp.PP[hi] - sp.PP[lo], n_dp - fcnt, sp.bw_sync, sp.intval);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (ok) {
                    const T base = sim_lockstep_n<T, 1>(S0, m, &F, &B, &xt, sp.sched);
                    const T t_sync = warp_max<T>(sync_i);
                    T extra = (T)0;   // summed in stage order, affected stages only
                    for (int s = 0; s < S0; ++s) {
                        const T e = __shfl_sync(0xffffffffu, extra_i, s);
                        const int c = __shfl_sync(0xffffffffu, fcnt, s);
                        if (c > 0) extra = extra + e;
                    }
                    out = Num<T>::bits((base + extra) + t_sync);
                }
            } else if (lane == 0) {
                int fcnt[kMaxS];
                for (int i = 0; i < S0; ++i) fcnt[i] = 0;
                for (uint32_t f = 0; f < sc.n_failed; ++f) fcnt[failed[f] % S0]++;
                bool ok = m >= 1;
                for (int i = 0; i < S0; ++i) ok = ok && fcnt[i] < n_dp;
                for (int i = 0; i < S0 && ok; ++i) {
                    const int lo = base_cuts[i], hi = base_cuts[i + 1];
                    ok = stage_fits(sp.PS[hi] - sp.PS[lo], sp.PA[hi] - sp.PA[lo], i, S0, m, sp.cap, sp.sched);
                }
                if (ok) {
                    T extra = (T)0, t_sync = (T)0;
                    for (int i = 0; i < S0; ++i) {
                        const int lo = base_cuts[i], hi = base_cuts[i + 1];
                        Fs[i] = sp.PF[hi] - sp.PF[lo];
                        Bs[i] = sp.PB[hi] - sp.PB[lo];
                        const int tier = (i / dpn == (i + 1) / dpn) ? 0 : 1;
                        xts[i] = i < S0 - 1 ? sp.XT[tier][hi - 1] : (T)0;
                        if (fcnt[i] > 0) extra = extra + Num<T>::reroute_extra(m * fcnt[i], Fs[i] + Bs[i], n_dp - fcnt[i], sp.intval);
                        t_sync = tmax(t_sync, Num<T>::sync(sp.PP[hi] - sp.PP[lo], n_dp - fcnt[i], sp.bw_sync, sp.intval));
                    }
                    const T base = sim_pipe<T>(S0, m, Fs, Bs, xts, clk, pnd, sp.sched);
                    out = Num<T>::bits((base + extra) + t_sync);
                }
            }
        }
        if (lane == 0) bd.pol_cost[2 * b + 0] = out;
    } else if (warp - 1 < n_dp) {
        // ------------------------------------------------- redundant computation, pipeline k
        const int k = warp - 1;
        uint64_t dead = 0;
        for (uint32_t f = 0; f < sc.n_failed; ++f)
            if ((int)(failed[f] / S0) == k) dead |= 1ull << (failed[f] % S0);
        bool ok = m >= 1 && !(dead & 1ull) && !(dead & (dead >> 1));   // warp-uniform
        const uint64_t all = S0 >= 64 ? ~0ull : ((1ull << S0) - 1);
        const uint64_t alive = ~dead & all;
        const int S = __popcll(alive);
        uint64_t bits = inf_bits<T>();
        if (ok && !wide) {
            // lane j = j-th surviving stage
            const int j = lane;
            int orig = 0;
            {
                uint64_t a = alive;
                for (int q = 0; q < j && a; ++q) a &= a - 1;
                orig = a ? __ffsll((long long)a) - 1 : 0;
            }
            T f = (T)0, bw = (T)0, xt = (T)0;
            long long stat = 0, act = 0, g = 0;
            int lo = 0, hi = 1, dev = 0;
            if (j < S) {
                lo = base_cuts[orig];
                hi = base_cuts[orig + 1];
                if (orig + 1 < S0 && ((dead >> (orig + 1)) & 1ull)) hi = base_cuts[orig + 2];
                dev = k * S0 + orig;
                f = sp.PF[hi] - sp.PF[lo];
                bw = sp.PB[hi] - sp.PB[lo];
                stat = sp.PS[hi] - sp.PS[lo];
                act = sp.PA[hi] - sp.PA[lo];
                g = sp.PP[hi] - sp.PP[lo];
            }
            // the successor's work and state ride along on every stage but the last
            const T f2 = __shfl_down_sync(0xffffffffu, f, 1), b2 = __shfl_down_sync(0xffffffffu, bw, 1);
            const long long stat2 = __shfl_down_sync(0xffffffffu, stat, 1), act2 = __shfl_down_sync(0xffffffffu, act, 1);
            const int dev2 = __shfl_down_sync(0xffffffffu, dev, 1);
            bool fits = true;
            if (j < S) {
                if (j < S - 1) {
                    f = f + f2;
                    bw = bw + b2;
                    stat = stat + stat2;
                    act = act + act2;
                    xt = sp.XT[(dev / dpn == dev2 / dpn) ? 0 : 1][hi - 1];
                }
                fits = stage_fits(stat, act, j, S, m, sp.cap, sp.sched);
            }
            ok = __all_sync(0xffffffffu, fits);
            if (ok) {
                const T t = sim_lockstep_n<T, 1>(S, m, &f, &bw, &xt, sp.sched);
                const long long g_max = warp_max<long long>(g);
                bits = Num<T>::bits(t + Num<T>::sync(g_max, n_dp, sp.bw_sync, sp.intval));
            }
        } else if (ok && lane == 0) {
            // deeper than a warp: lane 0 walks the surviving stages in order, each read off the
            // alive mask exactly as the lanes do above (stage j = j-th set bit; its range runs to
            // the end of a failed stage right behind it; the stage behind it rides along)
            uint64_t rest = alive;
            long long g_max = 0;
            bool fits = true;
            int n = 0;
            int orig = __ffsll((long long)rest) - 1;
            rest &= rest - 1;
            int lo = base_cuts[orig];
            int hi = base_cuts[orig + 1 + ((orig + 1 < S0 && ((dead >> (orig + 1)) & 1ull)) ? 1 : 0)];
            while (fits) {
                T f = sp.PF[hi] - sp.PF[lo], bw = sp.PB[hi] - sp.PB[lo];
                long long stat = sp.PS[hi] - sp.PS[lo], act = sp.PA[hi] - sp.PA[lo];
                const long long gb = sp.PP[hi] - sp.PP[lo];
                g_max = gb > g_max ? gb : g_max;
                xts[n] = (T)0;
                const bool last = rest == 0;
                int orig2 = 0, lo2 = 0, hi2 = 0;
                if (!last) {
                    orig2 = __ffsll((long long)rest) - 1;
                    rest &= rest - 1;
                    lo2 = base_cuts[orig2];
                    hi2 = base_cuts[orig2 + 1 + ((orig2 + 1 < S0 && ((dead >> (orig2 + 1)) & 1ull)) ? 1 : 0)];
                    f = f + (sp.PF[hi2] - sp.PF[lo2]);
                    bw = bw + (sp.PB[hi2] - sp.PB[lo2]);
                    stat = stat + (sp.PS[hi2] - sp.PS[lo2]);
                    act = act + (sp.PA[hi2] - sp.PA[lo2]);
                    xts[n] = sp.XT[((k * S0 + orig) / dpn == (k * S0 + orig2) / dpn) ? 0 : 1][hi - 1];
                }
                Fs[n] = f;
                Bs[n] = bw;
                fits = stage_fits(stat, act, n, S, m, sp.cap, sp.sched);
                ++n;
                if (last) break;
                orig = orig2; lo = lo2; hi = hi2;
            }
            if (fits) bits = Num<T>::bits(sim_pipe<T>(n, m, Fs, Bs, xts, clk, pnd, sp.sched) + Num<T>::sync(g_max, n_dp, sp.bw_sync, sp.intval));
        }
        if (wide) bits = __shfl_sync(0xffffffffu, bits, 0);
        if (lane == 0 && k < kMaxP) { rc_bits[k] = bits; rc_S[k] = (uint16_t)S; }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // the slowest pipeline sets the step; an infeasible pipeline (inf) wins the max
        uint64_t worst = 0;
        for (int k = 0; k < n_dp && k < kMaxP; ++k) {
            worst = rc_bits[k] > worst ? rc_bits[k] : worst;
            bd.rc_stages[b * kMaxP + k] = rc_S[k];
        }
        bd.pol_cost[2 * b + 1] = (sc.policy_mask & (1u << CM_REDUNDANT)) ? worst : inf_bits<T>();
    }
}

cudaError_t launch_policies(const Tables &t, const BatchDev &b, int n_dp, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    const int threads = 32 * (1 + (n_dp < kMaxP ? n_dp : kMaxP));
    if (native_i64(b)) cm_policy_kernel<long long><<<b.B, threads, 0, st>>>(t, b);
    else cm_policy_kernel<double><<<b.B, threads, 0, st>>>(t, b);
    return cudaGetLastError();
}

}  // namespace cm
