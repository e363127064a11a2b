"""Benchmark of the execution-plan search: candidate plans evaluated per second and
plan-search latency per failure on B200.

A step is one pass of the whole hot path (descriptor tables -> min-max partitions ->
rerouting / redundant-computation plans -> cost kernel over every pipeline-plan ->
split reduction -> tie-break pass -> policy pick -> plans on the host) over one batch
of synthetic failure scenarios.  Default workload: the failure-scenario sweep, the largest
configuration that fits one GPU (256 devices DP8 x PP32, L=96, 1024 failure sets of 1-16
devices, every policy); the other configurations are timed as context under "workloads".

  python bench.py --gpus 1 --steps K --warmup W            # this library
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle on the host cores
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate_plans_evaluated_per_sec"
UNIT = "plans/s"
N_SM = 148
SM_MAX_MHZ_FALLBACK = 1965.0
# The search pass is issue bound (no algorithmic HBM traffic, no contraction).  Its bound is
#   cells/s <= N_SM x 4 schedulers x 32 lanes x f_clk / I_cell
# with I_cell = executed thread-instructions per recurrence cell of the kernel class that
# dominates the workload, taken from the ncu capture summarised in the named file under
# profiles/ (instruction counters of one launch / its cells); `issue_active` is that capture's
# issue-slot utilisation.  f_clk is the median SM clock sampled while the timed region ran.
# class: "regs" = cm_cost_regs_kernel (pipelines of <= 16 stages), "wide" = the deep-pipeline
# kernel (17 .. 64 stages); arithmetic 0 = fp64 (also the exact integer-valued mode), 1 = int64.
KERNEL_PROFILES = {
    ("regs", 0): {"i_cell": 5.85, "issue_active": 0.650, "fp64_pipe_active": 0.646, "dram_bytes_per_cell": 660480 / 8.54e9,
                  "profile": "profiles/cm_cost_regs_kernel_paper-scale-512.md"},
    ("regs", 1): {"i_cell": 8.64, "issue_active": 0.630, "fp64_pipe_active": 0.0, "dram_bytes_per_cell": 620000 / 8.53e9,
                  "profile": "profiles/cm_cost_regs_kernel_int64_paper-scale-512.md"},
    ("wide", 0): {"i_cell": 6.14, "issue_active": 0.574, "fp64_pipe_active": 0.558, "dram_bytes_per_cell": 173056 / 6.199e9,
                  "profile": "profiles/cm_cost_wide_kernel_175b-like-8.md"},
    ("regs_pair", 0): {"i_cell": 5.80, "issue_active": 0.628, "fp64_pipe_active": 0.631, "dram_bytes_per_cell": 957184 / 4.992e9,
                       "profile": "profiles/cm_cost_regs_pair_kernel_paper-scale-512.md"},
    # the deep pipelines of a batch with micro-batch pairs on (the default): cm_cost_pair_kernel
    ("pair", 0): {"i_cell": 6.57, "issue_active": 0.546, "fp64_pipe_active": 0.496, "dram_bytes_per_cell": 6529024 / 3.653e9,
                  "profile": "profiles/cm_cost_pair_kernel_175b-like-8.md"},
}
KERNEL_NAMES = {"regs": "cm_cost_regs_kernel", "regs_pair": "cm_cost_regs_pair_kernel", "wide": "cm_cost_wide_kernel",
                "pair": "cm_cost_pair_kernel"}
FP64_INSTR_PER_CELL = 3.0          # 2 DADD + 1 DSETP; an FP64 warp instruction occupies its pipe for 2 cycles


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": SM_MAX_MHZ_FALLBACK}, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def rank_workload(name: str, rank: int):
    """The workload of one rank.  Ranks beyond 0 draw their random failure sets from their
    own seeds, so that N GPUs search N different batches of the same shape (weak scaling;
    no data-path collective: the scenarios are independent)."""
    from paper_2508_21613_b200 import workloads as W
    w = W.ALL_WORKLOADS[name]()
    if rank > 0:
        rng = W.SplitMix64(0xBEEF + 7919 * rank)
        n = w.profile.n_devices
        w.scenarios = [rng.sample_distinct(n, max(1, len(s))) for s in w.scenarios]
    return w


def aggregate(per_rank):
    """Whole-job numbers from per-rank (plans, seconds) pairs: units summed, time = max."""
    plans = sum(p for p, _ in per_rank)
    seconds = max(s for _, s in per_rank)
    return plans, seconds


def gather_rows(values, world: int, device: str):
    """Every rank's list of numbers on every rank (one all_gather; a list of one row when
    there is a single rank).  The only collective of the benchmark: the search itself
    exchanges nothing between GPUs."""
    if world <= 1:
        return [list(values)]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    gathered = [torch.zeros_like(t) for _ in range(world)]
    dist.all_gather(gathered, t)
    return [g.cpu().tolist() for g in gathered]


ORACLE_SAMPLE = 65536   # candidates the oracle evaluates per sampled scenario


def oracle_sample(orc, w, k: int, n_cand_sample: int = ORACLE_SAMPLE):
    """A bounded sample of the workload for the CPU oracle, as it stands, single thread:
    scenario k's rerouting and redundant-computation plans plus `n_cand_sample` of its
    dynamic-parallelism candidates drawn uniformly (seeded) from its whole candidate space.
    A full oracle search of one sweep scenario takes 10-30 s, too long for a bench step; the
    sample keeps the workload's mix of pipeline shapes.  -> (plans evaluated, seconds)."""
    import numpy as np
    from paper_2508_21613_b200 import workloads as W
    failed = w.scenarios[k % len(w.scenarios)]
    t0 = time.perf_counter()
    n = orc.count(failed)[0]
    plans = 0
    if n > 0:
        if n <= n_cand_sample:
            orc.evaluate(failed)
            plans += n
        else:
            rng = W.SplitMix64(0x0A11CE + k)
            idx = np.sort(np.asarray([rng.below(n) for _ in range(n_cand_sample)], dtype=np.uint64))
            orc.evaluate(failed, idx=idx)
            plans += n_cand_sample
    orc.search_policy(failed, 0)
    orc.search_policy(failed, 1)
    return plans + 2, time.perf_counter() - t0


def oracle_describe(w, n_scen: int) -> str:
    return (f"{n_scen} failure scenario(s) of '{w.name}': the rerouting and the redundant-computation plan and a seeded "
            f"uniform sample of {ORACLE_SAMPLE} dynamic-parallelism pipeline-plans each, single thread")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2508_21613_b200 import workloads as W
    from oracle.oracle import Oracle
    w = W.ALL_WORKLOADS[args.workload]()
    orc = Oracle(w.profile, w.options.with_cost_mode(args.cost_mode))
    per_step = max(1, args.ref_scenarios)
    for k in range(args.warmup):
        oracle_sample(orc, w, len(w.scenarios) - 1 - k)
    plans, seconds = 0, 0.0
    for k in range(args.steps):
        for j in range(per_step):
            p, s = oracle_sample(orc, w, k * per_step + j)
            plans += p
            seconds += s
    value = plans / seconds
    sample = oracle_describe(w, per_step) + " per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * seconds / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "i64" if args.cost_mode else "f64",
            "data": "synthetic",
            "config": {"workload": w.name, "scenarios_per_step": per_step,
                       "cost_mode": "int64ns" if args.cost_mode else "fp64"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def measure(binding, torch, w, mode, steps, warmup, local_rank, barrier, flush, latency_scenarios, sample_clocks=True,
            native_i64=False, cold_latency=True):
    """One workload on this rank: device-resident arm, end-to-end arm, per-failure latency."""
    import numpy as np
    opts = w.options.with_cost_mode(mode)
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    if native_i64:
        binding.cm_set_int64_arithmetic(ctx, True)
    packed = binding.PackedScenarios(w.scenarios)
    out = {}
    try:
        # ---- device-resident arm: descriptors already in HBM when the timed region starts
        batch, n_cand = packed.prepare(ctx, opts)
        for _ in range(warmup):
            packed.search_prepared(ctx, batch)
        sampler = ClockSampler(local_rank) if sample_clocks else None
        barrier()
        if sampler:
            sampler.start()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        stats_sum = {}
        for k in range(steps):
            flush.fill_(float(k))                       # evict L2 between timed iterations (untimed)
            ev[k][0].record()
            packed.search_prepared(ctx, batch)          # kernels + plans back on the host
            ev[k][1].record()
            for key, v in binding.cm_last_stats(ctx).items():
                stats_sum[key] = stats_sum.get(key, 0) + v
        barrier()
        out["clocks"] = sampler.stop() if sampler else None
        out["dev_seconds"] = sum(a.elapsed_time(b) for a, b in ev) * 1e-3
        out["plans_per_step"] = n_cand + 2 * len(w.scenarios)   # + one rerouting and one redundant plan each
        out["stats"] = stats_sum
        # the arithmetic the recurrence ran in: the integer mode runs in fp64 whenever that is exact
        out["arith"] = 0 if (mode == 0 or binding.cm_int64_runs_in_fp64(ctx)) else 1
        binding.cm_batch_free(batch)

        # ---- end-to-end arm: host failure sets in, host plans out, every step
        for _ in range(warmup):
            packed.search(ctx, opts)
        barrier()
        e2e_seconds = 0.0
        for k in range(steps):
            flush.fill_(float(k))
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            packed.search(ctx, opts)                    # cm_search_batch: build, H2D, kernels, D2H, sync
            e2e_seconds += time.perf_counter() - t0
            st = binding.cm_last_stats(ctx)
            out["h2d"], out["d2h"] = st["h2d_bytes"] + packed.ids.nbytes + packed.offsets.nbytes, st["d2h_bytes"]
        barrier()
        out["e2e_seconds"] = e2e_seconds

        # ---- search latency per failure: scenarios searched one at a time
        n_lat = max(1, min(latency_scenarios, len(w.scenarios)))
        lat_pack = binding.PackedScenarios(w.scenarios[:: max(1, len(w.scenarios) // n_lat)][:n_lat])
        for _ in range(3):   # two warm passes: resident batches are built, then their graphs captured
            lat_pack.search(ctx, opts, latency=True)
        lat = np.sort(lat_pack.latency[:lat_pack.B].astype(np.float64))
        out["latency_us"] = {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)),
                             "max": float(lat[-1]), "scenarios": int(lat_pack.B),
                             "what": "one failure set, all policies, descriptor build to plan on host; third pass over "
                                     "the scenarios: the batch of that survivor count is resident and its launch "
                                     "sequence replays as a CUDA graph"}
        # the same with sharing on: a failure set's duplicate pipelines (equal stages, micro-batches,
        # peers and link tiers) are searched once where that saves enough to pay for launching the
        # sequence directly instead of replaying the resident graph
        binding.cm_set_sharing(ctx, True)
        for _ in range(2):
            lat_pack.search(ctx, opts, latency=True)
        binding.cm_set_sharing(ctx, False)
        lat = np.sort(lat_pack.latency[:lat_pack.B].astype(np.float64))
        out["latency_us"]["shared_segments"] = {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)),
                                                "max": float(lat[-1])}
    finally:
        binding.cm_destroy(ctx)
    if cold_latency:
        out["latency_us"]["cold"] = measure_cold_latency(binding, w, opts, local_rank, native_i64)
        cold = measure_cold_latency(binding, w, opts, local_rank, native_i64, share=True)
        out["latency_us"]["shared_segments"]["cold"] = {k: cold[k] for k in ("p50", "p99", "max", "scenarios")}
    return out


def measure_cold_latency(binding, w, opts, local_rank, native_i64=False, max_sizes=16, share=False):
    """A failure is a first occurrence: the latency of the FIRST search of a survivor count on a
    context that has searched nothing yet (profile loaded; no resident batch, no captured graph,
    min-max partitions not computed).  One fresh context and one scenario per failure-set size of
    the workload; the process itself is warm (kernels were loaded by the legs before)."""
    import numpy as np
    by_size = {}
    for sc in w.scenarios:
        by_size.setdefault(len(sc), sc)
    lat = []
    for size in sorted(by_size)[:max_sizes]:
        ctx = binding.cm_create(local_rank)
        try:
            binding.cm_load_profile(ctx, w.profile)
            if native_i64:
                binding.cm_set_int64_arithmetic(ctx, True)
            binding.cm_set_sharing(ctx, share)
            pack = binding.PackedScenarios([by_size[size]])
            pack.search(ctx, opts, latency=True)
            lat.append(float(pack.latency[0]))
        finally:
            binding.cm_destroy(ctx)
    lat = np.sort(np.asarray(lat))
    return {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)), "max": float(lat[-1]),
            "scenarios": int(len(lat)),
            "what": "first search of a failure-set size on a fresh context (one per size), descriptor build to plan on host"}


def measure_objective(binding, torch, w, mode, steps, warmup, local_rank, flush):
    """The full-objective search (search + shortlist + weight-transfer matchings + ranking by
    steps before the next fault) through cm_search_objective, host buffers in and out."""
    import numpy as np
    from paper_2508_21613_b200 import workloads as W
    opts = w.options.with_cost_mode(mode)
    obj = W.ObjectiveOptions()
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    packed = binding.PackedScenarios(w.scenarios)
    try:
        for _ in range(warmup):
            res = packed.search_objective(ctx, opts, obj, shortlist=True)
        wall, phases = 0.0, {}
        search_ns = 0
        for k in range(steps):
            flush.fill_(float(k))
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            res = packed.search_objective(ctx, opts, obj, shortlist=True)
            wall += time.perf_counter() - t0
            for key, v in binding.cm_objective_stats(ctx).items():
                phases[key] = phases.get(key, 0) + v
            search_ns += binding.cm_last_stats(ctx)["device_ns"]
        best, trans, _, sb, _ = res
        packed.search(ctx, opts)
        plain = packed.best
        policies = [0, 0, 0]
        changed = 0
        for b in range(packed.B):
            policies[trans[b].policy] += 1
            changed += int(plain[b].policy != best[b].policy or plain[b].strategy != best[b].strategy
                           or plain[b].split_rank != best[b].split_rank)
        matchings = int((sb >= 0).sum())
        out = {
            "topk": obj.topk, "t_gap_s": obj.t_gap_ns * 1e-9, "t_restart_s": obj.t_restart_ns * 1e-9,
            "bw_xfer_GBps": obj.bw_xfer_Bpns, "scenarios": packed.B,
            "e2e_ms_per_call": 1e3 * wall / steps,
            "search_device_ms": 1e-6 * search_ns / steps,
            "objective_pass_device_ms": 1e-6 * phases["device_ns"] / steps,
            "phase_ms": {k[:-3]: 1e-6 * phases[k] / steps for k in ("shortlist_ns", "complete_ns", "matching_ns", "objective_ns")},
            "matchings_per_call": matchings,
            "matchings_per_s": matchings / (1e-9 * phases["matching_ns"] / steps) if phases["matching_ns"] else None,
            "devices_per_matching": int(trans[0].n_survivors),
            "chosen_policy_counts": {"reroute": policies[0], "redundant": policies[1], "dynpar": policies[2]},
            "choices_changed_by_transition_time": changed,
            "gpu_launches": int(phases["launches"] / steps),
        }
        # the same with the asymmetric-synchronisation rounds in the step time
        obj_r = W.ObjectiveOptions(sync_rounds=1)
        packed.search_objective(ctx, opts, obj_r, shortlist=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        best_r, trans_r, _, _, sr = packed.search_objective(ctx, opts, obj_r, shortlist=True)
        wall_r = time.perf_counter() - t0
        ph = binding.cm_objective_stats(ctx)
        dyn = [b for b in range(packed.B) if trans_r[b].policy == 2]
        out["sync_rounds"] = {
            "e2e_ms_per_call": 1e3 * wall_r,
            "matching_plus_rounds_kernel_ms": 1e-6 * ph["matching_ns"],
            "plans_coloured": int((sr > 0).sum()),
            "rounds_mean": float(sr[sr > 0].mean()) if (sr > 0).any() else None,
            "rounds_max": int(sr.max()),
            "layers": int(w.profile.L),
            "domains_mean_of_chosen": float(np.mean([trans_r[b].domains for b in dyn])) if dyn else None,
            "chosen_policy_counts": {"reroute": sum(trans_r[b].policy == 0 for b in range(packed.B)),
                                     "redundant": sum(trans_r[b].policy == 1 for b in range(packed.B)),
                                     "dynpar": len(dyn)},
            "choices_changed_vs_without_rounds": sum(
                int(best[b].policy != best_r[b].policy or best[b].strategy != best_r[b].strategy
                    or best[b].split_rank != best_r[b].split_rank) for b in range(packed.B)),
        }
        return out
    finally:
        binding.cm_destroy(ctx)


def measure_shared(binding, torch, w, mode, local_rank, flush, steps=5):
    """The same batch with sharing on: failure sets that leave the same survivor count and node
    boundaries have identical dynamic-parallelism searches and are searched once, and every
    distinct segment (stages, micro-batches, peers, link tiers) of the batch is searched once for
    all the scenarios and strategies it occurs in.  Not the headline: `value` above evaluates
    every scenario's plans."""
    opts = w.options.with_cost_mode(mode)
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    packed = binding.PackedScenarios(w.scenarios)
    try:
        binding.cm_set_sharing(ctx, True)
        for _ in range(3):
            packed.search(ctx, opts)
        wall = 0.0
        for k in range(steps):
            flush.fill_(float(k))
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            packed.search(ctx, opts)
            wall += time.perf_counter() - t0
        st = binding.cm_last_stats(ctx)
        return {"scenarios": packed.B, "e2e_ms_per_step": 1e3 * wall / steps, "device_ms_per_step": 1e-6 * st["device_ns"],
                "plans_of_searched_scenarios_per_step": st["plans"], "plans_simulated_per_step": st["plans_simulated"],
                "scenarios_per_s": packed.B / (wall / steps),
                "host_ms_per_step": {"descriptors": 1e-6 * st["host_build_ns"], "upload_and_segment_keys": 1e-6 * st["host_upload_ns"]}}
    finally:
        binding.cm_destroy(ctx)


def measure_trace(binding, w, mode, local_rank, seed=7, hours=9.0, rate=0.10):
    """The paper's simulated experiment in the library's model: devices fail at 10 % per hour for
    9 hours; reroute-first, always-reconfigure and the full objective are replayed over the same
    seeded trace (states the search windows cannot plan produce nothing)."""
    from paper_2508_21613_b200 import trace as T, workloads as W
    opts = w.options.with_cost_mode(mode)
    n = w.profile.n_dp * w.profile.n_pp
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    try:
        events = T.make_trace(n, rate, hours, seed)
        objective = W.ObjectiveOptions(t_gap_ns=3600e9 / (rate * n))
        base, _, _ = binding.cm_search_batch(ctx, [[]], opts, per_policy=True)
        fault_free = float(base[0].cost_ns if mode else base[0].cost)     # nothing failed: rerouting = the base configuration
        t0 = time.perf_counter()
        r = T.replay(T.gpu_planner(binding, ctx, opts, objective), events, hours, fault_free)
        dt = time.perf_counter() - t0
        return {"devices": n, "failure_rate_per_device_hour": rate, "hours": hours, "seed": seed, "failures": r["events"],
                "relative_work": {k: v["relative_work"] for k, v in r["rules"].items()},
                "full_objective_vs_always_dynpar": r["full_objective_vs_always_dynpar"],
                "full_objective_vs_reroute_first": r["full_objective_vs_reroute_first"],
                "choices_of_full_objective": [t[2] for t in r["rules"]["full-objective"]["timeline"]],
                "planning_ms_all_states": 1e3 * dt}
    finally:
        binding.cm_destroy(ctx)


def measure_stretch(binding, torch, mode, local_rank, picks=(63,), reps=2):
    """Stretch case: 70b-like with no cap on the layer compositions per pipeline (up to
    C(32,16) = 6e8 of them): the whole search of one failure set of 8 devices, 4.7e9 pipeline-plans
    (sets that leave more survivors have up to 1.2e10 plans, most of them memory-feasible, and take
    tens of seconds: too long for a default run)."""
    import copy
    from paper_2508_21613_b200 import workloads as W
    w = W.llama70b_like()
    opts = copy.copy(w.options.with_cost_mode(mode))
    opts.kappa_cap = 1 << 62
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    out = {"workload": "70b-like, kappa_cap unbounded", "failure_sets": []}
    try:
        for k in picks:
            pack = binding.PackedScenarios([w.scenarios[k]])
            pack.search(ctx, opts)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(reps):
                pack.search(ctx, opts)
            dt = (time.perf_counter() - t0) / reps
            st = binding.cm_last_stats(ctx)
            out["failure_sets"].append({"scenario": k, "failed_devices": len(w.scenarios[k]), "pipeline_plans": st["plans"],
                                        "plans_simulated": st["plans_simulated"], "e2e_ms": 1e3 * dt,
                                        "plans_per_s": st["plans"] / dt})
    finally:
        binding.cm_destroy(ctx)
    return out


def measure_cache(binding, w, mode, local_rank, sizes=(2, 3, 4)):
    """Plan cache: every failure set of at most k devices searched ahead of time; lookups."""
    from paper_2508_21613_b200 import workloads as W
    opts = w.options.with_cost_mode(mode)
    ctx = binding.cm_create(local_rank)
    binding.cm_load_profile(ctx, w.profile)
    out = {}
    try:
        binding.cm_cache_free(binding.cm_cache_build(ctx, 1, opts)[0])           # warm-up
        rng = W.SplitMix64(99)
        n_dev = w.profile.n_dp * w.profile.n_pp
        for k in sizes:
            t0 = time.perf_counter()
            cache, n = binding.cm_cache_build(ctx, k, opts)
            dt = time.perf_counter() - t0
            sets = [rng.sample_distinct(n_dev, 1 + rng.below(k)) for _ in range(2000)]
            t0 = time.perf_counter()
            for f in sets:
                binding.cm_cache_lookup(cache, f)
            lk = (time.perf_counter() - t0) / len(sets)
            binding.cm_cache_free(cache)
            out[f"up_to_{k}_failures"] = {"failure_sets": n, "build_ms": 1e3 * dt, "sets_per_s": n / dt,
                                          "lookup_us_through_ctypes": 1e6 * lk}
    finally:
        binding.cm_destroy(ctx)
    return out


def kernel_class(w) -> str:
    """Search-pass kernel that carries a workload: pipelines of the search window deeper than
    16 stages run the deep-pipeline kernel, the others the register-resident one."""
    if not (w.options.pp_hi > 16 and w.profile.n_pp > 16):
        # shallow pipelines pair up under the same conditions once a group of them holds enough plans
        big = len(w.scenarios) >= 256 and getattr(w.options, "schedule", 0) == 0
        return "regs_pair" if big and w.profile.n_micro * w.profile.n_dp // max(1, w.options.dp_hi) >= w.options.pp_hi else "regs"
    # 1F1B, remainder split of the micro-batches, stage counts of 17-48 with at least as many
    # micro-batches: the pipelines come as (m, m+1) pairs and the pair kernel carries the batch
    paired = (getattr(w.options, "schedule", 0) == 0 and w.options.pp_hi <= 48 and
              w.profile.n_micro * w.profile.n_dp // max(1, w.options.dp_hi) >= w.options.pp_hi)
    return "pair" if paired else "wide"


def roofline_of(stats_sum, dev_seconds, arith, kclass, clocks, sm_max, peak_kind):
    prof = KERNEL_PROFILES.get((kclass, arith)) or KERNEL_PROFILES[(kclass, 0)]
    f_mhz = float((clocks or {}).get("sm_mhz") or sm_max)
    lanes_per_s = N_SM * 4 * 32 * f_mhz * 1e6
    peak_cells = lanes_per_s / prof["i_cell"]
    cost_s = stats_sum["cost_kernel_ns"] * 1e-9
    achieved = stats_sum["cells"] / cost_s if cost_s > 0 else 0.0
    launches = max(1, stats_sum["cost_kernel_launches"])
    return {
        "bound": "alu", "kernel": KERNEL_NAMES[kclass] + " (search pass)",
        "achieved": achieved / 1e9, "peak": peak_cells / 1e9, "unit": "Gcell/s",
        "frac": achieved / peak_cells if peak_cells else None,
        "peak_kind": f"148 SM x 4 schedulers x 32 lanes x {f_mhz:.0f} MHz (median SM clock sampled during the timed region; "
                     f"{peak_kind} max {sm_max:.0f}) / I_cell",
        "i_cell": prof["i_cell"],
        "i_cell_source": f"executed thread-instructions per recurrence cell, ncu capture in {prof['profile']}",
        "issue_active_profiled": prof["issue_active"],
        # against the FP64 pipe alone: 3 FP64 instructions per cell, each holding the pipe of a
        # scheduler (16 lanes) for 2 cycles
        "frac_of_fp64_pipe": (achieved / (lanes_per_s / (2.0 * FP64_INSTR_PER_CELL))) if arith == 0 else None,
        # an FP64 warp instruction holds the dispatch slot for two cycles, so issue-active cannot pass
        # I_cell / (I_cell + 3): the bound of this instruction stream in cells is lanes / (I_cell + 3)
        "frac_of_dispatch_bound": (achieved / (lanes_per_s / (prof["i_cell"] + FP64_INSTR_PER_CELL))) if arith == 0 else None,
        "fp64_pipe_active_profiled": prof["fp64_pipe_active"],
        "cells_per_launch": stats_sum["cells"] / launches,
        "ms_per_launch": 1e3 * cost_s / launches,
        "share_of_step": cost_s / dev_seconds if dev_seconds else None,
        # the search pass reads only the small descriptor tables: ~0 algorithmic bytes.  Not
        # measured in this run: dram__bytes_read + write of the ncu capture named above, per
        # recurrence cell of that launch, times this run's cells per launch.
        "traffic": prof["dram_bytes_per_cell"] * stats_sum["cells"] / launches,
        "traffic_source": f"scaled by cells from the ncu capture in {prof['profile']} (not measured in this run)",
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sweep")
    ap.add_argument("--cost-mode", type=int, default=0, choices=[0, 1])
    ap.add_argument("--ref-scenarios", type=int, default=1, help="sampled oracle scenarios per step (--impl reference)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--latency-scenarios", type=int, default=4096, help="scenarios searched one by one for latency")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads / cost mode summary")
    ap.add_argument("--scenarios", type=int, default=0, help="use only the first N scenarios (profiling runs)")
    ap.add_argument("--native-int64", action="store_true",
                    help="with --cost-mode 1: force the 64-bit integer kernels (default: exact double arithmetic)")
    ap.add_argument("--objective", action="store_true",
                    help="also time the full-objective search on the selected workload (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2508_21613_b200 import binding, build
    build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the plan search has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = rank_workload(args.workload, rank)
    if args.scenarios > 0:
        w.scenarios = w.scenarios[:args.scenarios]
    flush = torch.empty(256 * 1024 * 1024 // 4, dtype=torch.float32, device="cuda")  # > 126 MB L2
    m = measure(binding, torch, w, args.cost_mode, args.steps, args.warmup, local_rank, barrier, flush,
                args.latency_scenarios, native_i64=args.native_int64)
    rows = gather_rows([float(m["plans_per_step"] * args.steps), m["dev_seconds"], m["e2e_seconds"]], world, "cuda")
    total_plans, max_dev = aggregate([(r[0], r[1]) for r in rows])
    _, max_e2e = aggregate([(r[0], r[2]) for r in rows])

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        sm_max = float(peaks.get("sm_max_mhz") or SM_MAX_MHZ_FALLBACK)
        line = {
            "metric": METRIC, "value": total_plans / max_dev, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * max_dev / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": ("f64 (integer-valued, exact)" if m["arith"] == 0 else "i64") if args.cost_mode else "f64",
            "data": "synthetic",
            "config": {"workload": w.name, "scenarios": len(w.scenarios), "plans_per_step": m["plans_per_step"],
                       # plans_per_step counts every pipeline-plan of the search space, i.e. every
                       # (strategy, pipeline, micro-batch count, layer composition), as the oracle
                       # enumerates them.  Of these: plans_reused belong to pipelines that another
                       # strategy of the same survivor count has as well and are not searched again;
                       # plans_memory_rejected fail the memory estimator; plans_simulated ran the recurrence.
                       "plans_reused_per_step": (m["stats"]["plans"] - m["stats"]["plans_own"]) // args.steps,
                       "plans_memory_rejected": (m["stats"]["plans_own"] - m["stats"]["plans_simulated"]) // args.steps,
                       "plans_simulated_per_step": m["stats"]["plans_simulated"] // args.steps + 2 * len(w.scenarios),
                       "policies": 3, "cost_mode": "int64ns" if args.cost_mode else "fp64",
                       "l2": "flushed between timed iterations (256 MB write)",
                       "parallelism": "replicas, scenarios independent" if world > 1 else "1 gpu"},
            "e2e": {"value": total_plans / max_e2e, "unit": UNIT, "ms_per_step": 1e3 * max_e2e / args.steps,
                    "h2d_bytes_per_step": int(m["h2d"]), "d2h_bytes_per_step": int(m["d2h"]),
                    "timing": "wall clock around cm_search_batch (host descriptor build inside)"},
            # the same rate counted on the pipeline-plans that are searched in their own right only
            "value_without_reused_plans": (m["stats"]["plans_own"] + 2 * len(w.scenarios) * args.steps) * world / max_dev,
            "latency_us": m["latency_us"],
            "gpu_launches": int(m["stats"]["launches"]),
            "clocks": m["clocks"],
            "roofline": roofline_of(m["stats"], m["dev_seconds"], m["arith"], kernel_class(w), m["clocks"], sm_max, peak_kind),
        }
        if not args.no_cpu_baseline:
            from oracle.oracle import Oracle
            orc = Oracle(w.profile, w.options.with_cost_mode(args.cost_mode))
            p_sum, s_sum, n = 0, 0.0, 0
            while s_sum < args.cpu_budget and n < len(w.scenarios):
                p, s = oracle_sample(orc, w, n)
                p_sum, s_sum, n = p_sum + p, s_sum + s, n + 1
            line["cpu_baseline"] = {"value": p_sum / s_sum, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": oracle_describe(w, n) + f", {s_sum:.1f} s"}
        if not args.no_extra and world == 1 and args.scenarios == 0:
            # the other configurations (and the other cost mode), two timed steps each: context
            # for the headline line above, same measurement code
            from paper_2508_21613_b200 import workloads as W
            extra = {}
            todo = [(args.workload, 1 - args.cost_mode)]
            todo += [(name, args.cost_mode) for name in ("tiny", "paper-scale", "70b-like", "175b-like", "sweep") if name != args.workload]
            n_extra = 5
            for name, mode in todo:
                ew = W.ALL_WORKLOADS[name]()
                em = measure(binding, torch, ew, mode, n_extra, 3, local_rank, barrier, flush, args.latency_scenarios)
                r = roofline_of(em["stats"], em["dev_seconds"], em["arith"], kernel_class(ew), em["clocks"], sm_max, peak_kind)
                extra[f"{name}/{'int64ns' if mode else 'fp64'}"] = {
                    "scenarios": len(ew.scenarios), "steps": n_extra, "plans_per_step": em["plans_per_step"],
                    "plans_reused_per_step": (em["stats"]["plans"] - em["stats"]["plans_own"]) // n_extra,
                    "plans_memory_rejected": (em["stats"]["plans_own"] - em["stats"]["plans_simulated"]) // n_extra,
                    "plans_per_s": em["plans_per_step"] * n_extra / em["dev_seconds"],
                    "ms_per_step": 1e3 * em["dev_seconds"] / n_extra, "e2e_ms_per_step": 1e3 * em["e2e_seconds"] / n_extra,
                    "latency_us_p50": em["latency_us"]["p50"], "latency_us_p99": em["latency_us"]["p99"],
                    "latency_us_cold_p50": em["latency_us"]["cold"]["p50"], "latency_us_cold_p99": em["latency_us"]["cold"]["p99"],
                    "latency_us_shared_segments_p50": em["latency_us"]["shared_segments"]["p50"],
                    "latency_us_shared_segments_p99": em["latency_us"]["shared_segments"]["p99"],
                    "latency_scenarios": em["latency_us"]["scenarios"],
                    "search_pass_kernel": r["kernel"], "search_pass_gcell_s": r["achieved"],
                    "search_pass_frac": r["frac"], "search_pass_frac_of_fp64_pipe": r["frac_of_fp64_pipe"],
                    "clocks_sm_mhz": (em["clocks"] or {}).get("sm_mhz")}
            line["workloads"] = extra
            # widening beyond the plan search: transition time in the objective
            line["full_objective"] = {
                name: measure_objective(binding, torch, W.ALL_WORKLOADS[name](), args.cost_mode, 3, 3, local_rank, flush)
                for name in dict.fromkeys((args.workload, "paper-scale", "175b-like"))}
        if not args.no_extra and world == 1 and args.scenarios == 0:
            line["shared_search"] = measure_shared(binding, torch, w, args.cost_mode, local_rank, flush)
        if not args.no_extra and world == 1 and args.scenarios == 0:
            # plan cache and failure-trace replay at the scale of the paper's cluster (32 devices)
            from paper_2508_21613_b200 import workloads as W
            small = w if w.profile.n_dp * w.profile.n_pp <= 64 else W.paper_scale(0, 0)
            line["plan_cache"] = dict(measure_cache(binding, small, args.cost_mode, local_rank), workload=small.name)
            line["failure_trace"] = dict(measure_trace(binding, small, args.cost_mode, local_rank), workload=small.name)
            line["stretch_uncapped"] = measure_stretch(binding, torch, args.cost_mode, local_rank)
        if args.objective and "full_objective" not in line:
            line["full_objective"] = {w.name: measure_objective(binding, torch, w, args.cost_mode, args.steps,
                                                                args.warmup, local_rank, flush)}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
