"""Failure-trace replay on top of the plan search (Section "Simulation Results": failures are
injected at a fixed per-device rate and the systems are compared by average throughput).

Three selection rules are replayed over the same seeded trace; they are the paper's policy
abstractions, not re-implementations of other systems:

  reroute-first   data rerouting whenever it is feasible, otherwise a reconfiguration
  always-dynpar   a reconfiguration (dynamic parallelism, least step time) at every failure
  full-objective  the plan of greatest ``(t_gap - t_trans) / t_step`` among all three policies

What the replay models, and what it does not: failures accumulate, and every state is planned
for its cumulative failure set from the ORIGINAL grid -- its step time depends on the survivors
only, but the transfer of a reconfiguration is priced against the original placement, not
against the previous reconfigured one (the library plans from a DP x PP grid).  Throughput is
relative to the fault-free step time; a reconfiguration costs its transition time in lost work;
a state without a feasible plan produces nothing.

This module holds no model arithmetic beyond that bookkeeping: plans, step times and transition
times come from a ``planner`` callable (the CUDA library in use, a plain CPU implementation in the tests).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Sequence, Tuple

from .workloads import SplitMix64

RULES = ("reroute-first", "always-dynpar", "full-objective")


@dataclass
class Event:
    minute: int
    device: int


@dataclass
class StatePlan:
    """What a planner returns for one cumulative failure set: step time per policy (None if
    infeasible), transition time of the best dynamic-parallelism plan and the full-objective
    choice as (policy, step time, transition time) or None."""
    step: Tuple[object, object, object]
    dynpar_transition: float
    chosen: object


def make_trace(n_devices: int, rate_per_hour: float, hours: float, seed: int) -> List[Event]:
    """Every minute each live device fails with probability rate/60 (libm-free Bernoulli draws,
    one per live device and minute, devices in ascending order)."""
    rng = SplitMix64(seed)
    alive = list(range(n_devices))
    p = rate_per_hour / 60.0
    out: List[Event] = []
    for minute in range(int(round(hours * 60))):
        for d in list(alive):
            if rng.uniform01() < p:
                alive.remove(d)
                out.append(Event(minute, d))
    return out


def replay(planner: Callable[[Sequence[Sequence[int]]], List[StatePlan]], trace: Sequence[Event], hours: float,
           fault_free_step: float) -> Dict[str, object]:
    """Replay ``trace``; ``planner`` plans all cumulative failure sets in one call.  Returns, per
    rule, the work done relative to a fault-free run of the same length, plus the timeline."""
    sets: List[List[int]] = []
    failed: List[int] = []
    for ev in trace:
        failed = sorted(failed + [ev.device])
        sets.append(list(failed))
    plans = planner(sets) if sets else []
    horizon = hours * 3600e9                                   # ns
    starts = [ev.minute * 60e9 for ev in trace] + [horizon]
    result: Dict[str, object] = {"events": len(trace), "rules": {}}
    for rule in RULES:
        work = starts[0] if trace else horizon                  # fault-free until the first failure
        timeline = []
        mode = "grid"                                           # reroute-first: still on the original grid?
        for k, st in enumerate(plans):
            span = starts[k + 1] - starts[k]
            step, trans, label = None, 0.0, "none"
            if rule == "reroute-first":
                if mode == "grid" and st.step[0] is not None:
                    step, label = st.step[0], "reroute"
                elif st.step[2] is not None:
                    step, label = st.step[2], "dynpar"
                    trans = st.dynpar_transition                # pays again at every later failure
                    mode = "reconfigured"
            elif rule == "always-dynpar":
                if st.step[2] is not None:
                    step, trans, label = st.step[2], st.dynpar_transition, "dynpar"
            else:
                if st.chosen is not None:
                    pol, step, trans = st.chosen
                    label = ("reroute", "redundant", "dynpar")[pol]
            if step is not None:
                work += max(0.0, span - trans) * (fault_free_step / step)
            timeline.append((trace[k].minute, len(sets[k]), label, None if step is None else fault_free_step / step))
        result["rules"][rule] = {"relative_work": work / horizon, "timeline": timeline}
    r = result["rules"]
    result["full_objective_vs_always_dynpar"] = (r["full-objective"]["relative_work"] / r["always-dynpar"]["relative_work"]
                                                 if r["always-dynpar"]["relative_work"] else None)
    result["full_objective_vs_reroute_first"] = (r["full-objective"]["relative_work"] / r["reroute-first"]["relative_work"]
                                                 if r["reroute-first"]["relative_work"] else None)
    return result


def gpu_planner(binding, ctx, opts, objective):
    """Planner backed by the CUDA library: one cm_search_objective over all states (its t_gap is
    the caller's; the shortlist's first plan is the least-step-time reconfiguration)."""
    def plan(sets):
        best, trans, sl, sb, _ = binding.cm_search_objective(ctx, sets, opts, objective, shortlist=True)
        plain, pol, _ = binding.cm_search_batch(ctx, sets, opts, per_policy=True)
        mode = opts.cost_mode
        cost = lambda p: float(p.cost_ns if mode else p.cost)
        out = []
        # the library prices the least-step-time reconfiguration (shortlist rank 0) itself
        t_f64, t_i64 = binding.cm_transition_time(objective, sb[:, 0])
        for b in range(len(sets)):
            per = [pol[3 * b + q] for q in range(3)]
            step = tuple(cost(p) if p.feasible else None for p in per)
            dyn_trans = 0.0
            if sb[b, 0] >= 0:
                dyn_trans = float(t_i64[b] if mode else t_f64[b])
            tr = trans[b]
            chosen = None
            if tr.feasible:
                chosen = (tr.policy, cost(best[b]), float(tr.t_trans_ns if mode else tr.t_trans))
            out.append(StatePlan(step, dyn_trans, chosen))
        return out
    return plan
