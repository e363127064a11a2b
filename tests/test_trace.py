"""Failure-trace replay (Section "Simulation Results"): the bookkeeping on hand numbers, the
seeded trace generator, and -- on the GPU -- the same replay planned by the CUDA library and by
the CPU oracle."""
import pytest

from paper_2508_21613_b200 import trace as T
from paper_2508_21613_b200 import workloads as W


def test_trace_generator_is_seeded_and_never_repeats_a_device():
    a = T.make_trace(32, 0.10, 9, seed=7)
    b = T.make_trace(32, 0.10, 9, seed=7)
    assert [(e.minute, e.device) for e in a] == [(e.minute, e.device) for e in b]
    assert len({e.device for e in a}) == len(a) and all(0 <= e.device < 32 for e in a)
    assert [e.minute for e in a] == sorted(e.minute for e in a)
    assert T.make_trace(32, 0.10, 9, seed=8) != a
    # 32 devices at 10 %/h for 9 h: 32 (1 - 0.9^9) = 19.6 failures expected
    counts = [len(T.make_trace(32, 0.10, 9, seed=s)) for s in range(40)]
    assert 16 < sum(counts) / len(counts) < 23
    assert T.make_trace(8, 0.0, 3, seed=1) == []


def test_replay_bookkeeping_on_hand_numbers():
    # 2 hours, one failure after 60 minutes.  Fault-free step 1 s.  Rerouting: 1.25 s per step,
    # no transition.  Reconfiguration: 1.0 s per step after a 10-minute transition.
    trace = [T.Event(60, 3)]
    hour = 3600e9

    def planner(sets):
        assert sets == [[3]]
        return [T.StatePlan((1.25e9, None, 1.0e9), 600e9, (2, 1.0e9, 600e9))]
    r = T.replay(planner, trace, 2, 1.0e9)
    rules = r["rules"]
    assert rules["reroute-first"]["relative_work"] == pytest.approx((hour + hour / 1.25) / (2 * hour))      # 0.9
    assert rules["always-dynpar"]["relative_work"] == pytest.approx((hour + (hour - 600e9)) / (2 * hour))   # 0.9167
    assert rules["full-objective"]["relative_work"] == rules["always-dynpar"]["relative_work"]
    assert r["full_objective_vs_reroute_first"] == pytest.approx(0.916666666 / 0.9, rel=1e-6)
    assert rules["reroute-first"]["timeline"] == [(60, 1, "reroute", 0.8)]

    # rerouting stops being feasible at the second failure: reroute-first reconfigures then and
    # pays a transition at every failure from there on; a state nobody can plan produces nothing
    trace = [T.Event(30, 1), T.Event(60, 2), T.Event(90, 5)]

    def planner2(sets):
        return [T.StatePlan((2.0e9, None, 1.0e9), 300e9, (0, 2.0e9, 0.0)),
                T.StatePlan((None, None, 1.0e9), 300e9, (2, 1.0e9, 300e9)),
                T.StatePlan((None, None, None), 0.0, None)]
    r = T.replay(planner2, trace, 2, 1.0e9)
    half = 1800e9
    assert r["rules"]["reroute-first"]["relative_work"] == pytest.approx((half + half / 2 + (half - 300e9)) / (4 * half))
    assert r["rules"]["always-dynpar"]["relative_work"] == pytest.approx((half + 2 * (half - 300e9)) / (4 * half))
    assert r["rules"]["full-objective"]["relative_work"] == pytest.approx((half + half / 2 + (half - 300e9)) / (4 * half))
    assert [t[2] for t in r["rules"]["full-objective"]["timeline"]] == ["reroute", "dynpar", "none"]
    # no failure at all: every rule does the fault-free work
    r = T.replay(lambda sets: [], [], 1, 1.0e9)
    assert all(v["relative_work"] == 1.0 for v in r["rules"].values())


def _oracle_planner(o, opts, objective):
    def plan(sets):
        out = []
        for failed in sets:
            best, tr = o.search_objective(failed, objective, opts)
            _, per = o.search(failed, opts)
            mode = opts.cost_mode
            cost = lambda p: float(p.cost_ns if mode else p.cost)
            step = tuple(cost(p) if p.feasible else None for p in per)
            dyn = 0.0
            if tr.shortlist_bytes:
                b = tr.shortlist_bytes[0]
                dyn = float(objective.t_restart_ns) + ((b // objective.bw_xfer_Bpns) if mode else float(b) / float(objective.bw_xfer_Bpns))
            chosen = None if best is None else (tr.policy, cost(best), float(tr.t_trans_ns if mode else tr.t_trans))
            out.append(T.StatePlan(step, dyn, chosen))
        return out
    return plan


@pytest.mark.gpu
@pytest.mark.parametrize("mode", [0, 1])
def test_replay_planned_by_the_library_equals_replay_planned_by_the_oracle(oracle_factory, mode):
    import torch
    from paper_2508_21613_b200 import binding, build
    build.build()
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; there is no CPU path")
    w = W.paper_scale(0, 0)
    opts = w.options.with_cost_mode(mode)
    o = oracle_factory(w.profile, opts)
    trace = T.make_trace(32, 0.10, 9, seed=7)[:12]           # the first twelve failures: 31 .. 20 survivors
    hours = (trace[-1].minute + 30) / 60.0
    n_alive = 32
    objective = W.ObjectiveOptions(t_gap_ns=3600e9 / (0.10 * n_alive))
    _, base_ns, base_i, _ = o.pipe(list(w.profile.base_cuts), w.profile.n_micro, list(range(w.profile.n_pp)),
                                   w.profile.n_dp, mode)
    fault_free = float(base_i if mode else base_ns)
    want = T.replay(_oracle_planner(o, opts, objective), trace, hours, fault_free)
    ctx = binding.cm_create(0)
    try:
        binding.cm_load_profile(ctx, w.profile)
        got = T.replay(T.gpu_planner(binding, ctx, opts, objective), trace, hours, fault_free)
    finally:
        binding.cm_destroy(ctx)
    assert got["events"] == want["events"] == 12
    for rule in T.RULES:
        assert got["rules"][rule]["timeline"] == want["rules"][rule]["timeline"], rule
        assert got["rules"][rule]["relative_work"] == want["rules"][rule]["relative_work"], rule
    assert got["full_objective_vs_always_dynpar"] == want["full_objective_vs_always_dynpar"]
    assert got["rules"]["full-objective"]["relative_work"] >= got["rules"]["always-dynpar"]["relative_work"] * 0.999
