"""Pins for the oracle's search (Algorithm 1: keep the plan with the least estimated
time; step time = slowest pipeline): the three-step separable rule against the flat
brute force over the full product, a re-derivation of the selection from per-candidate
costs, and the invariants the search must keep."""
import math

import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W


def _cost(plan, mode):
    return plan.cost_ns if mode else plan.cost


@pytest.mark.parametrize("mode", [0, 1])
def test_separable_search_equals_flat_brute_force_on_tiny(oracle_factory, mode):
    for w, scen in ((W.tiny(), [[0], [5]]), (W.tiny(mem_bound=True), [[2], [7]])):
        o = oracle_factory(w.profile, w.options.with_cost_mode(mode))
        for failed in scen:
            fast = o.search_policy(failed, W.POLICY_DYNPAR)
            flat, n_flat = o.search_policy(failed, W.POLICY_DYNPAR, flat=True)
            assert n_flat > 100000
            assert fast.key() == flat.key()
            assert _cost(fast, mode) == _cost(flat, mode)


@pytest.mark.parametrize("mode", [0, 1])
def test_separable_search_equals_flat_brute_force_on_random_small(oracle_factory, mode):
    for seed in range(6):
        w = W.random_small(seed, L=5 + seed % 3, n_dp=2, n_pp=2 + seed % 2, n_micro=3,
                           tight_memory=bool(seed % 2))
        opts = W.SearchOptions(1, 3, 1, 4, W.LAYERS_FULL if seed % 3 else W.LAYERS_REMAINDER,
                               W.BATCH_FULL if seed % 2 else W.BATCH_REMAINDER, 1 << 62, mode)
        o = oracle_factory(w.profile, opts)
        for failed in w.scenarios[:3]:
            fast = o.search_policy(failed, W.POLICY_DYNPAR)
            flat, _ = o.search_policy(failed, W.POLICY_DYNPAR, flat=True)
            assert fast.key() == flat.key()
            assert _cost(fast, mode) == _cost(flat, mode)


def _select_from_candidate_costs(o, failed, profile, opts):
    """Re-derive the winner from the per-candidate costs alone (python, no oracle search)."""
    cost, cost_ns, feas = o.evaluate(failed)
    vals = cost_ns.astype(object) if opts.cost_mode else cost
    segs = []
    s = 0
    while True:
        d = o.segment(failed, s)
        if d is None:
            break
        segs.append(d)
        s += 1
    n_surv = profile.n_dp * profile.n_pp - len(failed)
    G = profile.n_dp * profile.n_micro
    strategies = o.strategies(n_surv)
    best = None
    for si, stages in enumerate(strategies):
        for beta in range(o.split_count(opts.batch_mode, G, n_surv, stages)):
            ok, micro = o.split_unrank(opts.batch_mode, G, n_surv, stages, beta)
            if not ok:
                continue
            T = 0
            usable = True
            for p, m in enumerate(micro):
                d = next((d for d in segs if d["strategy"] == si and d["pipe"] == p and d["m"] == m), None)
                if d is None:
                    usable = False
                    break
                n = d["K"] + 1 if d["K"] else 1
                sl = slice(d["first"], d["first"] + n)
                f = feas[sl].astype(bool)
                if not f.any():
                    usable = False
                    break
                T = max(T, min(v for v, ff in zip(vals[sl], f) if ff))
            if usable and (best is None or T < best[0]):
                best = (T, si, beta, micro)
    return best, segs, vals, feas


@pytest.mark.parametrize("mode", [0, 1])
def test_search_agrees_with_selection_rederived_from_candidate_costs(oracle_factory, mode):
    w = W.tiny()
    opts = w.options.with_cost_mode(mode)
    o = oracle_factory(w.profile, opts)
    for failed in ([3], [6]):
        plan = o.search_policy(failed, W.POLICY_DYNPAR)
        best, segs, vals, feas = _select_from_candidate_costs(o, failed, w.profile, opts)
        assert best is not None and plan.feasible
        T, si, beta, micro = best
        assert (_cost(plan, mode), plan.strategy, plan.split_rank, list(plan.micro)) == (T, si, beta, micro)
        for p, m in enumerate(micro):
            d = next(d for d in segs if d["strategy"] == si and d["pipe"] == p and d["m"] == m)
            n = d["K"] + 1 if d["K"] else 1
            lowest = next(k for k in range(n) if feas[d["first"] + k] and vals[d["first"] + k] <= T)
            assert plan.kappa[p] == lowest


def test_infeasible_candidates_are_never_selected_and_carry_infinite_cost(oracle_factory):
    w = W.tiny(mem_bound=True)
    o = oracle_factory(w.profile, w.options)
    failed = [1]
    cost, cost_ns, feas = o.evaluate(failed)
    assert 0 < feas.sum() < len(feas)                         # the capacity check binds
    assert np.all(np.isinf(cost[feas == 0])) and np.all(np.isfinite(cost[feas == 1]))
    plan = o.search_policy(failed, W.POLICY_DYNPAR)
    cuts = o.decode(failed, plan)
    surv = [d for d in range(8) if d not in failed]
    off = 0
    for p in range(plan.n_pipes):
        ok, c, _, peak = o.pipe(cuts[p], plan.micro[p], surv[off:off + plan.stages[p]], plan.n_pipes)
        assert ok and max(peak) <= w.profile.mem_capacity_bytes and c <= plan.cost
        off += plan.stages[p]
    # with a capacity nothing fits in, nothing is feasible
    w.profile.mem_capacity_bytes = 1000
    o = oracle_factory(w.profile, w.options)
    best, per = o.search(failed)
    assert best is None and not any(p.feasible for p in per)


@pytest.mark.parametrize("mode", [0, 1])
def test_fault_free_search_contains_the_baseline_plan(oracle_factory, mode):
    for w in (W.tiny(), W.paper_scale(0, 0)):
        p = w.profile
        opts = w.options.with_cost_mode(mode)
        o = oracle_factory(p, opts)
        base_ok, base_cost, base_ns, _ = o.pipe(list(p.base_cuts), p.n_micro, list(range(p.n_pp)), p.n_dp, mode)
        assert base_ok
        base = base_ns if mode else base_cost
        best, per = o.search([])
        assert _cost(per[W.POLICY_REROUTE], mode) == base       # nothing failed: rerouting is the baseline
        assert _cost(per[W.POLICY_DYNPAR], mode) <= base        # the baseline is one of the candidates
        assert _cost(best, mode) <= base
        # the identity plan (same grid, same split, same layers) costs exactly the baseline
        strategies = o.strategies(p.n_dp * p.n_pp)
        si = strategies.index((p.n_pp,) * p.n_dp)
        cost, cost_ns, feas = o.evaluate([])
        vals = cost_ns if mode else cost
        s = 0
        found = 0
        while True:
            d = o.segment([], s)
            if d is None:
                break
            s += 1
            if d["strategy"] != si or d["m"] != p.n_micro:
                continue
            for k in range(d["K"]):
                if o.layer_unrank(opts.layer_mode, d["S"], k) == list(p.base_cuts):
                    devs = list(range(d["off"], d["off"] + d["S"]))
                    want = o.pipe(list(p.base_cuts), p.n_micro, devs, p.n_dp, mode)
                    assert vals[d["first"] + k] == (want[2] if mode else want[1])
                    found += 1
        assert found == p.n_dp


def test_policy_tie_break_and_redundant_computation_rules(oracle_factory):
    w = W.paper_scale(0, 0)
    o = oracle_factory(w.profile, w.options)
    # stage 0 has no predecessor to take over; adjacent failures in a pipeline lose the replica
    assert not o.search_policy([0], W.POLICY_REDUNDANT).feasible
    assert not o.search_policy([8], W.POLICY_REDUNDANT).feasible
    assert not o.search_policy([3, 4], W.POLICY_REDUNDANT).feasible
    plan = o.search_policy([3, 12], W.POLICY_REDUNDANT)
    assert plan.feasible and plan.stages == (7, 7, 8, 8)
    cuts = o.decode([3, 12], plan)
    assert cuts[0] == [0, 4, 8, 16, 20, 24, 28, 32] and cuts[1] == [0, 4, 8, 12, 20, 24, 28, 32]
    assert cuts[2] == list(w.profile.base_cuts)
    # every stage but the last carries its successor's work: the fault-free redundant cost
    # equals a plain pipeline whose stage times are those pairwise sums
    none_failed = o.search_policy([], W.POLICY_REDUNDANT)
    p = w.profile
    PF = [0.0]
    PB = [0.0]
    for l in range(p.L):
        PF.append(PF[-1] + float(p.fwd_ns[l]))
        PB.append(PB[-1] + float(p.bwd_ns[l]))
    F = [PF[4 * i + 4] - PF[4 * i] for i in range(8)]
    B = [PB[4 * i + 4] - PB[4 * i] for i in range(8)]
    F2 = [F[i] + F[i + 1] for i in range(7)] + [F[7]]
    B2 = [B[i] + B[i + 1] for i in range(7)] + [B[7]]
    xt = [float(p.p2p_bytes[4 * i + 3]) / float(p.bw_intra_Bpns) for i in range(7)]
    sync = ((2.0 * 3.0) * float(4 * int(p.param_bytes[0]))) / (4.0 * float(p.bw_inter_Bpns))
    assert none_failed.feasible
    assert none_failed.cost == o.pipe_time(F2, B2, xt, p.n_micro) + sync
    base = o.search_policy([], W.POLICY_REROUTE)
    assert none_failed.cost > base.cost * 1.5                  # "nearly double"
    # overall winner: least cost, ties to the lowest policy id
    best, per = o.search([3, 12])
    feas = [q for q in per if q.feasible]
    assert best.cost == min(q.cost for q in feas)
    assert best.policy == min(q.policy for q in feas if q.cost == best.cost)
