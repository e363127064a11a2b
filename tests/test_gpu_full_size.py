"""Parity at the full sizes of the workloads, in the launch configuration bench.py times
(one cm_search_batch over every failure scenario): the selected plan of EVERY scenario is
compared with the stored result of the CPU oracle -- policy, feasibility, cost and a
fingerprint of the whole plan tuple plus cost bits (tests/golden/search_*.txt, written by
tests/golden/make_search_goldens.py, which calls only the oracle)."""
import importlib.util
import os

import pytest

from paper_2508_21613_b200 import workloads as W

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
_spec = importlib.util.spec_from_file_location("make_search_goldens", os.path.join(GOLDEN, "make_search_goldens.py"))
goldens = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(goldens)


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2508_21613_b200 import binding, build
    build.build()
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; there is no CPU path")
    return binding


def _stored(name, mode):
    path = goldens.golden_path(name, mode)
    assert os.path.exists(path), f"{path} is missing: run tests/golden/make_search_goldens.py {name}"
    return [l.strip() for l in open(path) if l.strip() and not l.startswith("#")]


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("name", ["paper-scale", "70b-like", "175b-like", "sweep"])
def test_every_scenario_matches_the_stored_oracle_result(gpu, name, mode):
    w = W.ALL_WORKLOADS[name]()
    want = _stored(name, mode)
    assert len(want) == len(w.scenarios)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, w.options.with_cost_mode(mode))
        got = [goldens.line_of(p, mode) for p in gpu.plans_from_array(best)]
        wrong = [b for b in range(len(want)) if got[b] != want[b]]
        assert not wrong, (f"{len(wrong)} of {len(want)} scenarios differ, first: scenario {wrong[0]} "
                           f"{w.scenarios[wrong[0]]}: got {got[wrong[0]]} want {want[wrong[0]]}")
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("share", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
def test_every_paper_scale_scenario_under_the_second_order(gpu, mode, share):
    """The same comparison with the time model under the all-forward-all-backward order
    (tests/golden/search_paper-scale_gpipe_*.txt, `make_search_goldens.py paper-scale --schedule gpipe`)."""
    w = W.paper_scale()
    path = goldens.golden_path(w.name, mode, W.SCHED_GPIPE)
    assert os.path.exists(path), f"{path} is missing"
    want = [l.strip() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(want) == len(w.scenarios)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        gpu.cm_set_sharing(ctx, share)
        best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, w.options.with_cost_mode(mode).with_schedule(W.SCHED_GPIPE))
        got = [goldens.line_of(p, mode) for p in gpu.plans_from_array(best)]
        wrong = [b for b in range(len(want)) if got[b] != want[b]]
        assert not wrong, f"{len(wrong)} of {len(want)} scenarios differ, first: {wrong[0]}: got {got[wrong[0]]} want {want[wrong[0]]}"
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("share", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("name,picks", [("70b-like", range(64)), ("175b-like", range(0, 64, 3)), ("sweep", range(0, 256, 7))])
def test_one_failure_at_a_time_matches_the_stored_oracle_result(gpu, name, picks, mode, share):
    """The per-failure path (cm_search_batch with a latency buffer handles one failure set at a time: its own launch classes --
    a warp per plan where the memory screen leaves few deep plans -- the lock-step tie-break
    pass and, from the second search of a survivor count on, the replayed launch graph), each
    scenario searched three times in a row, against the same stored oracle results.  With
    sharing on, a failure set whose duplicate pipelines are worth removing is searched over its
    distinct segments instead (keyed on the host, launched directly)."""
    w = W.ALL_WORKLOADS[name]()
    want = _stored(name, mode)
    opts = w.options.with_cost_mode(mode)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        gpu.cm_set_sharing(ctx, share)
        saved = 0
        for b in picks:
            for rep in range(3):
                best, _, lat = gpu.cm_search_batch(ctx, [w.scenarios[b]], opts, latency=True)
                assert lat[0] > 0
                got = goldens.line_of(gpu.plans_from_array(best)[0], mode)
                assert got == want[b], f"scenario {b} {w.scenarios[b]} (search {rep}): got {got} want {want[b]}"
                st = gpu.cm_last_stats(ctx)
                if rep == 2 and share and name != "70b-like":
                    saved += st["plans"] > 3 * st["plans_simulated"]
        if share and name != "70b-like":
            assert saved > 0   # some failure sets of these jobs repeat most of their pipelines
    finally:
        gpu.cm_destroy(ctx)


def _stored_objective(name, mode):
    path = goldens.objective_path(name, mode)
    assert os.path.exists(path), f"{path} is missing: run tests/golden/make_search_goldens.py {name} --objective"
    return [l.strip() for l in open(path) if l.strip() and not l.startswith("#")]


@pytest.mark.parametrize("name,mode", [("paper-scale", 0), ("paper-scale", 1), ("70b-like", 0), ("70b-like", 1),
                                       ("175b-like", 0), ("175b-like", 1), ("sweep", 0)])
def test_full_objective_of_every_scenario_matches_the_stored_oracle_result(gpu, name, mode):
    """cm_search_objective with the default options over the whole workload: chosen policy,
    shortlist rank, matched bytes, transition time, objective, the chosen plan and the whole
    shortlist (plan tuples, costs, matched bytes) of every scenario against the oracle's."""
    from types import SimpleNamespace
    w = W.ALL_WORKLOADS[name]()
    want = _stored_objective(name, mode)
    assert len(want) == len(w.scenarios)
    obj = W.ObjectiveOptions()
    k = obj.topk
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        best, trans, sl, sb, _ = gpu.cm_search_objective(ctx, w.scenarios, w.options.with_cost_mode(mode), obj,
                                                      shortlist=True)
        plans = gpu.plans_from_array(best)
        short = gpu.plans_from_array(sl)
        wrong = []
        for b in range(len(want)):
            used = [r for r in range(k) if sb[b, r] >= 0]
            tr = SimpleNamespace(policy=trans[b].policy, rank=trans[b].rank, xfer_bytes=trans[b].xfer_bytes,
                                 t_trans=trans[b].t_trans, t_trans_ns=trans[b].t_trans_ns,
                                 objective=trans[b].objective,
                                 shortlist=[short[b * k + r] for r in used],
                                 shortlist_bytes=[int(sb[b, r]) for r in used])
            got = goldens.objective_line(plans[b] if trans[b].feasible else None, tr, mode)
            if got != want[b]:
                wrong.append((b, got))
        assert not wrong, (f"{len(wrong)} of {len(want)} scenarios differ, first: scenario {wrong[0][0]} "
                           f"{w.scenarios[wrong[0][0]]}: got {wrong[0][1]} want {want[wrong[0][0]]}")
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("name", ["paper-scale", "70b-like", "175b-like", "sweep"])
def test_shared_search_matches_the_stored_oracle_results(gpu, name, mode):
    """With sharing on, scenarios whose dynamic-parallelism spaces coincide are searched once,
    and so is every distinct segment (stages, micro-batches, peers, link tiers) of the batch;
    every scenario must still come out exactly as the oracle has it, in the plain search and
    in the full-objective search."""
    from types import SimpleNamespace
    w = W.ALL_WORKLOADS[name]()
    want = _stored(name, mode)
    want_obj = _stored_objective(name, mode) if os.path.exists(goldens.objective_path(name, mode)) else None
    obj = W.ObjectiveOptions()
    k = obj.topk
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        opts = w.options.with_cost_mode(mode)
        gpu.cm_search_batch(ctx, w.scenarios, opts)
        plain_plans, plain_simulated = (gpu.cm_last_stats(ctx)[k_] for k_ in ("plans", "plans_simulated"))
        gpu.cm_set_sharing(ctx, True)
        for _ in range(2):   # the distinct segments are listed in whatever order the atomics give: twice
            best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, opts)
            shared_plans, shared_simulated = (gpu.cm_last_stats(ctx)[k_] for k_ in ("plans", "plans_simulated"))
            got = [goldens.line_of(p, mode) for p in gpu.plans_from_array(best)]
            assert got == want
        assert shared_plans <= plain_plans
        if name == "paper-scale":
            assert shared_plans * 20 < plain_plans        # 2576 failure sets fall into a few dozen classes
        if name != "70b-like":                            # (there the memory screen leaves almost nothing to share)
            assert shared_simulated * 10 < plain_simulated    # few distinct segments among the scenarios' pipelines
        if want_obj is None:
            return
        best, trans, sl, sb, _ = gpu.cm_search_objective(ctx, w.scenarios, opts, obj, shortlist=True)
        plans = gpu.plans_from_array(best)
        short = gpu.plans_from_array(sl)
        for b in range(len(want_obj)):
            used = [r for r in range(k) if sb[b, r] >= 0]
            tr = SimpleNamespace(policy=trans[b].policy, rank=trans[b].rank, xfer_bytes=trans[b].xfer_bytes,
                                 t_trans=trans[b].t_trans, t_trans_ns=trans[b].t_trans_ns, objective=trans[b].objective,
                                 shortlist=[short[b * k + r] for r in used], shortlist_bytes=[int(sb[b, r]) for r in used])
            assert goldens.objective_line(plans[b] if trans[b].feasible else None, tr, mode) == want_obj[b], f"scenario {b}"
        gpu.cm_set_sharing(ctx, False)
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("name", ["paper-scale", "175b-like"])
def test_pipeline_reuse_changes_the_work_not_the_result(gpu, name, mode):
    """A pipeline that several strategies of a survivor count have in common searched once (the
    default) and once per strategy: every scenario equals the stored oracle result either way,
    batched and one failure at a time; with reuse fewer recurrences run for the same search space."""
    w = W.ALL_WORKLOADS[name]()
    want = _stored(name, mode)
    opts = w.options.with_cost_mode(mode)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        work = {}
        for reuse in (True, False):
            gpu.cm_set_pipeline_reuse(ctx, reuse)
            best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, opts)
            st = gpu.cm_last_stats(ctx)
            work[reuse] = (st["plans"], st["plans_simulated"])
            assert [goldens.line_of(p, mode) for p in gpu.plans_from_array(best)] == want
            for b in range(0, len(w.scenarios), max(1, len(w.scenarios) // 24)):
                for _ in range(2):
                    one, _, _ = gpu.cm_search_batch(ctx, [w.scenarios[b]], opts, latency=True)
                assert goldens.line_of(gpu.plans_from_array(one)[0], mode) == want[b], f"scenario {b} reuse={reuse}"
        assert work[True][0] == work[False][0]             # the same search space ...
        assert work[True][1] * 2 < work[False][1]          # ... with under half the recurrences
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("mode", [0, 1])
def test_micro_batch_pairs_change_the_work_not_the_result(gpu, mode):
    """A pipeline's m and m+1 micro-batch variants evaluated in one recurrence (the default) and
    each on its own: every 175b-like scenario equals the stored oracle result either way, and
    the paired search runs fewer recurrence cells for the same plans."""
    w = W.gpt175b_like()
    want = _stored(w.name, mode)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        cells = {}
        for pairs in (True, False):
            gpu.cm_set_micro_batch_pairs(ctx, pairs)
            best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, w.options.with_cost_mode(mode))
            st = gpu.cm_last_stats(ctx)
            cells[pairs] = (st["cells"], st["plans_simulated"])
            assert [goldens.line_of(p, mode) for p in gpu.plans_from_array(best)] == want
        assert cells[True][1] == cells[False][1]            # the same plans ...
        assert cells[True][0] * 3 < cells[False][0] * 2     # ... in under two thirds of the cells
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("name", ["paper-scale", "175b-like"])
def test_forced_integer_kernels_match_the_stored_oracle_results(gpu, name):
    """The integer mode normally runs in double arithmetic (exact for these profiles); the
    64-bit integer kernels stay covered by forcing them."""
    w = W.ALL_WORKLOADS[name]()
    want = _stored(name, 1)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        assert gpu.cm_int64_runs_in_fp64(ctx)
        gpu.cm_set_int64_arithmetic(ctx, True)
        assert not gpu.cm_int64_runs_in_fp64(ctx)
        best, _, _ = gpu.cm_search_batch(ctx, w.scenarios, w.options.with_cost_mode(1))
        got = [goldens.line_of(p, 1) for p in gpu.plans_from_array(best)]
        assert got == want
    finally:
        gpu.cm_destroy(ctx)
