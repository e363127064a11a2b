"""The plan cache (Section "Planner": plans for the loss of 1..k devices computed ahead of
time) returns, for every failure set it covers, exactly what the search returns -- checked
against the stored oracle results and against the oracle itself."""
import importlib.util
import itertools
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


@pytest.mark.parametrize("mode", [0, 1])
def test_cache_of_all_single_and_double_failures_matches_stored_oracle_results(gpu, mode):
    w = W.paper_scale(0, 0)          # its 528 scenarios are all sets of one and of two devices
    want = [l.strip() for l in open(goldens.golden_path("paper-scale", mode)) if l.strip() and not l.startswith("#")]
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        cache, n = gpu.cm_cache_build(ctx, 2, w.options.with_cost_mode(mode))
        assert n == 1 + 32 + 32 * 31 // 2
        for b, failed in enumerate(w.scenarios):
            plan = gpu.cm_cache_lookup(cache, list(reversed(failed)))       # any order
            assert goldens.line_of(plan, mode) == want[b], f"scenario {b} {failed}"
        # the empty set: nothing failed, rerouting is the unchanged base configuration
        plan, per = gpu.cm_cache_lookup(cache, [], per_policy=True)
        assert plan.feasible and per[W.POLICY_REROUTE].feasible
        # not covered / malformed
        assert gpu.cm_cache_lookup(cache, [1, 2, 3]) is None
        for bad in ([32], [3, 3]):
            with pytest.raises(gpu.ChameleonError):
                gpu.cm_cache_lookup(cache, bad)
        gpu.cm_cache_free(cache)
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_cache_build(ctx, 9, w.options)                           # C(32,9) sets: too many
    finally:
        gpu.cm_destroy(ctx)


def test_cache_equals_search_and_oracle_on_tiny(gpu, oracle_factory):
    w = W.tiny()
    o = oracle_factory(w.profile, w.options)
    ctx = gpu.cm_create(0)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        cache, n = gpu.cm_cache_build(ctx, 3, w.options)
        assert n == 1 + 8 + 28 + 56
        sets = [list(c) for k in range(4) for c in itertools.combinations(range(8), k)]
        best, pol, _ = gpu.cm_search_batch(ctx, sets, w.options, per_policy=True)
        direct = gpu.plans_from_array(best)
        for b, failed in enumerate(sets):
            plan, per = gpu.cm_cache_lookup(cache, failed, per_policy=True)
            assert plan.key() == direct[b].key() and plan.cost == direct[b].cost
            for q in range(3):
                assert per[q].key() == gpu.plans_from_array([pol[3 * b + q]])[0].key()
        for failed in ([5], [1, 6], [0, 3, 7]):
            want, _ = o.search(failed)
            got = gpu.cm_cache_lookup(cache, failed)
            assert (want is None and not got.feasible) or (got.key() == want.key() and got.cost == want.cost)
        gpu.cm_cache_free(cache)
    finally:
        gpu.cm_destroy(ctx)
