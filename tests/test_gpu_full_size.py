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
