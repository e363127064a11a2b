"""Stretch case: the 70b-like workload with NO cap on the layer compositions per pipeline
(up to C(32,16) = 6e8 of them, 1e10 pipeline-plans for one failure set).  The oracle cannot
search such a space; what it can do one by one: count the candidates, evaluate a seeded
sample of them, and re-evaluate the selected plan from its decoded cuts.  Properties that
hold at any size close the gap: the uncapped space contains every candidate of the capped
one, so its best plan cannot be slower; no sampled candidate of a winning segment may beat
the selected composition's bound."""
import copy

import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W

from test_gpu_parity import Session, assert_same_candidates, evaluate_on_gpu, gpu  # noqa: F401

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1])
def test_uncapped_compositions_on_70b_like(gpu, oracle_factory, mode):
    w = W.llama70b_like()
    failed = w.scenarios[63]
    capped = w.options.with_cost_mode(mode)
    opts = copy.copy(capped)
    opts.kappa_cap = 1 << 62
    o = oracle_factory(w.profile, opts)
    s = Session(gpu, w.profile)
    try:
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, opts)
        assert n == o.count(failed)[0] and n > 4_000_000_000
        # a seeded sample of candidate indices, element by element
        rng = W.SplitMix64(4242 + mode)
        idx = sorted({rng.below(n) for _ in range(1500)} | {0, n - 1})
        assert_same_candidates(evaluate_on_gpu(s, space, n, mode, idx), o.evaluate(failed, idx=idx), mode)
        # the search itself
        got = gpu.cm_select(s.ctx, [space])
        assert got.feasible
        cost = got.cost_ns if mode else got.cost
        cuts = gpu.cm_decode_plan(s.ctx, space, got)
        surv = [d for d in range(w.profile.n_devices) if d not in failed]
        off, worst = 0, 0
        for p in range(got.n_pipes):
            ok, c, c_ns, peak = o.pipe(cuts[p], got.micro[p], surv[off:off + got.stages[p]], got.n_pipes, mode)
            assert ok and max(peak) <= w.profile.mem_capacity_bytes
            worst = max(worst, c_ns if mode else c)
            off += got.stages[p]
        assert worst == cost and sum(got.stages) == len(surv)
        # superset of the capped space: cannot be slower than its optimum (stored oracle result path)
        cspace, _ = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, capped)
        cgot = gpu.cm_select(s.ctx, [cspace])
        assert cost <= (cgot.cost_ns if mode else cgot.cost)
        # sampled candidates of the winning pipelines' segments: none that precedes the selected
        # composition may be feasible within the winning step time (the tie-break rule), none at
        # all may beat the step time on the slowest pipeline's own segment minimum
        for p in range(got.n_pipes):
            seg = next(g for g in (o.segment(failed, k) for k in range(o.count(failed)[2]))
                       if g["strategy"] == got.strategy and g["pipe"] == p and g["m"] == got.micro[p])
            ks = sorted({rng.below(seg["K"] + 1) for _ in range(300)})
            c, c_ns, f = o.evaluate(failed, idx=[seg["first"] + k for k in ks])
            vals = c_ns if mode else c
            for k, v, ok in zip(ks, vals, f):
                if ok and k < got.kappa[p]:
                    assert v > cost
        gpu.cm_space_free(space)
        gpu.cm_space_free(cspace)
    finally:
        s.close()
