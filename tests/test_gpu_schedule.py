"""Parity of the CUDA path with the CPU oracle under the second execution order (all forwards,
then all backwards; every micro-batch in flight): the same element-by-element comparisons as
for 1F1B -- every candidate's cost and feasibility flag, every policy's plan, the selected plan
-- on the small workloads in full and on the large ones by sample.  Same bar: plan tuple and
flags bit-exact, integer costs bit-exact, fp64 costs within 1e-12 relative (in fact equal)."""
import pytest

from paper_2508_21613_b200 import workloads as W

from test_gpu_parity import Session, _sampled_candidate_parity, assert_same_plan, full_parity, gpu  # noqa: F401

pytestmark = pytest.mark.gpu

GPIPE = W.SCHED_GPIPE


def _gpipe(w):
    w.options = w.options.with_schedule(GPIPE)
    return w


def test_tiny_and_random_small_in_full(gpu, oracle_factory):
    w = _gpipe(W.tiny())
    full_parity(gpu, oracle_factory, w, w.scenarios[:3] + [[]])
    w = _gpipe(W.tiny(mem_bound=True))
    full_parity(gpu, oracle_factory, w, w.scenarios[:2] + [[0, 5]])
    for seed in range(4):
        w = W.random_small(seed, L=6 + seed, n_dp=2, n_pp=2 + seed % 3, n_micro=3 + seed % 3, tight_memory=bool(seed % 2))
        for lm, bm in ((W.LAYERS_FULL, W.BATCH_FULL), (W.LAYERS_REMAINDER, W.BATCH_REMAINDER), (W.LAYERS_MINMAX, W.BATCH_REMAINDER)):
            w.options = W.SearchOptions(1, 4, 1, 6, lm, bm, 1 << 62 if seed % 2 else 12, schedule=GPIPE)
            full_parity(gpu, oracle_factory, w, w.scenarios[:2] + w.scenarios[-1:])


def test_paper_scale_sampled_scenarios(gpu, oracle_factory):
    w = _gpipe(W.paper_scale())
    full_parity(gpu, oracle_factory, w, [w.scenarios[i] for i in (0, 31, 200, 528, 1552, 2575)])


def test_deep_pipelines(gpu, oracle_factory):
    w = _gpipe(W.deep_pipeline())
    full_parity(gpu, oracle_factory, w, w.scenarios[:4])


def test_large_workloads_by_sample(gpu, oracle_factory):
    w = _gpipe(W.llama70b_like())
    _sampled_candidate_parity(gpu, oracle_factory, w, [w.scenarios[0], w.scenarios[44]], 2000)
    w = _gpipe(W.gpt175b_like())
    w.profile.mem_capacity_bytes = 160_000_000_000       # all micro-batches in flight: 120 GB holds nothing here
    _sampled_candidate_parity(gpu, oracle_factory, w, [w.scenarios[0], w.scenarios[40]], 300)
    full_parity(gpu, oracle_factory, w, [w.scenarios[35]], modes=(0,), candidates=False)


def test_the_two_orders_share_a_context(gpu, oracle_factory):
    """Min-max partitions and feasible-composition lists are kept per order: alternating the
    order on one context must give each order's own results."""
    w = W.tiny(mem_bound=True)
    s = Session(gpu, w.profile)
    try:
        for sched in (W.SCHED_1F1B, GPIPE, W.SCHED_1F1B, GPIPE):
            for mode in (0, 1):
                opts = w.options.with_cost_mode(mode).with_schedule(sched)
                o = oracle_factory(w.profile, opts)
                best, _, _ = gpu.cm_search_batch(s.ctx, w.scenarios, opts, per_policy=True)
                for b, failed in enumerate(w.scenarios):
                    assert_same_plan(gpu.plans_from_array(best)[b], o.search(failed)[0], mode, f"order {sched} {failed}")
    finally:
        s.close()


def test_full_objective_with_rounds_under_gpipe(gpu, oracle_factory):
    w = _gpipe(W.tiny())
    s = Session(gpu, w.profile)
    try:
        for mode in (0, 1):
            for rounds in (0, 1):
                opts = w.options.with_cost_mode(mode)
                obj = W.ObjectiveOptions(topk=4, sync_rounds=rounds)
                o = oracle_factory(w.profile, opts)
                best, trans, _, sb, _ = gpu.cm_search_objective(s.ctx, w.scenarios[:4], opts, obj, shortlist=True)
                for b, failed in enumerate(w.scenarios[:4]):
                    want, wt = o.search_objective(failed, obj)
                    got = gpu.plans_from_array(best)[b]
                    assert_same_plan(got, want, mode, f"objective {failed} rounds {rounds}")
                    assert trans[b].policy == wt.policy and trans[b].xfer_bytes == wt.xfer_bytes and trans[b].rounds == wt.rounds
    finally:
        s.close()
