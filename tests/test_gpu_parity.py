"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded
inputs.  Bar: selected plan tuple and feasibility flags bit-exact; fp64 costs within
1e-12 relative (the kernels follow the oracle's operation order, so they are in fact
compared for equality as well); integer-nanosecond costs bit-exact."""
import math

import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W

pytestmark = pytest.mark.gpu

REL_TOL = 1e-12


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2508_21613_b200 import binding, build
    build.build()
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; there is no CPU path")
    return binding


class Session:
    def __init__(self, binding, profile):
        self.b = binding
        self.ctx = binding.cm_create(0)
        binding.cm_load_profile(self.ctx, profile)

    def close(self):
        self.b.cm_destroy(self.ctx)


def _plan_cost(plan, mode):
    return plan.cost_ns if mode else plan.cost


def assert_same_plan(got, want, mode, what=""):
    if want is None or not want.feasible:
        assert got is None or not got.feasible, what
        return
    assert got is not None and got.feasible, what
    assert got.key() == want.key(), f"{what}: {got} != {want}"
    a, b = _plan_cost(got, mode), _plan_cost(want, mode)
    if mode:
        assert a == b, what
    else:
        assert abs(a - b) <= REL_TOL * abs(b), what
        assert a == b, f"{what}: costs differ in the last bits ({a!r} vs {b!r})"


def evaluate_on_gpu(s, space, n, mode, idx=None):
    import torch
    count = n if idx is None else len(idx)
    cost = torch.zeros(max(count, 1), dtype=torch.float64, device="cuda")
    cost_ns = torch.zeros(max(count, 1), dtype=torch.int64, device="cuda")
    feas = torch.zeros(max(count, 1), dtype=torch.uint8, device="cuda")
    idx_dev = None
    if idx is not None:
        idx_dev = torch.tensor(np.asarray(idx, dtype=np.int64), device="cuda")
    s.b.cm_evaluate(s.ctx, space, 0, count, idx_dev, cost, cost_ns, feas)
    torch.cuda.synchronize()
    return cost.cpu().numpy()[:count], cost_ns.cpu().numpy()[:count], feas.cpu().numpy()[:count]


def assert_same_candidates(gpu_res, orc_res, mode):
    gc, gn, gf = gpu_res
    oc, on, of = orc_res
    assert np.array_equal(gf, of)                       # feasibility flags bit-exact
    if mode:
        assert np.array_equal(gn, on)                   # integer nanoseconds bit-exact
    else:
        fin = of.astype(bool)
        assert np.all(np.isinf(gc[~fin]))
        assert np.all(np.abs(gc[fin] - oc[fin]) <= REL_TOL * np.abs(oc[fin]))
        assert np.array_equal(gc[fin], oc[fin])         # stronger than required: identical bits


def full_parity(gpu, oracle_factory, w, scenarios, modes=(0, 1), candidates=True):
    s = Session(gpu, w.profile)
    try:
        for mode in modes:
            opts = w.options.with_cost_mode(mode)
            o = oracle_factory(w.profile, opts)
            for failed in scenarios:
                want_best, want_per = o.search(failed)
                spaces = []
                for pol in range(3):
                    space, n = gpu.cm_enumerate(s.ctx, pol, failed, opts)
                    spaces.append(space)
                    got = gpu.cm_select(s.ctx, [space])
                    assert_same_plan(got, want_per[pol], mode, f"{w.name} {failed} policy {pol} mode {mode}")
                    if pol == W.POLICY_DYNPAR:
                        assert n == o.count(failed)[0]
                        if candidates:
                            assert_same_candidates(evaluate_on_gpu(s, space, n, mode), o.evaluate(failed), mode)
                        if got is not None:
                            assert gpu.cm_decode_plan(s.ctx, space, got) == o.decode(failed, want_per[pol])
                    else:
                        gc, gn, gf = evaluate_on_gpu(s, space, 1, mode)
                        assert bool(gf[0]) == want_per[pol].feasible
                        if want_per[pol].feasible:
                            assert (gn[0] if mode else gc[0]) == _plan_cost(want_per[pol], mode)
                got = gpu.cm_select(s.ctx, spaces)
                assert_same_plan(got, want_best, mode, f"{w.name} {failed} overall mode {mode}")
                for space in spaces:
                    gpu.cm_space_free(space)
            # the same scenarios in one launch sequence
            best, per, _ = gpu.cm_search_batch(s.ctx, scenarios, opts, per_policy=True)
            best, per = gpu.plans_from_array(best), gpu.plans_from_array(per)
            for b, failed in enumerate(scenarios):
                want_best, want_per = o.search(failed)
                assert_same_plan(best[b], want_best, mode, f"{w.name} batch {failed}")
                for pol in range(3):
                    assert_same_plan(per[3 * b + pol], want_per[pol], mode, f"{w.name} batch {failed} policy {pol}")
    finally:
        s.close()


def test_tiny_every_single_failure_full_enumeration(gpu, oracle_factory):
    w = W.tiny()
    full_parity(gpu, oracle_factory, w, w.scenarios)


def test_tiny_with_binding_memory(gpu, oracle_factory):
    w = W.tiny(mem_bound=True)
    full_parity(gpu, oracle_factory, w, w.scenarios[:4] + [[], [0, 5]])


def test_random_small_profiles_all_modes(gpu, oracle_factory):
    for seed in range(6):
        w = W.random_small(seed, L=6 + seed, n_dp=2, n_pp=2 + seed % 3, n_micro=3 + seed % 3,
                           tight_memory=bool(seed % 2))
        for lm, bm in ((W.LAYERS_FULL, W.BATCH_FULL), (W.LAYERS_REMAINDER, W.BATCH_REMAINDER),
                       (W.LAYERS_MINMAX, W.BATCH_REMAINDER), (W.LAYERS_REMAINDER, W.BATCH_FULL)):
            w.options = W.SearchOptions(1, 4, 1, 6, lm, bm, 1 << 62 if seed % 2 else 12)
            full_parity(gpu, oracle_factory, w, w.scenarios[:2] + w.scenarios[-2:])


def test_paper_scale_sampled_scenarios(gpu, oracle_factory):
    w = W.paper_scale()
    pick = [0, 7, 31, 32, 200, 527, 528, 1000, 1551, 1552, 2000, 2575]
    full_parity(gpu, oracle_factory, w, [w.scenarios[i] for i in pick])


def test_paper_scale_whole_batch_against_oracle(gpu, oracle_factory):
    # every 8th failure set of the 2576 of this configuration, searched in one launch
    # sequence (the configuration bench.py times)
    w = W.paper_scale()
    scen = w.scenarios[::8]
    s = Session(gpu, w.profile)
    try:
        for mode in (0, 1):
            opts = w.options.with_cost_mode(mode)
            o = oracle_factory(w.profile, opts)
            best, per, _ = gpu.cm_search_batch(s.ctx, w.scenarios, opts, per_policy=True)
            best = gpu.plans_from_array(best)
            for b in range(0, len(w.scenarios), 8):
                want_best, _ = o.search(w.scenarios[b])
                assert_same_plan(best[b], want_best, mode, f"paper-scale batch scenario {b}")
            assert len(scen) == 322
    finally:
        s.close()


def test_70b_like_memory_decides(gpu, oracle_factory):
    w = W.llama70b_like()
    full_parity(gpu, oracle_factory, w, [w.scenarios[i] for i in (0, 9, 23, 40, 63)], modes=(0,), candidates=False)
    full_parity(gpu, oracle_factory, w, [w.scenarios[i] for i in (5, 58)], modes=(1,), candidates=False)


def test_deep_pipelines_beyond_a_warp_and_beyond_the_register_kernels(gpu, oracle_factory):
    # fault-free pipelines of 40 stages (policy kernel's serial path) and candidates of up to
    # 61 stages (generic cost kernel), next to 18..48-stage ones with few segments per bucket
    w = W.deep_pipeline()
    full_parity(gpu, oracle_factory, w, w.scenarios)


def _sampled_candidate_parity(gpu, oracle_factory, w, scenarios, n_samples, modes=(0, 1)):
    s = Session(gpu, w.profile)
    try:
        for mode in modes:
            opts = w.options.with_cost_mode(mode)
            o = oracle_factory(w.profile, opts)
            for k, failed in enumerate(scenarios):
                space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, opts)
                assert n == o.count(failed)[0]
                rng = W.SplitMix64(1000 + k)
                idx = sorted({rng.below(n) for _ in range(n_samples)} | {0, n - 1})
                assert_same_candidates(evaluate_on_gpu(s, space, n, mode, idx), o.evaluate(failed, idx=idx), mode)
                gpu.cm_space_free(space)
    finally:
        s.close()


def test_70b_like_sampled_candidates(gpu, oracle_factory):
    w = W.llama70b_like()
    _sampled_candidate_parity(gpu, oracle_factory, w, [w.scenarios[i] for i in (0, 17, 44)], 3000)


def test_175b_like_sampled_candidates_and_one_full_search(gpu, oracle_factory):
    w = W.gpt175b_like()
    _sampled_candidate_parity(gpu, oracle_factory, w, [w.scenarios[0], w.scenarios[40]], 400)
    full_parity(gpu, oracle_factory, w, [w.scenarios[3]], modes=(0,), candidates=False)


def test_sweep_selected_plans_hold_against_the_oracle(gpu, oracle_factory):
    """At the sweep's full size the oracle cannot search every scenario in seconds.  What
    it can do one by one: re-evaluate each selected plan's pipelines from their decoded
    cuts (cost equals the slowest pipeline, every stage fits), check that no sampled
    candidate of the winning strategy beats the selection, and search in full the
    scenarios whose spaces are small."""
    w = W.sweep(64)
    s = Session(gpu, w.profile)
    try:
        opts = w.options
        o = oracle_factory(w.profile, opts)
        best, per, _ = gpu.cm_search_batch(s.ctx, w.scenarios, opts, per_policy=True)
        best, per = gpu.plans_from_array(best), gpu.plans_from_array(per)
        searched = 0
        for b, failed in enumerate(w.scenarios):
            dyn = per[3 * b + W.POLICY_DYNPAR]
            rr = o.search_policy(failed, W.POLICY_REROUTE)
            rc = o.search_policy(failed, W.POLICY_REDUNDANT)
            assert_same_plan(per[3 * b + 0], rr, 0)
            assert_same_plan(per[3 * b + 1], rc, 0)
            if dyn.feasible:
                space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, opts)
                cuts = gpu.cm_decode_plan(s.ctx, space, dyn)
                assert cuts == o.decode(failed, _as_oracle_plan(dyn))
                surv = [d for d in range(w.profile.n_devices) if d not in failed]
                off, worst = 0, 0.0
                for p in range(dyn.n_pipes):
                    ok, c, _, peak = o.pipe(cuts[p], dyn.micro[p], surv[off:off + dyn.stages[p]], dyn.n_pipes)
                    assert ok and max(peak) <= w.profile.mem_capacity_bytes
                    worst = max(worst, c)
                    off += dyn.stages[p]
                assert sum(dyn.stages) == len(surv) and sum(dyn.micro) == w.profile.n_dp * w.profile.n_micro
                assert worst == dyn.cost
                gpu.cm_space_free(space)
            if o.count(failed)[0] < 120000 and searched < 3:
                want_best, want_per = o.search(failed)
                assert_same_plan(dyn, want_per[2], 0, f"sweep scenario {b}")
                assert_same_plan(best[b], want_best, 0, f"sweep scenario {b}")
                searched += 1
            feas = [q for q in per[3 * b:3 * b + 3] if q.feasible]
            if feas:
                assert best[b].feasible and best[b].cost == min(q.cost for q in feas)
                assert best[b].policy == min(q.policy for q in feas if q.cost == best[b].cost)
    finally:
        s.close()


def _as_oracle_plan(plan):
    from oracle.oracle import Plan
    return Plan(plan.policy, plan.feasible, plan.cost, plan.cost_ns, plan.strategy, plan.n_pipes,
                plan.split_rank, plan.stages, plan.micro, plan.kappa)


def test_edge_cases(gpu, oracle_factory):
    w = W.tiny()
    s = Session(gpu, w.profile)
    try:
        opts = w.options
        # argument checks
        for bad in ([8], [1, 1]):
            with pytest.raises(gpu.ChameleonError) as e:
                gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, bad, opts)
            assert e.value.status == gpu.CM_EINVAL
        with pytest.raises(gpu.ChameleonError) as e:
            gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [0], W.SearchOptions(1, 17, 1, 8, 0, 0, 1 << 62))
        assert e.value.status == gpu.CM_EINVAL
        # one survivor left: a single one-stage pipeline holding all layers
        o = oracle_factory(w.profile, opts)
        failed = list(range(7))
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, opts)
        assert n == o.count(failed)[0]
        assert_same_plan(gpu.cm_select(s.ctx, [space]), o.search_policy(failed, 2), 0)
        gpu.cm_space_free(space)
        # nothing fails: the baseline is among the candidates
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [], opts)
        assert_same_plan(gpu.cm_select(s.ctx, [space]), o.search_policy([], 2), 0)
        gpu.cm_space_free(space)
        # empty batch
        best, _, _ = gpu.cm_search_batch(s.ctx, [], opts)
        # a window no strategy fits in: zero candidates, not an error; select says no plan
        narrow = W.SearchOptions(2, 2, 1, 2, W.LAYERS_FULL, W.BATCH_FULL, 1 << 62)
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [0], narrow)
        assert n == 0
        assert gpu.cm_select(s.ctx, [space]) is None
        gpu.cm_space_free(space)
    finally:
        s.close()
    # no plan fits in memory anywhere
    w = W.tiny()
    w.profile.mem_capacity_bytes = 1000
    s = Session(gpu, w.profile)
    try:
        best, per, _ = gpu.cm_search_batch(s.ctx, [[1], [2, 6]], w.options, per_policy=True)
        assert not any(p.feasible for p in gpu.plans_from_array(best) + gpu.plans_from_array(per))
    finally:
        s.close()
    # split counts that do not fit 64 bits are refused, not wrapped
    w = W.gpt175b_like()
    s = Session(gpu, w.profile)
    try:
        o2 = W.SearchOptions(7, 9, 30, 34, W.LAYERS_REMAINDER, W.BATCH_FULL, 1 << 13)
        with pytest.raises(gpu.ChameleonError) as e:
            gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [3], o2)
        assert e.value.status == gpu.CM_EOVERFLOW
    finally:
        s.close()


def test_latency_mode_gives_the_same_plans(gpu):
    w = W.paper_scale(8, 8)
    s = Session(gpu, w.profile)
    try:
        scen = w.scenarios[:40]
        a, _, _ = gpu.cm_search_batch(s.ctx, scen, w.options)
        b, _, lat = gpu.cm_search_batch(s.ctx, scen, w.options, latency=True)
        assert [p.key() for p in gpu.plans_from_array(a)] == [p.key() for p in gpu.plans_from_array(b)]
        assert [p.cost for p in gpu.plans_from_array(a)] == [p.cost for p in gpu.plans_from_array(b)]
        assert np.all(lat[:40] > 0)
    finally:
        s.close()


# ---- arithmetic of the integer-nanosecond mode ----

def test_integer_mode_runs_in_double_arithmetic_when_exact_and_both_paths_agree(gpu, oracle_factory):
    """By default the integer mode is evaluated in double arithmetic on the integer-valued
    inputs; the 64-bit integer kernels can be forced.  Both must reproduce the oracle."""
    for w in (W.tiny(), W.tiny(mem_bound=True), W.random_small(3, L=9, n_dp=3, n_pp=3, n_micro=6)):
        opts = w.options.with_cost_mode(1)
        o = oracle_factory(w.profile, opts)
        s = Session(gpu, w.profile)
        try:
            assert gpu.cm_int64_runs_in_fp64(s.ctx)
            for native in (False, True):
                gpu.cm_set_int64_arithmetic(s.ctx, native)
                assert gpu.cm_int64_runs_in_fp64(s.ctx) == (not native)
                best, pol, _ = gpu.cm_search_batch(s.ctx, w.scenarios, opts, per_policy=True)
                plans = gpu.plans_from_array(best)
                per = gpu.plans_from_array(pol)
                for b, failed in enumerate(w.scenarios):
                    want, want_per = o.search(failed)
                    assert_same_plan(plans[b], want, 1, f"{w.name} {failed} native={native}")
                    for q in range(3):
                        assert_same_plan(per[3 * b + q], want_per[q] if want_per[q].feasible else None, 1,
                                         f"{w.name} {failed} policy {q} native={native}")
                # per-candidate costs through cm_evaluate as well
                failed = w.scenarios[1]
                space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, failed, opts)
                assert_same_candidates(evaluate_on_gpu(s, space, n, 1), o.evaluate(failed), 1)
                gpu.cm_space_free(space)
        finally:
            s.close()


def test_integer_mode_falls_back_to_integer_kernels_when_values_exceed_2_pow_52(gpu, oracle_factory):
    # layer times near 2^39 ns, 24 layers, 1600 global micro-batches: pipeline times pass 2^52,
    # where doubles no longer hold every integer
    L, n_dp, n_pp, n_micro = 24, 2, 3, 800
    rng = W.SplitMix64(77)
    fwd = [float(int(rng.uniform(0.5, 1.0) * (1 << 39))) for _ in range(L)]
    bwd = [float(int(f * rng.uniform(1.5, 2.0))) for f in fwd]
    prof = W.make_profile_ns(L, n_dp, n_pp, n_micro, fwd, bwd, act=1_000_000, param=50_000_000, opt=300_000_000,
                             p2p=[int(rng.uniform(1e6, 6e7)) for _ in range(L)], base_cuts=[0, 8, 16, 24],
                             cap=80_000_000_000, dev_per_node=4, bw_intra=300, bw_inter=20)
    opts = W.SearchOptions(1, 3, 1, 4, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 62, 1)
    o = oracle_factory(prof, opts)
    s = Session(gpu, prof)
    try:
        assert not gpu.cm_int64_runs_in_fp64(s.ctx)
        scen = [[0], [4], [1, 5]]
        best, _, _ = gpu.cm_search_batch(s.ctx, scen, opts)
        plans = gpu.plans_from_array(best)
        for b, failed in enumerate(scen):
            want, _ = o.search(failed)
            assert want.cost_ns > (1 << 52)
            assert_same_plan(plans[b], want, 1, f"big values {failed}")
    finally:
        s.close()


@pytest.mark.parametrize("graphs", [True, False])
def test_per_failure_searches_reuse_resident_batches_and_match_the_batched_search(gpu, oracle_factory, graphs):
    """Latency mode keeps one prepared batch per survivor count and, with graphs on, replays its
    launch sequence; interleaved survivor counts, repeated sets, both cost modes and a profile
    reload in between must all give what the batched search and the oracle give."""
    w = W.paper_scale(6, 6)
    scen = [w.scenarios[i] for i in (0, 5, 31, 40, 41, 300, 527, 528, 529, 533, 534, 539, 5, 300)]
    scen += [[], [7, 3], [3, 7]]                                 # nothing failed; ids in either order
    s = Session(gpu, w.profile)
    try:
        gpu.cm_set_latency_graphs(s.ctx, graphs)
        for mode in (0, 1, 0):
            opts = w.options.with_cost_mode(mode)
            batched, _, _ = gpu.cm_search_batch(s.ctx, scen, opts)
            single, pol, lat = gpu.cm_search_batch(s.ctx, scen, opts, per_policy=True, latency=True)
            a, b = gpu.plans_from_array(batched), gpu.plans_from_array(single)
            for i in range(len(scen)):
                assert a[i].key() == b[i].key() and a[i].cost == b[i].cost and a[i].cost_ns == b[i].cost_ns, (mode, scen[i])
            assert np.all(lat[:len(scen)] > 0)
        o = oracle_factory(w.profile, w.options)
        for i in (3, 9, 16):
            want, _ = o.search(scen[i])
            assert_same_plan(b[i], want, 0, f"latency mode {scen[i]}")
        # another profile on the same context: resident batches of the old one must not survive
        t = W.tiny()
        gpu.cm_load_profile(s.ctx, t.profile)
        ot = oracle_factory(t.profile, t.options)
        for rep in range(2):
            got, _, _ = gpu.cm_search_batch(s.ctx, t.scenarios, t.options, latency=True)
            for i, failed in enumerate(t.scenarios):
                want, _ = ot.search(failed)
                assert_same_plan(gpu.plans_from_array(got)[i], want, 0, f"after reload {failed}")
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_search_batch(s.ctx, [[1, 1]], t.options, latency=True)
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_search_batch(s.ctx, [[99]], t.options, latency=True)
    finally:
        s.close()


def test_searches_on_a_caller_owned_stream(gpu, oracle_factory):
    """cm_create takes the caller's CUDA stream: batched, per-failure (resident batch + graph
    replay) and full-objective searches enqueue there and give the usual results."""
    import torch
    w = W.paper_scale(4, 4)
    o = oracle_factory(w.profile, w.options)
    stream = torch.cuda.Stream()
    ctx = gpu.cm_create(0, stream.cuda_stream)
    try:
        gpu.cm_load_profile(ctx, w.profile)
        scen = [w.scenarios[i] for i in (1, 2, 3, 40, 41, 42, 530, 531)]
        a, _, _ = gpu.cm_search_batch(ctx, scen, w.options)
        for rep in range(3):
            b, _, _ = gpu.cm_search_batch(ctx, scen, w.options, latency=True)
            assert [p.key() for p in gpu.plans_from_array(a)] == [p.key() for p in gpu.plans_from_array(b)]
        best, trans, _, _, _ = gpu.cm_search_objective(ctx, scen, w.options, W.ObjectiveOptions(topk=3, sync_rounds=1))
        for i in (0, 5):
            want, _ = o.search(scen[i])
            assert_same_plan(gpu.plans_from_array(a)[i], want, 0, f"stream {scen[i]}")
            wo, wt = o.search_objective(scen[i], W.ObjectiveOptions(topk=3, sync_rounds=1))
            assert gpu.plans_from_array(best)[i].key() == wo.key() and trans[i].objective == wt.objective
        stream.synchronize()
    finally:
        gpu.cm_destroy(ctx)


@pytest.mark.parametrize("seed", [100, 101])
def test_deep_pipelines_across_every_switch(gpu, oracle_factory, seed):
    """Pipelines of 18..64 stages (one-plan segments walked by a warp, per-lane and transposed
    kernels, the local-memory fallback) under every combination of cost mode, sharing, forced
    integer kernels, batched and per-failure (resident batch + graph) search."""
    import itertools
    w = W.deep_pipeline(seed)
    base = w.options
    for mode, (cap, lm) in itertools.product((0, 1), ((40, W.LAYERS_REMAINDER), (5000, W.LAYERS_REMAINDER),
                                                      (1 << 62, W.LAYERS_MINMAX))):
        opts = W.SearchOptions(base.dp_lo, base.dp_hi, base.pp_lo, base.pp_hi, lm, base.batch_mode, cap, mode)
        o = oracle_factory(w.profile, opts)
        want = [o.search(f) for f in w.scenarios]
        for share, native, latency in itertools.product((False, True), (False, True), (False, True)):
            if native and mode == 0:
                continue
            s = Session(gpu, w.profile)
            try:
                gpu.cm_set_sharing(s.ctx, share)
                gpu.cm_set_int64_arithmetic(s.ctx, native)
                for _ in range(3 if latency else 1):
                    best, pol, _ = gpu.cm_search_batch(s.ctx, w.scenarios, opts, per_policy=True, latency=latency)
                plans, per = gpu.plans_from_array(best), gpu.plans_from_array(pol)
                for b, failed in enumerate(w.scenarios):
                    what = f"{w.name} {failed} mode={mode} cap={cap} share={share} native={native} latency={latency}"
                    assert_same_plan(plans[b], want[b][0], mode, what)
                    for q in range(3):
                        assert_same_plan(per[3 * b + q], want[b][1][q] if want[b][1][q].feasible else None, mode, what)
            finally:
                s.close()


@pytest.mark.parametrize("sched", [W.SCHED_1F1B, W.SCHED_GPIPE])
def test_pipelines_of_62_to_64_stages(gpu, oracle_factory, sched):
    """The deepest pipelines the library takes: 16, 17 and 18 failures leave one pipeline of
    64, 63 and 62 stages (both stages of the last lane in use, one, none), batched and one
    failure at a time (a warp per plan and per tie-break composition), both cost modes."""
    w = W.deep_pipeline(7)
    rng = W.SplitMix64(62_64)
    scen = [sorted(rng.sample_distinct(80, k)) for k in (16, 17, 18)]
    base = w.options
    for cap in (40, 3000):
        w.options = W.SearchOptions(1, 2, 18, 64, base.layer_mode, base.batch_mode, cap, schedule=sched)
        full_parity(gpu, oracle_factory, w, scen, candidates=cap == 40)
        for mode in (0, 1):
            opts = w.options.with_cost_mode(mode)
            o = oracle_factory(w.profile, opts)
            s = Session(gpu, w.profile)
            try:
                for _ in range(3):
                    best, _, _ = gpu.cm_search_batch(s.ctx, scen, opts, latency=True)
                for b, failed in enumerate(scen):
                    want = o.search(failed)[0]
                    assert_same_plan(gpu.plans_from_array(best)[b], want, mode, f"{failed} cap {cap} mode {mode} one at a time")
            finally:
                s.close()


@pytest.mark.parametrize("layer_mode,batch_mode", [(W.LAYERS_FULL, W.BATCH_FULL), (W.LAYERS_FULL, W.BATCH_REMAINDER)])
def test_micro_batch_pairs_on_shallow_pipelines_against_the_oracle(gpu, oracle_factory, layer_mode, batch_mode):
    """Pairs of consecutive micro-batch counts in the register-resident kernels, under the full
    enumeration of splits (every count from 1 up: pairs (m, m+1), (m+2, m+3), .. wherever
    m >= stages) and under the remainder rule: a batch large enough for the shallow pair
    kernel (every failure set of one or two of the twelve devices, a third of the triples), non-uniform stage
    times, tight and loose memory; every scenario against the oracle, pairs on and off."""
    import itertools
    for tight in (False, True):
        w = W.random_small(11 + tight, L=13, n_dp=3, n_pp=4, n_micro=7, tight_memory=tight)
        scen = [list(c) for k in (1, 2) for c in itertools.combinations(range(12), k)]
        scen += [list(c) for c in itertools.combinations(range(12), 3)][::3]
        for mode in (0, 1):
            opts = W.SearchOptions(1, 3, 2, 6, layer_mode, batch_mode, 1 << 62, mode)
            o = oracle_factory(w.profile, opts)
            want = [o.search(f)[0] for f in scen]
            cells = {}
            s = Session(gpu, w.profile)
            try:
                for pairs in (True, False):
                    gpu.cm_set_micro_batch_pairs(s.ctx, pairs)
                    best, _, _ = gpu.cm_search_batch(s.ctx, scen, opts)
                    cells[pairs] = gpu.cm_last_stats(s.ctx)["cells"]
                    for b, failed in enumerate(scen):
                        assert_same_plan(gpu.plans_from_array(best)[b], want[b], mode, f"{failed} pairs={pairs} tight={tight}")
            finally:
                s.close()
            assert cells[True] < cells[False]   # some groups were large enough to be paired


def test_micro_batch_pairs_on_deep_pipelines_against_the_oracle(gpu, oracle_factory):
    """The transposed pair kernel on strongly non-uniform stages: every single failure of the
    deep, narrow job in one batch (80 scenarios of one survivor count, so groups of pair heads
    fill transposed warps), pipelines of 18-61 stages, each scenario against the oracle with
    pairs on and off; then three of them one at a time (the per-lane pair kernel)."""
    w = W.deep_pipeline(3)
    scen = [[d] for d in range(80)]
    for mode in (0, 1):
        opts = W.SearchOptions(1, 3, 18, 64, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 600, mode)
        o = oracle_factory(w.profile, opts)
        want = [o.search(f) for f in scen]
        cells = {}
        s = Session(gpu, w.profile)
        try:
            for pairs in (True, False):
                gpu.cm_set_micro_batch_pairs(s.ctx, pairs)
                best, per, _ = gpu.cm_search_batch(s.ctx, scen, opts, per_policy=True)
                cells[pairs] = gpu.cm_last_stats(s.ctx)["cells"]
                for b, failed in enumerate(scen):
                    assert_same_plan(gpu.plans_from_array(best)[b], want[b][0], mode, f"{failed} pairs={pairs}")
                    assert_same_plan(gpu.plans_from_array(per)[3 * b + 2], want[b][1][2], mode, f"{failed} dynpar pairs={pairs}")
                for _ in range(2):
                    best, _, _ = gpu.cm_search_batch(s.ctx, scen[:3], opts, latency=True)
                    for b in range(3):
                        assert_same_plan(gpu.plans_from_array(best)[b], want[b][0], mode, f"{scen[b]} alone pairs={pairs}")
        finally:
            s.close()
        assert cells[True] * 10 < cells[False] * 9   # (many of these pipelines have fewer micro-batches than stages)


def test_handworked_readings_rerouting_redundant_memory_minmax_ties(gpu, oracle_factory):
    """The hand-worked cases that fix the readings taken where the paper prints no formula
    (``tests/golden/*_handworked.txt``): the library must give the fixtures' own numbers, not
    merely agree with the oracle."""
    import reading_cases as R
    for mode in (0, 1):
        for prof, failed, expected in R.reroute_cases():
            s = Session(gpu, prof)
            try:
                space, n = gpu.cm_enumerate(s.ctx, W.POLICY_REROUTE, failed, R.options(mode))
                got = gpu.cm_select(s.ctx, [space])
                assert n == 1 and got.feasible and _plan_cost(got, mode) == expected
                want = oracle_factory(prof, R.options(mode)).search_policy(failed, W.POLICY_REROUTE)
                assert_same_plan(got, want, mode, "rerouting, non-uniform stages")
                gpu.cm_space_free(space)
            finally:
                s.close()
        for prof, failed, feasible in R.redundant_cases():
            s = Session(gpu, prof)
            try:
                space, _ = gpu.cm_enumerate(s.ctx, W.POLICY_REDUNDANT, failed, R.options(mode))
                got = gpu.cm_select(s.ctx, [space])
                assert (got is not None and bool(got.feasible)) == feasible
                want = oracle_factory(prof, R.options(mode)).search_policy(failed, W.POLICY_REDUNDANT)
                assert_same_plan(got, want, mode, "redundant computation, memory binding")
                gpu.cm_space_free(space)
            finally:
                s.close()
        for prof, S, bottleneck, cuts in R.minmax_tie_cases():
            s = Session(gpu, prof)
            try:
                opts = R.minmax_only_options(S, mode)
                space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [], opts)
                got = gpu.cm_select(s.ctx, [space])
                assert n == 1 and got.feasible
                assert gpu.cm_decode_plan(s.ctx, space, got) == [cuts]
                want = oracle_factory(prof, opts).search_policy([], W.POLICY_DYNPAR)
                assert_same_plan(got, want, mode, "min-max tie")
                gpu.cm_space_free(space)
            finally:
                s.close()


def test_spaces_and_batches_of_an_earlier_profile_are_refused(gpu):
    """A space or prepared batch describes the L, G and min-max partitions of the profile it was
    built under; after cm_load_profile replaces that profile every call that takes it must fail
    with CM_EINVAL instead of evaluating old descriptors against new tables."""
    import torch
    big, small = W.paper_scale(0, 0), W.tiny()
    s = Session(gpu, big.profile)
    try:
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [3], big.options)
        packed = gpu.PackedScenarios([[3], [4, 9]])
        batch, _ = packed.prepare(s.ctx, big.options)
        plan = gpu.cm_select(s.ctx, [space])
        assert plan.feasible
        gpu.cm_load_profile(s.ctx, small.profile)          # fewer layers, fewer micro-batches
        cost = torch.zeros(16, dtype=torch.float64, device="cuda")
        calls = [lambda: gpu.cm_evaluate(s.ctx, space, 0, 16, None, cost, None, None),
                 lambda: gpu.cm_select(s.ctx, [space]),
                 lambda: gpu.cm_decode_plan(s.ctx, space, plan),
                 lambda: gpu.cm_evaluate_argmin_noalloc(s.ctx, space, 0, 16, cost, None, None),
                 lambda: packed.search_prepared(s.ctx, batch)]
        for call in calls:
            with pytest.raises(gpu.ChameleonError) as e:
                call()
            assert e.value.status == gpu.CM_EINVAL and "earlier profile" in str(e.value)
        gpu.cm_space_free(space)
        gpu.cm_batch_free(batch)
        # the context itself is fine: a space enumerated under the new profile works
        space, n = gpu.cm_enumerate(s.ctx, W.POLICY_DYNPAR, [1], small.options)
        assert gpu.cm_select(s.ctx, [space]).feasible
        gpu.cm_space_free(space)
    finally:
        s.close()


def test_memory_screen_changes_the_work_not_the_result(gpu, oracle_factory):
    """With the screen on (default) the passes walk the listed memory-feasible compositions;
    with it off they test every composition.  Plans, costs and the count of plans whose
    recurrence ran must be identical; the oracle pins the plans themselves."""
    for w, scen in ((W.tiny(mem_bound=True), None), (W.llama70b_like(), 6), (W.random_small(1, tight_memory=True), None)):
        scenarios = w.scenarios if scen is None else w.scenarios[:scen]
        for mode in (0, 1):
            opts = w.options.with_cost_mode(mode)
            results = []
            for screen in (True, False):
                s = Session(gpu, w.profile)
                try:
                    gpu.cm_set_memory_screen(s.ctx, screen)
                    best, per, _ = gpu.cm_search_batch(s.ctx, scenarios, opts, per_policy=True)
                    st = gpu.cm_last_stats(s.ctx)
                    results.append((gpu.plans_from_array(best), gpu.plans_from_array(per), st["plans"], st["plans_simulated"]))
                    # one at a time as well (resident batches, graph replay on the second pass)
                    for _ in range(2):
                        one = gpu.PackedScenarios(scenarios[:3])
                        one.search(s.ctx, opts, latency=True)
                        for b in range(3):
                            assert_same_plan(gpu.plans_from_array(one.best)[b], results[-1][0][b], mode, "one by one")
                finally:
                    s.close()
            on, off = results
            assert on[2] == off[2] and on[3] == off[3] and on[3] <= on[2]
            for a, b in zip(on[0] + on[1], off[0] + off[1]):
                assert a.key() == b.key() and a.cost == b.cost and a.cost_ns == b.cost_ns
            if w.name != "70b-like":
                o = oracle_factory(w.profile, opts)
                for b, failed in enumerate(scenarios):
                    assert_same_plan(on[0][b], o.search(failed)[0], mode, f"{w.name} {failed}")
