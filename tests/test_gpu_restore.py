"""Parity of the CUDA weight-transfer matching and full-objective search (through the C
ABI) with the CPU oracle on the same seeded inputs.  Bar: matched bytes, shortlisted plan
tuples, chosen policy / rank and integer transition times bit-exact; fp64 transition time
and objective within 1e-12 relative (compared for equality as well, the kernels follow the
oracle's operation order).  A matching itself may differ where several are optimal: it is
checked to be a permutation whose cost is the unique optimum."""
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


def _random_ranges(rng, n, L, kind):
    out = []
    for _ in range(n):
        if kind == "stage":                       # a pipeline-like partition: few distinct ranges
            S = int(rng.integers(1, min(L, 12) + 1))
            cuts = [0] + sorted(rng.choice(np.arange(1, L), size=S - 1, replace=False).tolist()) + [L]
            i = int(rng.integers(0, S))
            out.append((cuts[i], cuts[i + 1]))
        else:                                     # arbitrary, empty ranges included
            a = int(rng.integers(0, L + 1))
            out.append((a, int(rng.integers(a, L + 1))))
    return out


def test_matching_parity_on_random_ranges(gpu, oracle_factory):
    w = W.gpt175b_like()
    o = oracle_factory(w.profile, w.options)
    s = Session(gpu, w.profile)
    try:
        rng = np.random.default_rng(3)
        L = w.profile.L
        problems = []
        for n in (1, 2, 3, 7, 31, 32, 33, 64, 65, 100, 200, 255, 256):
            for kind in ("stage", "any"):
                problems.append((_random_ranges(rng, n, L, kind), _random_ranges(rng, n, L, kind)))
        total, assign = gpu.cm_transfer_matching(s.ctx, problems)
        for q, (old, new) in enumerate(problems):
            c = o.transfer_cost_matrix(old, new)
            want, _ = o.assign(c)
            assert int(total[q]) == want, f"problem {q} (n={len(old)})"
            a = assign[q]
            assert sorted(a) == list(range(len(old)))
            assert sum(int(c[a[j], j]) for j in range(len(old))) == want
    finally:
        s.close()


def test_matching_of_the_papers_worked_example(gpu):
    # 9 layers of one unit each: (3,3,3) x 3 pipelines minus one device -> (2,2,2,3) x 2
    p = W.make_profile_ns(9, 3, 3, 4, [1.0] * 9, [2.0] * 9, act=1, param=1, opt=0, p2p=1,
                          base_cuts=[0, 3, 6, 9], cap=1 << 40, dev_per_node=8, bw_intra=1, bw_inter=1)
    s = Session(gpu, p)
    try:
        old = ([(0, 3), (3, 6), (6, 9)] * 3)[:8]
        new = [(0, 2), (2, 4), (4, 6), (6, 9)] * 2
        total, assign = gpu.cm_transfer_matching(s.ctx, [(old, new), ([(0, 3)], [(0, 2)]), ([(0, 3)], [(2, 4)])])
        assert total.tolist() == [2, 0, 1]
        assert sorted(assign[0]) == list(range(8))
    finally:
        s.close()


def test_matching_rejects_bad_problems(gpu):
    w = W.tiny()
    s = Session(gpu, w.profile)
    try:
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_transfer_matching(s.ctx, [([(0, 9)], [(0, 1)])])          # layer index above L = 8
        with pytest.raises(gpu.ChameleonError):
            gpu.cm_transfer_matching(s.ctx, [([(0, 1)] * 257, [(0, 1)] * 257)])
        total, _ = gpu.cm_transfer_matching(s.ctx, [])
        assert len(total) == 0
    finally:
        s.close()


def _check_objective(gpu, o, w, scenarios, opts, obj, mode, res):
    best, trans, sl, sb, sr = res
    p = w.profile
    wts = o.state_bytes()
    for b, failed in enumerate(scenarios):
        want, wt = o.search_objective(failed, obj, opts)
        got = gpu.plans_from_array([best[b]])[0]
        tr = trans[b]
        what = f"{w.name} scenario {b} {failed} mode {mode}"
        if want is None:
            assert not got.feasible and not tr.feasible, what
            continue
        assert got.feasible and tr.feasible, what
        assert got.key() == want.key(), what
        assert (got.cost_ns if mode else got.cost) == (want.cost_ns if mode else want.cost), what
        assert (tr.policy, tr.rank, tr.n_survivors, tr.xfer_bytes) == (wt.policy, wt.rank, wt.n_surv, wt.xfer_bytes), what
        if mode:
            assert tr.t_trans_ns == wt.t_trans_ns, what
        else:
            assert abs(tr.t_trans - wt.t_trans) <= REL_TOL * abs(wt.t_trans), what
            assert tr.t_trans == wt.t_trans, what
        assert abs(tr.objective - wt.objective) <= REL_TOL * abs(wt.objective), what
        assert tr.objective == wt.objective, what
        assert (tr.rounds, tr.domains, tr.t_sync_ns) == (wt.rounds, wt.domains, wt.t_sync_ns), what
        assert tr.t_sync == wt.t_sync, what
        # the shortlist, slot by slot
        k = obj.topk
        plans = gpu.plans_from_array([sl[b * k + r] for r in range(k)])
        for r in range(k):
            if r < len(wt.shortlist):
                assert plans[r].feasible and plans[r].key() == wt.shortlist[r].key(), f"{what} rank {r}"
                assert int(sb[b, r]) == wt.shortlist_bytes[r], f"{what} rank {r}"
                assert int(sr[b, r]) == wt.shortlist_rounds[r], f"{what} rank {r}"
                a, c = (plans[r].cost_ns, wt.shortlist[r].cost_ns) if mode else (plans[r].cost, wt.shortlist[r].cost)
                assert a == c, f"{what} rank {r}: step time {a!r} != {c!r}"
            else:
                assert not plans[r].feasible and int(sb[b, r]) == -1, f"{what} rank {r}"
        # the migration scheme: a permutation of the survivors whose cost is the matched bytes
        if tr.policy == W.POLICY_DYNPAR:
            n = tr.n_survivors
            a = [int(x) for x in tr.assign[:n]]
            assert sorted(a) == list(range(n)), what
            surv = [d for d in range(p.n_dp * p.n_pp) if d not in failed]
            old = [(int(p.base_cuts[d % p.n_pp]), int(p.base_cuts[d % p.n_pp + 1])) for d in surv]
            new = []
            for cuts in o.decode(failed, want, opts):
                new += list(zip(cuts[:-1], cuts[1:]))
            cost = sum(sum(int(wts[l]) for l in range(new[j][0], new[j][1]) if not old[a[j]][0] <= l < old[a[j]][1])
                       for j in range(n))
            assert cost == tr.xfer_bytes, what


@pytest.mark.parametrize("mode", [0, 1])
def test_objective_parity_tiny(gpu, oracle_factory, mode):
    for w in (W.tiny(), W.tiny(mem_bound=True)):
        opts = w.options.with_cost_mode(mode)
        o = oracle_factory(w.profile, opts)
        s = Session(gpu, w.profile)
        try:
            for obj in (W.ObjectiveOptions(topk=1), W.ObjectiveOptions(topk=6, t_gap_ns=40e9, bw_xfer_Bpns=1),
                        W.ObjectiveOptions(topk=16, t_gap_ns=1e14, t_restart_ns=0.0),
                        W.ObjectiveOptions(topk=7, sync_rounds=1)):
                res = gpu.cm_search_objective(s.ctx, w.scenarios, opts, obj, shortlist=True)
                _check_objective(gpu, o, w, w.scenarios, opts, obj, mode, res)
        finally:
            s.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_objective_parity_random_small(gpu, oracle_factory, mode):
    for seed in range(8):
        w = W.random_small(seed, L=6 + seed % 5, n_dp=2 + seed % 2, n_pp=2 + seed % 3, n_micro=3 + seed % 4,
                           tight_memory=bool(seed % 2))
        opts = W.SearchOptions(1, 4, 1, 5, W.LAYERS_FULL if seed % 3 else W.LAYERS_REMAINDER,
                               W.BATCH_FULL if seed % 2 else W.BATCH_REMAINDER, 1 << 62, mode)
        o = oracle_factory(w.profile, opts)
        s = Session(gpu, w.profile)
        try:
            obj = W.ObjectiveOptions(topk=1 + seed % 5, t_gap_ns=[1e9, 30e9, 1125e9][seed % 3],
                                     t_restart_ns=[0.0, 2e9][seed % 2], bw_xfer_Bpns=1 + seed,
                                     sync_rounds=(seed // 2) % 2)
            res = gpu.cm_search_objective(s.ctx, w.scenarios, opts, obj, shortlist=True)
            _check_objective(gpu, o, w, w.scenarios, opts, obj, mode, res)
        finally:
            s.close()


@pytest.mark.parametrize("rounds", [0, 1])
@pytest.mark.parametrize("mode", [0, 1])
def test_objective_parity_paper_scale_sampled(gpu, oracle_factory, mode, rounds):
    w = W.paper_scale()
    opts = w.options.with_cost_mode(mode)
    o = oracle_factory(w.profile, opts)
    s = Session(gpu, w.profile)
    try:
        obj = W.ObjectiveOptions(sync_rounds=rounds)
        # the whole batch runs in the launch configuration the bench times; a sample is checked one by one
        res = gpu.cm_search_objective(s.ctx, w.scenarios, opts, obj, shortlist=True)
        pick = list(range(0, len(w.scenarios), 97))[:28]
        best, trans, sl, sb, sr = res
        k = obj.topk
        sub = ([best[b] for b in pick], [trans[b] for b in pick],
               [sl[b * k + r] for b in pick for r in range(k)], sb[pick], sr[pick])
        _check_objective(gpu, o, w, [w.scenarios[b] for b in pick], opts, obj, mode, sub)
        # properties that hold for every scenario of the batch
        for b in range(len(w.scenarios)):
            tr = trans[b]
            assert tr.feasible
            assert tr.n_survivors == w.profile.n_dp * w.profile.n_pp - len(w.scenarios[b])
            good = sb[b][sb[b] >= 0]
            assert len(good) >= 1 and np.all(good >= 0)
            if tr.policy == W.POLICY_DYNPAR:
                assert tr.xfer_bytes == sb[b, tr.rank]
                assert sorted(tr.assign[:tr.n_survivors]) == list(range(tr.n_survivors))
    finally:
        s.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_objective_parity_minmax_only_and_capped_segments(gpu, oracle_factory, mode):
    # segments whose only candidate is the min-max partition (layer mode MINMAX, or more
    # compositions than kappa_cap): the completed plan carries kappa = 0 = that partition
    w = W.tiny()
    for lm, cap in ((W.LAYERS_MINMAX, 1 << 62), (W.LAYERS_FULL, 20), (W.LAYERS_REMAINDER, 3)):
        opts = W.SearchOptions(1, 4, 1, 6, lm, W.BATCH_REMAINDER, cap, mode)
        o = oracle_factory(w.profile, opts)
        s = Session(gpu, w.profile)
        try:
            for obj in (W.ObjectiveOptions(topk=5), W.ObjectiveOptions(topk=5, sync_rounds=1)):
                res = gpu.cm_search_objective(s.ctx, w.scenarios, opts, obj, shortlist=True)
                _check_objective(gpu, o, w, w.scenarios, opts, obj, mode, res)
        finally:
            s.close()


def test_objective_parity_deep_pipelines_sampled(gpu, oracle_factory):
    w = W.llama70b_like()
    opts = w.options
    o = oracle_factory(w.profile, opts)
    s = Session(gpu, w.profile)
    try:
        obj = W.ObjectiveOptions(topk=4)
        scen = [w.scenarios[0], w.scenarios[33]]
        res = gpu.cm_search_objective(s.ctx, scen, opts, obj, shortlist=True)
        _check_objective(gpu, o, w, scen, opts, obj, 0, res)
    finally:
        s.close()


def test_objective_parity_255_device_matchings(gpu, oracle_factory):
    # 175B-like grid: 256 devices, matchings of 248 and 255 survivors inside the search
    w = W.gpt175b_like()
    opts = w.options
    o = oracle_factory(w.profile, opts)
    s = Session(gpu, w.profile)
    try:
        obj = W.ObjectiveOptions(topk=3, sync_rounds=1)
        scen = [w.scenarios[0], w.scenarios[40]]
        res = gpu.cm_search_objective(s.ctx, scen, opts, obj, shortlist=True)
        _check_objective(gpu, o, w, scen, opts, obj, 0, res)
    finally:
        s.close()


def test_objective_limits_and_errors(gpu):
    w = W.paper_scale(2, 2)
    s = Session(gpu, w.profile)
    try:
        scen = w.scenarios[:16]
        plain, _, _ = gpu.cm_search_batch(s.ctx, scen, w.options)
        # faults far apart: the plain search's choice stands
        best, trans, _, _, _ = gpu.cm_search_objective(s.ctx, scen, w.options, W.ObjectiveOptions(topk=4, t_gap_ns=1e18))
        assert [p.key() for p in gpu.plans_from_array(best)] == [p.key() for p in gpu.plans_from_array(plain)]
        # faults closer together than a restart: no reconstruction
        best, trans, _, _, _ = gpu.cm_search_objective(s.ctx, scen, w.options,
                                                    W.ObjectiveOptions(topk=4, t_gap_ns=4e9, t_restart_ns=5e9))
        assert all(trans[b].policy != W.POLICY_DYNPAR and trans[b].xfer_bytes == 0 for b in range(len(scen)))
        for bad in (W.ObjectiveOptions(topk=0), W.ObjectiveOptions(topk=17), W.ObjectiveOptions(bw_xfer_Bpns=0),
                    W.ObjectiveOptions(sync_rounds=2),
                    W.ObjectiveOptions(t_gap_ns=0.0), W.ObjectiveOptions(t_restart_ns=-1.0)):
            with pytest.raises(gpu.ChameleonError):
                gpu.cm_search_objective(s.ctx, scen, w.options, bad)
        best, trans, _, _, _ = gpu.cm_search_objective(s.ctx, [], w.options, W.ObjectiveOptions())
        st = gpu.cm_objective_stats(s.ctx)
        assert st["launches"] == 0
    finally:
        s.close()
