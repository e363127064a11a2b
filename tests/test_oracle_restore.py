"""Pins for the oracle's weight-transfer matching and full objective (Section "Restorer",
Weight Transfer; Section "Problem Formulation", the arg max over the next state): the
paper's worked cost entries, brute force over permutations, an independent library
solver, set arithmetic for the matrix, exact rational arithmetic for the ranking, and
invariants of the shortlist."""
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy.optimize import linear_sum_assignment

from paper_2508_21613_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden", "weight_transfer_paper_values.txt")


def _tiny_oracle(oracle_factory, mode=0):
    w = W.tiny()
    return w, oracle_factory(w.profile, w.options.with_cost_mode(mode))


def test_cost_entries_of_the_papers_worked_example(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    rows = [ln for ln in open(GOLD) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for ln in rows:
        lhs, rhs = ln.split("|")
        olo, ohi, nlo, nhi = (int(x) for x in lhs.split())
        c = o.transfer_cost_matrix([(olo, ohi)], [(nlo, nhi)], weights=[1] * 9)
        assert int(c[0, 0]) == int(rhs)


def test_whole_matrix_of_the_worked_example_and_its_matching(oracle_factory):
    # all 8 survivors of the 3 x 3 grid (device 8 failed) against the 2 x 4 plan (2,2,2,3)
    _, o = _tiny_oracle(oracle_factory)
    old = ([(0, 3), (3, 6), (6, 9)] * 3)[:8]
    new = [(0, 2), (2, 4), (4, 6), (6, 9)] * 2
    c = o.transfer_cost_matrix(old, new, weights=[1] * 9)
    # rows repeat with the old stage, columns with the new stage
    assert c[0].tolist() == [0, 1, 2, 3, 0, 1, 2, 3]     # held 0-2
    assert c[1].tolist() == [2, 1, 0, 3, 2, 1, 0, 3]     # held 3-5
    assert c[2].tolist() == [2, 2, 2, 0, 2, 2, 2, 0]     # held 6-8
    total, match = o.assign(c)
    # by hand: the two positions (6,9) go to the two holders of 6-8 (0 each); the positions (0,2)
    # go to holders of 0-2 (0 each); the positions (4,6) to holders of 3-5 (0 each); the two
    # positions (2,4) are left with one holder of 0-2 and one of 3-5, each fetching one layer
    assert total == 2
    assert sorted(match) == list(range(8))
    assert o.assign_brute(c) == 2


def test_cost_matrix_equals_set_difference(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    rng = np.random.default_rng(11)
    L = 12
    w = rng.integers(1, 1000, size=L)
    for _ in range(30):
        n = int(rng.integers(1, 7))
        def ranges():
            out = []
            for _ in range(n):
                a = int(rng.integers(0, L))
                b = int(rng.integers(a, L + 1))       # empty ranges allowed
                out.append((a, b))
            return out
        old, new = ranges(), ranges()
        c = o.transfer_cost_matrix(old, new, weights=w)
        for i, (a, b) in enumerate(old):
            for j, (x, y) in enumerate(new):
                missing = set(range(x, y)) - set(range(a, b))
                assert int(c[i, j]) == sum(int(w[l]) for l in missing)


def test_matching_equals_brute_force_over_permutations(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    rng = np.random.default_rng(5)
    for n in range(1, 9):
        for trial in range(40):
            hi = 4 if trial % 2 else 1000                 # many ties / few ties
            c = rng.integers(0, hi, size=(n, n))
            total, match = o.assign(c)
            assert total == o.assign_brute(c)
            assert sorted(match) == list(range(n))
            assert sum(int(c[match[j], j]) for j in range(n)) == total


def test_matching_equals_library_solver(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    rng = np.random.default_rng(6)
    for n, hi in ((17, 50), (64, 10**6), (100, 3), (255, 10**12), (255, 2)):
        c = rng.integers(0, hi, size=(n, n))
        total, match = o.assign(c)
        r, k = linear_sum_assignment(c)
        assert total == int(c[r, k].sum())
        assert sorted(match) == list(range(n))
        assert sum(int(c[match[j], j]) for j in range(n)) == total


def test_matching_invariants(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    rng = np.random.default_rng(7)
    c = rng.integers(0, 100, size=(9, 9))
    total, _ = o.assign(c)
    assert o.assign(c.T)[0] == total                       # rows and columns swap roles
    shifted = c.copy()
    shifted[3] += 17                                       # a row offset moves every matching alike
    assert o.assign(shifted)[0] == total + 17
    perm = rng.permutation(9)
    assert o.assign(c[perm])[0] == total                   # renaming devices changes nothing
    # a lone asymmetric entry tells rows from columns: only row 0 may take column 1 for free
    a = np.full((3, 3), 5, dtype=np.int64)
    a[0, 1] = 0
    t, match = o.assign(a)
    assert t == 10 and match[1] == 0


def test_unchanged_placement_moves_nothing(oracle_factory):
    # nobody failed and the plan is the old grid: the identity matching costs 0
    w, o = _tiny_oracle(oracle_factory)
    p = w.profile
    strategies = o.strategies(p.n_dp * p.n_pp)
    si = strategies.index((p.n_pp,) * p.n_dp)
    best = o.search_policy([], W.POLICY_DYNPAR)
    # build the identity plan by hand: the layer composition that reproduces base_cuts
    K = o.layer_count(w.options.layer_mode, p.n_pp)
    kappa = next(k for k in range(K) if o.layer_unrank(w.options.layer_mode, p.n_pp, k) == list(p.base_cuts))
    from oracle.oracle import Plan
    ident = Plan(W.POLICY_DYNPAR, True, 0.0, 0, si, p.n_dp, best.split_rank if best.strategy == si else 0,
                 (p.n_pp,) * p.n_dp, (p.n_micro,) * p.n_dp, (kappa,) * p.n_dp)
    total, match = o.plan_transfer([], ident)
    assert total == 0
    # every device keeps a position of its own old stage
    for j, u in enumerate(match):
        assert j % p.n_pp == u % p.n_pp


def test_plan_transfer_equals_library_solver_on_the_plans_matrix(oracle_factory):
    w = W.paper_scale(4, 4)
    o = oracle_factory(w.profile, w.options)
    p = w.profile
    wts = o.state_bytes()
    for failed in (w.scenarios[0], w.scenarios[40], w.scenarios[-1]):
        plan = o.search_policy(failed, W.POLICY_DYNPAR)
        total, match = o.plan_transfer(failed, plan)
        surv = [d for d in range(p.n_dp * p.n_pp) if d not in failed]
        old = [(int(p.base_cuts[d % p.n_pp]), int(p.base_cuts[d % p.n_pp + 1])) for d in surv]
        new = []
        for cuts in o.decode(failed, plan):
            new += list(zip(cuts[:-1], cuts[1:]))
        assert len(new) == len(surv)
        c = np.zeros((len(surv), len(surv)), dtype=np.int64)
        for i, (a, b) in enumerate(old):
            for j, (x, y) in enumerate(new):
                c[i, j] = sum(int(wts[l]) for l in range(x, y) if not a <= l < b)
        r, k = linear_sum_assignment(c)
        assert total == int(c[r, k].sum())
        assert sorted(match) == list(range(len(surv)))
        assert sum(int(c[match[j], j]) for j in range(len(surv))) == total


def _pairs_from_candidate_costs(o, failed, profile, opts):
    """Step time of every (strategy, split) pair from the per-candidate costs alone."""
    cost, cost_ns, feas = o.evaluate(failed)
    vals = cost_ns.astype(object) if opts.cost_mode else cost
    segs, s = [], 0
    while (d := o.segment(failed, s)) is not None:
        segs.append(d)
        s += 1
    n_surv = profile.n_dp * profile.n_pp - len(failed)
    G = profile.n_dp * profile.n_micro
    pairs = []
    order = 0
    for si, stages in enumerate(o.strategies(n_surv)):
        for beta in range(o.split_count(opts.batch_mode, G, n_surv, stages)):
            order += 1
            ok, micro = o.split_unrank(opts.batch_mode, G, n_surv, stages, beta)
            if not ok:
                continue
            T, kap = 0, []
            for p, m in enumerate(micro):
                d = next((d for d in segs if d["strategy"] == si and d["pipe"] == p and d["m"] == m), None)
                if d is None:
                    T = None
                    break
                n = d["K"] + 1 if d["K"] else 1
                good = [vals[d["first"] + k] for k in range(n) if feas[d["first"] + k]]
                if not good:
                    T = None
                    break
                T = max(T, min(good))
                kap.append((d, n))
            if T is None:
                continue
            kappa = tuple(next(k for k in range(n) if feas[d["first"] + k] and vals[d["first"] + k] <= T)
                          for d, n in kap)
            pairs.append((T, order, si, beta, tuple(micro), kappa))
    pairs.sort(key=lambda t: (t[0], t[1]))
    return pairs


@pytest.mark.parametrize("mode", [0, 1])
def test_shortlist_rederived_from_candidate_costs(oracle_factory, mode):
    w, o = _tiny_oracle(oracle_factory, mode)
    opts = w.options.with_cost_mode(mode)
    obj = W.ObjectiveOptions(topk=6)
    for failed in ([2], [7]):
        _, tr = o.search_objective(failed, obj)
        pairs = _pairs_from_candidate_costs(o, failed, w.profile, opts)
        assert len(tr.shortlist) == 6
        for plan, ref in zip(tr.shortlist, pairs):
            T, _, si, beta, micro, kappa = ref
            assert (plan.cost_ns if mode else plan.cost) == T
            assert (plan.strategy, plan.split_rank, plan.micro, plan.kappa) == (si, beta, micro, kappa)
        # the head of the shortlist is the plain search's plan
        assert tr.shortlist[0].key() == o.search_policy(failed, W.POLICY_DYNPAR).key()
        # and every shortlisted plan's transfer is the matching of that plan
        for plan, b in zip(tr.shortlist, tr.shortlist_bytes):
            assert o.plan_transfer(failed, plan)[0] == b


@pytest.mark.parametrize("mode", [0, 1])
def test_objective_ranking_in_exact_rational_arithmetic(oracle_factory, mode):
    for w in (W.tiny(), W.paper_scale(2, 2)):
        opts = w.options.with_cost_mode(mode)
        o = oracle_factory(w.profile, opts)
        for t_gap, t_restart, bw in ((1125e9, 5e9, 25), (20e9, 5e9, 1), (3e9, 5e9, 25), (1e15, 0.0, 400)):
            obj = W.ObjectiveOptions(topk=5, t_gap_ns=t_gap, t_restart_ns=t_restart, bw_xfer_Bpns=bw)
            for failed in (w.scenarios[1], w.scenarios[-1]):
                best, tr = o.search_objective(failed, obj)
                _, per = o.search(failed)
                cands = []   # (objective, policy, rank)
                for pol in (W.POLICY_REROUTE, W.POLICY_REDUNDANT):
                    if per[pol].feasible:
                        step = per[pol].cost_ns if mode else per[pol].cost
                        cands.append((Fraction(int(t_gap)) / Fraction(step), pol, -1, 0))
                for r, (plan, b) in enumerate(zip(tr.shortlist, tr.shortlist_bytes)):
                    if mode:
                        t_trans = int(t_restart) + b // bw
                        j = Fraction(int(t_gap) - t_trans, plan.cost_ns)
                    else:
                        t_trans = float(t_restart) + float(b) / float(bw)       # one rounding each, as the model
                        j = Fraction((t_gap - t_trans) / plan.cost)             # the rounded quotient ranks
                    cands.append((j, W.POLICY_DYNPAR, r, t_trans))
                top = max(c[0] for c in cands)
                first = next(c for c in cands if c[0] == top)                   # ties: policy id, then rank
                assert (tr.policy, tr.rank) == (first[1], first[2])
                assert best.policy == tr.policy
                if tr.policy == W.POLICY_DYNPAR:
                    assert best.key() == tr.shortlist[tr.rank].key()
                    assert (tr.t_trans_ns if mode else tr.t_trans) == first[3]
                    assert tr.xfer_bytes == tr.shortlist_bytes[tr.rank]
                    assert sorted(tr.assign) == list(range(tr.n_surv))
                else:
                    assert tr.xfer_bytes == 0 and tr.t_trans == 0 and tr.t_trans_ns == 0
                assert tr.objective == pytest.approx(float(top), rel=1e-12)


def test_objective_limits(oracle_factory):
    w = W.paper_scale(2, 2)
    o = oracle_factory(w.profile, w.options)
    for failed in w.scenarios[:3]:
        plain, per = o.search(failed)
        # faults far apart: the transition does not matter, the plain search's choice stands
        best, tr = o.search_objective(failed, W.ObjectiveOptions(topk=4, t_gap_ns=1e18))
        assert best.key() == plain.key()
        # faults closer together than a restart: a reconstruction never pays off
        best, tr = o.search_objective(failed, W.ObjectiveOptions(topk=4, t_gap_ns=4e9, t_restart_ns=5e9))
        assert tr.policy != W.POLICY_DYNPAR
        assert best.key() == min((p for p in per[:2] if p.feasible), key=lambda p: p.cost).key()
        # a longer gap never lowers the objective, a slower transfer never raises it
        j = [o.search_objective(failed, W.ObjectiveOptions(topk=4, t_gap_ns=g))[1].objective
             for g in (50e9, 200e9, 1125e9)]
        assert j[0] <= j[1] <= j[2]
        k = [o.search_objective(failed, W.ObjectiveOptions(topk=4, t_gap_ns=60e9, bw_xfer_Bpns=b))[1].objective
             for b in (400, 25, 1)]
        assert k[0] >= k[1] >= k[2]


# ---- asymmetric communication: rounds by greedy colouring (Section "Restorer") ----

def _stage_of(cuts_per_pipeline, L):
    out = []
    for cuts in cuts_per_pipeline:
        row = [0] * L
        for i in range(len(cuts) - 1):
            for l in range(cuts[i], cuts[i + 1]):
                row[l] = i
        out.append(row)
    return out


def test_rounds_equal_library_greedy_colouring_in_layer_order(oracle_factory):
    import networkx as nx
    _, o = _tiny_oracle(oracle_factory)
    rng = np.random.default_rng(21)
    for trial in range(60):
        L = int(rng.integers(2, 25))
        dp = int(rng.integers(1, 5))
        pipes = []
        for _ in range(dp):
            S = int(rng.integers(1, L + 1))
            inner = sorted(rng.choice(np.arange(1, L), size=S - 1, replace=False).tolist()) if S > 1 else []
            pipes.append([0] + inner + [L])
        st = _stage_of(pipes, L)
        rounds, colour, domains = o.comm_rounds(st)
        g = nx.Graph()
        g.add_nodes_from(range(L))
        for a in range(L):
            for b in range(a + 1, L):
                if any(st[p][a] == st[p][b] for p in range(dp)):
                    g.add_edge(a, b)
        ref = nx.coloring.greedy_color(g, strategy=lambda graph, colors: list(range(L)))
        assert colour == [ref[l] for l in range(L)]
        assert rounds == max(colour) + 1
        # a proper colouring, at least as many colours as the fullest device holds layers
        assert all(colour[a] != colour[b] for a, b in g.edges)
        fullest = max(max(c[i + 1] - c[i] for i in range(len(c) - 1)) for c in pipes)
        assert fullest <= rounds <= max(dict(g.degree).values(), default=0) + 1
        # domains: one per distinct cut position of any pipeline
        assert domains == len(set().union(*[set(c) for c in pipes])) - 1


def test_rounds_of_symmetric_and_shifted_layouts(oracle_factory):
    _, o = _tiny_oracle(oracle_factory)
    # symmetric: every pipeline cuts alike -> rounds = layers of the fullest stage, domains = stages
    st = _stage_of([[0, 2, 4, 6, 9]] * 3, 9)
    rounds, colour, domains = o.comm_rounds(st)
    assert (rounds, domains) == (3, 4)
    assert colour == [0, 1, 0, 1, 0, 1, 0, 1, 2]
    # by hand: 4 stages (2,2,2,2) next to 3 stages (3,3,2) over 8 layers.  Layer 2 shares a
    # device with layers 0,1 (second pipeline) and 3 (first), layer 3 with 2 and 4,5, ...
    st = _stage_of([[0, 2, 4, 6, 8], [0, 3, 6, 8]], 8)
    rounds, colour, domains = o.comm_rounds(st)
    assert colour == [0, 1, 2, 0, 1, 2, 0, 1]
    assert (rounds, domains) == (3, 5)      # domains: cut positions {0,2,3,4,6,8} -> 5 runs
    # one pipeline alone: its stages are disjoint cliques
    rounds, colour, domains = o.comm_rounds(_stage_of([[0, 1, 5, 7]], 7))
    assert (rounds, domains) == (4, 3) and colour == [0, 0, 1, 2, 3, 0, 1]


@pytest.mark.parametrize("mode", [0, 1])
def test_async_step_time_by_hand_composition(oracle_factory, mode):
    w = W.paper_scale(2, 2)
    opts = w.options.with_cost_mode(mode)
    o = oracle_factory(w.profile, opts)
    p = w.profile
    for failed in (w.scenarios[3], w.scenarios[-1]):
        plan = o.search_policy(failed, W.POLICY_DYNPAR)
        step, rounds, domains, t_sync = o.plan_async_step(failed, plan)
        cuts = o.decode(failed, plan)
        surv = [d for d in range(p.n_dp * p.n_pp) if d not in failed]
        # slowest bare pipeline (one participant: no synchronisation term)
        off, t_pipe = 0, 0
        for q in range(plan.n_pipes):
            ok, c, c_ns, _ = o.pipe(cuts[q], plan.micro[q], surv[off:off + plan.stages[q]], 1, mode)
            assert ok
            t_pipe = max(t_pipe, c_ns if mode else c)
            off += plan.stages[q]
        r2, colour, d2 = o.comm_rounds(_stage_of(cuts, p.L))
        assert (rounds, domains) == (r2, d2)
        n = plan.n_pipes
        bw = p.bw_inter_Bpns if p.n_dp * p.n_pp > p.devices_per_node else p.bw_intra_Bpns
        total = 0
        for c in range(r2):
            sizes = [int(p.param_bytes[l]) for l in range(p.L) if colour[l] == c]
            big = max(sizes)
            total = total + ((2 * (n - 1) * big) // (n * bw) if mode else ((2.0 * (n - 1)) * big) / (float(n) * bw))
        assert t_sync == total
        assert step == t_pipe + total
        if mode:   # uniform layers: the rounds cost exactly rounds x one layer's all-reduce
            one = (2 * (n - 1) * int(p.param_bytes[0])) // (n * bw)
            assert len(set(int(x) for x in p.param_bytes)) == 1 and t_sync == rounds * one


@pytest.mark.parametrize("mode", [0, 1])
def test_objective_with_sync_rounds_ranks_by_the_async_step(oracle_factory, mode):
    w = W.paper_scale(2, 2)
    opts = w.options.with_cost_mode(mode)
    o = oracle_factory(w.profile, opts)
    obj0 = W.ObjectiveOptions(topk=6)
    obj1 = W.ObjectiveOptions(topk=6, sync_rounds=1)
    for failed in (w.scenarios[0], w.scenarios[7], w.scenarios[-2]):
        _, t0 = o.search_objective(failed, obj0)
        best, t1 = o.search_objective(failed, obj1)
        _, per = o.search(failed)
        assert [p.key() for p in t0.shortlist] == [p.key() for p in t1.shortlist]     # same shortlist
        assert t0.shortlist_bytes == t1.shortlist_bytes
        cands = []
        for pol in (W.POLICY_REROUTE, W.POLICY_REDUNDANT):
            if per[pol].feasible:
                cands.append((Fraction(int(obj1.t_gap_ns)) / Fraction(per[pol].cost_ns if mode else per[pol].cost), pol, -1))
        for r, (plan, b) in enumerate(zip(t1.shortlist, t1.shortlist_bytes)):
            step, rounds, _, _ = o.plan_async_step(failed, t0.shortlist[r])
            assert (plan.cost_ns if mode else plan.cost) == step and t1.shortlist_rounds[r] == rounds
            if mode:
                j = Fraction(int(obj1.t_gap_ns) - (int(obj1.t_restart_ns) + b // obj1.bw_xfer_Bpns), plan.cost_ns)
            else:
                j = Fraction((obj1.t_gap_ns - (obj1.t_restart_ns + float(b) / float(obj1.bw_xfer_Bpns))) / plan.cost)
            cands.append((j, W.POLICY_DYNPAR, r))
        top = max(c[0] for c in cands)
        first = next(c for c in cands if c[0] == top)
        assert (t1.policy, t1.rank) == (first[1], first[2])
        if t1.policy == W.POLICY_DYNPAR:
            assert best.key() == t1.shortlist[t1.rank].key()
            assert t1.rounds == t1.shortlist_rounds[t1.rank] and t1.rounds >= 1
