"""Pins for the second execution order of the time estimator.  The paper's transition equation
(Section "Estimator") leaves the order of the computations on a stage -- f_2 -- to the
execution that is profiled; besides non-interleaved 1F1B the oracle knows the
all-forward-all-backward order.  Pinned by hand-worked values, the permutation flow-shop
closed form (identical jobs: sum of the stage times + (m-1) * the slowest stage), an
independently formulated longest-path computation, the memory rule (all m micro-batches in
flight) and brute force over the whole plan space."""
import os

import pytest

from paper_2508_21613_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GPIPE = W.SCHED_GPIPE


@pytest.fixture(scope="module")
def orc(oracle_factory):
    w = W.tiny()
    return oracle_factory(w.profile, w.options)


def _rows(name):
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [[float(x) for x in part.split()] for part in line.split("|")]


def test_handworked_gpipe_times(orc):
    n = 0
    for (S, m), F, B, xt, (expected,) in _rows("pipe_time_gpipe_handworked.txt"):
        for mode in (0, 1):
            if mode == 1 and any(x != int(x) for x in F + B + xt):
                continue
            assert orc.pipe_time(F, B, xt, int(m), mode, GPIPE) == expected
        n += 1
    assert n == 7


@pytest.mark.parametrize("mode", [0, 1])
def test_flow_shop_closed_forms(orc, mode):
    """m identical jobs through S machines in a fixed order finish at sum(p_i) + (m-1) max(p_i)
    (permutation flow shop, identical jobs).  With zero backward times the iteration is the
    forward wave plus the transfers on the way back; with zero forward times it is the backward
    wave alone."""
    rng = W.SplitMix64(11)
    for _ in range(100):
        S, m = 1 + rng.below(7), 1 + rng.below(9)
        p = [1 + rng.below(20) for _ in range(S)]
        x = [rng.below(5) for _ in range(S - 1)]
        zero = [0] * S
        wave = sum(p) + (m - 1) * max(p)
        assert orc.pipe_time(p, zero, x, m, mode, GPIPE) == wave + 2 * sum(x)
        assert orc.pipe_time(zero, p, x, m, mode, GPIPE) == wave + 2 * sum(x)
        # uniform stages: the symmetric closed form of the paper holds for this order too
        assert orc.pipe_time([p[0]] * S, [2 * p[0]] * S, [0] * S, m, mode, GPIPE) == (S + m - 1) * 3 * p[0]


def _longest_path(S, m, F, B, xt, order):
    """Pipeline time as the longest path through the DAG of the 2*S*m computations: edges 'next
    on the same stage' (per `order`) and 'depends on the neighbouring stage' (+ transfer)."""
    dur, edges = {}, []
    for i in range(S):
        seq = order(i)
        for n, (kind, j) in enumerate(seq):
            node = (kind, i, j)
            dur[node] = F[i] if kind == "F" else B[i]
            if n > 0:
                edges.append(((seq[n - 1][0], i, seq[n - 1][1]), node, 0))
            if kind == "F" and i > 0:
                edges.append((("F", i - 1, j), node, xt[i - 1]))
            if kind == "B":
                edges.append(((("B", i + 1, j), node, xt[i]) if i < S - 1 else (("F", i, j), node, 0)))
    end = dict(dur)
    for _ in range(len(dur) + 1):
        changed = False
        for a, b, wgt in edges:
            cand = end[a] + wgt + dur[b]
            if cand > end[b]:
                end[b], changed = cand, True
        if not changed:
            break
    return max(end.values())


def test_gpipe_recurrence_equals_longest_path(orc):
    rng = W.SplitMix64(78)
    for _ in range(300):
        S, m = 1 + rng.below(6), 1 + rng.below(7)
        F = [1 + rng.below(9) for _ in range(S)]
        B = [1 + rng.below(17) for _ in range(S)]
        xt = [rng.below(4) for _ in range(S)]
        want = _longest_path(S, m, F, B, xt, lambda i: [("F", j) for j in range(m)] + [("B", j) for j in range(m)])
        assert orc.pipe_time(F, B, xt, m, 0, GPIPE) == want
        assert orc.pipe_time(F, B, xt, m, 1, GPIPE) == want


def test_all_micro_batches_are_in_flight(oracle_factory):
    """Every stage has run its m forwards before its first backward: peak = static + m * act,
    whatever the stage's position (under 1F1B it is min(S - i, m))."""
    par, act = [1000, 2000, 3000], [100, 200, 300]
    prof = W.make_profile_ns(3, 2, 3, 5, [1000.0] * 3, [2000.0] * 3, act=act, param=par, opt=[6 * g for g in par],
                             p2p=0, base_cuts=[0, 1, 2, 3], cap=10**12, dev_per_node=8, bw_intra=100, bw_inter=100)
    o = oracle_factory(prof, None)
    assert o.pipe([0, 1, 2, 3], 5, [0, 1, 2], 2, 0, GPIPE)[3] == [8000 + 500, 16000 + 1000, 24000 + 1500]
    assert o.pipe([0, 1, 2, 3], 5, [0, 1, 2], 2, 0, W.SCHED_1F1B)[3] == [8000 + 300, 16000 + 400, 24000 + 300]
    assert o.pipe([0, 2, 3], 2, [0, 1], 2, 0, GPIPE)[3] == [24000 + 2 * 300, 24000 + 2 * 300]
    # the capacity threshold follows: 25500 holds the last stage of the 3-stage plan, 25499 does not
    for cap, feasible in ((25500, True), (25499, False)):
        prof.mem_capacity_bytes = cap
        assert oracle_factory(prof, None).pipe([0, 1, 2, 3], 5, [0, 1, 2], 2, 0, GPIPE)[0] == feasible
        assert oracle_factory(prof, None).pipe([0, 1, 2, 3], 5, [0, 1, 2], 2, 0, W.SCHED_1F1B)[0]


@pytest.mark.parametrize("mode", [0, 1])
def test_search_under_gpipe_equals_flat_brute_force(oracle_factory, mode):
    cases = [(W.tiny(), [3]), (W.tiny(mem_bound=True), [6])]
    cases += [(W.random_small(s, L=6, n_dp=2, n_pp=2, n_micro=3, tight_memory=bool(s % 2)), None) for s in range(3)]
    for w, failed in cases:
        if w.name.startswith("tiny"):
            w.options = W.SearchOptions(1, 3, 1, 4, W.LAYERS_FULL, W.BATCH_FULL, 1 << 62)
        opts = w.options.with_cost_mode(mode).with_schedule(GPIPE)
        o = oracle_factory(w.profile, opts)
        for f in ([failed] if failed is not None else w.scenarios[:3]):
            fast = o.search_policy(f, W.POLICY_DYNPAR)
            flat, n_flat = o.search_policy(f, W.POLICY_DYNPAR, flat=True)
            assert n_flat > 0 and fast.key() == flat.key()
            assert fast.cost == flat.cost and fast.cost_ns == flat.cost_ns


def test_the_order_changes_times_and_memory_but_not_the_candidate_space(oracle_factory):
    w = W.tiny(mem_bound=True)
    a = oracle_factory(w.profile, w.options)
    b = oracle_factory(w.profile, w.options.with_schedule(GPIPE))
    failed = [2]
    assert a.count(failed) == b.count(failed)
    ca, _, fa = a.evaluate(failed)
    cb, _, fb = b.evaluate(failed)
    assert (fb <= fa).all() and fb.sum() < fa.sum()        # more activations in flight: fewer plans fit
    both = (fa & fb).astype(bool)
    assert (ca[both] != cb[both]).any()
    # rerouting follows the order too: without a failure it is the base pipeline under that order
    w = W.tiny()
    p = w.profile
    for sched in (W.SCHED_1F1B, GPIPE):
        o = oracle_factory(p, w.options.with_schedule(sched))
        plan = o.search_policy([], W.POLICY_REROUTE)
        ok, cost, _, _ = o.pipe(list(p.base_cuts), p.n_micro, list(range(p.n_pp)), p.n_dp, 0, sched)
        assert ok and plan.feasible and plan.cost == cost
    assert (oracle_factory(p, w.options).search_policy([], W.POLICY_REROUTE).cost
            != oracle_factory(p, w.options.with_schedule(GPIPE)).search_policy([], W.POLICY_REROUTE).cost)
