"""Pins for the oracle's time estimator (Section "Estimator"): values worked by hand,
the symmetric closed form, an independently formulated longest-path computation, the
data-rerouting formulas as printed, and invariants."""
import itertools
import math
import os

import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _uniform_profile(L, n_dp, n_pp, n_micro, tf, tb, act=0, param=0, p2p=0, cap=10**15):
    base = [i * (L // n_pp) for i in range(n_pp + 1)]
    return W.make_profile_ns(L, n_dp, n_pp, n_micro, [float(tf)] * L, [float(tb)] * L, act, param,
                             6 * param, p2p, base, cap, 8, 100, 100)


@pytest.fixture(scope="module")
def orc(oracle_factory):
    w = W.tiny()
    return oracle_factory(w.profile, w.options)


def _rows(name):
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [[float(x) for x in part.split()] for part in line.split("|")]


def test_handworked_pipeline_times(orc):
    n = 0
    for (S, m), F, B, xt, (expected,) in _rows("pipe_time_handworked.txt"):
        for mode in (0, 1):
            if mode == 1 and any(x != int(x) for x in F + B + xt):
                continue
            assert orc.pipe_time(F, B, xt, int(m), mode) == expected
        n += 1
    assert n >= 10


@pytest.mark.parametrize("mode", [0, 1])
def test_uniform_pipeline_matches_symmetric_closed_form(orc, mode):
    # (N_pp + N_m - 1)(T_f + T_b), Section "Estimator"; also holds when N_m < N_pp
    for S in range(1, 7):
        for m in range(1, 10):
            for tf, tb in ((1, 2), (3, 5), (7, 7)):
                got = orc.pipe_time([tf] * S, [tb] * S, [0] * S, m, mode)
                assert got == (S + m - 1) * (tf + tb)


def _longest_path_time(S, m, F, B, xt):
    """Independent formulation: the pipeline time is the longest path through the DAG whose
    nodes are the 2*S*m computations (weight = duration) and whose edges are 'next on the
    same stage' (weight 0) and 'depends on neighbour stage' (weight = transfer time).
    Solved by repeated relaxation over an explicit edge list."""
    order = {}
    for i in range(S):
        w = min(S - 1 - i, m)
        seq = [("F", j) for j in range(w)]
        for k in range(m - w):
            seq += [("F", w + k), ("B", k)]
        seq += [("B", j) for j in range(m - w, m)]
        order[i] = seq
    dur = {}
    edges = []
    for i in range(S):
        for n, (kind, j) in enumerate(order[i]):
            node = (kind, i, j)
            dur[node] = F[i] if kind == "F" else B[i]
            if n > 0:
                pk, pj = order[i][n - 1]
                edges.append(((pk, i, pj), node, 0.0))
            if kind == "F" and i > 0:
                edges.append((("F", i - 1, j), node, xt[i - 1]))
            if kind == "B":
                if i < S - 1:
                    edges.append((("B", i + 1, j), node, xt[i]))
                else:
                    edges.append((("F", i, j), node, 0.0))
    end = {node: dur[node] for node in dur}
    for _ in range(len(dur) + 1):
        changed = False
        for a, b, wgt in edges:
            cand = end[a] + wgt + dur[b]
            if cand > end[b]:
                end[b] = cand
                changed = True
        if not changed:
            break
    return max(end.values())


def test_recurrence_equals_longest_path_on_random_small_pipelines(orc):
    rng = W.SplitMix64(77)
    for _ in range(300):
        S = 1 + rng.below(6)
        m = 1 + rng.below(7)
        # small integers: every sum is exact, so the two formulations must agree exactly
        F = [1 + rng.below(9) for _ in range(S)]
        B = [1 + rng.below(17) for _ in range(S)]
        xt = [rng.below(4) for _ in range(S)]
        expect = _longest_path_time(S, m, F, B, xt)
        assert orc.pipe_time(F, B, xt, m, 0) == expect
        assert orc.pipe_time(F, B, xt, m, 1) == expect


def test_pipeline_time_is_monotone_and_respects_path_bounds(orc):
    rng = W.SplitMix64(5)
    for _ in range(200):
        S = 1 + rng.below(7)
        m = 1 + rng.below(9)
        F = [rng.uniform(0.5, 3.0) for _ in range(S)]
        B = [rng.uniform(0.5, 6.0) for _ in range(S)]
        xt = [rng.uniform(0.0, 0.7) for _ in range(S)]
        t = orc.pipe_time(F, B, xt, m)
        i = rng.below(S)
        for arr in (F, B, xt):
            bumped = list(arr)
            bumped[i] += 0.25
            args = [F, B, xt]
            args[[id(F), id(B), id(xt)].index(id(arr))] = bumped
            assert orc.pipe_time(args[0], args[1], args[2], m) >= t
        # every stage must run its m forwards and backwards after the forwards before it
        for b in range(S):
            bound = m * (F[b] + B[b]) + sum(F[:b])
            assert t >= bound * (1 - 1e-12)
        # one micro-batch goes up and down the whole pipeline
        assert t >= (sum(F) + sum(B)) * (1 - 1e-12)


def test_single_stage_runs_back_to_back(orc):
    assert orc.pipe_time([3.5], [7.25], [0.0], 6) == 6 * (3.5 + 7.25)


def _reroute_cases():
    for (n_pp, n_m, n_dp, tf, tb), Fcnt, (expected,) in _rows("reroute_paper_values.txt"):
        yield int(n_pp), int(n_m), int(n_dp), tf, tb, [int(x) for x in Fcnt], expected


@pytest.mark.parametrize("mode", [0, 1])
def test_rerouting_matches_the_printed_formulas(oracle_factory, mode):
    for n_pp, n_m, n_dp, tf, tb, Fcnt, expected in _reroute_cases():
        prof = _uniform_profile(n_pp, n_dp, n_pp, n_m, tf, tb)
        opts = W.SearchOptions(1, 2, 1, 8, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 16, mode)
        o = oracle_factory(prof, opts)
        failed = []
        for stage, cnt in enumerate(Fcnt):
            failed += [k * n_pp + stage for k in range(cnt)]
        plan = o.search_policy(sorted(failed), W.POLICY_REROUTE)
        assert plan.feasible
        got = plan.cost_ns if mode else plan.cost
        if mode:
            assert got == math.floor(expected)  # every quotient floors in integer mode
        else:
            assert got == pytest.approx(expected, rel=1e-14)


def test_rerouting_unrecoverable_when_a_stage_loses_all_peers(oracle_factory):
    prof = _uniform_profile(4, 2, 4, 8, 1, 2)
    opts = W.SearchOptions(1, 2, 1, 8, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 16)
    o = oracle_factory(prof, opts)
    assert o.search_policy([1], W.POLICY_REROUTE).feasible
    assert not o.search_policy([1, 5], W.POLICY_REROUTE).feasible  # stage 1 of both pipelines


@pytest.mark.parametrize("mode", [0, 1])
def test_no_failure_rerouting_equals_baseline_pipeline(oracle_factory, mode):
    for w in (W.tiny(), W.paper_scale(0, 0), W.random_small(3)):
        o = oracle_factory(w.profile, w.options.with_cost_mode(mode))
        p = w.profile
        plan = o.search_policy([], W.POLICY_REROUTE)
        ok, cost, cost_ns, _ = o.pipe(list(p.base_cuts), p.n_micro, list(range(p.n_pp)), p.n_dp, mode)
        assert ok and plan.feasible
        assert (plan.cost_ns == cost_ns) if mode else (plan.cost == cost)


def test_integer_and_double_builds_agree_on_integer_inputs(oracle_factory):
    # integer nanoseconds, bandwidths that divide the bytes: both builds are exact
    L, n_pp, n_dp, n_m = 12, 4, 3, 6
    rng = W.SplitMix64(123)
    fwd = [float(1000 + rng.below(500)) for _ in range(L)]
    bwd = [float(2000 + rng.below(900)) for _ in range(L)]
    prof = W.make_profile_ns(L, n_dp, n_pp, n_m, fwd, bwd, act=1 << 20, param=3 * (1 << 22),
                           opt=6 * 3 * (1 << 22), p2p=1 << 16, base_cuts=[0, 3, 6, 9, 12],
                           cap=10**12, dev_per_node=4, bw_intra=64, bw_inter=16)
    assert np.array_equal(prof.fwd_ns, prof.fwd_ns_i.astype(np.float64))
    for cuts in ([0, 3, 6, 9, 12], [0, 1, 5, 6, 12], [0, 6, 12]):
        S = len(cuts) - 1
        devs = list(range(2, 2 + S))
        for n_sync in (1, 3):
            # 2(n-1)G/(n bw) with n=3, G a multiple of 3*2^22, bw=16: exact in both
            a = oracle_factory(prof, None).pipe(cuts, n_m, devs, n_sync, 0)
            b = oracle_factory(prof, None).pipe(cuts, n_m, devs, n_sync, 1)
            assert a[0] and b[0]
            assert a[1] == float(b[2])


@pytest.mark.parametrize("mode", [0, 1])
def test_transfer_and_sync_terms_on_a_two_stage_pipeline(oracle_factory, mode):
    """S=2, m=1 has a single path: F0, transfer, F1, B1, transfer, B0 -- so the pipeline
    time is their plain sum, and the step adds the slower stage's gradient all-reduce
    (ring lower bound 2(n-1)/n * bytes / bandwidth, a textbook figure).  Pins that the
    transfer is paid in both directions, that the link tier follows the two devices'
    nodes, and which bandwidth the synchronisation uses."""
    L, dpn = 4, 4
    fwd = [1000.0, 3000.0, 5000.0, 7000.0]
    bwd = [2000.0, 6000.0, 10000.0, 14000.0]
    par = [4 * 3 * 5 * 1000, 8 * 3 * 5 * 1000, 1000 * 3 * 5, 1000 * 3 * 5]
    p2p = [0, 600 * 20 * 7, 0, 0]                      # the cut sits after layer 1
    prof = W.make_profile_ns(L, 3, 2, 1, fwd, bwd, 0, par, [6 * v for v in par], p2p, [0, 2, 4],
                             10**15, dpn, 600, 20)
    o = oracle_factory(prof, None)
    F0, F1, B0, B1 = 4000.0, 12000.0, 8000.0, 24000.0
    g0 = par[0] + par[1]                               # stage 0 holds the larger gradients
    for devs, bw in (([0, 1], 600), ([3, 4], 20), ([4, 3], 20), ([5, 6], 600)):
        xt = p2p[1] / bw                               # exact: 600*20*7 divides by both tiers
        for n_sync in (1, 3):
            # 6 devices > 4 per node: the job spans nodes, sync runs on the inter-node tier
            sync = 0.0 if n_sync == 1 else 2 * (n_sync - 1) * g0 / (n_sync * 20)
            assert sync == int(sync)
            ok, cost, cost_ns, _ = o.pipe([0, 2, 4], 1, devs, n_sync, mode)
            want = F0 + xt + F1 + B1 + xt + B0 + sync
            assert ok and (cost_ns == int(want) if mode else cost == want)
    # a job inside one node synchronises over the intra-node tier
    prof1 = W.make_profile_ns(L, 2, 2, 1, fwd, bwd, 0, par, [6 * v for v in par], p2p, [0, 2, 4],
                              10**15, dpn, 600, 20)
    ok, cost, cost_ns, _ = oracle_factory(prof1, None).pipe([0, 2, 4], 1, [0, 1], 2, mode)
    want = F0 + F1 + B1 + B0 + 2 * p2p[1] / 600 + 2 * 1 * g0 / (2 * 600)
    assert ok and (cost_ns == int(want) if mode else cost == want)
