"""Pins for the oracle's candidate space (Section "Planner", Algorithm 1) and memory
estimator (Section "Estimator"): the paper's worked examples, closed forms, brute force
on tiny inputs and invariants."""
import itertools
import math

import numpy as np
import pytest

from paper_2508_21613_b200 import workloads as W


@pytest.fixture(scope="module")
def orc(oracle_factory):
    w = W.tiny()
    return oracle_factory(w.profile, w.options)


# ---------------------------------------------------------------- combinatorics

def test_binomials_against_math_comb(orc):
    for n in range(0, 70):
        for k in range(0, n + 2):
            want = math.comb(n, k)
            assert orc.binom(n, k) == min(want, 2**64 - 1)
    assert orc.binom(127, 63) == 2**64 - 1          # saturates
    assert orc.binom(1023, 3) == math.comb(1023, 3)


def test_subset_unranking_is_the_colex_bijection(orc):
    for n, t in ((6, 0), (6, 1), (7, 3), (9, 4), (8, 8), (12, 5)):
        K = math.comb(n, t)
        seen = []
        for rank in range(K):
            c = orc.unrank_subset(rank, t)
            assert len(c) == t and all(0 <= x < n for x in c)
            assert all(c[i] < c[i + 1] for i in range(t - 1))
            assert orc.rank_subset(c) == rank
            seen.append(tuple(reversed(c)))   # colex = lexicographic on the reversed tuple
        assert seen == sorted(seen)
        assert len(set(seen)) == K
        if t:
            assert orc.unrank_subset(0, t) == list(range(t))


def _partitions(n, parts, lo, hi, minimum=None):
    """Independent recursive generator of non-decreasing tuples."""
    minimum = lo if minimum is None else minimum
    if parts == 0:
        if n == 0:
            yield ()
        return
    for first in range(minimum, hi + 1):
        if first * parts > n:
            break
        for rest in _partitions(n - first, parts - 1, lo, hi, first):
            yield (first,) + rest


def test_strategies_cover_the_papers_examples_and_match_a_partition_counter(oracle_factory):
    # Section "Memory Analysis": 8 cards DP4 x PP2, one failure -> pipelines [2, 2, 3]
    prof = W.make_profile_ns(8, 4, 2, 4, 1.0, 2.0, 0, 0, 0, 0, [0, 4, 8], 10**15, 8, 1, 1)
    o = oracle_factory(prof, W.SearchOptions(3, 5, 1, 4, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 16))
    assert (2, 2, 3) in o.strategies(7)
    # Section "Restorer", weight transfer: DP3 x PP3 with 9 layers, one failure -> DP2 x PP4
    prof = W.make_profile_ns(9, 3, 3, 4, 1.0, 2.0, 0, 0, 0, 0, [0, 3, 6, 9], 10**15, 8, 1, 1)
    o = oracle_factory(prof, W.SearchOptions(2, 4, 1, 9, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 16))
    assert (4, 4) in o.strategies(8)
    cuts = [o.layer_unrank(W.LAYERS_REMAINDER, 4, k) for k in range(o.layer_count(W.LAYERS_REMAINDER, 4))]
    assert [0, 2, 4, 6, 9] in cuts                       # layers (2,2,2,3) is a candidate
    # every window: same list as an independent generator, all survivors used
    for n_surv, (dlo, dhi, plo, phi), L in ((7, (1, 7, 1, 8), 8), (31, (3, 5, 4, 12), 32),
                                            (255, (7, 9, 30, 34), 96), (60, (1, 3, 16, 48), 80),
                                            (13, (2, 3, 2, 9), 6)):
        prof = W.make_profile_ns(L, 2, 2, 4, 1.0, 2.0, 0, 0, 0, 0, [0, L // 2, L], 10**15, 8, 1, 1)
        o = oracle_factory(prof, W.SearchOptions(dlo, dhi, plo, phi, 1, 1, 1 << 16))
        got = o.strategies(n_surv)
        want = [t for dp in range(dlo, dhi + 1) for t in _partitions(n_surv, dp, plo, min(phi, L))]
        assert got == want
        assert all(sum(t) == n_surv for t in got)


def _paper_batch_rule(G, stages):
    """Section "Planner", batch distribution, restated independently: pre-allocate in
    proportion to the nodes, then hand the leftovers out one by one."""
    n = sum(stages)
    m = [G * s // n for s in stages]
    p = 0
    while sum(m) < G:
        m[p % len(m)] += 1
        p += 1
    return m


def test_batch_split_invariants(orc):
    for G, stages in ((16, (3, 4)), (128, (7, 8, 8, 8)), (128, (4, 4, 5, 6, 12)), (1024, (30,) * 3 + (32,) * 5),
                      (16, (1, 1, 1, 1, 1, 2)), (5, (1, 6))):
        n = sum(stages)
        for mode in (W.BATCH_REMAINDER, W.BATCH_FULL):
            cnt = orc.split_count(mode, G, n, stages)
            if mode == W.BATCH_FULL:
                assert cnt == math.comb(G - 1, len(stages) - 1)
                if cnt > 20000:
                    continue
            seen = set()
            for beta in range(cnt):
                ok, m = orc.split_unrank(mode, G, n, stages, beta)
                assert sum(m) == G                       # Definition 1 (iii)
                assert ok == all(x >= 1 for x in m)      # no pipeline left idle
                seen.add(tuple(m))
            assert len(seen) == cnt
            if mode == W.BATCH_REMAINDER:
                assert orc.split_unrank(mode, G, n, stages, 0)[1] == _paper_batch_rule(G, stages)
            else:
                want = {c for c in itertools.product(range(1, G + 1), repeat=len(stages)) if sum(c) == G} \
                    if G <= 16 and len(stages) <= 3 else None
                if want is not None:
                    assert seen == want


def test_layer_compositions(oracle_factory):
    for L in (8, 9, 32, 80, 96):
        prof = W.make_profile_ns(L, 2, 2, 4, 1.0, 2.0, 0, 0, 0, 0, [0, L // 2, L], 10**15, 8, 1, 1)
        o = oracle_factory(prof, None)
        for S in range(1, min(L, 12) + 1):
            K = o.layer_count(W.LAYERS_REMAINDER, S)
            assert K == math.comb(S, L % S)          # Section "Planner": C(N_pp, r) placements
            if K <= 5000:
                seen = set()
                for k in range(K):
                    cuts = o.layer_unrank(W.LAYERS_REMAINDER, S, k)
                    n = np.diff(cuts)
                    assert cuts[0] == 0 and cuts[-1] == L
                    assert set(n) <= {L // S, L // S + 1} and n.min() >= 1
                    seen.add(tuple(cuts))
                assert len(seen) == K
            Kf = o.layer_count(W.LAYERS_FULL, S)
            assert Kf == math.comb(L - 1, S - 1)
            if Kf <= 5000:
                seen = set()
                for k in range(Kf):
                    cuts = o.layer_unrank(W.LAYERS_FULL, S, k)
                    assert cuts[0] == 0 and cuts[-1] == L and all(np.diff(cuts) >= 1)
                    seen.add(tuple(cuts))
                assert len(seen) == Kf


# --------------------------------------------------------------------- memory

def test_peak_memory_closed_form_and_capacity_threshold(oracle_factory):
    # M_peak,i = N_l (m_p + m_o + m_g) + (N_pp - i) N_l m_a with m_g = m_p (Section "Estimator")
    L, S, m = 12, 4, 8
    m_p, m_a = 50_000_000, 8_000_000
    m_o = 6 * m_p
    cuts = [0, 2, 5, 9, 12]
    want = [(cuts[i + 1] - cuts[i]) * (m_p + m_o + m_p) + (S - i) * (cuts[i + 1] - cuts[i]) * m_a
            for i in range(S)]
    prof = W.make_profile_ns(L, 2, S, m, 1.0, 2.0, m_a, m_p, m_o, 0, [0, 3, 6, 9, 12], max(want), 8, 1, 1)
    o = oracle_factory(prof, None)
    for mode in (0, 1):
        ok, _, _, peak = o.pipe(cuts, m, [0, 1, 2, 3], 2, mode)
        assert peak == want and ok                      # exactly at capacity still fits
    prof.mem_capacity_bytes = max(want) - 1
    o = oracle_factory(prof, None)
    for mode in (0, 1):
        ok, cost, cost_ns, _ = o.pipe(cuts, m, [0, 1, 2, 3], 2, mode)
        assert not ok and cost == math.inf and cost_ns == 2**63 - 1
    # fewer micro-batches than stages: at most m activations are ever in flight
    ok, _, _, peak = oracle_factory(prof, None).pipe(cuts, 2, [0, 1, 2, 3], 2)
    assert peak[0] == 2 * (m_p + m_o + m_p) + 2 * 2 * m_a
    # more layers in a stage never lowers its peak
    p2 = oracle_factory(prof, None).pipe([0, 3, 5, 9, 12], m, [0, 1, 2, 3], 2)[3]
    assert p2[0] > want[0] and p2[1] < want[1]


# ----------------------------------------------------------- min-max partition

def _brute_minmax(prof, S, m, mode):
    L = prof.L
    f = prof.fwd_ns_i if mode else prof.fwd_ns
    b = prof.bwd_ns_i if mode else prof.bwd_ns
    PF = [0]
    PB = [0]
    for l in range(L):
        PF.append(PF[-1] + (int(f[l]) if mode else float(f[l])))
        PB.append(PB[-1] + (int(b[l]) if mode else float(b[l])))
    best = None
    for inner in itertools.combinations(range(1, L), S - 1):
        cuts = (0,) + inner + (L,)
        ok = True
        worst = 0
        for i in range(S):
            lo, hi = cuts[i], cuts[i + 1]
            stat = 2 * int(prof.param_bytes[lo:hi].sum()) + int(prof.opt_bytes[lo:hi].sum())
            peak = stat + min(S - i, m) * int(prof.act_bytes[lo:hi].sum())
            if peak > prof.mem_capacity_bytes:
                ok = False
                break
            worst = max(worst, (PF[hi] - PF[lo]) + (PB[hi] - PB[lo]))
        if ok and (best is None or worst < best):
            best = worst
    return best


def _bottleneck(prof, cuts, mode):
    f = prof.fwd_ns_i if mode else prof.fwd_ns
    b = prof.bwd_ns_i if mode else prof.bwd_ns
    PF, PB = [0], [0]
    for l in range(prof.L):
        PF.append(PF[-1] + (int(f[l]) if mode else float(f[l])))
        PB.append(PB[-1] + (int(b[l]) if mode else float(b[l])))
    return max((PF[hi] - PF[lo]) + (PB[hi] - PB[lo]) for lo, hi in zip(cuts[:-1], cuts[1:]))


@pytest.mark.parametrize("mode", [0, 1])
def test_minmax_partition_against_brute_force(oracle_factory, mode):
    checked_infeasible = 0
    for seed in range(12):
        for tight in (False, True):
            w = W.random_small(seed, L=6 + seed % 5, tight_memory=tight)
            o = oracle_factory(w.profile, w.options)
            for S in range(1, 6):
                for m in (1, 3, 7):
                    ok, cuts, val = o.minmax(S, m, mode)
                    want = _brute_minmax(w.profile, S, m, mode)
                    assert ok == (want is not None)
                    if not ok:
                        checked_infeasible += 1
                        continue
                    assert val == want                          # same bottleneck, exactly
                    assert _bottleneck(w.profile, cuts, mode) == want   # and the partition attains it
                    feasible, _, _, peak = o.pipe(cuts, m, list(range(S)), 1, mode)
                    assert feasible and max(peak) <= w.profile.mem_capacity_bytes
                    assert cuts[0] == 0 and cuts[-1] == w.profile.L and all(np.diff(cuts) >= 1)
    assert checked_infeasible > 0                               # the memory cap did bind somewhere
