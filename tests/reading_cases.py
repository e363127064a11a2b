"""Inputs of the hand-worked cases under ``tests/golden/`` that fix the readings taken where
the paper gives no formula (data rerouting on non-uniform stages, the memory of redundant
computation, ties of the min-max partition).  Only builds profiles from the fixture rows;
the expected values are the fixtures' own, derived by hand in their headers."""
import os

from paper_2508_21613_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [part.split() for part in line.split("|")]


def _options(mode):
    return W.SearchOptions(1, 2, 1, 8, W.LAYERS_REMAINDER, W.BATCH_REMAINDER, 1 << 16, mode)


def reroute_cases():
    """-> (profile, failed ids, expected cost in ns); one layer per stage, two devices per
    node so that the job spans nodes and synchronises over the slow tier (10 B/ns)."""
    for (n_pp, n_m, n_dp), fwd, bwd, grad, fcnt, (expected,) in _rows("reroute_nonuniform_handworked.txt"):
        n_pp, n_m, n_dp = int(n_pp), int(n_m), int(n_dp)
        par = [int(g) for g in grad]
        prof = W.make_profile_ns(n_pp, n_dp, n_pp, n_m, [float(x) for x in fwd], [float(x) for x in bwd],
                                 act=0, param=par, opt=[6 * g for g in par], p2p=0,
                                 base_cuts=list(range(n_pp + 1)), cap=10**15, dev_per_node=2,
                                 bw_intra=1000, bw_inter=10)
        failed = sorted(k * n_pp + stage for stage, cnt in enumerate(fcnt) for k in range(int(cnt)))
        yield prof, failed, int(expected)


def redundant_cases():
    """-> (profile, failed ids, feasible)."""
    par = [1000, 2000, 3000]
    for failed, (cap,), (feasible,) in _rows("redundant_memory_handworked.txt"):
        prof = W.make_profile_ns(3, 2, 3, 4, [1000.0, 1000.0, 1000.0], [2000.0, 2000.0, 2000.0],
                                 act=[100, 200, 300], param=par, opt=[6 * g for g in par], p2p=0,
                                 base_cuts=[0, 1, 2, 3], cap=int(cap), dev_per_node=8,
                                 bw_intra=100, bw_inter=100)
        yield prof, [int(x) for x in failed if x != "-"], bool(int(feasible))


def minmax_tie_cases():
    """-> (profile of L uniform layers of 1000 + 2000 ns, S, expected bottleneck ns, expected cuts)."""
    for (L, S), (layers,), cuts in _rows("minmax_ties_handworked.txt"):
        L, S = int(L), int(S)
        # one pipeline of S devices, so that a search restricted to (1 pipeline, S stages, min-max
        # layers, no failure) has exactly this partition as its only candidate
        prof = W.make_profile_ns(L, 1, S, 4, [1000.0] * L, [2000.0] * L, act=0, param=8, opt=48, p2p=0,
                                 base_cuts=list(range(S)) + [L], cap=10**15, dev_per_node=8,
                                 bw_intra=100, bw_inter=100)
        yield prof, S, 3000 * int(layers), [int(c) for c in cuts]


options = _options


def minmax_only_options(S, mode):
    return W.SearchOptions(1, 1, S, S, W.LAYERS_MINMAX, W.BATCH_REMAINDER, 1 << 16, mode)
