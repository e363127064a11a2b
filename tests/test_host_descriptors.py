"""The host-side descriptor builder of the CUDA library (strategies, micro-batch splits,
segments, candidate counts, survivor placement) against the oracle's own enumeration, on the
CPU: ``cm_host_describe`` makes no CUDA call, so these run without a GPU."""
import math

import pytest

from paper_2508_21613_b200 import workloads as W


@pytest.fixture(scope="module")
def lib():
    from paper_2508_21613_b200 import binding, build
    build.build()
    return binding


def _node_crossings(profile, failed):
    surv = [d for d in range(profile.n_dp * profile.n_pp) if d not in failed]
    return sum(1 for a, b in zip(surv[:-1], surv[1:]) if a // profile.devices_per_node != b // profile.devices_per_node)


@pytest.mark.parametrize("name", ["tiny", "paper-scale", "70b-like", "175b-like", "sweep"])
def test_candidate_strategy_and_segment_counts_equal_the_oracles(lib, oracle_factory, name):
    w = W.ALL_WORKLOADS[name]()
    o = oracle_factory(w.profile, w.options)
    step = max(1, len(w.scenarios) // 12)
    for failed in w.scenarios[::step][:12] + [[]]:
        got = lib.cm_host_describe(w.profile, failed, w.options)
        n, n_strat, n_seg = o.count(failed)
        assert (got["candidates"], got["strategies"], got["segments"]) == (n, n_strat, n_seg), (name, failed)
        assert got["survivors"] == w.profile.n_dp * w.profile.n_pp - len(failed)
        assert got["node_crossings"] == _node_crossings(w.profile, failed)
        # (strategy, split) pairs: re-counted from the oracle's strategies and split counts
        G = w.profile.n_dp * w.profile.n_micro
        pairs = sum(o.split_count(w.options.batch_mode, G, got["survivors"], st) for st in o.strategies(got["survivors"]))
        assert got["splits"] == pairs
        assert 1 <= got["launch_classes"] <= got["buckets"] <= max(got["segments"], 1)


def test_counts_on_random_small_workloads_in_every_mode(lib, oracle_factory):
    for seed in range(10):
        w = W.random_small(seed, L=5 + seed % 6, n_dp=2 + seed % 3, n_pp=2 + seed % 3, n_micro=2 + seed % 4)
        for lm in (W.LAYERS_FULL, W.LAYERS_REMAINDER, W.LAYERS_MINMAX):
            for bm in (W.BATCH_FULL, W.BATCH_REMAINDER):
                opts = W.SearchOptions(1, 5, 1, 6, lm, bm, [1 << 62, 5][seed % 2])
                o = oracle_factory(w.profile, opts)
                for failed in w.scenarios[:4]:
                    got = lib.cm_host_describe(w.profile, failed, opts)
                    n, n_strat, n_seg = o.count(failed, opts)
                    assert (got["candidates"], got["strategies"], got["segments"]) == (n, n_strat, n_seg), (seed, lm, bm, failed)


def test_host_describe_rejects_what_the_search_rejects(lib):
    w = W.tiny()
    for bad in ([8], [1, 1]):
        with pytest.raises(lib.ChameleonError):
            lib.cm_host_describe(w.profile, bad, w.options)
    wide = W.SearchOptions(1, 17, 1, 8, W.LAYERS_FULL, W.BATCH_FULL, 1 << 62)       # dp_hi above CM_MAX_PIPES
    with pytest.raises(lib.ChameleonError):
        lib.cm_host_describe(w.profile, [0], wide)
    # a space whose candidate count does not fit the index type is refused, not wrapped
    big = W.gpt175b_like()
    opts = W.SearchOptions(7, 9, 30, 34, W.LAYERS_FULL, W.BATCH_FULL, 1 << 63)
    with pytest.raises(lib.ChameleonError) as e:
        lib.cm_host_describe(big.profile, [3], opts)
    assert e.value.args[0] == lib.CM_EOVERFLOW or "overflow" in str(e.value)
