"""Pins for the readings the oracle takes where the paper prints no formula.  Every expected
value is worked by hand in the header of its fixture under ``tests/golden/``; each case is
built so that the neighbouring reading (the other stage's time, all N_dp peers, a sum instead
of a maximum, memory not doubled, the other optimal partition) gives a different number."""
import pytest

from paper_2508_21613_b200 import workloads as W

import reading_cases as R


@pytest.mark.parametrize("mode", [0, 1])
def test_rerouting_on_nonuniform_stages_with_synchronisation(oracle_factory, mode):
    n = 0
    for prof, failed, expected in R.reroute_cases():
        plan = oracle_factory(prof, R.options(mode)).search_policy(failed, W.POLICY_REROUTE)
        assert plan.feasible
        assert (plan.cost_ns if mode else plan.cost) == expected
        n += 1
    assert n == 2


@pytest.mark.parametrize("mode", [0, 1])
def test_redundant_computation_holds_the_successors_memory(oracle_factory, mode):
    n = 0
    for prof, failed, feasible in R.redundant_cases():
        o = oracle_factory(prof, R.options(mode))
        assert o.search_policy(failed, W.POLICY_REDUNDANT).feasible == feasible
        # the plain configuration itself fits either way: only the replica's share decides
        assert o.search_policy([], W.POLICY_REROUTE).feasible
        n += 1
    assert n == 4


@pytest.mark.parametrize("mode", [0, 1])
def test_minmax_partition_ties_put_surplus_layers_last(oracle_factory, mode):
    n = 0
    for prof, S, bottleneck, cuts in R.minmax_tie_cases():
        ok, got_cuts, value = oracle_factory(prof, None).minmax(S, 4, mode)
        assert ok and value == bottleneck and got_cuts == cuts
        n += 1
    assert n == 4
