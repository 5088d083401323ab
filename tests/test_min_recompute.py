"""Least recomputation under a memory budget (plan(sizes, costs) -> checkpoint set): among the sets whose Eq. (memory)
value fits the budget - by default the optimum of Algorithms 5/6, which many sets reach - the one whose non-checkpoint
units are cheapest to run again in the backward pass of Algorithm 4.  The oracle's enumeration is pinned by a hand
example, a closed form on uniform chains and monotonicity; the library's search is compared with the enumeration."""
import random

import numpy as np
import pytest

from oracle import planner_oracle as po
from paper_2502_12499_b200 import binding as ck


# ------------------------------------------------------------------------------------------------ oracle pins

def test_hand_example():
    # d = 1, 2, 3, 4: Eq. (memory) gives {0,3} -> 5 + 5 + 3 = 13, {0,1,3} -> 13, {0,2,3} -> max(8, 11) = 11, all -> 13.
    d, cost = [1, 2, 3, 4], [0, 5, 1, 0]
    assert [po.eval_dynamic(d, C) for C in ([0, 3], [0, 1, 3], [0, 2, 3], [0, 1, 2, 3])] == [13, 13, 11, 13]
    assert po.brute_force_min_recompute(d, cost, 10) is None
    for budget in (11, 12):
        got = po.brute_force_min_recompute(d, cost, budget)
        assert got["set"] == [0, 2, 3] and got["cost"] == 5 and got["feasible_sets"] == 1
    got = po.brute_force_min_recompute(d, cost, 13)
    assert got["cost"] == 0 and got["set"] == [0, 1, 2, 3] and got["feasible_sets"] == 4
    assert po.recompute_cost(cost, [0, 3]) == 6 and po.recompute_cost(cost, [0, 1, 3]) == 1


def uniform_min_noncheckpoints(n, P):
    """Uniform chain (every d = 1) under budget P: the p-th checkpoint after d_0 may end a segment of at most P - 2 - p
    tensors (Eq. (memory): 1 + p checkpoints, the segment, one gradient buffer), so K checkpoints cover the chain iff
    n - K <= K (P - 2) - K (K + 1) / 2 and K <= P - 2; the fewest non-checkpoints are n - max K."""
    best = None
    for K in range(1, min(n, P - 2) + 1):
        if n - K <= K * (P - 2) - K * (K + 1) // 2:
            best = K
    return None if best is None else n - best


def test_uniform_chain_closed_form():
    for n in range(2, 11):
        d, cost = [1] * (n + 1), [0] + [1] * n
        optimum = po.brute_force_dynamic(d)["value"]
        for P in range(optimum - 1, n + 4):
            got = po.brute_force_min_recompute(d, cost, P)
            want = uniform_min_noncheckpoints(n, P)
            assert (got is None) == (want is None), (n, P)
            if got is not None:
                assert got["cost"] == want, (n, P)


def test_monotone_in_the_budget_and_consistent_with_the_optimum():
    rng = random.Random(11)
    for _ in range(60):
        n = rng.randint(2, 9)
        d = [rng.randint(1, 30) for _ in range(n + 1)]
        cost = [0] + [rng.randint(0, 20) for _ in range(n)]
        bf = po.brute_force_dynamic(d)
        assert po.brute_force_min_recompute(d, cost, bf["value"] - 1) is None
        at_optimum = po.brute_force_min_recompute(d, cost, bf["value"])
        assert at_optimum["peak"] == bf["value"]
        assert at_optimum["cost"] <= po.recompute_cost(cost, bf["set"])
        assert at_optimum["cost"] == po.recompute_cost(cost, at_optimum["set"])
        everything = po.eval_dynamic(d, list(range(n + 1)))
        assert po.brute_force_min_recompute(d, cost, everything)["cost"] == 0
        last = None
        for budget in range(bf["value"], everything + 1, max(1, (everything - bf["value"]) // 7)):
            c = po.brute_force_min_recompute(d, cost, budget)["cost"]
            assert last is None or c <= last
            last = c


# ------------------------------------------------------------------------------------------------ library vs oracle

def test_library_equals_enumeration():
    rng = random.Random(12)
    for trial in range(200):
        n = rng.randint(1, 10)
        d = [rng.randint(1, 40) for _ in range(n + 1)]
        cost = [0] + [rng.randint(0, 25) for _ in range(n)]
        optimum = po.brute_force_dynamic(d)["value"]
        everything = po.eval_dynamic(d, list(range(n + 1)))
        for budget in {0, optimum, optimum + rng.randint(0, 30), (optimum + everything) // 2, everything}:
            want = po.brute_force_min_recompute(d, cost, optimum if budget == 0 else budget)
            mask, peak, rec = ck.plan_min_recompute(d, cost, budget)
            C = [int(i) for i in np.nonzero(mask)[0]]
            assert rec == want["cost"], (d, cost, budget)
            assert po.recompute_cost(cost, C) == rec
            assert peak == po.eval_dynamic(d, C) <= (optimum if budget == 0 else budget)
        if n >= 2:
            with pytest.raises(ck.CkptError) as e:
                ck.plan_min_recompute(d, cost, optimum - 1)
            assert e.value.code == -6 and "budget" in str(e.value)


def test_library_on_long_chains():
    rng = random.Random(13)
    for n in (60, 400):
        d = [rng.randint(1, 1 << 20) for _ in range(n + 1)]
        cost = [0] + [rng.randint(1, 1000) for _ in range(n)]
        mask6, peak6 = ck.plan(ck.ALGO_DYNAMIC_N, d)
        mask, peak, rec = ck.plan_min_recompute(d, cost)
        assert peak <= peak6 and ck.eval(ck.MODEL_DYNAMIC, d, mask) == peak
        assert rec == int(np.asarray(cost)[1:-1][mask[1:-1] == 0].sum())
        assert rec <= int(np.asarray(cost)[1:-1][mask6[1:-1] == 0].sum())
        # more room, less recomputation; the whole chain fits at the store-all-like peak of "every tensor a checkpoint"
        looser = ck.plan_min_recompute(d, cost, int(peak6 * 1.3))[2]
        assert looser <= rec
        assert ck.plan_min_recompute(d, cost, ck.eval(ck.MODEL_DYNAMIC, d, np.ones(n + 1, dtype=np.uint8)))[2] == 0


def test_library_errors_and_chain_costs():
    with pytest.raises(ck.CkptError) as e:
        ck.plan_min_recompute([1, 2, 3], [0, -1, 0])
    assert e.value.code == -6
    with pytest.raises(ck.CkptError) as e:
        ck.plan_min_recompute([1, 0, 3], [0, 1, 0])
    assert e.value.code == -3
    from paper_2502_12499_b200 import workloads as wl
    chain = ck.Chain(wl.config(2))
    cost = chain.unit_costs()
    assert cost[0] == 0 and np.all(cost[1:] > 0)
    # the second 3x3 layer at 224 x 224 is the most expensive unit of the VGG-16 chain, the pools are cheap
    assert int(np.argmax(cost)) == 2 and cost[3] < cost[2] / 3
    d = chain.sizes()
    mask6, peak6 = ck.plan(ck.ALGO_DYNAMIC_N, d)
    mask, peak, rec = ck.plan_min_recompute(d, cost)
    assert peak == peak6 and int(mask.sum()) > int(mask6.sum())
