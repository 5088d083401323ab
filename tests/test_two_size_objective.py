"""Eq. (memory) with separate sizes for a checkpoint, a segment tensor and a gradient (the allocator model that
Section 6 leaves as future work): the oracle pinned against hand values, closed forms and Eq. (memory) itself, then
the library's planners against the oracle's enumeration."""
import random

import numpy as np
import pytest

from oracle import planner_oracle as po
from paper_2502_12499_b200 import binding as ck


def random_sizes(rng, n, live_at_least_kept):
    kept = [rng.randint(1, 40) for _ in range(n + 1)]
    live = [k + rng.randint(0, 30) if live_at_least_kept else rng.randint(1, 40) for k in kept]
    grad = [rng.randint(1, 40) for _ in range(n + 1)]
    return kept, live, grad


# ------------------------------------------------------------------------------------------------ oracle pins

def test_hand_example():
    # n = 3: the only segment of C = {0, 3} holds live_1 + live_2, the output-gradient buffer max(g_0, g_1, g_2) and,
    # when counted, the incoming-gradient buffer max(g_1, g_2, g_3)
    kept, live, grad = [1, 2, 3, 4], [9, 5, 6, 9], [1, 1, 2, 7]
    assert po.eval_two_size(kept, live, grad, [0, 3]) == (1 + 4) + (5 + 6) + 2
    assert po.eval_two_size(kept, live, grad, [0, 3], incoming=True) == (1 + 4) + (5 + 6) + 2 + 7
    # C = {0, 2, 3}: at checkpoint 2: kept_0 + kept_2 + live_1 + max(g_0, g_1) = 1 + 3 + 5 + 1; at 3: all kept + g_2
    assert po.eval_two_size(kept, live, grad, [0, 2, 3]) == max(1 + 3 + 5 + 1, 1 + 3 + 4 + 2)
    assert po.eval_two_size(kept, live, grad, [0, 2, 3], incoming=True) == max(1 + 3 + 5 + 1 + 2, 1 + 3 + 4 + 2 + 7)


def test_reduces_to_eq_memory():
    rng = random.Random(3)
    for _ in range(200):
        n = rng.randint(1, 9)
        d = [rng.randint(1, 50) for _ in range(n + 1)]
        C = [0] + [i for i in range(1, n) if rng.random() < 0.4] + [n]
        assert po.eval_two_size(d, d, d, C) == po.eval_dynamic(d, C)
    d = [rng.randint(1, 50) for _ in range(11)]
    assert po.brute_force_two_size(d, d, d)["value"] == po.brute_force_dynamic(d)["value"]
    assert po.brute_force_two_size(d, d, d)["set"] == po.brute_force_dynamic(d)["set"]


def test_closed_forms_of_the_extreme_sets():
    rng = random.Random(4)
    for _ in range(50):
        n = rng.randint(2, 12)
        kept, live, grad = random_sizes(rng, n, False)
        for incoming in (False, True):
            # no interior checkpoint: every interior tensor is live at once
            want = kept[0] + kept[n] + sum(live[1:n]) + max(grad[:n]) + (max(grad[1:]) if incoming else 0)
            assert po.eval_two_size(kept, live, grad, [0, n], incoming) == want
            # every tensor a checkpoint: no segment tensor, buffers of one gradient each
            want = max(sum(kept[: i + 1]) + grad[i - 1] + (grad[i] if incoming else 0) for i in range(1, n + 1))
            assert po.eval_two_size(kept, live, grad, range(n + 1), incoming) == want


def test_uniform_chain_with_heavier_segment_tensors():
    # kept = grad = 1, live = a: a segment of s interior tensors costs a*s + 1 on top of the checkpoints so far.
    # With P checkpoints after d_0 ending segments of s_1..s_P interior tensors the peak is
    # max_p (1 + p + a*s_p + 1); the optimum by enumeration must equal the recursion's.
    for a in (1, 2, 5):
        for n in (6, 9, 12):
            kept, live, grad = [1] * (n + 1), [a] * (n + 1), [1] * (n + 1)
            bf = po.brute_force_two_size(kept, live, grad)
            assert po.dp_two_size_reference(kept, live, grad)[0] == bf["value"]
    # a = 1 is the paper's uniform chain: least P with (P-1)(P-2)/2 >= n
    n = 12
    P = next(p for p in range(1, 50) if (p - 1) * (p - 2) // 2 >= n)
    assert po.brute_force_two_size([1] * (n + 1), [1] * (n + 1), [1] * (n + 1))["value"] == P


def test_recursion_equals_enumeration_and_monotonicity():
    rng = random.Random(5)
    for trial in range(120):
        n = rng.randint(1, 10)
        kept, live, grad = random_sizes(rng, n, trial % 2 == 0)
        for incoming in (False, True):
            bf = po.brute_force_two_size(kept, live, grad, incoming)
            v, C = po.dp_two_size_reference(kept, live, grad, incoming)
            assert v == bf["value"] and C == bf["set"]
            assert po.eval_two_size(kept, live, grad, C, incoming) == v
            # a heavier segment tensor or a counted incoming buffer never lowers the optimum
            heavier = list(live)
            heavier[rng.randint(0, n)] += 7
            assert po.brute_force_two_size(kept, heavier, grad, incoming)["value"] >= v
        assert po.brute_force_two_size(kept, live, grad, True)["value"] >= po.brute_force_two_size(kept, live, grad, False)["value"]


def test_lemma_1_needs_live_at_least_kept():
    # U(i,j) = s(i,j) + kept_j increases with j when live >= kept (Lemma 1 of Section 4.2 on the generalised sizes)
    rng = random.Random(6)
    for _ in range(100):
        n = rng.randint(3, 12)
        kept, live, grad = random_sizes(rng, n, True)
        for incoming in (False, True):
            for i in range(n - 1):
                u = [po.s_term_two_size(live, grad, i, j, incoming) + kept[j] for j in range(i + 1, n + 1)]
                assert all(b > a for a, b in zip(u, u[1:]))
    # and can fail otherwise: a large checkpoint followed by a small one
    kept, live, grad = [1, 50, 1, 1], [1, 1, 1, 1], [1, 1, 1, 1]
    u = [po.s_term_two_size(live, grad, 0, j, False) + kept[j] for j in (1, 2, 3)]
    assert u[1] < u[0]


# ------------------------------------------------------------------------------------------------ library vs oracle

def test_library_planners_equal_enumeration():
    rng = random.Random(7)
    for trial in range(150):
        n = rng.randint(1, 11)
        ordered = trial % 3 != 0
        kept, live, grad = random_sizes(rng, n, ordered)
        for incoming in (False, True):
            bf = po.brute_force_two_size(kept, live, grad, incoming)
            mask, peak = ck.plan_sizes(ck.ALGO_DYNAMIC_N2, kept, live, grad, incoming)
            assert peak == bf["value"] and [int(i) for i in np.nonzero(mask)[0]] == bf["set"]
            assert ck.eval_sizes(kept, live, grad, mask, incoming) == peak
            if ordered:
                mask6, peak6 = ck.plan_sizes(ck.ALGO_DYNAMIC_N, kept, live, grad, incoming)
                assert peak6 == peak and np.array_equal(mask6, mask)
            C = [0] + [i for i in range(1, n) if rng.random() < 0.5] + [n]
            assert ck.eval_sizes(kept, live, grad, ck.mask_from_set(n, C), incoming) == po.eval_two_size(kept, live, grad, C, incoming)


def test_library_queue_search_equals_recursion_on_long_chains():
    rng = random.Random(8)
    for n in (50, 333, 1200):
        kept = [rng.randint(1, 1 << 20) for _ in range(n + 1)]
        live = [k + rng.randint(0, 1 << 20) for k in kept]
        grad = [rng.randint(1, 1 << 20) for _ in range(n + 1)]
        for incoming in (False, True):
            m5, p5 = ck.plan_sizes(ck.ALGO_DYNAMIC_N2, kept, live, grad, incoming)
            m6, p6 = ck.plan_sizes(ck.ALGO_DYNAMIC_N, kept, live, grad, incoming)
            assert p5 == p6 and np.array_equal(m5, m6)
            if n <= 333:
                v, C = po.dp_two_size_reference(kept, live, grad, incoming)
                assert v == p5 and [int(i) for i in np.nonzero(m5)[0]] == C


def test_library_equal_sizes_is_ckpt_plan():
    rng = random.Random(9)
    for _ in range(40):
        n = rng.randint(1, 60)
        d = [rng.randint(1, 1000) for _ in range(n + 1)]
        m, p = ck.plan(ck.ALGO_DYNAMIC_N, d)
        m2, p2 = ck.plan_sizes(ck.ALGO_DYNAMIC_N, d, d, d, False)
        assert p == p2 and np.array_equal(m, m2)


def test_library_errors():
    with pytest.raises(ck.CkptError) as e:
        ck.plan_sizes(ck.ALGO_DYNAMIC_N, [1, 50, 1, 1], [1, 1, 1, 1], [1, 1, 1, 1])
    assert e.value.code == -6 and "live" in str(e.value)
    with pytest.raises(ck.CkptError) as e:
        ck.plan_sizes(ck.ALGO_STATIC_N3, [1, 2, 3], [1, 2, 3], [1, 2, 3])
    assert e.value.code == -6
    with pytest.raises(ck.CkptError) as e:
        ck.plan_sizes(ck.ALGO_DYNAMIC_N2, [1, 2, 3], [1, 0, 3], [1, 2, 3])
    assert e.value.code == -3
    with pytest.raises(ck.CkptError) as e:
        ck.eval_sizes([1, 2, 3], [1, 2, 3], [1, 2, 3], [1, 1, 0])
    assert e.value.code == -5
