"""Pins for the planner oracle: closed forms, the paper's printed VGG-19 values, and the
agreement of definition (enumeration), recursion and allocation-event list."""
import random

import pytest

from oracle import planner_oracle as po

MIB = 1024 * 1024


def rand_chain(rng, n, lo=1, hi=50):
    return [rng.randint(lo, hi) for _ in range(n + 1)]


# ---------------------------------------------------------------- closed forms, Eq. (cost)

def test_static_all_and_none_equal_total():
    rng = random.Random(1)
    for n in range(1, 12):
        d = rand_chain(rng, n)
        assert po.eval_static(d, range(n + 1)) == sum(d)
        assert po.eval_static(d, [0, n]) == sum(d)


def test_static_hand_example_fig1():
    # Fig. 1: checkpoints {0,2,5}, segments {d1} and {d3,d4}
    d = [7, 11, 13, 17, 19, 23]
    assert po.eval_static(d, [0, 2, 5]) == (7 + 13 + 23) + max(11, 17 + 19)


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 12])
def test_static_uniform_optimum_closed_form(n):
    # uniform sizes: k segments -> k checkpoints besides d_0 plus a segment of ceil(n/k)-1,
    # so optimum = d * min_k (k + ceil(n/k))
    d = [3] * (n + 1)
    want = 3 * min(k + -(-n // k) for k in range(1, n + 1))
    assert po.brute_force_static(d)["value"] == want
    assert po.dp_static_reference(d)[0] == want


def test_static_uniform_n8_is_6d_n1000_is_64d():
    assert min(k + -(-8 // k) for k in range(1, 9)) == 6
    assert min(k + -(-1000 // k) for k in range(1, 1001)) == 64


# ---------------------------------------------------------------- closed forms, Eq. (memory)

def test_dynamic_extremes_closed_form():
    rng = random.Random(2)
    for n in range(1, 12):
        d = rand_chain(rng, n)
        assert po.eval_dynamic(d, [0, n]) == sum(d) + max(d[:n])
        want_all = max(sum(d[: i + 1]) + d[i - 1] for i in range(1, n + 1))
        assert po.eval_dynamic(d, range(n + 1)) == want_all


def test_dynamic_hand_example():
    d = [4, 9, 2, 6, 5]
    # C={0,2,4}: m(2)=d0+d2 + d1 + max(d0,d1); m(4)=d0+d2+d4 + d3 + max(d2,d3)
    assert po.eval_dynamic(d, [0, 2, 4]) == max(4 + 2 + 9 + 9, 4 + 2 + 5 + 6 + 6)


@pytest.mark.parametrize("n", [1, 2, 3, 6, 8, 10, 11])
def test_dynamic_uniform_optimum_closed_form(n):
    # uniform sizes: optimum = P*d with P the least integer with (P-1)(P-2)/2 >= n
    P = 2
    while (P - 1) * (P - 2) // 2 < n:
        P += 1
    d = [5] * (n + 1)
    assert po.brute_force_dynamic(d)["value"] == 5 * P
    assert po.dp_dynamic_reference(d)[0] == 5 * P


def test_dynamic_uniform_n100_and_n1000():
    assert po.dp_dynamic_reference([7] * 101)[0] == 7 * 16
    v, C, _ = po.dp_dynamic_reference([1] * 1001)
    assert v == 47
    assert po.eval_dynamic([1] * 1001, C) == 47


# ---------------------------------------------------------------- definition == recursion == events

def test_event_simulators_match_objectives():
    rng = random.Random(3)
    for trial in range(300):
        n = rng.randint(1, 12)
        d = rand_chain(rng, n)
        C = [0] + [i for i in range(1, n) if rng.random() < 0.4] + [n]
        assert po.simulate_alg2(d, C)[0] == po.eval_static(d, C)
        assert po.simulate_alg4(d, C)[0] == po.eval_dynamic(d, C)
    assert po.simulate_alg1([3, 4, 5])[0] == 12


def test_alg4_listing_order_would_overshoot():
    # keeping the old gradient buffer during the recompute (the listing's literal order)
    # exceeds Eq. (memory) on this chain; the adopted order does not.
    d = [1, 1, 1, 10, 1, 1, 1, 1, 1]
    C = [0, 4, 8]
    assert po.simulate_alg4(d, C)[0] == po.eval_dynamic(d, C)


def test_bruteforce_equals_recursions_random():
    rng = random.Random(4)
    for trial in range(120):
        n = rng.randint(1, 10)
        d = rand_chain(rng, n, 1, 30 if trial % 2 else 4)   # small range -> many ties
        bs = po.brute_force_static(d)
        vs, Cs = po.dp_static_reference(d)
        assert vs == bs["value"]
        assert Cs == bs["set"]
        assert po.eval_static(d, Cs) == vs
        bd = po.brute_force_dynamic(d)
        vd, Cd, M = po.dp_dynamic_reference(d)
        assert vd == bd["value"]
        assert Cd == bd["set"]
        assert M == bd["suffix_values"]
        assert po.eval_dynamic(d, Cd) == vd
        assert bs["n_evaluated"] == 2 ** (n - 1) and bs["n_masks"] == 2 ** n


def test_n8_config_all_256_masks():
    d = [49152] + [262144] * 8
    bs = po.brute_force_static(d)
    bd = po.brute_force_dynamic(d)
    assert bs["n_masks"] == 256 and bs["n_evaluated"] == 128
    # uniform tail: 6 tensors' worth of d_1..8 minus the smaller d_0 adjustment
    assert bd["value"] == po.dp_dynamic_reference(d)[0]
    assert bs["value"] == po.dp_static_reference(d)[0]
    assert bs["value"] == 49152 + 5 * 262144
    assert bd["value"] == 49152 + 5 * 262144


def test_scaling_leaves_set_unchanged():
    # Section 5.5: the batch size multiplies every d_i and does not change the sets
    rng = random.Random(5)
    for _ in range(40):
        n = rng.randint(2, 9)
        d = rand_chain(rng, n)
        d4 = [4 * v for v in d]
        assert po.brute_force_static(d)["set"] == po.brute_force_static(d4)["set"]
        assert po.brute_force_dynamic(d)["set"] == po.brute_force_dynamic(d4)["set"]


# ---------------------------------------------------------------- lemmas of Section 4.2

def test_lemmas_U_monotone():
    rng = random.Random(6)
    for _ in range(100):
        n = rng.randint(3, 12)
        d = rand_chain(rng, n)

        def U(i, j):
            return po.s_term(d, i, j) + d[j]

        for i in range(0, n):
            for j in range(i + 1, n):
                assert U(i, j + 1) > U(i, j)            # Lemma 1
        for i in range(1, n):
            for j in range(i + 1, n + 1):
                assert U(i - 1, j) > U(i, j)            # Eq. (U-update) inequality


# ---------------------------------------------------------------- the paper's VGG-19 numbers

def test_vgg19_static_plan_is_3_6_24(vgg19_golden):
    d = vgg19_golden["sizes_per_image"]
    assert len(d) == 25
    v, C = po.dp_static_reference(d)
    assert C[1:] == vgg19_golden["alg3_set"]            # paper lists indices without 0
    assert v == po.eval_static(d, [0] + vgg19_golden["alg3_set"])
    assert v == 7778280
    # one 64x224x224 fp32 tensor at batch 128 is the 1.53125 GiB step of the printed series
    assert d[1] * 128 * 4 == int(1.53125 * 1024 * MIB)


def test_vgg19_dynamic_value_and_printed_set(vgg19_golden):
    d = vgg19_golden["sizes_per_image"]
    v, C, _ = po.dp_dynamic_reference(d)
    printed = [0] + vgg19_golden["alg6_set"]
    assert po.eval_dynamic(d, printed) == v             # the printed set is one of the optima
    assert po.eval_dynamic(d, C) == v
    assert v * 128 * 4 == int(4777.5 * MIB)


def test_vgg19_table2_column_differences(vgg19_golden):
    d = [v * 128 * 4 for v in vgg19_golden["sizes_per_image"]]
    opt = po.dp_dynamic_reference(d)[0]
    acg = po.eval_dynamic(d, [0] + vgg19_golden["alg3_set"])
    sqrtn = po.eval_dynamic(d, [0] + vgg19_golden["sqrtn_set"])
    t = vgg19_golden["table2_b128_mib"]
    assert (acg - opt) == vgg19_golden["saving_vs_acg_mib"][0] * MIB
    assert abs((acg - opt) / MIB - (t[1] - t[0])) <= 1          # 6835-6444 printed as rounded MiB
    assert (sqrtn - opt) / MIB == t[3] - t[0]                   # 8404-6444 = 1960
    assert po.sqrt_n_plan(24)[1:] == vgg19_golden["sqrtn_set"]


def test_vgg19_fig2_segment_start_jump(vgg19_golden):
    # Soft pin of Algorithm 4's event order.  Stage 37 -> 38 of the printed prediction rises by
    # (recomputed d_4..d_10) - (old gradient buffer) + (new gradient buffer); the printed series
    # differs from that by one d_24 (0.49 MiB), so the tolerance is 1 MiB on a 3920 MiB jump.
    d = [v * 128 * 4 for v in vgg19_golden["sizes_per_image"]]
    C = [0] + vgg19_golden["fig2_set"]
    GIB = 1024 * MIB
    rise = (vgg19_golden["fig2_stage38_gib"][0] - vgg19_golden["fig2_stage37_gib"][0]) * GIB
    old_r = max(d[11:24])
    new_r = max(d[3:11])
    assert abs(rise - (sum(d[4:11]) - old_r + new_r)) < 1 * MIB
    # the simulator takes the same jump between "old buffer released" and "new buffer allocated"
    _, events = po.simulate_alg4(d, C)
    idx = [k for k, e in enumerate(events) if e[1] == "r"]
    free_old, alloc_new = idx[1], idx[2]
    assert events[free_old][0] == "free" and events[alloc_new][0] == "alloc"
    sim_rise = events[alloc_new][3] - events[free_old - 1][3]
    assert abs(rise - sim_rise) < 1 * MIB
    # stage 37 of the print (input excluded: it sits in the constant base) is the level before that
    base = vgg19_golden["fig2_stage0_gib"][0] * GIB
    assert abs(events[free_old - 1][3] - d[0] + base - vgg19_golden["fig2_stage37_gib"][0] * GIB) < 1


def test_stage_trace_consistent_with_events_and_print(vgg19_golden):
    rng = random.Random(8)
    for _ in range(100):
        n = rng.randint(1, 12)
        d = rand_chain(rng, n)
        C = [0] + [i for i in range(1, n) if rng.random() < 0.4] + [n]
        t4 = po.stage_trace(d, C, "alg4")
        t2 = po.stage_trace(d, C, "alg2")
        assert len(t4) == len(t2) == 2 * n + 2 and t4[0] == t4[-1] == d[0]
        assert max(t2) <= po.eval_static(d, C) and max(t4) <= po.eval_dynamic(d, C)
        assert t4[n] == t2[n] == sum(d[c] for c in C)           # end of the forward phase: checkpoints only
        assert t2[2 * n] == po.simulate_alg2(d, C)[1][-1][3]    # last event of the event list
    # Fig. 2 (VGG-19, b = 128, C = {3,11,24}): forward stages 3 and 11 (ends of stages whose output is a
    # checkpoint) and the whole run of backward stages 26..37, relative to the printed constant base.
    # The printed series excludes the input (it sits in the base) and carries one d_24 (0.49 MiB) of
    # the loss gradient through the backward phase.
    d = [v * 128 * 4 for v in vgg19_golden["sizes_per_image"]]
    t = po.stage_trace(d, [0] + vgg19_golden["fig2_set"], "alg4")
    GIB = 1024 * MIB
    base = vgg19_golden["fig2_stage0_gib"][0] * GIB
    assert abs((t[37] - d[0]) - (vgg19_golden["fig2_stage37_gib"][0] * GIB - base)) < 1
    assert abs((t[45] - d[0] + d[24]) - (vgg19_golden["fig2_stage45_gib"][0] * GIB - base)) < 1 * MIB
