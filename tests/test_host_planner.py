"""Host side of the library (no GPU): planners, objective evaluation, arena schedule, C ABI surface.
Everything is compared with the oracle bit for bit."""
import os
import random
import re

import numpy as np
import pytest

from oracle import numeric_oracle as no
from oracle import planner_oracle as po
from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def as_set(mask):
    return [int(i) for i in np.nonzero(mask)[0]]


def oracle_sizes(chain):
    es = 2 if chain["dtype"] == "bf16" else 4
    return [-(-(chain["batch"] * h * w * c * es) // 256) * 256 for h, w, c in no.output_shapes(chain)]


# ---------------------------------------------------------------- C ABI surface

def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "ckpt_b200.h")).read()
    names = set(re.findall(r"CKPT_API\s+[\w\s\*]+?\b(ckpt_\w+)\s*\(", header))
    assert len(names) >= 20
    lib = ck.lib()
    for name in sorted(names):
        assert hasattr(lib, name), name


def test_error_codes():
    with pytest.raises(ck.CkptError) as e:
        ck.plan(ck.ALGO_DYNAMIC_N, [5])
    assert e.value.code == -2
    with pytest.raises(ck.CkptError) as e:
        ck.plan(ck.ALGO_DYNAMIC_N, [5, 0, 3])
    assert e.value.code == -3
    with pytest.raises(ck.CkptError) as e:
        ck.plan(ck.ALGO_STATIC_N3, [2 ** 62, 2 ** 62, 5])
    assert e.value.code == -4
    with pytest.raises(ck.CkptError) as e:
        ck.eval(ck.MODEL_DYNAMIC, [1, 2, 3], [1, 1, 0])
    assert e.value.code == -5
    with pytest.raises(ck.CkptError) as e:
        ck.plan(7, [1, 2, 3])
    assert e.value.code == -6
    assert "unknown algorithm" in str(e.value)


# ---------------------------------------------------------------- planners vs brute force

@pytest.mark.parametrize("seed", range(6))
def test_plans_match_brute_force(seed):
    rng = random.Random(100 + seed)
    for trial in range(60):
        n = rng.randint(1, 11)
        hi = [3, 6, 40, 1000][trial % 4]
        d = [rng.randint(1, hi) for _ in range(n + 1)]
        bs = po.brute_force_static(d)
        m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
        assert peak == bs["value"] and as_set(m) == bs["set"], (d, as_set(m), bs)
        bd = po.brute_force_dynamic(d)
        for algo in (ck.ALGO_DYNAMIC_N2, ck.ALGO_DYNAMIC_N):
            m, peak = ck.plan(algo, d)
            assert peak == bd["value"] and as_set(m) == bd["set"], (algo, d, as_set(m), bd)
        assert ck.eval(ck.MODEL_STATIC, d, m) == po.eval_static(d, as_set(m))
        assert ck.eval(ck.MODEL_DYNAMIC, d, m) == po.eval_dynamic(d, as_set(m))
        assert ck.eval(ck.MODEL_STORE_ALL, d, None) == sum(d)


def test_n16_brute_force_once():
    rng = random.Random(7)
    d = [rng.randint(1, 9) for _ in range(17)]
    bd = po.brute_force_dynamic(d)
    m, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
    assert (peak, as_set(m)) == (bd["value"], bd["set"])
    bs = po.brute_force_static(d)
    m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
    assert (peak, as_set(m)) == (bs["value"], bs["set"])
    assert bs["n_masks"] == 65536


@pytest.mark.parametrize("seed", range(4))
def test_plans_match_reference_recursions_longer_chains(seed):
    rng = random.Random(200 + seed)
    for trial in range(12):
        n = rng.randint(12, 90)
        kind = trial % 3
        if kind == 0:
            d = [rng.randint(1, 5) for _ in range(n + 1)]
        elif kind == 1:
            d = [rng.randint(1, 10 ** 9) for _ in range(n + 1)]
        else:                                               # CNN-like: plateaus that shrink
            d, v = [], 2 ** 20
            for i in range(n + 1):
                if rng.random() < 0.2:
                    v = max(256, v // 2)
                d.append(v)
        vs, Cs = po.dp_static_reference(d)
        m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
        assert (peak, as_set(m)) == (vs, Cs)
        vd, Cd, _ = po.dp_dynamic_reference(d)
        for algo in (ck.ALGO_DYNAMIC_N2, ck.ALGO_DYNAMIC_N):
            m, peak = ck.plan(algo, d)
            assert (peak, as_set(m)) == (vd, Cd), (algo, d)


def test_alg6_work_is_linear():
    # Algorithm 6's queue/pointer steps must grow linearly, Algorithm 5's pairs quadratically.
    rng = random.Random(11)
    for n in (500, 2000, 8000):
        d = [rng.randint(1, 10 ** 6) for _ in range(n + 1)]
        _, p6, w6 = ck.plan_counted(ck.ALGO_DYNAMIC_N, d)
        assert w6 <= 8 * n, (n, w6)
        if n <= 2000:
            _, p5, w5 = ck.plan_counted(ck.ALGO_DYNAMIC_N2, d)
            assert p5 == p6 and w5 == n * (n + 1) // 2


def test_vgg19_paper_values(vgg19_golden):
    d = [v * 128 * 4 for v in vgg19_golden["sizes_per_image"]]
    m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
    assert as_set(m)[1:] == vgg19_golden["alg3_set"]
    m6, peak6 = ck.plan(ck.ALGO_DYNAMIC_N, d)
    assert peak6 == int(4777.5 * 2 ** 20)
    assert ck.eval(ck.MODEL_DYNAMIC, d, ck.mask_from_set(24, [0] + vgg19_golden["alg6_set"])) == peak6
    assert ck.eval(ck.MODEL_DYNAMIC, d, m) - peak6 == 392 * 2 ** 20


# ---------------------------------------------------------------- the benchmark configurations

@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_config_plans(index):
    chain = wl.config(index)
    d = oracle_sizes(chain)
    n = len(d) - 1
    vd, Cd, _ = po.dp_dynamic_reference(d)
    for algo in (ck.ALGO_DYNAMIC_N2, ck.ALGO_DYNAMIC_N):
        m, peak = ck.plan(algo, d)
        assert (peak, as_set(m)) == (vd, Cd)
    vs, Cs = po.dp_static_reference(d)
    m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
    assert (peak, as_set(m)) == (vs, Cs)
    if index == 1:
        assert n == 8 and vd == po.brute_force_dynamic(d)["value"] and vs == po.brute_force_static(d)["value"]
    if index == 5:
        assert n == 1000 and vd == 47 * d[1] and vs == 64 * d[1]
        assert sum(d) > 20 * vd                                  # >20x less than storing everything


def test_chain_sizes_match_oracle_shapes():
    for index in (1, 2, 3, 4, 5):
        spec = wl.config(index)
        chain = ck.Chain(spec)
        assert list(chain.sizes()) == oracle_sizes(spec)
        assert [tuple(s) for s in chain.shapes()] == no.output_shapes(spec)
        flat = ck.flatten_params(spec, wl.make_params(spec) if index in (1, 2) else
                                 [{k: np.zeros(s, np.float32) for k, s in wl.param_shapes(u).items()} for u in spec["units"]])
        assert chain.num_params() == len(flat)
        for p, (ui, name, arr) in enumerate(flat):
            unit, elems, dt = chain.param_info(p)
            assert unit == ui + 1 and elems == arr.size
            assert dt == (chain.dtype if name.startswith("w") else ck.DTYPE_F32)
        assert chain.workspace_bytes() > 2 * max(chain.sizes())


def test_chain_rejects_inconsistent_units():
    spec = wl.plain_chain(2, 8, 3, (8, 8), 2, "f32")
    spec["units"][1]["cin"] = 5
    with pytest.raises(ck.CkptError) as e:
        ck.Chain(spec)
    assert e.value.code == -6


# ---------------------------------------------------------------- arena schedule

def check_events(events, capacity, n):
    live = {}
    for kind, tid, off, size in events:
        if kind == 1:
            assert off >= 0 and off + size <= capacity
            for o2, s2 in live.values():
                assert off + size <= o2 or o2 + s2 <= off, "overlap"
            live[tid] = (off, size)
        else:
            assert live.pop(tid) == (off, size)
    return live


@pytest.mark.parametrize("seed", range(5))
def test_arena_schedule_matches_event_simulators(seed):
    rng = random.Random(300 + seed)
    for trial in range(80):
        n = rng.randint(1, 14)
        d = [256 * rng.randint(1, 40) for _ in range(n + 1)]
        C = [0] + [i for i in range(1, n) if rng.random() < 0.45] + [n]
        mask = ck.mask_from_set(n, C)
        for policy, sim, model in ((ck.POLICY_STATIC, po.simulate_alg2, po.eval_static),
                                   (ck.POLICY_DYNAMIC, po.simulate_alg4, po.eval_dynamic)):
            r = ck.arena_dry_run(policy, d, mask)
            hw, ev = sim(d, C)
            assert r["high_water"] == hw == model(d, C)
            assert r["extent"] == hw                                 # no fragmentation
            check_events(r["events"], hw, n)
            # same alloc/free sequence as the oracle's event list
            names = [(e[0], e[1]) for e in ev]
            mine = [("alloc" if k == 1 else "free", "r" if t == n + 1 else "d%d" % t) for k, t, _, _ in r["events"]]
            assert mine == names
        r = ck.arena_dry_run(ck.POLICY_STORE_ALL, d, None)
        assert r["high_water"] == r["extent"] == po.simulate_alg1(d)[0] == sum(d)


def test_arena_schedule_on_optimal_plans_of_configs():
    for index in (1, 2, 5):
        d = oracle_sizes(wl.config(index))
        n = len(d) - 1
        m, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
        r = ck.arena_dry_run(ck.POLICY_DYNAMIC, d, m)
        assert r["high_water"] == r["extent"] == peak
        check_events(r["events"], peak, n)
        m, peak = ck.plan(ck.ALGO_STATIC_N3, d)
        r = ck.arena_dry_run(ck.POLICY_STATIC, d, m)
        assert r["high_water"] == r["extent"] == peak


def test_stage_trace_and_sqrt_plan_match_oracle(vgg19_golden):
    rng = random.Random(400)
    for _ in range(150):
        n = rng.randint(1, 14)
        d = [256 * rng.randint(1, 40) for _ in range(n + 1)]
        C = [0] + [i for i in range(1, n) if rng.random() < 0.45] + [n]
        mask = ck.mask_from_set(n, C)
        assert list(ck.arena_stage_trace(ck.POLICY_DYNAMIC, d, mask)) == po.stage_trace(d, C, "alg4")
        assert list(ck.arena_stage_trace(ck.POLICY_STATIC, d, mask)) == po.stage_trace(d, C, "alg2")
        m, peak = ck.plan(ck.ALGO_SQRT_N, d)
        assert as_set(m) == po.sqrt_n_plan(n) and peak == po.eval_dynamic(d, po.sqrt_n_plan(n))
    d = [v * 128 * 4 for v in vgg19_golden["sizes_per_image"]]
    m, peak = ck.plan(ck.ALGO_SQRT_N, d)
    assert as_set(m)[1:] == vgg19_golden["sqrtn_set"]
    assert peak - ck.plan(ck.ALGO_DYNAMIC_N, d)[1] == 1960 * 2 ** 20      # Table 2: 8404 - 6444 MiB


def test_split_units_chain_and_plan():
    """Finer granularity (Section 5.4): the split VGG-16 chain has 47 units; conv, bn and relu outputs
    have the size of the fused unit's output; the O(n) planner still matches the O(n^2) recursion, and
    its optimum is below that of the same chain with every tensor stored."""
    coarse = wl.config(2)
    fine, origin = wl.split_units(coarse)
    assert len(fine["units"]) == 21 + 2 * 13 == len(origin)
    chain = ck.Chain(fine)
    d = [int(v) for v in chain.sizes()]
    assert d == oracle_sizes(fine)
    dc = oracle_sizes(coarse)
    k = 1
    for ui, u in enumerate(coarse["units"]):
        if u["kind"] == "conv_bn_relu":
            assert d[k] == d[k + 1] == d[k + 2] == dc[ui + 1]
            k += 3
        else:
            assert d[k] == dc[ui + 1]
            k += 1
    vd, Cd, _ = po.dp_dynamic_reference(d)
    m, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
    assert (peak, as_set(m)) == (vd, Cd)
    assert peak < sum(d) / 2
    r = ck.arena_dry_run(ck.POLICY_DYNAMIC, d, m)
    assert r["high_water"] == r["extent"] == peak
    # the parameters of the fused chain re-file one to one
    shapes = [{k2: np.zeros(s, np.float32) for k2, s in wl.param_shapes(u).items()} for u in coarse["units"]]
    flat_c = ck.flatten_params(coarse, shapes)
    flat_f = ck.flatten_params(fine, wl.split_params(origin, shapes))
    assert [(origin[fi][0], name) for fi, name, _ in flat_f] == [(ui, name) for ui, name, _ in flat_c]
    assert chain.num_params() == len(flat_f)


def test_launch_log_is_empty_without_launches():
    ck.launch_log(True)
    assert ck.launch_log_read() == {}
    ck.launch_log(False)


def test_chain_option_errors_need_no_device():
    """Argument checks of the chain options (host only: nothing is launched or dereferenced)."""
    import ctypes as C
    from paper_2502_12499_b200 import workloads as wl
    chain = ck.Chain(wl.config(1))
    need = int(sum(chain.sizes()[1:]))
    lib = ck.lib()
    fake = C.c_void_p(0x1000)                       # never dereferenced: the call only records the address
    assert lib.ckpt_chain_set_gradient_tap(chain._h, fake, C.c_int64(need - 1)) == -8       # E_WORKSPACE: tap too small
    assert "tap" in lib.ckpt_last_error().decode()
    assert lib.ckpt_chain_set_gradient_tap(chain._h, fake, C.c_int64(need)) == 0
    assert lib.ckpt_chain_set_gradient_tap(chain._h, None, C.c_int64(0)) == 0
    assert lib.ckpt_chain_set_sgd(chain._h, C.c_double(-1.0)) == -6
    assert lib.ckpt_chain_set_sgd(chain._h, C.c_double(float("nan"))) == -6
    assert lib.ckpt_chain_set_sgd(chain._h, C.c_double(0.01)) == 0
    assert lib.ckpt_chain_set_sgd(None, C.c_double(0.01)) == -1
    assert lib.ckpt_chain_set_selftest(None, 1) == -1
    assert lib.ckpt_selftest_bounded_wait(C.c_int64(0), None) in (-6, -1)                   # limit out of range (or no status word)
    # input staging: null pointers, slot, labels and buffer size are checked before any device call
    need_stage = chain.staging_bytes()
    assert need_stage >= 2 * (int(chain.sizes()[0]) + 4 * wl.config(1)["batch"])
    out_b, out_l = C.c_void_p(0), C.c_void_p(0)
    args = lambda slot, batch, labels, size: lib.ckpt_chain_stage_batch(  # noqa: E731
        chain._h, C.c_int(slot), batch, labels, fake, C.c_int64(size), C.byref(out_b), C.byref(out_l))
    assert args(0, None, fake, need_stage) == -1
    assert args(2, fake, fake, need_stage) == -6 and "slot" in lib.ckpt_last_error().decode()
    labelled = ck.Chain(wl.config(2))               # softmax loss: labels are required
    assert lib.ckpt_chain_stage_batch(labelled._h, C.c_int(0), fake, None, fake, C.c_int64(labelled.staging_bytes()), C.byref(out_b),
                                      C.byref(out_l)) == -1 and "labels" in lib.ckpt_last_error().decode()
    assert args(1, fake, fake, need_stage - 1) == -8 and "staging" in lib.ckpt_last_error().decode()
    assert lib.ckpt_chain_staging_bytes(chain._h, None) == -1
    # workspace per schedule: Algorithm 4's is a prefix of the full one
    assert chain.workspace_bytes_for(ck.POLICY_STORE_ALL) == chain.workspace_bytes_for(ck.POLICY_STATIC) == chain.workspace_bytes()
    assert 0 < chain.workspace_bytes_for(ck.POLICY_DYNAMIC) < chain.workspace_bytes()
    out_bytes = C.c_int64(0)
    assert lib.ckpt_chain_workspace_bytes_for(chain._h, C.c_int(3), C.byref(out_bytes)) == -6
    assert lib.ckpt_chain_workspace_bytes_for(chain._h, C.c_int(2), None) == -1
