"""GPU parity of the whole training step (ckpt_train_step) against the oracle's store-all step.

Checked for every case: weight gradients within tolerance of the float64 oracle; gradients of every
checkpointed run bit-identical to the GPU's own store-all run; arena high-water mark == highest
offset used == the planner's predicted peak, with an arena of exactly that many bytes."""
import random

import numpy as np
import pytest

from oracle import numeric_oracle as no
from oracle import planner_oracle as po
from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import StepRunner, max_rel_err

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-3, "bf16": 3e-2}


def mini_vgg(dtype, batch=4):
    return wl.vgg16_chain(batch, hw=(32, 32), dtype=dtype, widths=(8, 16, 24, 32, 32), fc_width=48, classes=10,
                          name="mini_vgg_" + dtype)


def oracle_step(spec, params, x, labels, storage="exact"):
    p64 = [{k: v.astype(np.float64) for k, v in p.items()} for p in params]
    return no.chain_forward_backward(spec, p64, x.astype(np.float64), labels, storage=storage)


def compare_with_oracle(runner, grads, ref, tol):
    worst = 0.0
    for (ui, name, _), g in zip(runner.flat, grads):
        want = ref["grads"][ui][name]
        assert np.all(np.isfinite(g)), (ui, name)
        err = max_rel_err(g.reshape(want.shape), want)
        assert err <= tol, (ui, name, err)
        worst = max(worst, err)
    return worst


def all_policies_agree(runner, x, labels, masks_dynamic, masks_static):
    rep0, g0 = runner.run(ck.POLICY_STORE_ALL, None, x, labels)
    assert rep0["peak_bytes"] == rep0["extent_bytes"] == rep0["predicted_bytes"] == int(sum(runner.d))
    assert rep0["recomputed_units"] == 0 and rep0["launches"] > 0 and rep0["device_status"] == 0
    for policy, masks in ((ck.POLICY_DYNAMIC, masks_dynamic), (ck.POLICY_STATIC, masks_static)):
        for mask in masks:
            rep, g = runner.run(policy, mask, x, labels)
            C = [int(i) for i in np.nonzero(mask)[0]]
            want = (po.eval_dynamic if policy == ck.POLICY_DYNAMIC else po.eval_static)([int(v) for v in runner.d], C)
            assert rep["peak_bytes"] == rep["extent_bytes"] == rep["predicted_bytes"] == want
            assert rep["recomputed_units"] == runner.n + 1 - len(C)
            assert rep["loss"] == rep0["loss"]
            for a, b in zip(g, g0):
                assert np.array_equal(a, b)            # bit-identical to the store-all run
    return rep0, g0


def test_config1_plain8_fp32_all_masks():
    spec = wl.config(1)
    params = wl.make_params(spec, seed=0)
    x, _ = wl.make_batch(spec, seed=1)
    runner = StepRunner(spec, params)
    d = [int(v) for v in runner.d]
    assert d == [49152] + [262144] * 8
    # the planners' sets (checked against brute force over all 256 masks on the CPU side)
    m6, peak6 = ck.plan(ck.ALGO_DYNAMIC_N, d)
    m3, peak3 = ck.plan(ck.ALGO_STATIC_N3, d)
    assert peak6 == po.brute_force_dynamic(d)["value"] and peak3 == po.brute_force_static(d)["value"]
    masks = [m6, m3]
    rng = random.Random(0)
    every = [ck.mask_from_set(8, [0] + [i for i in range(1, 8) if (bits >> (i - 1)) & 1] + [8]) for bits in range(128)]
    masks += rng.sample(every, 12)
    rep0, g0 = all_policies_agree(runner, x, None, masks, masks)
    ref = oracle_step(spec, params, x, None)
    assert abs(rep0["loss"] - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    compare_with_oracle(runner, g0, ref, TOL["f32"])
    # the high-water mark of all 128 feasible masks equals Eq. (memory) (arena of exactly that size)
    for mask in every:
        rep, _ = runner.run(ck.POLICY_DYNAMIC, mask, x, None)
        assert rep["peak_bytes"] == rep["need"] == rep["extent_bytes"]


def rel_l2(got, want):
    want = np.asarray(want, dtype=np.float64)
    return float(np.linalg.norm(np.asarray(got, dtype=np.float64).reshape(want.shape) - want) / max(np.linalg.norm(want), 1e-300))


def test_mini_vgg_fp32_against_exact_oracle():
    """16 units deep (13 conv units, 5 pools, 3 FC), every policy, float32: max relative error 1e-3."""
    spec = mini_vgg("f32")
    params = wl.make_params(spec, seed=3, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=4)
    runner = StepRunner(spec, params)
    d = [int(v) for v in runner.d]
    n = runner.n
    m6, _ = ck.plan(ck.ALGO_DYNAMIC_N, d)
    m3, _ = ck.plan(ck.ALGO_STATIC_N3, d)
    rng = random.Random(1)
    extra = [ck.mask_from_set(n, [0] + [i for i in range(1, n) if rng.random() < 0.4] + [n]) for _ in range(4)]
    extra.append(ck.mask_from_set(n, [0, n]))
    extra.append(ck.mask_from_set(n, range(n + 1)))
    rep0, g0 = all_policies_agree(runner, x, labels, [m6] + extra, [m3] + extra)
    ref = oracle_step(spec, params, x, labels)
    assert abs(rep0["loss"] - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    compare_with_oracle(runner, g0, ref, TOL["f32"])


@pytest.mark.parametrize("seed", [3, 0])
def test_mini_vgg_bf16_statistical_parity(seed):
    """A 16-unit bfloat16 chain cannot be compared element-wise with any independent reference:
    every stored tensor is rounded to bfloat16, one element that rounds the other way (float32 vs
    float64 accumulation) changes ReLU masks and pooling arg-max decisions downstream, and the
    differences multiply from layer to layer - the oracle's own exact and bfloat16-storage modes
    differ by tens of percent on this chain.  What is fixed is the *size* of that deviation: the
    executor (float32 accumulation, bfloat16 storage) must be no further from the exact result than
    1.5 x the oracle run with the same storage rounding, per tensor in relative L2 norm (+0.02).
    Element-wise bfloat16 parity is asserted on the shallow chains below and per operation."""
    spec = mini_vgg("bf16", batch=8)
    params = wl.make_params(spec, seed=seed, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=seed + 1)
    runner = StepRunner(spec, params)
    n = runner.n
    m6, _ = ck.plan(ck.ALGO_DYNAMIC_N, runner.d)
    m3, _ = ck.plan(ck.ALGO_STATIC_N3, runner.d)
    rep0, g0 = all_policies_agree(runner, x, labels, [m6, ck.mask_from_set(n, [0, n])], [m3])
    exact = oracle_step(spec, params, x, labels)
    stored = oracle_step(spec, params, x, labels, storage="bf16")
    assert abs(rep0["loss"] - exact["loss"]) <= 2e-2 * abs(exact["loss"])
    for (ui, name, _), g in zip(runner.flat, g0):
        assert np.all(np.isfinite(g))
        mine = rel_l2(g, exact["grads"][ui][name])
        theirs = rel_l2(stored["grads"][ui][name], exact["grads"][ui][name])
        assert mine <= 1.5 * theirs + 0.02, (ui, name, mine, theirs)


def shallow_chains():
    s = wl.plain_chain(1, 32, 16, (24, 20), 16, "bf16", "softmax_ce", name="conv+fc")
    s["units"].append({"kind": "fc", "cin": 24 * 20 * 32, "cout": 10, "relu": False})
    yield s
    s = wl.plain_chain(1, 24, 8, (16, 16), 32, "bf16", "softmax_ce", name="conv+pool+fc")
    s["units"] += [{"kind": "maxpool", "k": 2, "stride": 2, "pad": 0}, {"kind": "fc", "cin": 8 * 8 * 24, "cout": 10, "relu": False}]
    yield s
    s = dict(units=[{"kind": "fc", "cin": 6 * 6 * 8, "cout": 40, "relu": True}, {"kind": "fc", "cin": 40, "cout": 12, "relu": False}],
             input_hwc=(6, 6, 8), batch=16, dtype="bf16", loss="softmax_ce", name="fc+fc")
    yield s
    s = dict(units=[{"kind": "fc", "cin": 2 * 2 * 64, "cout": 128, "relu": True}, {"kind": "fc", "cin": 128, "cout": 64, "relu": False}],
             input_hwc=(2, 2, 64), batch=24, dtype="bf16", loss="softmax_ce", name="fc+fc on tensor cores")
    yield s
    s = dict(units=[{"kind": "fc", "cin": 4 * 4 * 128, "cout": 200, "relu": True}, {"kind": "fc", "cin": 200, "cout": 16, "relu": False}],
             input_hwc=(4, 4, 128), batch=40, dtype="bf16", loss="softmax_ce", name="wide fc (matrix on M, split reduction)+fc")
    yield s
    s = wl.plain_chain(2, 64, 64, (12, 12), 8, "bf16", "softmax_ce", name="conv64+conv64+fc")
    s["units"].append({"kind": "fc", "cin": 12 * 12 * 64, "cout": 10, "relu": False})
    yield s


@pytest.mark.parametrize("spec", list(shallow_chains()), ids=lambda s: s["name"])
def test_shallow_bf16_chains(spec):
    """bfloat16 storage with float32 accumulation, max relative error 3e-2 per gradient tensor.
    The stored tensors are quantised codes and the ReLU masks / pooling arg-max are decisions taken
    on those codes, so the oracle takes them in the kernel's precision: float64 arithmetic with
    every stored tensor rounded to bfloat16 where the executor stores it.  Against the oracle
    without that rounding the same bound holds wherever the rounding itself moves the exact
    gradient by less than 1e-2 (it moves the conv gradient of the pooled chain by 5-8 %)."""
    params = wl.make_params(spec, seed=11, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=12)
    runner = StepRunner(spec, params)
    n = runner.n
    masks = [ck.mask_from_set(n, [0, n]), ck.plan(ck.ALGO_DYNAMIC_N, runner.d)[0]]
    rep0, g0 = all_policies_agree(runner, x, labels, masks, masks)
    stored = oracle_step(spec, params, x, labels, storage="bf16")
    exact = oracle_step(spec, params, x, labels)
    assert abs(rep0["loss"] - stored["loss"]) <= 1e-4 * abs(stored["loss"])
    assert abs(rep0["loss"] - exact["loss"]) <= 5e-3 * abs(exact["loss"])
    compare_with_oracle(runner, g0, stored, TOL["bf16"])
    for (ui, name, _), g in zip(runner.flat, g0):
        moved = max_rel_err(stored["grads"][ui][name], exact["grads"][ui][name])
        if moved <= 1e-2:
            assert max_rel_err(g.reshape(exact["grads"][ui][name].shape), exact["grads"][ui][name]) <= TOL["bf16"], (ui, name)


def test_ragged_chain_fp32():
    # odd spatial sizes and channel counts: nothing is a multiple of a tile or a vector width
    units = [wl.conv_unit(3, 7), wl.conv_unit(7, 13, k=3, stride=2, pad=1), {"kind": "maxpool", "k": 3, "stride": 2, "pad": 1},
             wl.conv_unit(13, 10, k=1, stride=1, pad=0), {"kind": "avgpool"}, {"kind": "fc", "cin": 10, "cout": 6, "relu": False}]
    spec = dict(units=units, input_hwc=(19, 23, 3), batch=3, dtype="f32", loss="softmax_ce", name="ragged")
    params = wl.make_params(spec, seed=5, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=6)
    runner = StepRunner(spec, params)
    n = runner.n
    masks = [ck.mask_from_set(n, [0, n]), ck.mask_from_set(n, [0, 2, 4, n]), ck.plan(ck.ALGO_DYNAMIC_N, runner.d)[0]]
    rep0, g0 = all_policies_agree(runner, x, labels, masks, masks)
    ref = oracle_step(spec, params, x, labels)
    compare_with_oracle(runner, g0, ref, TOL["f32"])


def mini_resnet(dtype, batch=4):
    """Stem (7x7 stride 2), 3x3 stride-2 max-pool, bottleneck blocks with and without projection and
    stride, global average pool, classifier: every unit kind of the ResNet configurations."""
    units = [wl.conv_unit(3, 8, k=7, stride=2, pad=3), {"kind": "maxpool", "k": 3, "stride": 2, "pad": 1},
             {"kind": "bottleneck", "cin": 8, "mid": 4, "cout": 16, "stride": 1, "project": True},
             {"kind": "bottleneck", "cin": 16, "mid": 4, "cout": 16, "stride": 1, "project": False},
             {"kind": "bottleneck", "cin": 16, "mid": 8, "cout": 32, "stride": 2, "project": True},
             {"kind": "bottleneck", "cin": 32, "mid": 8, "cout": 32, "stride": 1, "project": False},
             {"kind": "avgpool"}, {"kind": "fc", "cin": 32, "cout": 10, "relu": False}]
    return dict(units=units, input_hwc=(40, 36, 3), batch=batch, dtype=dtype, loss="softmax_ce", name="mini_resnet_" + dtype)


def test_mini_resnet_fp32_against_exact_oracle():
    spec = mini_resnet("f32")
    params = wl.make_params(spec, seed=21, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=22)
    runner = StepRunner(spec, params)
    n = runner.n
    masks = [ck.plan(ck.ALGO_DYNAMIC_N, runner.d)[0], ck.mask_from_set(n, [0, n]), ck.mask_from_set(n, [0, 3, 5, n])]
    rep0, g0 = all_policies_agree(runner, x, labels, masks, masks + [ck.plan(ck.ALGO_STATIC_N3, runner.d)[0]])
    ref = oracle_step(spec, params, x, labels)
    assert abs(rep0["loss"] - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    compare_with_oracle(runner, g0, ref, TOL["f32"])


def test_bottleneck_bf16_on_tensor_cores():
    """One block wide enough for the tcgen05 kernels (1x1 and 3x3, 64/256 channels), bf16, against the
    oracle with the same storage rounding."""
    units = [{"kind": "bottleneck", "cin": 64, "mid": 64, "cout": 256, "stride": 1, "project": True},
             {"kind": "bottleneck", "cin": 256, "mid": 64, "cout": 256, "stride": 1, "project": False},
             {"kind": "avgpool"}, {"kind": "fc", "cin": 256, "cout": 10, "relu": False}]
    spec = dict(units=units, input_hwc=(12, 12, 64), batch=8, dtype="bf16", loss="softmax_ce", name="blocks_bf16")
    params = wl.make_params(spec, seed=31, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=32)
    runner = StepRunner(spec, params)
    n = runner.n
    masks = [ck.mask_from_set(n, [0, n]), ck.plan(ck.ALGO_DYNAMIC_N, runner.d)[0]]
    rep0, g0 = all_policies_agree(runner, x, labels, masks, masks)
    exact = oracle_step(spec, params, x, labels)
    stored = oracle_step(spec, params, x, labels, storage="bf16")
    assert abs(rep0["loss"] - exact["loss"]) <= 2e-2 * abs(exact["loss"])
    for (ui, name, _), g in zip(runner.flat, g0):
        assert np.all(np.isfinite(g))
        mine = rel_l2(g, exact["grads"][ui][name])
        theirs = rel_l2(stored["grads"][ui][name], exact["grads"][ui][name])
        assert mine <= 1.5 * theirs + 0.02, (ui, name, mine, theirs)


def test_split_mini_vgg_fp32_against_exact_oracle():
    """Finer granularity (Section 5.4): conv, bn and relu as chain units of their own (39 + 8 units).
    Same function as the fused chain, so the oracle of the *split* chain and of the fused chain both
    apply; the arena follows the planner's prediction on the longer chain."""
    coarse = mini_vgg("f32")
    spec, origin = wl.split_units(coarse)
    cparams = wl.make_params(coarse, seed=3, bn_affine="random")
    params = wl.split_params(origin, cparams)
    x, labels = wl.make_batch(coarse, seed=4)
    runner = StepRunner(spec, params)
    n = runner.n
    assert n == len(coarse["units"]) + 2 * 13
    d = [int(v) for v in runner.d]
    m6, _ = ck.plan(ck.ALGO_DYNAMIC_N, d)
    m3, _ = ck.plan(ck.ALGO_STATIC_N3, d)
    rng = random.Random(2)
    extra = [ck.mask_from_set(n, [0] + [i for i in range(1, n) if rng.random() < 0.35] + [n]) for _ in range(4)]
    extra.append(ck.mask_from_set(n, [0, n]))
    rep0, g0 = all_policies_agree(runner, x, labels, [m6] + extra, [m3] + extra)
    ref = oracle_step(spec, params, x, labels)
    assert abs(rep0["loss"] - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    compare_with_oracle(runner, g0, ref, TOL["f32"])
    # and against the fused chain's oracle gradients, re-filed
    fused = oracle_step(coarse, cparams, x, labels)
    for (fi, name, _), g in zip(runner.flat, g0):
        want = fused["grads"][origin[fi][0]][name]
        assert max_rel_err(g.reshape(want.shape), want) <= TOL["f32"]


def test_split_shallow_bf16_chain():
    """bfloat16 split chain on the tensor-core kernels, element-wise against the storage-rounded oracle."""
    coarse = [c for c in shallow_chains() if c["name"] == "conv64+conv64+fc"][0]
    spec, origin = wl.split_units(coarse)
    params = wl.split_params(origin, wl.make_params(coarse, seed=11, bn_affine="random"))
    x, labels = wl.make_batch(coarse, seed=12)
    runner = StepRunner(spec, params)
    n = runner.n
    m6, _ = ck.plan(ck.ALGO_DYNAMIC_N, runner.d)
    rep0, g0 = all_policies_agree(runner, x, labels, [m6, ck.mask_from_set(n, [0, n]), ck.mask_from_set(n, [0, 2, 5, n])],
                                  [ck.mask_from_set(n, [0, 3, n])])
    ref = oracle_step(spec, params, x, labels, storage="bf16")
    assert abs(rep0["loss"] - ref["loss"]) <= 1e-2 * abs(ref["loss"])
    compare_with_oracle(runner, g0, ref, TOL["bf16"])


def test_arena_too_small_is_rejected_before_any_launch():
    spec = wl.config(1)
    runner = StepRunner(spec, wl.make_params(spec, seed=0))
    x, _ = wl.make_batch(spec, seed=1)
    mask, peak = ck.plan(ck.ALGO_DYNAMIC_N, runner.d)
    with pytest.raises(ck.CkptError) as e:
        runner.run(ck.POLICY_DYNAMIC, mask, x, None, arena_bytes=peak - 256)
    assert e.value.code == -7
    rep, _ = runner.run(ck.POLICY_DYNAMIC, mask, x, None, arena_bytes=peak)
    assert rep["peak_bytes"] == peak


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_graph_replay_is_bit_identical(dtype):
    """ckpt_chain_set_graph: the first step with a set of arguments runs launch by launch, the second is
    recorded, later ones replay the recording.  Same buffers, new batch contents each step: gradients,
    loss and report must equal those of a chain that never records."""
    import torch
    spec = mini_vgg(dtype)
    params = wl.make_params(spec, seed=41, bn_affine="random")
    plain, graphed = StepRunner(spec, params), StepRunner(spec, params)
    graphed.chain.set_graph(True)
    mask = ck.plan(ck.ALGO_DYNAMIC_N, plain.d)[0]
    peak = ck.eval(ck.MODEL_DYNAMIC, plain.d, mask)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    xb = torch.empty((spec["batch"],) + tuple(spec["input_hwc"]), dtype=tdt, device="cuda")
    lab = torch.empty(spec["batch"], dtype=torch.int32, device="cuda")
    arenas = [torch.empty(peak, dtype=torch.uint8, device="cuda") for _ in range(2)]
    replayed = []
    for step in range(5):
        x, labels = wl.make_batch(spec, seed=50 + step)
        xb.copy_(torch.from_numpy(x).to(tdt))
        lab.copy_(torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)))
        out = []
        for runner, arena in ((plain, arenas[0]), (graphed, arenas[1])):
            arena.fill_(0xFF)
            for g in runner.grads:
                g.fill_(float("nan"))
            rep = ck.train_step(runner.chain, mask, ck.POLICY_DYNAMIC, xb, lab, runner.params, runner.grads, arena, runner.workspace)
            torch.cuda.synchronize()
            out.append((rep, [g.detach().cpu().numpy().copy() for g in runner.grads]))
        (rep_a, g_a), (rep_b, g_b) = out
        replayed.append(rep_b["replayed"])
        assert rep_a["replayed"] == 0
        for key in ("peak_bytes", "extent_bytes", "predicted_bytes", "launches", "recomputed_units", "loss", "device_status"):
            assert rep_a[key] == rep_b[key], (step, key)
        for a, b in zip(g_a, g_b):
            assert np.array_equal(a, b)
    assert replayed == [0, 1, 1, 1, 1]
    # another plan is another recording; switching the feature off drops them
    mask2 = ck.mask_from_set(plain.n, [0, plain.n])
    arena2 = torch.empty(ck.eval(ck.MODEL_DYNAMIC, plain.d, mask2), dtype=torch.uint8, device="cuda")
    seq = [ck.train_step(graphed.chain, mask2, ck.POLICY_DYNAMIC, xb, lab, graphed.params, graphed.grads, arena2, graphed.workspace)["replayed"]
           for _ in range(3)]
    assert seq == [0, 1, 1]
    g_two = [g.detach().cpu().numpy().copy() for g in graphed.grads]
    graphed.chain.set_graph(False)
    rep = ck.train_step(graphed.chain, mask2, ck.POLICY_DYNAMIC, xb, lab, graphed.params, graphed.grads, arena2, graphed.workspace)
    torch.cuda.synchronize()
    assert rep["replayed"] == 0
    for a, b in zip(g_two, graphed.grads):
        assert np.array_equal(a, b.detach().cpu().numpy())


@pytest.mark.parametrize("graph", [False, True])
def test_staged_batches_equal_direct_steps(graph):
    """ckpt_chain_stage_batch: batches copied from pinned host memory on the chain's copy stream, one step ahead, give
    the gradients, loss and report of steps that are handed the same batches directly - launch by launch and through
    graph replay (one recording per staging slot)."""
    import torch
    spec = mini_vgg("bf16")
    params = wl.make_params(spec, seed=43, bn_affine="random")
    direct, staged = StepRunner(spec, params), StepRunner(spec, params)
    staged.chain.set_graph(graph)
    mask = ck.plan(ck.ALGO_DYNAMIC_N, direct.d)[0]
    peak = ck.eval(ck.MODEL_DYNAMIC, direct.d, mask)
    arenas = [torch.empty(peak, dtype=torch.uint8, device="cuda") for _ in range(2)]
    staging = torch.empty(staged.chain.staging_bytes(), dtype=torch.uint8, device="cuda")
    staging.fill_(0xFF)
    batches = []
    for step in range(6):
        x, labels = wl.make_batch(spec, seed=70 + step)
        batches.append((torch.from_numpy(x).to(torch.bfloat16).pin_memory(),
                        torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).pin_memory()))
    nxt = staged.chain.stage_batch(0, batches[0][0], batches[0][1], staging)
    replayed = []
    for step in range(6):
        cur = nxt
        if step + 1 < 6:
            nxt = staged.chain.stage_batch((step + 1) % 2, batches[step + 1][0], batches[step + 1][1], staging)
        for g in staged.grads + direct.grads:
            g.fill_(float("nan"))
        rep_s = ck.train_step(staged.chain, mask, ck.POLICY_DYNAMIC, cur[0], cur[1], staged.params, staged.grads, arenas[0], staged.workspace)
        rep_d = ck.train_step(direct.chain, mask, ck.POLICY_DYNAMIC, batches[step][0].cuda(), batches[step][1].cuda(), direct.params,
                              direct.grads, arenas[1], direct.workspace)
        torch.cuda.synchronize()
        replayed.append(rep_s["replayed"])
        for key in ("peak_bytes", "extent_bytes", "predicted_bytes", "recomputed_units", "loss", "device_status"):
            assert rep_s[key] == rep_d[key], (step, key)
        assert np.isfinite(rep_s["loss"])
        for a, b in zip(staged.grads, direct.grads):
            assert torch.equal(a, b)
    assert replayed == ([0, 0, 1, 1, 1, 1] if graph else [0] * 6)
    with pytest.raises(ck.CkptError) as e:
        staged.chain.stage_batch(0, batches[0][0], batches[0][1], staging[:-256])
    assert e.value.code == -8


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_store_all_that_keeps_block_interiors(dtype):
    """ckpt_chain_set_keep_interiors: a store-all step in which every residual block keeps its interior tensors from the
    forward pass (a region of its own per block) instead of re-deriving them in its backward gives the same loss and
    bit-identical gradients, launches fewer kernels, and leaves the checkpointed schedules as they were."""
    import torch
    if dtype == "f32":
        spec = mini_resnet("f32")
    else:
        units = [{"kind": "bottleneck", "cin": 64, "mid": 64, "cout": 256, "stride": 1, "project": True},
                 {"kind": "bottleneck", "cin": 256, "mid": 64, "cout": 256, "stride": 1, "project": False},
                 {"kind": "bottleneck", "cin": 256, "mid": 128, "cout": 512, "stride": 2, "project": True},
                 {"kind": "avgpool"}, {"kind": "fc", "cin": 512, "cout": 10, "relu": False}]
        spec = dict(units=units, input_hwc=(12, 12, 64), batch=8, dtype="bf16", loss="softmax_ce", name="blocks_keep")
    params = wl.make_params(spec, seed=51, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=52)
    plain, keeping = StepRunner(spec, params), StepRunner(spec, params)
    base_ws = keeping.chain.workspace_bytes()
    keeping.chain.set_keep_interiors(True)
    assert keeping.chain.workspace_bytes() > base_ws
    assert keeping.chain.workspace_bytes_for(ck.POLICY_DYNAMIC) == plain.chain.workspace_bytes_for(ck.POLICY_DYNAMIC)
    with pytest.raises(ck.CkptError) as e:                   # the old workspace is too small for the store-all policy now
        keeping.run(ck.POLICY_STORE_ALL, None, x, labels)
    assert e.value.code == -8
    keeping.workspace = torch.empty(keeping.chain.workspace_bytes(), dtype=torch.uint8, device="cuda")
    keeping.workspace.fill_(0xFF)
    rep_a, g_a = plain.run(ck.POLICY_STORE_ALL, None, x, labels)
    rep_b, g_b = keeping.run(ck.POLICY_STORE_ALL, None, x, labels)
    assert rep_a["loss"] == rep_b["loss"] and rep_b["device_status"] == 0
    assert rep_b["launches"] < rep_a["launches"]
    for a, b in zip(g_a, g_b):
        assert np.array_equal(a, b)
    mask = ck.plan(ck.ALGO_DYNAMIC_N, plain.d)[0]
    rep_c, g_c = keeping.run(ck.POLICY_DYNAMIC, mask, x, labels)
    rep_d, _ = plain.run(ck.POLICY_DYNAMIC, mask, x, labels)
    assert rep_c["launches"] == rep_d["launches"] and rep_c["peak_bytes"] == rep_d["peak_bytes"]
    for a, b in zip(g_a, g_c):
        assert np.array_equal(a, b)
