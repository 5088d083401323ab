"""ckpt_chain_set_sgd: the step's parameter update ("update w_i with g_i", last line of the backward loop of
Algorithms 1, 2 and 4) against the oracle's w - lr*g, and the gradients unchanged by it."""
import numpy as np
import pytest

from oracle import numeric_oracle as no
from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import StepRunner, max_rel_err

pytestmark = pytest.mark.gpu


def chains():
    yield wl.vgg16_chain(4, hw=(32, 32), dtype="f32", widths=(8, 16, 24, 32, 32), fc_width=48, classes=10, name="mini_vgg_f32")
    # tensor-core kernels: split wgrad with the fused update (128 channels: shared-taps kernel; 64: pixel pairs), first layer, FC
    s = dict(units=[wl.conv_unit(3, 64), wl.conv_unit(64, 64), {"kind": "maxpool", "k": 2, "stride": 2, "pad": 0}, wl.conv_unit(64, 128),
                    wl.conv_unit(128, 128), {"kind": "avgpool"}, {"kind": "fc", "cin": 128, "cout": 10, "relu": False}],
             input_hwc=(32, 32, 3), batch=8, dtype="bf16", loss="softmax_ce", name="convs_bf16")
    yield s
    s = dict(units=[{"kind": "bottleneck", "cin": 64, "mid": 64, "cout": 256, "stride": 1, "project": True},
                    {"kind": "bottleneck", "cin": 256, "mid": 128, "cout": 512, "stride": 2, "project": True},
                    {"kind": "avgpool"}, {"kind": "fc", "cin": 512, "cout": 10, "relu": False}],
             input_hwc=(16, 16, 64), batch=8, dtype="bf16", loss="softmax_ce", name="blocks_bf16")
    yield s


@pytest.mark.parametrize("spec", list(chains()), ids=lambda s: s["name"])
def test_step_updates_parameters(spec):
    import torch
    lr = 0.05
    params = wl.make_params(spec, seed=7, bn_affine="random")
    x, labels = wl.make_batch(spec, seed=8)
    runner = StepRunner(spec, params)
    mask = ck.plan(ck.ALGO_DYNAMIC_N, runner.d)[0]
    before = [t.detach().float().cpu().numpy().astype(np.float64) for t in runner.params]
    rep0, g0 = runner.run(ck.POLICY_DYNAMIC, mask, x, labels)                  # no update: parameters untouched
    for a, t in zip(before, runner.params):
        assert np.array_equal(a, t.detach().float().cpu().numpy())
    runner.chain.set_sgd(lr)
    ck.launch_log(True)
    rep1, g1 = runner.run(ck.POLICY_DYNAMIC, mask, x, labels)
    kernels = ck.launch_log_read()
    ck.launch_log(False)
    assert rep1["loss"] == rep0["loss"]
    for a, b in zip(g0, g1):
        assert np.array_equal(a, b)                                            # same gradients, bit for bit
    storage = "bf16" if spec["dtype"] == "bf16" else "exact"
    grads = [dict() for _ in spec["units"]]
    olds = [dict() for _ in spec["units"]]
    for (ui, name, _), g, w in zip(runner.flat, g1, before):
        grads[ui][name] = g.astype(np.float64)
        olds[ui][name] = w.reshape(g.shape)
    want = no.sgd_update(olds, grads, lr, storage)
    for (ui, name, _), t in zip(runner.flat, runner.params):
        got = t.detach().float().cpu().numpy().astype(np.float64).reshape(want[ui][name].shape)
        scale = np.abs(want[ui][name]).max()
        if t.dtype == torch.bfloat16:
            # float32 arithmetic before the rounding: at most the neighbouring bfloat16 code
            assert np.abs(got - want[ui][name]).max() <= 2.0 ** -7 * scale, (ui, name)
            assert np.mean(got != want[ui][name]) <= 1e-3, (ui, name)
        else:
            assert np.abs(got - want[ui][name]).max() <= 1e-6 * max(scale, 1e-30), (ui, name)
        assert np.any(got != olds[ui][name]), (ui, name)                        # every parameter moved
    if spec["dtype"] == "bf16":
        assert any("slice_sum" in k or "pairview_fold" in k for k in kernels), sorted(kernels)
    # a second step starts from the updated parameters: its loss is that of the oracle at those parameters
    runner.chain.set_sgd(0.0)
    rep2, _ = runner.run(ck.POLICY_STORE_ALL, None, x, labels)
    new_params = [{k: v for k, v in q.items()} for q in want]
    ref = no.chain_forward_backward(spec, new_params, x.astype(np.float64), labels, storage=storage)
    assert abs(rep2["loss"] - ref["loss"]) <= (1e-4 if storage == "exact" else 2e-2) * abs(ref["loss"])
    assert rep2["loss"] != rep0["loss"]
