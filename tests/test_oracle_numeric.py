"""Pins for the numeric oracle: things fixed by mathematics or by an independent routine."""
import math

import numpy as np
import pytest
from scipy.signal import correlate2d

from oracle import numeric_oracle as no
from paper_2502_12499_b200 import workloads as wl


def test_round_bf16_bit_patterns():
    # 1 + 2^-8 is exactly halfway between two bfloat16 values: ties go to even (1.0);
    # 1 + 3*2^-8 is halfway as well and goes up to 1 + 2^-6.
    assert no.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert no.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert no.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -20]))[0] == 1.0 + 2.0 ** -7
    assert no.round_bf16(np.array([-3.140625]))[0] == -3.140625          # already representable
    x = np.random.default_rng(0).standard_normal(1000)
    r = no.round_bf16(x)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(r.astype(np.float32), wl.to_bf16_representable(x.astype(np.float32)))


def conv_loops(x, w, stride, pad):
    n, h, wd, cin = x.shape
    cout, k, _, _ = w.shape
    ho = (h + 2 * pad - k) // stride + 1
    wo = (wd + 2 * pad - k) // stride + 1
    z = np.zeros((n, ho, wo, cout))
    for b in range(n):
        for oh in range(ho):
            for ow in range(wo):
                for co in range(cout):
                    acc = 0.0
                    for r in range(k):
                        for s in range(k):
                            ih, iw = oh * stride - pad + r, ow * stride - pad + s
                            if 0 <= ih < h and 0 <= iw < wd:
                                for ci in range(cin):
                                    acc += x[b, ih, iw, ci] * w[co, r, s, ci]
                    z[b, oh, ow, co] = acc
    return z


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (1, 1, 0), (1, 2, 0), (5, 2, 2)])
def test_conv_against_loop_definition(k, stride, pad):
    rng = np.random.default_rng(k * 10 + stride)
    x = rng.standard_normal((2, 6, 5, 3))
    w = rng.standard_normal((4, k, k, 3))
    assert np.allclose(no.conv2d_fwd(x, w, stride, pad), conv_loops(x, w, stride, pad), atol=1e-12)


def test_conv_against_scipy_correlate():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 9, 7, 1))
    w = rng.standard_normal((1, 3, 3, 1))
    got = no.conv2d_fwd(x, w, 1, 1)[0, :, :, 0]
    want = correlate2d(x[0, :, :, 0], w[0, :, :, 0], mode="same", boundary="fill")
    assert np.allclose(got, want, atol=1e-12)
    # a transposed or flipped filter must not pass
    assert not np.allclose(got, correlate2d(x[0, :, :, 0], w[0, ::-1, ::-1, 0], mode="same"))


def test_maxpool_against_loops_and_first_max_rule():
    rng = np.random.default_rng(4)
    x = rng.integers(0, 3, size=(2, 7, 6, 2)).astype(np.float64)          # many ties
    for k, stride, pad in [(2, 2, 0), (3, 2, 1)]:
        y, arg = no.maxpool_fwd(x, k, stride, pad)
        dy = rng.standard_normal(y.shape)
        dx = no.maxpool_bwd(dy, arg, x.shape, k, stride, pad)
        want = np.zeros_like(x)
        n, h, w, c = x.shape
        for b in range(n):
            for oh in range(y.shape[1]):
                for ow in range(y.shape[2]):
                    for ch in range(c):
                        best, pos = -math.inf, None
                        for r in range(k):
                            for s in range(k):
                                ih, iw = oh * stride - pad + r, ow * stride - pad + s
                                if 0 <= ih < h and 0 <= iw < w and x[b, ih, iw, ch] > best:
                                    best, pos = x[b, ih, iw, ch], (ih, iw)
                        assert y[b, oh, ow, ch] == best
                        want[b, pos[0], pos[1], ch] += dy[b, oh, ow, ch]
        assert np.allclose(dx, want)


def test_batchnorm_properties():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((3, 4, 5, 6)) * 3 + 1
    gamma = rng.uniform(0.5, 1.5, 6)
    beta = rng.standard_normal(6)
    y, cache = no.bn_fwd(z, gamma, beta)
    # normalised output has mean beta and biased variance gamma^2 * var/(var+eps)
    assert np.allclose(y.mean(axis=(0, 1, 2)), beta, atol=1e-12)
    var = z.var(axis=(0, 1, 2))
    assert np.allclose(y.var(axis=(0, 1, 2)), gamma ** 2 * var / (var + no.EPS), rtol=1e-12)
    # a constant upstream gradient carries no information through the normalisation
    dz, dgamma, dbeta = no.bn_bwd(np.full_like(z, 0.7), cache, gamma)
    assert np.allclose(dz, 0.0, atol=1e-12)
    assert np.allclose(dbeta, 0.7 * 60)
    assert np.allclose(dgamma, 0.0, atol=1e-10)


def test_softmax_hand_values():
    logits = np.array([[0.0, math.log(3.0)], [math.log(2.0), 0.0]]).reshape(2, 1, 1, 2)
    loss, g = no.softmax_ce(logits, np.array([1, 1]))
    assert math.isclose(loss, 0.5 * (-math.log(0.75) - math.log(1.0 / 3.0)))
    assert np.allclose(g.reshape(2, 2), np.array([[0.25, -0.25], [2 / 3, -2 / 3]]) / 2)


def tiny_chains():
    yield wl.plain_chain(3, 4, 2, (5, 4), 3, "f32", "sum", name="plain3")
    units = [wl.conv_unit(2, 4), {"kind": "maxpool", "k": 2, "stride": 2, "pad": 0},
             wl.conv_unit(4, 4, k=3, stride=2, pad=1),
             {"kind": "fc", "cin": 2 * 2 * 4, "cout": 6, "relu": True},
             {"kind": "fc", "cin": 6, "cout": 5, "relu": False}]
    yield dict(units=units, input_hwc=(8, 6, 2), batch=3, dtype="f32", loss="softmax_ce", name="mini_vgg")
    units = [wl.conv_unit(2, 4, k=5, stride=2, pad=2), {"kind": "maxpool", "k": 3, "stride": 2, "pad": 1},
             {"kind": "bottleneck", "cin": 4, "mid": 2, "cout": 8, "stride": 1, "project": True},
             {"kind": "bottleneck", "cin": 8, "mid": 2, "cout": 8, "stride": 1, "project": False},
             {"kind": "bottleneck", "cin": 8, "mid": 4, "cout": 16, "stride": 2, "project": True},
             {"kind": "avgpool"}, {"kind": "fc", "cin": 16, "cout": 5, "relu": False}]
    yield dict(units=units, input_hwc=(16, 12, 2), batch=2, dtype="f32", loss="softmax_ce", name="mini_resnet")


@pytest.mark.parametrize("chain", list(tiny_chains()), ids=lambda c: c["name"])
def test_gradients_by_central_differences(chain):
    params = wl.make_params(chain, seed=7, bn_affine="random")
    params = [{k: v.astype(np.float64) for k, v in p.items()} for p in params]
    x, labels = wl.make_batch(chain, seed=8)
    x = x.astype(np.float64)
    out = no.chain_forward_backward(chain, params, x, labels)
    rng = np.random.default_rng(9)
    h = 1e-6

    def loss_at():
        d, _, _ = no.chain_forward(chain, params, x)
        return no.loss_and_grad(chain, d[-1], labels)[0]

    checked = 0
    for ui, p in enumerate(params):
        for name, arr in p.items():
            flat = arr.reshape(-1)
            for idx in rng.choice(flat.size, size=min(3, flat.size), replace=False):
                keep = flat[idx]
                flat[idx] = keep + h
                lp = loss_at()
                flat[idx] = keep - h
                lm = loss_at()
                flat[idx] = keep
                fd = (lp - lm) / (2 * h)
                an = out["grads"][ui][name].reshape(-1)[idx]
                assert abs(fd - an) <= 2e-5 * max(1.0, abs(an)), (chain["name"], ui, name, idx, fd, an)
                checked += 1
    # gradient w.r.t. the input as well (exercises every dgrad)
    flat = x.reshape(-1)
    for idx in rng.choice(flat.size, size=4, replace=False):
        keep = flat[idx]
        flat[idx] = keep + h
        lp = loss_at()
        flat[idx] = keep - h
        lm = loss_at()
        flat[idx] = keep
        assert abs((lp - lm) / (2 * h) - out["input_grad"].reshape(-1)[idx]) <= 2e-5
    assert checked >= 9


def test_output_shapes_match_forward():
    for chain in tiny_chains():
        params = wl.make_params(chain, seed=1)
        x, _ = wl.make_batch(chain, seed=2)
        d, _, _ = no.chain_forward(chain, params, x)
        assert [t.shape[1:] for t in d] == no.output_shapes(chain)


def test_bf16_storage_mode_rounds_stored_tensors_only():
    """storage="bf16": every stored tensor is a bfloat16 code, the arithmetic stays float64, and on
    a one-unit chain the result stays within a few roundings of the exact one."""
    spec = wl.plain_chain(1, 8, 4, (6, 6), 8, "bf16", "softmax_ce")
    spec["units"].append({"kind": "fc", "cin": 6 * 6 * 8, "cout": 5, "relu": False})
    params = wl.make_params(spec, seed=1, bn_affine="random")
    params = [{k: v.astype(np.float64) for k, v in p.items()} for p in params]
    x, labels = wl.make_batch(spec, seed=2)
    exact = no.chain_forward_backward(spec, params, x.astype(np.float64), labels)
    stored = no.chain_forward_backward(spec, params, x.astype(np.float64), labels, storage="bf16")
    for t in stored["d"]:
        assert np.array_equal(t, no.round_bf16(t))
    assert not np.array_equal(exact["d"][1], no.round_bf16(exact["d"][1]))
    # conv output of unit 1: stored = round(exact conv), nothing else
    z_exact = no.conv2d_fwd(x.astype(np.float64), params[0]["w"], 1, 1)
    y_stored, _ = no.bn_fwd(no.round_bf16(z_exact), params[0]["gamma"], params[0]["beta"])
    assert np.array_equal(stored["d"][1], no.round_bf16(np.maximum(y_stored, 0)))
    for ge, gs in zip(exact["grads"], stored["grads"]):
        for k in ge:
            assert np.abs(ge[k] - gs[k]).max() <= 3e-2 * np.abs(ge[k]).max()
    assert abs(exact["loss"] - stored["loss"]) <= 5e-3 * abs(exact["loss"])


def test_split_chain_equals_fused_chain():
    """Finer granularity (Section 5.4): conv, bn and relu as chain units of their own compute the same
    function as the fused unit, so every gradient agrees to rounding; and the central-difference check
    runs on the split chain too (it exercises the three new unit kinds by themselves)."""
    for chain in tiny_chains():
        if not any(u["kind"] == "conv_bn_relu" for u in chain["units"]):
            continue
        fine, origin = wl.split_units(chain)
        params = [{k: v.astype(np.float64) for k, v in p.items()} for p in wl.make_params(chain, seed=3, bn_affine="random")]
        fparams = wl.split_params(origin, params)
        x, labels = wl.make_batch(chain, seed=4)
        a = no.chain_forward_backward(chain, params, x.astype(np.float64), labels)
        b = no.chain_forward_backward(fine, fparams, x.astype(np.float64), labels)
        assert len(fine["units"]) > len(chain["units"])
        assert abs(a["loss"] - b["loss"]) <= 1e-12 * max(1.0, abs(a["loss"]))
        np.testing.assert_allclose(a["input_grad"], b["input_grad"], rtol=0, atol=1e-12)
        for fi, (ui, names) in enumerate(origin):
            for name in names:
                if name in params[ui]:
                    np.testing.assert_allclose(b["grads"][fi][name], a["grads"][ui][name], rtol=0, atol=1e-11)
        shapes = no.output_shapes(fine)
        assert [t.shape[1:] for t in b["d"]] == shapes
        # a relu unit's output is its input clipped; a bn unit's output has per-channel mean beta
        for fi, u in enumerate(fine["units"]):
            if u["kind"] == "relu":
                assert np.array_equal(b["d"][fi + 1], np.maximum(b["d"][fi], 0))
            if u["kind"] == "bn":
                np.testing.assert_allclose(b["d"][fi + 1].mean(axis=(0, 1, 2)), fparams[fi]["beta"], atol=1e-12)


def test_sgd_update_is_a_descent_step():
    """"Update w_i with g_i" as w - lr*g: hand values, and along -g the float64 loss of a tiny chain goes down by
    lr * |g|^2 to first order."""
    new = no.sgd_update([{"w": np.array([1.0, -2.0]), "b": np.array([0.5])}], [{"w": np.array([0.5, 0.25]), "b": np.array([-1.0])}], 0.1)
    assert np.allclose(new[0]["w"], [0.95, -2.025]) and np.allclose(new[0]["b"], [0.6])
    rounded = no.sgd_update([{"w": np.array([1.0 + 2.0 ** -9]), "gamma": np.array([1.0 + 2.0 ** -9])}],
                            [{"w": np.array([0.0]), "gamma": np.array([0.0])}], 0.1, storage="bf16")
    assert rounded[0]["w"][0] == 1.0 and rounded[0]["gamma"][0] == 1.0 + 2.0 ** -9      # only matrices are stored in bf16
    from paper_2502_12499_b200 import workloads as wl
    spec = wl.plain_chain(2, 4, 3, (6, 6), 2, "f32", "softmax_ce", name="tiny")
    spec["units"].append({"kind": "fc", "cin": 6 * 6 * 4, "cout": 5, "relu": False})
    params = [{k: v.astype(np.float64) for k, v in p.items()} for p in wl.make_params(spec, seed=2, bn_affine="random")]
    x, labels = wl.make_batch(spec, seed=3)
    ref = no.chain_forward_backward(spec, params, x.astype(np.float64), labels)
    lr = 1e-4
    after = no.chain_forward_backward(spec, no.sgd_update(params, ref["grads"], lr), x.astype(np.float64), labels)
    g2 = sum(float((g ** 2).sum()) for unit in ref["grads"] for g in unit.values())
    assert after["loss"] < ref["loss"]
    assert abs((ref["loss"] - after["loss"]) - lr * g2) <= 0.05 * lr * g2
