"""Full-size checks, in the launch configuration bench.py times.

* the tensor-core convolution kernels at the VGG-16 / batch-64 layer shapes, on sampled outputs that
  the oracle computes one by one (a cropped neighbourhood for forward/dgrad, one (c_out, c_in)
  channel pair over all pixels for wgrad), and the fully connected layers of the VGG-16 head on
  sampled output rows and input columns; the same for the layer shapes of the residual networks at their
  benchmark batches (7x7 stride-2 stem, 1x1 layers, strided 3x3 and 1x1 layers);
* the whole checkpointed step of configurations 2, 3, 4 and 5 through properties that hold at any size:
  arena high-water == highest offset == planner's prediction (arena of exactly that size),
  gradients bit-identical between the checkpointed and the store-all schedule, finite loss;
* configuration 2 as bench.py submits it: replayed from its recorded CUDA graph, and fed from pinned host buffers."""
import time

import numpy as np
import pytest

from oracle import numeric_oracle as no
from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import StepRunner

pytestmark = pytest.mark.gpu

LAYERS = [
    # n, h, w, cin, cout   (3x3, stride 1, padding 1)
    (64, 224, 224, 3, 64),       # first layer: operand tiles gathered by threads
    (64, 224, 224, 64, 64),
    (64, 112, 112, 64, 128),
    (64, 112, 112, 128, 128),
    (64, 56, 56, 128, 256),
    (64, 56, 56, 256, 256),
    (64, 28, 28, 256, 512),
    (64, 28, 28, 512, 512),
    (64, 14, 14, 512, 512),
    (32, 56, 56, 64, 64),        # the unit of the 1000-layer chain
]


def bf16_host(t):
    """Exact float64 copy of a bf16 device tensor."""
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("layer", LAYERS, ids=lambda l: "x".join(map(str, l)))
def test_conv_kernels_full_size_sampled(layer):
    import torch
    n, h, w, cin, cout = layer
    dt = ck.DTYPE_BF16
    gen = torch.Generator(device="cuda").manual_seed(n * h + cin)
    x = torch.randn(n, h, w, cin, device="cuda", generator=gen).bfloat16()
    wt = (torch.randn(cout, 3, 3, cin, device="cuda", generator=gen) / (3.0 * cin ** 0.5)).bfloat16()
    dz = torch.randn(n, h, w, cout, device="cuda", generator=gen).bfloat16()
    shape = ck.ConvShape(n, h, w, cin, cout, 3, 1, 1)
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, dt)), dtype=torch.uint8, device="cuda")
    z = torch.empty(n, h, w, cout, device="cuda", dtype=torch.bfloat16)
    dx = torch.empty_like(x)
    dw = torch.empty(cout, 3, 3, cin, device="cuda")
    ck.conv2d_forward(shape, dt, 0, x, wt, z, scratch)
    ck.conv2d_dgrad(shape, dt, 0, dz, wt, dx, scratch)
    ck.conv2d_wgrad(shape, dt, 0, dz, x, dw, scratch)
    torch.cuda.synchronize()
    w64 = bf16_host(wt)
    rng = np.random.default_rng(7)
    # corners, edges (tile and image borders) and random interior pixels
    picks = [(0, 0, 0), (n - 1, h - 1, w - 1), (n // 2, 0, w - 1), (n - 1, h - 1, 0), (1, h // 2, w // 2 + 1)]
    picks += [(int(rng.integers(n)), int(rng.integers(h)), int(rng.integers(w))) for _ in range(11)]
    scale_z = float(z.float().abs().max())
    scale_dx = float(dx.float().abs().max())
    for (b, i, j) in picks:
        lo_i, hi_i, lo_j, hi_j = max(i - 2, 0), min(i + 3, h), max(j - 2, 0), min(j + 3, w)
        xc = bf16_host(x[b:b + 1, lo_i:hi_i, lo_j:hi_j, :])
        dzc = bf16_host(dz[b:b + 1, lo_i:hi_i, lo_j:hi_j, :])
        z_ref = no.conv2d_fwd(xc, w64, 1, 1)[0, i - lo_i, j - lo_j, :]
        dx_ref = no.conv2d_bwd(xc, w64, dzc, 1, 1)[0][0, i - lo_i, j - lo_j, :]
        assert np.abs(bf16_host(z[b, i, j, :]) - z_ref).max() <= 6e-3 * scale_z
        assert np.abs(bf16_host(dx[b, i, j, :]) - dx_ref).max() <= 6e-3 * scale_dx
    scale_dw = float(dw.abs().max())
    for _ in range(3):
        co, ci = int(rng.integers(cout)), int(rng.integers(cin))
        xs = bf16_host(x[..., ci:ci + 1])
        dzs = bf16_host(dz[..., co:co + 1])
        dw_ref = no.conv2d_bwd(xs, np.zeros((1, 3, 3, 1)), dzs, 1, 1)[1][0, :, :, 0]
        assert np.abs(dw[co, :, :, ci].cpu().numpy().astype(np.float64) - dw_ref).max() <= 2e-5 * max(scale_dw, np.abs(dw_ref).max())


FC_LAYERS = [(64, 25088, 4096), (64, 4096, 4096), (64, 4096, 1000)]      # batch, inputs, outputs of the VGG-16 head


@pytest.mark.parametrize("layer", FC_LAYERS, ids=lambda l: "x".join(map(str, l)))
def test_fc_kernels_full_size_sampled(layer):
    """A fully connected layer is a 1x1 convolution on a 1x1 image: sampled outputs, input gradients and
    weight gradients against the oracle's convolution on the rows and columns they depend on."""
    import torch
    n, cin, cout = layer
    dt = ck.DTYPE_BF16
    gen = torch.Generator(device="cuda").manual_seed(cin + cout)
    x = torch.randn(n, 1, 1, cin, device="cuda", generator=gen).bfloat16()
    wt = (torch.randn(cout, 1, 1, cin, device="cuda", generator=gen) / cin ** 0.5).bfloat16()
    dz = torch.randn(n, 1, 1, cout, device="cuda", generator=gen).bfloat16()
    shape = ck.ConvShape(n, 1, 1, cin, cout, 1, 1, 0)
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, dt)), dtype=torch.uint8, device="cuda")
    z = torch.empty(n, 1, 1, cout, device="cuda", dtype=torch.bfloat16)
    dx = torch.empty_like(x)
    dw = torch.empty(cout, 1, 1, cin, device="cuda")
    ck.conv2d_forward(shape, dt, 0, x, wt, z, scratch)
    ck.conv2d_dgrad(shape, dt, 0, dz, wt, dx, scratch)
    ck.conv2d_wgrad(shape, dt, 0, dz, x, dw, scratch)
    torch.cuda.synchronize()
    rng = np.random.default_rng(11)
    x64, dz64 = bf16_host(x), bf16_host(dz)
    scale_z, scale_dx, scale_dw = float(z.float().abs().max()), float(dx.float().abs().max()), float(dw.abs().max())
    outs = sorted({0, cout - 1, 127, 128, *map(int, rng.integers(cout, size=12))})
    z_ref = no.conv2d_fwd(x64, bf16_host(wt[outs]), 1, 0)                              # [n,1,1,len(outs)]
    assert np.abs(bf16_host(z[..., outs]) - z_ref).max() <= 6e-3 * scale_z
    # weight gradient of the sampled output rows (all inputs), and input gradient of sampled input columns
    dw_ref = no.conv2d_bwd(x64, np.zeros((len(outs), 1, 1, cin)), dz64[..., outs], 1, 0)[1]
    assert np.abs(dw[outs].cpu().numpy().astype(np.float64) - dw_ref).max() <= 2e-5 * max(scale_dw, np.abs(dw_ref).max())
    ins = sorted({0, cin - 1, 63, 64, *map(int, rng.integers(cin, size=12))})
    dx_ref = no.conv2d_bwd(np.zeros((n, 1, 1, len(ins))), bf16_host(wt[..., ins]), dz64, 1, 0)[0]
    assert np.abs(bf16_host(dx[..., ins]) - dx_ref).max() <= 6e-3 * scale_dx


RESNET_LAYERS = [
    # n, h, w, cin, cout, k, stride, pad: layer shapes of the residual networks at their benchmark batches
    (128, 224, 224, 3, 64, 7, 2, 3),     # stem: operand tiles gathered from staged input rows
    (128, 56, 56, 64, 256, 1, 1, 0),     # 1x1, short reduction (role-swapped kernel, epilogue-bound)
    (128, 56, 56, 256, 64, 1, 1, 0),     # 1x1, 64 output channels
    (128, 56, 56, 128, 128, 3, 2, 1),    # 3x3 stride 2: strided boxes forward, parity classes for dgrad
    (128, 56, 56, 256, 512, 1, 2, 0),    # 1x1 stride-2 projection
    (256, 14, 14, 256, 1024, 1, 1, 0),   # the layers ResNet-152 spends its time in
    (256, 14, 14, 1024, 256, 1, 1, 0),
    (256, 14, 14, 256, 256, 3, 1, 1),
    (128, 7, 7, 512, 512, 3, 1, 1),
]


def crop_range(o, size_out, size_in, k, stride, pad, lo_out, hi_out):
    """Output rows [a, b) around [lo_out, hi_out] and the input rows [a * stride, end) such that the oracle's
    convolution of the cropped input (same stride and padding) has exactly the output rows a .. b - 1 of the full
    convolution, and is exact on rows lo_out .. hi_out: the crop starts on a multiple of the stride (or at the image
    border, where the oracle's zero padding is the real one) far enough above, and ends at the image border or after
    the last row the window of output b - 1 reads."""
    margin = -(-pad // stride) + 1
    a = max(0, lo_out - margin)
    b = min(size_out, hi_out + margin + 1)
    start = a * stride
    end = size_in if b == size_out else start + (b - a - 1) * stride + k - 2 * pad
    # rows the oracle pads below the crop stand for real rows: keep output hi_out's window inside the crop
    while b < size_out and hi_out * stride - pad + k > end:
        b += 1
        end = size_in if b == size_out else start + (b - a - 1) * stride + k - 2 * pad
    assert (end - start + 2 * pad - k) // stride + 1 == b - a
    return a, b, start, end


@pytest.mark.parametrize("layer", RESNET_LAYERS, ids=lambda l: "x".join(map(str, l)))
def test_resnet_conv_kernels_full_size_sampled(layer):
    """The convolution kernels at the residual networks' layer shapes and batches (7x7 stem, 1x1, strided 3x3 and
    1x1): sampled output pixels and input-gradient pixels against the oracle's convolution of a cropped neighbourhood,
    sampled (c_out, c_in) pairs of the weight gradient against the oracle over all pixels."""
    import torch
    n, h, w, cin, cout, k, stride, pad = layer
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    dt = ck.DTYPE_BF16
    gen = torch.Generator(device="cuda").manual_seed(n * h + cin + k)
    x = torch.randn(n, h, w, cin, device="cuda", generator=gen).bfloat16()
    wt = (torch.randn(cout, k, k, cin, device="cuda", generator=gen) / (k * cin ** 0.5)).bfloat16()
    dz = torch.randn(n, ho, wo, cout, device="cuda", generator=gen).bfloat16()
    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, dt)), dtype=torch.uint8, device="cuda")
    z = torch.empty(n, ho, wo, cout, device="cuda", dtype=torch.bfloat16)
    dx = torch.empty_like(x)
    dw = torch.empty(cout, k, k, cin, device="cuda")
    ck.launch_log(True)
    try:
        ck.conv2d_forward(shape, dt, 0, x, wt, z, scratch)
        if cin > 3:
            ck.conv2d_dgrad(shape, dt, 0, dz, wt, dx, scratch)
        ck.conv2d_wgrad(shape, dt, 0, dz, x, dw, scratch)
        torch.cuda.synchronize()
    finally:
        kernels = ck.launch_log_read()
        ck.launch_log(False)
    assert ck.op_status() == 0
    assert not [name for name in kernels if "CUDA cores" in name or "conv_gemm" in name], kernels
    w64 = bf16_host(wt)
    rng = np.random.default_rng(13)
    scale_z = float(z.float().abs().max())
    # forward: corners, borders and random output pixels
    picks = [(0, 0, 0), (n - 1, ho - 1, wo - 1), (n // 2, 0, wo - 1), (n - 1, ho - 1, 0), (1, ho // 2, wo // 2)]
    picks += [(int(rng.integers(n)), int(rng.integers(ho)), int(rng.integers(wo))) for _ in range(9)]
    for (b, oi, oj) in picks:
        a_i, b_i, s_i, e_i = crop_range(oi, ho, h, k, stride, pad, oi, oi)
        a_j, b_j, s_j, e_j = crop_range(oj, wo, w, k, stride, pad, oj, oj)
        z_crop = no.conv2d_fwd(bf16_host(x[b:b + 1, s_i:e_i, s_j:e_j, :]), w64, stride, pad)
        assert z_crop.shape[1:3] == (b_i - a_i, b_j - a_j)
        assert np.abs(bf16_host(z[b, oi, oj, :]) - z_crop[0, oi - a_i, oj - a_j, :]).max() <= 6e-3 * scale_z, (b, oi, oj)
    # input gradient: every output pixel whose window reaches the input pixel lies inside the crop
    if cin > 3:
        scale_dx = float(dx.float().abs().max())
        picks = [(0, 0, 0), (n - 1, h - 1, w - 1), (n // 2, 0, w - 1), (n - 1, h - 1, 0), (1, h // 2 + 1, w // 2)]
        picks += [(int(rng.integers(n)), int(rng.integers(h)), int(rng.integers(w))) for _ in range(9)]
        for (b, i, j) in picks:
            rng_o = []
            for pos, size_o in ((i, ho), (j, wo)):
                lo = max(0, -(-(pos + pad - k + 1) // stride))
                hi = min(size_o - 1, (pos + pad) // stride)
                rng_o.append((lo, max(lo, hi)))
            a_i, b_i, s_i, e_i = crop_range(i, ho, h, k, stride, pad, *rng_o[0])
            a_j, b_j, s_j, e_j = crop_range(j, wo, w, k, stride, pad, *rng_o[1])
            if not (s_i <= i < e_i and s_j <= j < e_j):
                continue                                    # an input pixel no window reaches (stride-2 1x1): checked below
            xc = np.zeros((1, e_i - s_i, e_j - s_j, cin))
            dx_crop = no.conv2d_bwd(xc, w64, bf16_host(dz[b:b + 1, a_i:b_i, a_j:b_j, :]), stride, pad)[0]
            assert np.abs(bf16_host(dx[b, i, j, :]) - dx_crop[0, i - s_i, j - s_j, :]).max() <= 6e-3 * scale_dx, (b, i, j)
        if k == 1 and stride == 2:
            assert float(dx[:, 1::2, :, :].float().abs().max()) == 0.0 and float(dx[:, :, 1::2, :].float().abs().max()) == 0.0
    # weight gradient: sampled (c_out, c_in) pairs over all pixels
    scale_dw = float(dw.abs().max())
    for _ in range(2):
        co, ci = int(rng.integers(cout)), int(rng.integers(cin))
        dw_ref = no.conv2d_bwd(bf16_host(x[..., ci:ci + 1]), np.zeros((1, k, k, 1)), bf16_host(dz[..., co:co + 1]), stride, pad)[1][0, :, :, 0]
        assert np.abs(dw[co, :, :, ci].cpu().numpy().astype(np.float64) - dw_ref).max() <= 2e-5 * max(scale_dw, np.abs(dw_ref).max()), (co, ci)
    del x, z, dx, dz, dw, scratch
    torch.cuda.empty_cache()


def step_properties(spec, seed=0, finite_last_units=None):

    import torch
    params = wl.make_params(spec, seed=seed)
    x, labels = wl.make_batch(spec, seed=seed + 1)
    runner = StepRunner(spec, params)
    del params
    d = runner.d
    mask, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
    if spec["loss"] != "softmax_ce":
        labels = None
    rep, g = runner.run(ck.POLICY_DYNAMIC, mask, x, labels)
    assert rep["peak_bytes"] == rep["extent_bytes"] == rep["predicted_bytes"] == peak
    assert rep["device_status"] == 0 and np.isfinite(rep["loss"])
    assert rep["recomputed_units"] == runner.n + 1 - int(mask.sum())
    rep0, g0 = runner.run(ck.POLICY_STORE_ALL, None, x, labels)
    assert rep0["peak_bytes"] == int(d.sum())
    assert rep0["loss"] == rep["loss"]
    for (ui, name, _), a, b in zip(runner.flat, g, g0):
        if finite_last_units is None or ui >= runner.n - finite_last_units:
            assert np.all(np.isfinite(a)), (ui, name)
        assert np.array_equal(a, b, equal_nan=True)     # checkpointed == store-all, bit for bit
    # the set bench.py runs: same peak, least recomputation (the canonical set above when nothing is cheaper)
    mask_mr, peak_mr, _ = ck.plan_min_recompute(d, runner.chain.unit_costs())
    assert peak_mr == peak and int(mask_mr.sum()) >= int(mask.sum())
    if not np.array_equal(mask_mr, mask):
        rep_mr, g_mr = runner.run(ck.POLICY_DYNAMIC, mask_mr, x, labels)
        assert rep_mr["peak_bytes"] == rep_mr["extent_bytes"] == rep_mr["predicted_bytes"] == peak
        assert rep_mr["recomputed_units"] == runner.n + 1 - int(mask_mr.sum()) and rep_mr["loss"] == rep0["loss"]
        for a, b in zip(g_mr, g0):
            assert np.array_equal(a, b, equal_nan=True)
    # Algorithm 4's schedule in the shorter workspace it asks for (no buffer for activated copies), filled with NaN patterns
    full_ws = runner.workspace
    lean_bytes = runner.chain.workspace_bytes_for(ck.POLICY_DYNAMIC)
    assert lean_bytes <= runner.chain.workspace_bytes_for(ck.POLICY_STORE_ALL) == runner.chain.workspace_bytes()
    runner.workspace = torch.empty(lean_bytes, dtype=torch.uint8, device="cuda")
    runner.workspace.fill_(0xFF)
    rep_lean, g_lean = runner.run(ck.POLICY_DYNAMIC, mask_mr, x, labels)
    assert rep_lean["peak_bytes"] == peak and rep_lean["workspace_bytes"] == lean_bytes and rep_lean["loss"] == rep0["loss"]
    for a, b in zip(g_lean, g0):
        assert np.array_equal(a, b, equal_nan=True)
    if lean_bytes < runner.chain.workspace_bytes():
        with pytest.raises(ck.CkptError) as e:
            runner.run(ck.POLICY_STORE_ALL, None, x, labels)
        assert e.value.code == -8
    runner.workspace = full_ws
    mask3, peak3 = ck.plan(ck.ALGO_STATIC_N3, d)
    rep3, g3 = runner.run(ck.POLICY_STATIC, mask3, x, labels)
    assert rep3["peak_bytes"] == rep3["extent_bytes"] == peak3
    for a, b in zip(g3, g0):
        assert np.array_equal(a, b, equal_nan=True)
    torch.cuda.empty_cache()
    return rep, rep0, peak


def test_config2_vgg16_full_size_step():
    rep, rep0, peak = step_properties(wl.config(2))
    assert peak < 0.65 * rep0["peak_bytes"]             # 1.17 GiB against 1.82 GiB
    assert abs(rep["loss"] - np.log(1000.0)) < 2.0      # random labels, random weights


def test_config2_vgg16_full_size_graph_replay_and_host_batch():
    """The two submissions bench.py times: the recorded step replayed as a CUDA graph, and the same step fed from
    pinned host buffers.  Both must reproduce the launch-by-launch step bit for bit."""
    import torch
    spec = wl.config(2)
    params = wl.make_params(spec, seed=0)
    runner = StepRunner(spec, params)
    del params
    mask, peak = ck.plan(ck.ALGO_DYNAMIC_N, runner.d)
    x, labels = wl.make_batch(spec, seed=1)
    x_host = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    lab_host = torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).pin_memory()
    xb, lab = x_host.cuda(), lab_host.cuda()
    arena = torch.empty(peak, dtype=torch.uint8, device="cuda")

    def step(batch, lbl):
        arena.fill_(0xFF)
        for g in runner.grads:
            g.fill_(float("nan"))
        rep = ck.train_step(runner.chain, mask, ck.POLICY_DYNAMIC, batch, lbl, runner.params, runner.grads, arena, runner.workspace)
        torch.cuda.synchronize()
        return rep, [g.detach().cpu().numpy().copy() for g in runner.grads]

    rep0, g0 = step(xb, lab)
    assert rep0["replayed"] == 0 and rep0["peak_bytes"] == peak and np.isfinite(rep0["loss"])
    runner.chain.set_graph(True)
    flags = []
    for batch, lbl in ((xb, lab), (xb, lab), (xb, lab), (x_host, lab_host), (x_host, lab_host), (x_host, lab_host)):
        rep, g = step(batch, lbl)
        flags.append(rep["replayed"])
        for key in ("peak_bytes", "extent_bytes", "predicted_bytes", "launches", "recomputed_units", "loss", "device_status"):
            assert rep[key] == rep0[key], key
        for a, b in zip(g, g0):
            assert np.array_equal(a, b, equal_nan=True)
    assert flags == [0, 1, 1, 0, 1, 1]          # each argument set: one plain step, then the recording
    torch.cuda.empty_cache()


def test_config2_vgg16_split_units_full_size_step():
    """Finer granularity (Section 5.4): the 47-unit split of the VGG-16 chain at full size."""
    fine, _ = wl.split_units(wl.config(2))
    rep, rep0, peak = step_properties(fine)
    assert rep0["peak_bytes"] == int(sum(ck.Chain(fine).sizes()))
    assert peak < 0.5 * rep0["peak_bytes"]
    assert abs(rep["loss"] - np.log(1000.0)) < 2.0


def test_config3_resnet50_full_size_step():
    rep, rep0, peak = step_properties(wl.config(3))
    assert peak == int(771.75 * 2 ** 20)                # planner value of the ResNet-50 chain at batch 128


def test_config4_resnet152_full_size_step():
    rep, rep0, peak = step_properties(wl.config(4))
    assert peak == int(1837.5 * 2 ** 20)
    assert rep0["peak_bytes"] > 3.7 * peak              # the O(n) plan stores 3.8x less than keeping everything


def test_config5_plain1000_full_size_step():
    spec = wl.config(5)
    chain = ck.Chain(spec)
    d = chain.sizes()
    t0 = time.perf_counter(); m6, p6 = ck.plan(ck.ALGO_DYNAMIC_N, d); t6 = time.perf_counter() - t0
    t0 = time.perf_counter(); m5, p5 = ck.plan(ck.ALGO_DYNAMIC_N2, d); t5 = time.perf_counter() - t0
    t0 = time.perf_counter(); m3, p3 = ck.plan(ck.ALGO_STATIC_N3, d); t3 = time.perf_counter() - t0
    assert p6 == p5 == 47 * int(d[1]) and np.array_equal(m6, m5)
    assert p3 == 64 * int(d[1])
    assert t6 < t3                                      # the O(n) planner beats the O(n^3) one at n = 1000
    # A BN+ReLU chain at random initialisation multiplies the gradient norm by about 1.18 per unit on
    # the way back (measured on the float64 oracle), i.e. by 1e70 over 1000 units: the gradients of
    # the early units lie outside the float32/bfloat16 range in any implementation.  They overflow
    # identically under every schedule; finiteness is required of the last 300 units only.
    rep, rep0, peak = step_properties(spec, finite_last_units=300)
    assert rep0["peak_bytes"] > 20 * peak               # 12 GiB stored against 0.56 GiB checkpointed
