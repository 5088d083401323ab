"""Run and time single operations of the library (roofline numbers for bench.py, and a command line for profiling).

    python bench_ops.py conv fwd|dgrad|wgrad N H W C_IN C_OUT K PAD [STRIDE] [--reps R]
    python bench_ops.py bn fwd|bwd ROWS C [--reps R]
    python bench_ops.py pool fwd|bwd N H W C [--reps R]
    python bench_ops.py convmix fwd|dgrad|wgrad CONFIG [--batch B]   (all conv layers of a benchmark configuration)

Prints one JSON line with the CUDA-event time per launch and the algorithmic throughput (TFLOP/s for convolutions,
GB/s for the memory-bound operations).  bf16 storage throughout.  Everything goes through the C ABI; torch only
owns the buffers.

Timing: every operation runs on a rotation of buffer sets that together exceed the L2 cache (so that no launch finds
its operands left there by the previous one), for at least 20 launches and at least 10 ms after the warm-up, between
CUDA events on the launching stream.  `--reps R` fixes the launch count instead (R = 1 for profiler captures).
"""
import argparse
import json
import math
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2502_12499_b200 import binding as ck  # noqa: E402

L2_BYTES = 126e6
MIN_LAUNCHES, MIN_MS, MAX_LAUNCHES, MAX_SETS = 20, 10.0, 400, 8
GRAPH_BELOW_MS = 0.06          # kernels shorter than this are timed from a recorded graph (see time_replayed)


def sets_beyond_l2(bytes_per_set):
    return int(max(1, min(MAX_SETS, math.ceil(1.3 * L2_BYTES / max(bytes_per_set, 1)))))


def time_rotating(fns, reps=None, warmup=3):
    """fns: one callable per buffer set.  Returns the mean milliseconds per launch."""
    import torch
    stream = torch.cuda.current_stream()
    k = 0

    def run(count):
        nonlocal k
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(count):
            fns[k % len(fns)]()
            k += 1
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    run(max(warmup, len(fns)) if reps != 1 else 1)
    if reps is None:
        est = run(3) / 3
        reps = int(min(MAX_LAUNCHES, max(MIN_LAUNCHES, math.ceil(MIN_MS / max(est, 1e-4)))))
        if est < GRAPH_BELOW_MS:
            ms = time_replayed(fns, reps)
            if ms is not None:
                return ms, reps
    return run(reps) / reps, reps


def time_replayed(fns, reps):
    """Short kernels: launched from Python they are bound by the host (two library calls cost more than a 15 us
    kernel runs), so one round over the buffer sets is recorded as a CUDA graph and replayed, as the training step
    itself is submitted.  Returns the mean milliseconds per launch, or None when recording is not possible."""
    import torch
    rounds = int(math.ceil(reps / len(fns)))
    try:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for fn in fns:
                fn()
    except Exception:
        torch.cuda.synchronize()
        return None
    stream = torch.cuda.current_stream()
    for _ in range(2):
        graph.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(rounds):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (rounds * len(fns))


def conv(what, n, h, w, cin, cout, k, pad, stride=1, reps=None, impl=0):
    """One convolution operation; returns dict(ms, tflops, flops, bytes): bytes = the tensors the operation must read
    and write once (bf16 activations and filter; the f32 gradient for wgrad)."""
    import torch
    dt = ck.DTYPE_BF16
    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    x_b, z_b, w_b = n * h * w * cin * 2.0, n * ho * wo * cout * 2.0, cout * k * k * cin * 2.0
    nbytes = x_b + z_b + (2 * w_b if what == "wgrad" else w_b)
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, dt), ck.bn_scratch_bytes(n * ho * wo, cout)), dtype=torch.uint8, device="cuda")
    fns = []
    for _ in range(1 if reps == 1 else sets_beyond_l2(nbytes)):
        x = torch.randn(n, h, w, cin, device="cuda").bfloat16()
        wt = (torch.randn(cout, k, k, cin, device="cuda") * 0.05).bfloat16()
        z = torch.empty(n, ho, wo, cout, device="cuda", dtype=torch.bfloat16)
        if what == "fwd":
            fns.append(lambda x=x, wt=wt, z=z: ck.conv2d_forward(shape, dt, impl, x, wt, z, scratch))
        elif what == "fwd_stats":
            # as a conv+BN+ReLU unit runs it: the batch-norm sums of the stored output gathered in the epilogue, then
            # the per-channel finalize
            gamma, beta = torch.ones(cout, device="cuda"), torch.zeros(cout, device="cuda")
            stats = torch.empty(4 * cout, device="cuda")
            fns.append(lambda x=x, wt=wt, z=z, g=gamma, b=beta, st=stats: ck.conv2d_bn_statistics(shape, dt, x, wt, z, g, b, st, scratch))
        elif what == "dgrad":
            z.normal_()
            dx = torch.empty_like(x)
            fns.append(lambda z=z, wt=wt, dx=dx: ck.conv2d_dgrad(shape, dt, impl, z, wt, dx, scratch))
        else:
            z.normal_()
            dw = torch.empty(cout, k, k, cin, device="cuda")
            fns.append(lambda z=z, x=x, dw=dw: ck.conv2d_wgrad(shape, dt, impl, z, x, dw, scratch))
    ms, launches = time_rotating(fns, reps)
    ck.op_status()
    flops = 2.0 * n * ho * wo * cout * k * k * cin
    return dict(op="conv " + what, shape=[n, h, w, cin, cout, k, pad] + ([stride] if stride != 1 else []), ms=ms,
                launches=launches, flops=flops, bytes=nbytes, tflops=flops / ms / 1e9, gbs=nbytes / ms / 1e6)


def bn(what, rows, c, reps=None):
    """Batch norm + ReLU forward (statistics + apply: 3 tensor passes) or backward (sums + apply: 5)."""
    import torch
    dt = ck.DTYPE_BF16
    gamma, beta = torch.ones(c, device="cuda"), torch.zeros(c, device="cuda")
    stats, dg, db = torch.empty(4 * c, device="cuda"), torch.empty(c, device="cuda"), torch.empty(c, device="cuda")
    scratch = torch.empty(ck.bn_scratch_bytes(rows, c), dtype=torch.uint8, device="cuda")
    passes = 3 if what == "fwd" else 5
    fns = []
    for _ in range(1 if reps == 1 else sets_beyond_l2((2 if what == "fwd" else 3) * rows * c * 2.0)):
        z = torch.randn(rows, c, device="cuda").bfloat16()
        y = torch.empty_like(z)
        if what == "fwd":
            fns.append(lambda z=z, y=y: ck.bn_relu_forward(dt, rows, c, z, gamma, beta, 1, y, stats, scratch))
        else:
            dy = torch.randn(rows, c, device="cuda").bfloat16()
            fns.append(lambda z=z, y=y, dy=dy: ck.bn_relu_backward(dt, rows, c, dy, z, gamma, stats, 1, y, dg, db, scratch))
    ck.bn_relu_forward(dt, rows, c, torch.randn(rows, c, device="cuda").bfloat16(), gamma, beta, 1,
                       torch.empty(rows, c, device="cuda", dtype=torch.bfloat16), stats, scratch)
    ms, launches = time_rotating(fns, reps)
    nbytes = passes * rows * c * 2.0
    return dict(op="bn " + what, shape=[rows, c], ms=ms, launches=launches, bytes=nbytes, gbs=nbytes / ms / 1e6)


def pool(what, n, h, w, c, reps=None):
    """2x2 max pooling forward (read x, write x/4) or backward (read x and dy, write dx)."""
    import torch
    dt = ck.DTYPE_BF16
    fns = []
    for _ in range(1 if reps == 1 else sets_beyond_l2(2.25 * n * h * w * c * 2.0)):
        x = torch.randn(n, h, w, c, device="cuda").bfloat16()
        y = torch.empty(n, h // 2, w // 2, c, device="cuda", dtype=torch.bfloat16)
        if what == "fwd":
            fns.append(lambda x=x, y=y: ck.maxpool_forward(dt, n, h, w, c, 2, 2, 0, x, y))
        else:
            dy, dx = torch.randn_like(y), torch.empty_like(x)
            fns.append(lambda x=x, dy=dy, dx=dx: ck.maxpool_backward(dt, n, h, w, c, 2, 2, 0, x, dy, dx))
    ms, launches = time_rotating(fns, reps)
    nbytes = (1.25 if what == "fwd" else 2.25) * n * h * w * c * 2.0
    return dict(op="pool " + what, shape=[n, h, w, c], ms=ms, launches=launches, bytes=nbytes, gbs=nbytes / ms / 1e6)


def chain_layers(spec):
    """Walks a chain description and lists what its step runs, with input sizes:
    convs = (n, h, w, c_in, c_out, k, pad, stride) of every convolution (units and bottleneck interiors), followed by
    the fully connected layers as 1x1 convolutions on a 1x1 image (h = w = 1), norms = (rows, channels) of every batch
    normalisation, pools = (n, h, w, c) of every 2x2 max-pool."""
    convs, norms, pools = [], [], []
    h, w, c = spec["input_hwc"]
    b = spec["batch"]

    def conv(cin, cout, k, pad, st, hh, ww):
        convs.append((b, hh, ww, cin, cout, k, pad, st))
        ho, wo = (hh + 2 * pad - k) // st + 1, (ww + 2 * pad - k) // st + 1
        return ho, wo

    for u in spec["units"]:
        kind = u["kind"]
        if kind in ("conv_bn_relu", "conv"):
            h, w = conv(u["cin"], u["cout"], u["k"], u["pad"], u["stride"], h, w)
            c = u["cout"]
            if kind == "conv_bn_relu":
                norms.append((b * h * w, c))
        elif kind == "bn":
            norms.append((b * h * w, c))
        elif kind == "bottleneck":
            st, mid = u["stride"], u["mid"]
            conv(u["cin"], mid, 1, 0, 1, h, w)
            norms.append((b * h * w, mid))
            ho, wo = conv(mid, mid, 3, 1, st, h, w)
            norms.append((b * ho * wo, mid))
            conv(mid, u["cout"], 1, 0, 1, ho, wo)
            norms.append((b * ho * wo, u["cout"]))
            if u["project"]:
                conv(u["cin"], u["cout"], 1, 0, st, h, w)
                norms.append((b * ho * wo, u["cout"]))
            h, w, c = ho, wo, u["cout"]
        elif kind == "maxpool":
            if u["k"] == 2 and u["stride"] == 2 and u["pad"] == 0:
                pools.append((b, h, w, c))
            h = (h + 2 * u["pad"] - u["k"]) // u["stride"] + 1
            w = (w + 2 * u["pad"] - u["k"]) // u["stride"] + 1
        elif kind == "avgpool":
            h = w = 1
        elif kind == "fc":
            convs.append((b, 1, 1, u["cin"], u["cout"], 1, 0, 1))
            h, w, c = 1, 1, u["cout"]
    return convs, norms, pools


def is_fc(shape):
    return shape[1] == 1 and shape[2] == 1 and shape[5] == 1


def conv_mix(what, spec, peaks, reps=None, min_cin=16, layers="conv"):
    """The kernels `what` over every convolution of a chain with at least `min_cin` input channels (the 3-channel
    first layers are gather kernels of their own), or over its fully connected layers (layers="fc": matrix-streaming
    kernels of their own, bound by HBM): per-shape numbers and the launch-weighted totals.
    Each shape is held against the roof that bounds it: time_roof = max(FLOPs / tensor peak, bytes / HBM bandwidth)
    with bytes = its operands and result once; frac = time_roof / measured time."""
    layers = [s for s in chain_layers(spec)[0] if s[3] >= min_cin and is_fc(s) == (layers == "fc")]
    if not layers:
        return None
    seen, per_layer = {}, []
    for s in layers:
        if s not in seen:
            seen[s] = conv(what, *s, reps=reps)
        per_layer.append(seen[s])
    flops = sum(r["flops"] for r in per_layer)
    ms = sum(r["ms"] for r in per_layer)
    tensor_peak, hbm = peaks["tflops_burst"] * 1e12, peaks["hbm_gbs"] * 1e9
    roof_ms = 0.0
    rows = []
    for r in per_layer:
        t_tensor, t_hbm = r["flops"] / tensor_peak * 1e3, r["bytes"] / hbm * 1e3
        roof_ms += max(t_tensor, t_hbm)
    for s, r in seen.items():
        t_tensor, t_hbm = r["flops"] / tensor_peak * 1e3, r["bytes"] / hbm * 1e3
        rows.append({"shape": r["shape"], "count": layers.count(s), "ms": round(r["ms"], 4), "tflops": round(r["tflops"], 1),
                     "gbs": round(r["gbs"], 1), "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                     "frac": round(max(t_tensor, t_hbm) / r["ms"], 3), "timed_launches": r["launches"]})
    return dict(op="conv " + what + " mix", launches=len(per_layer), ms=ms, flops=flops, tflops=flops / ms / 1e9,
                frac_of_tensor_peak=flops / ms / 1e9 / peaks["tflops_burst"], frac_of_roof=roof_ms / ms, per_shape=rows)


def elementwise_mix(spec, peaks, reps=None):
    """Batch-norm forward / backward over every normalised tensor of the chain and the 2x2 pools over every pooled
    one, launch-weighted: sum of algorithmic bytes / sum of time, against the measured copy bandwidth."""
    _, norms, pools = chain_layers(spec)
    out = {"unit": "GB/s", "peak": peaks["hbm_gbs"]}
    for name, shapes, fn, whats in (("bn", norms, bn, ("fwd", "bwd")), ("maxpool", pools, pool, ("fwd", "bwd"))):
        for what in whats:
            seen = {}
            nbytes = ms = 0.0
            worst = None
            for s in shapes:
                if s not in seen:
                    seen[s] = fn(what, *s, reps=reps)
                nbytes += seen[s]["bytes"]
                ms += seen[s]["ms"]
                if worst is None or seen[s]["gbs"] < worst["gbs"]:
                    worst = seen[s]
            if ms > 0:
                key = "%s_%s" % (name, "forward" if what == "fwd" else "backward")
                out[key] = {"gbs": nbytes / ms / 1e6, "frac": nbytes / ms / 1e6 / peaks["hbm_gbs"], "launches": len(shapes),
                            "distinct_shapes": len(seen), "slowest": {"shape": worst["shape"], "gbs": round(worst["gbs"], 1)}}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["conv", "bn", "pool", "convmix"])
    ap.add_argument("what")
    ap.add_argument("dims", type=int, nargs="+")
    ap.add_argument("--reps", type=int, default=None)
    ap.add_argument("--impl", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="convmix: run the configuration's layers at this batch (small profiler captures)")
    a = ap.parse_args()
    if a.kind == "convmix":
        from paper_2502_12499_b200 import workloads as wl
        peaks = dict(tflops_burst=1672.2, hbm_gbs=6549.4)
        path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(path):
            p = json.load(open(path))
            peaks = dict(tflops_burst=p["bf16_tflops"], hbm_gbs=p["hbm_gbs"])
        spec = wl.config(a.dims[0])
        if a.batch:
            spec = dict(spec, batch=a.batch)
        out = conv_mix(a.what, spec, peaks, reps=a.reps)
    elif a.kind == "conv":
        out = conv(a.what, *a.dims, reps=a.reps, impl=a.impl)
    elif a.kind == "bn":
        out = bn(a.what, *a.dims, reps=a.reps)
    else:
        out = pool(a.what, *a.dims, reps=a.reps)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
