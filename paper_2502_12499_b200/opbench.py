"""Run and time single operations of the library (for profiling and roofline numbers).

    python -m paper_2502_12499_b200.opbench conv fwd|dgrad|wgrad N H W C_IN C_OUT K PAD [STRIDE] [--reps R]
    python -m paper_2502_12499_b200.opbench bn fwd|bwd ROWS C [--reps R]
    python -m paper_2502_12499_b200.opbench pool fwd|bwd N H W C [--reps R]
    python -m paper_2502_12499_b200.opbench convmix fwd|dgrad|wgrad CONFIG [--reps R]   (all conv layers of a config)

Prints one JSON line with the CUDA-event time per launch and the algorithmic throughput
(TFLOP/s for convolutions, GB/s for the memory-bound operations).  bf16 storage throughout.
Everything goes through the C ABI; torch only owns the buffers.
"""
import argparse
import json

from . import binding as ck


def _time(fn, reps, warmup=2):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def conv(what, n, h, w, cin, cout, k, pad, stride=1, reps=3, impl=0):
    """One convolution operation; returns dict(ms, tflops, flops)."""
    import torch
    dt = ck.DTYPE_BF16
    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    x = torch.randn(n, h, w, cin, device="cuda").bfloat16()
    wt = (torch.randn(cout, k, k, cin, device="cuda") * 0.05).bfloat16()
    z = torch.empty(n, ho, wo, cout, device="cuda", dtype=torch.bfloat16)
    dz = torch.randn(n, ho, wo, cout, device="cuda").bfloat16()
    dx = torch.empty_like(x)
    dw = torch.empty(cout, k, k, cin, device="cuda")
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, dt)), dtype=torch.uint8, device="cuda")
    fn = {"fwd": lambda: ck.conv2d_forward(shape, dt, impl, x, wt, z, scratch),
          "dgrad": lambda: ck.conv2d_dgrad(shape, dt, impl, dz, wt, dx, scratch),
          "wgrad": lambda: ck.conv2d_wgrad(shape, dt, impl, dz, x, dw, scratch)}[what]
    ms = _time(fn, reps)
    flops = 2.0 * n * ho * wo * cout * k * k * cin
    return dict(op="conv " + what, shape=[n, h, w, cin, cout, k, pad] + ([stride] if stride != 1 else []), ms=ms, flops=flops, tflops=flops / ms / 1e9)


def bn(what, rows, c, reps=5):
    """Batch norm + ReLU forward (statistics + apply: 3 tensor passes) or backward (sums + apply: 5)."""
    import torch
    dt = ck.DTYPE_BF16
    z = torch.randn(rows, c, device="cuda").bfloat16()
    dy = torch.randn(rows, c, device="cuda").bfloat16()
    y, dz = torch.empty_like(z), torch.empty_like(z)
    gamma, beta = torch.ones(c, device="cuda"), torch.zeros(c, device="cuda")
    stats, dg, db = torch.empty(4 * c, device="cuda"), torch.empty(c, device="cuda"), torch.empty(c, device="cuda")
    scratch = torch.empty(ck.bn_scratch_bytes(rows, c), dtype=torch.uint8, device="cuda")
    ck.bn_relu_forward(dt, rows, c, z, gamma, beta, 1, y, stats, scratch)
    if what == "fwd":
        ms = _time(lambda: ck.bn_relu_forward(dt, rows, c, z, gamma, beta, 1, y, stats, scratch), reps)
        passes = 3
    else:
        ms = _time(lambda: ck.bn_relu_backward(dt, rows, c, dy, z, gamma, stats, 1, dz, dg, db, scratch), reps)
        passes = 5
    nbytes = passes * rows * c * 2.0
    return dict(op="bn " + what, shape=[rows, c], ms=ms, bytes=nbytes, gbs=nbytes / ms / 1e6)


def pool(what, n, h, w, c, reps=5):
    """2x2 max pooling forward (read x, write x/4) or backward (read x and dy, write dx)."""
    import torch
    dt = ck.DTYPE_BF16
    x = torch.randn(n, h, w, c, device="cuda").bfloat16()
    y = torch.empty(n, h // 2, w // 2, c, device="cuda", dtype=torch.bfloat16)
    dy, dx = torch.randn_like(y), torch.empty_like(x)
    if what == "fwd":
        ms = _time(lambda: ck.maxpool_forward(dt, n, h, w, c, 2, 2, 0, x, y), reps)
        nbytes = 1.25 * x.numel() * 2.0
    else:
        ms = _time(lambda: ck.maxpool_backward(dt, n, h, w, c, 2, 2, 0, x, dy, dx), reps)
        nbytes = 2.25 * x.numel() * 2.0
    return dict(op="pool " + what, shape=[n, h, w, c], ms=ms, bytes=nbytes, gbs=nbytes / ms / 1e6)


def conv_layers(spec):
    """(n, h, w, c_in, c_out, k, pad) of every stride-1 convolution of a chain description: the conv units and
    the convolutions inside bottleneck blocks (input size of each convolution)."""
    out = []
    h, w, c = spec["input_hwc"]
    b = spec["batch"]
    for u in spec["units"]:
        if u["kind"] in ("conv_bn_relu", "conv"):
            if u["stride"] == 1:
                out.append((b, h, w, u["cin"], u["cout"], u["k"], u["pad"]))
            h = (h + 2 * u["pad"] - u["k"]) // u["stride"] + 1
            w = (w + 2 * u["pad"] - u["k"]) // u["stride"] + 1
            c = u["cout"]
        elif u["kind"] == "bottleneck":
            st, mid = u["stride"], u["mid"]
            out.append((b, h, w, u["cin"], mid, 1, 0))
            if st == 1:
                out.append((b, h, w, mid, mid, 3, 1))
            h, w = (h + 2 - 3) // st + 1, (w + 2 - 3) // st + 1
            out.append((b, h, w, mid, u["cout"], 1, 0))
            if u["project"] and st == 1:
                out.append((b, h, w, u["cin"], u["cout"], 1, 0))
            c = u["cout"]
        elif u["kind"] == "maxpool":
            h = (h + 2 * u["pad"] - u["k"]) // u["stride"] + 1
            w = (w + 2 * u["pad"] - u["k"]) // u["stride"] + 1
        elif u["kind"] in ("fc", "avgpool"):
            h = w = 1
    return out


def conv_mix(what, config_index, reps=3, min_cin=16):
    """The conv kernel `what` over every conv layer shape of a benchmark configuration: per-layer
    numbers plus the launch-weighted total (sum of FLOPs / sum of time)."""
    from . import workloads as wl
    layers = [s for s in conv_layers(wl.config(config_index)) if s[3] >= min_cin]
    seen, per_layer = {}, []
    for s in layers:
        if s not in seen:
            seen[s] = conv(what, *s, reps=reps)
        per_layer.append(seen[s])
    flops = sum(r["flops"] for r in per_layer)
    ms = sum(r["ms"] for r in per_layer)
    return dict(op="conv " + what + " mix", config=config_index, launches=len(per_layer), ms=ms, flops=flops,
                tflops=flops / ms / 1e9,
                per_layer=[{"shape": r["shape"], "ms": round(r["ms"], 4), "tflops": round(r["tflops"], 1)} for r in per_layer])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["conv", "bn", "pool", "convmix"])
    ap.add_argument("what")
    ap.add_argument("dims", type=int, nargs="+")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--impl", type=int, default=0)
    a = ap.parse_args()
    if a.kind == "convmix":
        out = conv_mix(a.what, a.dims[0], reps=a.reps)
    elif a.kind == "conv":
        out = conv(a.what, *a.dims, reps=a.reps, impl=a.impl)
    elif a.kind == "bn":
        out = bn(a.what, *a.dims, reps=a.reps)
    else:
        out = pool(a.what, *a.dims, reps=a.reps)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
