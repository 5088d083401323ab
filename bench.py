"""Benchmark: checkpointed training-step throughput (images/s) of the VGG-16-shaped chain on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]

One "step" = one full pass of the hot path over one synthetic batch: forward keeping the planned
checkpoints, loss, backward with segment recomputation, all weight gradients.  The plan is the
O(n) dynamic planner's (Algorithm 6) and the schedule is Algorithm 4.  With N > 1 (torchrun) every
rank runs an independent replica on its own batch: the step has no exchange between GPUs.

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle instead, on rank 0 only.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2502_12499_b200 import workloads as wl  # noqa: E402

METRIC = "checkpointed_train_step_images_per_s"
UNIT = "images/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


def max_over_ranks(ms, world, device):
    """Replicas share nothing but the clock: the job's time per timed region is the slowest rank's."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_images_per_s(batch, world, steps, ms):
    """Every rank runs `steps` steps of `batch` images on its own batch within `ms` milliseconds."""
    return batch * world * steps / (ms * 1e-3)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, flag in zip(names, parts[2:6]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


def conv_flops(spec, plan_mask, shapes):
    """Algorithmic FLOPs of one step: 2*MAC x (forward + recompute of non-checkpoints + dgrad
    (units 2..n) + wgrad)."""
    fwd = []
    h, w, c = spec["input_hwc"]
    for u, (ho, wo, co) in zip(spec["units"], shapes[1:]):
        if u["kind"] in ("conv_bn_relu", "conv"):
            fwd.append(2.0 * spec["batch"] * ho * wo * co * u["k"] * u["k"] * u["cin"])
        elif u["kind"] == "bottleneck":
            st, mid = u["stride"], u["mid"]
            macs = ho * st * wo * st * u["cin"] * mid + ho * wo * 9 * mid * mid + ho * wo * mid * co
            if u["project"]:
                macs += ho * wo * u["cin"] * co
            fwd.append(2.0 * spec["batch"] * macs)
        elif u["kind"] == "fc":
            fwd.append(2.0 * spec["batch"] * u["cin"] * u["cout"])
        else:
            fwd.append(0.0)
    total = 0.0
    for i, f in enumerate(fwd, start=1):
        total += f                                   # forward
        if not plan_mask[i]:
            total += f                               # segment recompute
        total += f                                   # wgrad
        if i > 1:
            total += f                               # dgrad
    return total, fwd


def run_reference(args, spec, steps=None, warmup=None, budget_s=None):
    """The CPU oracle, as it stands, on a bounded sample of the same workload.  With a time budget the
    sample (images per step) is sized so that warmup + steps steps fit it (about 1.6 s per image of the
    VGG-16 chain on 16 cores)."""
    from oracle import numeric_oracle as no
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    steps = args.steps_cpu if steps is None else max(1, steps)
    warmup = args.warmup_cpu if warmup is None else max(0, warmup)
    sample_batch = min(spec["batch"], args.cpu_batch)
    if budget_s is not None:
        sample_batch = int(max(1, min(sample_batch, budget_s / (1.6 * (steps + warmup)))))
    small = dict(spec, batch=sample_batch)
    params = wl.make_params(small, seed=0)
    x, labels = wl.make_batch(small, seed=1)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        no.chain_forward_backward(small, params, x, labels)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    t = float(np.mean(times))
    return dict(value=sample_batch / t, unit=UNIT, cores=int(cores), kind="oracle",
                sample="store-all step of the same chain on a batch of %d of %d images, float64 numpy, %d timed step(s)"
                       % (sample_batch, spec["batch"], len(times)), seconds_per_step=t)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (debugging only)")
    ap.add_argument("--cpu-batch", type=int, default=4)
    ap.add_argument("--steps-cpu", type=int, default=1)
    ap.add_argument("--warmup-cpu", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel of every step from the host")
    ap.add_argument("--split-units", action="store_true",
                    help="finer granularity: conv, batch norm and ReLU as chain units of their own")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    spec = wl.config(args.config)
    if args.batch:
        spec = dict(spec, batch=args.batch)
    if args.split_units:
        spec, _ = wl.split_units(spec)
    config = {"workload": "%s: %d units, batch %d of %dx%dx%d %s, plan = Algorithm 6, schedule = Algorithm 4"
                          % (spec["name"], len(spec["units"]), spec["batch"], *spec["input_hwc"], spec["dtype"]),
              "l2": "inputs larger than L2 (every step streams > 1 GB of activations)",
              "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
              "submission": "launch by launch" if args.no_graph else "CUDA graph replay of the recorded step"}

    if args.impl == "reference":
        if rank != 0:
            return
        # the requested step counts, each step a sample of the batch sized so that the run ends within about two minutes
        cpu = run_reference(args, spec, steps=args.steps, warmup=args.warmup, budget_s=120.0)
        line = {"impl": "reference", "metric": METRIC, "value": cpu["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cpu["seconds_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": config, "cpu_baseline": cpu,
                "e2e": {"value": cpu["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    from paper_2502_12499_b200 import binding as ck

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")

    chain = ck.Chain(spec)
    if not args.no_graph:
        chain.set_graph(True)        # a step whose arguments repeat is recorded once and replayed
    d = chain.sizes()
    shapes = [tuple(int(v) for v in s) for s in chain.shapes()]
    t0 = time.perf_counter()
    mask, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
    plan_us = 1e6 * (time.perf_counter() - t0)
    # the three planners on this chain (host only; median of a few runs): Algorithm 3 is O(n^3), 5 O(n^2), 6 O(n)
    planner_us = {}
    for name, algo in (("algorithm_3", ck.ALGO_STATIC_N3), ("algorithm_5", ck.ALGO_DYNAMIC_N2), ("algorithm_6", ck.ALGO_DYNAMIC_N)):
        runs = []
        for _ in range(3 if len(d) > 200 else 15):
            t1 = time.perf_counter()
            ck.plan(algo, d)
            runs.append(1e6 * (time.perf_counter() - t1))
        planner_us[name] = round(sorted(runs)[len(runs) // 2], 1)
    store_all = ck.eval(ck.MODEL_STORE_ALL, d, None)

    params_h = wl.make_params(spec, seed=0)
    params, grads, _ = ck.upload_params(chain, params_h)
    del params_h
    x_h, labels_h = wl.make_batch(spec, seed=1 + rank)
    tdt = torch.bfloat16 if spec["dtype"] == "bf16" else torch.float32
    x_pinned = torch.from_numpy(x_h).to(tdt).pin_memory()
    labels_pinned = torch.from_numpy(labels_h).pin_memory()
    x_dev = x_pinned.cuda()
    labels_dev = labels_pinned.cuda()
    arena = torch.empty(peak, dtype=torch.uint8, device="cuda")
    workspace = torch.empty(chain.workspace_bytes(), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step(batch, labels):
        return ck.train_step(chain, mask, ck.POLICY_DYNAMIC, batch, labels, params, grads, arena, workspace, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(batch, labels, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        rep = None
        for _ in range(steps):
            rep = step(batch, labels)
        e1.record(stream)
        barrier()
        ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        return ms, rep

    for _ in range(max(args.warmup, 3)):
        rep = step(x_dev, labels_dev)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms, rep = timed(x_dev, labels_dev, args.steps)
    for _ in range(3):                       # the end-to-end leg has its own arguments: warm it up (and record it) too
        step(x_pinned, labels_pinned)
    ms_e2e, rep_e2e = timed(x_pinned, labels_pinned, args.steps)
    clocks = sampler.stop() if rank == 0 else None

    value = whole_job_images_per_s(spec["batch"], world, args.steps, ms)
    e2e_value = whole_job_images_per_s(spec["batch"], world, args.steps, ms_e2e)

    if rank == 0:
        peaks = measured_peaks()
        flops, _ = conv_flops(spec, mask, shapes)
        roofline = dominant_kernel_roofline(args.config, peaks, spec["batch"], shapes[1])
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": spec["dtype"], "data": "synthetic", "config": config,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_pinned.numel() * x_pinned.element_size() + labels_pinned.numel() * 4),
                        "d2h_bytes_per_step": 12},
                "gpu_launches": int(rep["launches"]) * args.steps, "clocks": clocks, "roofline": roofline,
                "peak_bytes": int(rep["peak_bytes"]), "predicted_bytes": int(peak), "store_all_bytes": int(store_all),
                "peak_gib": rep["peak_bytes"] / 2 ** 30, "workspace_gib": chain.workspace_bytes() / 2 ** 30,
                "recomputed_units": int(rep["recomputed_units"]), "plan_us": plan_us, "planner_us": planner_us, "loss": rep["loss"],
                "step_tflops": flops / (ms / args.steps * 1e-3) / 1e12,
                "step_tensor_frac_of_sustained": flops / (ms / args.steps * 1e-3) / 1e12 / peaks["tflops_sustained"],
                "peaks": peaks}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = run_reference(args, spec)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM traffic per launch of the conv-forward kernels over the layer mix of config 2, from one ncu pass
# (profiles/conv_forward_vgg16_b64_dram_traffic.md).  Valid only for the kernel source it was taken
# on: reported as null when csrc/conv_tc.cu has changed since.
CONV_FWD_TRAFFIC = {"source_sha256": "9fdcfc7547a05b6256d957c5f1e983fb78b6a0d1b4a819e2b4cb5d3a7524a1d5", "bytes_per_launch": 169731242}


def _kernel_source_sha():
    import hashlib
    path = os.path.join(ROOT, "paper_2502_12499_b200", "csrc", "conv_tc.cu")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()


def dominant_kernel_roofline(config_index, peaks, batch, first_shape):
    """The convolution-forward kernels (tcgen05; the role-swapped kernel for every layer but the two
    64-channel ones) hold the largest share of the step: they run in the forward phase, in segment
    recomputation and, on the transposed matrix, as dgrad.  Timed here on
    every conv layer shape of the workload with CUDA events; achieved = sum of algorithmic FLOPs /
    sum of launch times, against the measured dense-bf16 peak."""
    from paper_2502_12499_b200 import opbench
    mix = opbench.conv_mix("fwd", config_index, reps=3)
    traffic = CONV_FWD_TRAFFIC["bytes_per_launch"] if CONV_FWD_TRAFFIC["source_sha256"] == _kernel_source_sha() else None
    out = {"kernel": "tc_conv_tp_kernel / tc_conv_t_kernel (implicit-GEMM conv forward over the layer mix)", "bound": "tensor",
           "achieved": mix["tflops"], "peak": peaks["tflops_burst"], "unit": "TFLOP/s", "frac": mix["tflops"] / peaks["tflops_burst"],
           "peak_source": peaks["source"] + " (burst: kernels timed in isolation)", "traffic": traffic,
           "launch_shapes": mix["launches"], "flops_per_launch": mix["flops"] / mix["launches"],
           "ms_per_launch": mix["ms"] / mix["launches"], "per_layer": mix["per_layer"]}
    # the memory-bound side of the step, for the record: batch-norm and 2x2 pooling passes on the largest
    # activation of the chain (the output of its first unit)
    b, (h, w, c) = batch, first_shape
    f, g = opbench.bn("fwd", b * h * w, c), opbench.bn("bwd", b * h * w, c)
    pf, pb = opbench.pool("fwd", b, h, w, c), opbench.pool("bwd", b, h, w, c)
    out["elementwise"] = {"unit": "GB/s", "peak": peaks["hbm_gbs"],
                          "bn_forward": f["gbs"], "bn_backward": g["gbs"], "maxpool_forward": pf["gbs"], "maxpool_backward": pb["gbs"],
                          "frac": {"bn_forward": f["gbs"] / peaks["hbm_gbs"], "bn_backward": g["gbs"] / peaks["hbm_gbs"],
                                   "maxpool_forward": pf["gbs"] / peaks["hbm_gbs"], "maxpool_backward": pb["gbs"] / peaks["hbm_gbs"]}}
    return out


if __name__ == "__main__":
    main()
