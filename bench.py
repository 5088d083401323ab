"""Benchmark: checkpointed training-step throughput (images/s) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2] [--only]

One "step" = one full pass of the hot path over one synthetic batch: forward keeping the planned
checkpoints, loss, backward with segment recomputation, all weight gradients.  The plan is the
dynamic planner's (Algorithm 6) and the schedule is Algorithm 4.  With N > 1 (torchrun) every
rank runs an independent replica on its own batch: the step has no exchange between GPUs.

The top-level fields of the JSON line are those of the headline workload (--config, default the VGG-16-shaped
chain at batch 64).  At N = 1 the line also carries `configs`: the same measurements for every bf16 benchmark
configuration (VGG-16 b64, ResNet-50 b128, ResNet-152 b256, the 1000-unit chain b32) - checkpointed and
store-all (Algorithm 1) step times and the recompute overhead between them, end-to-end throughput from pinned
host batches, device footprint (arena + workspace + parameters) under the plan and under store-all, planner times,
and the roofline of its kernels: forward, dgrad and wgrad convolution mixes and the launch-weighted batch-norm
and pooling bandwidth.  `--only` restricts the run to the headline workload.

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
    """FLOPs of one step as executed: 2*MAC x (forward + recompute of non-checkpoints + dgrad (units 2..n) + wgrad),
    plus one more forward of every residual block: only a block's output is chain data, so its backward re-derives
    the interior tensors under every schedule, store-all included."""
    fwd = []
    rederived = []          # 1-based indices of units whose backward re-derives its interior tensors (one more forward)
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
            rederived.append(len(fwd))
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
        if i in rederived:
            total += f                               # a residual block's backward re-runs its convolutions (any schedule)
    return total, fwd


def host_cores():
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] + [1]))
    except Exception:
        return int(os.cpu_count() or 1)


def run_reference(spec, sample_batch, steps, warmup=0):
    """The CPU oracle, as it stands (float64 numpy, Algorithm 1 = store-all), on a bounded sample of the same workload:
    the same chain on the first `sample_batch` images of the batch.  Returns images/s over `steps` timed steps."""
    from oracle import numeric_oracle as no
    import numpy  # noqa: F401  (loaded before the thread count is read)
    small = dict(spec, batch=sample_batch)
    params = wl.make_params(small, seed=0)
    x, labels = wl.make_batch(small, seed=1)
    if spec["loss"] != "softmax_ce":
        labels = None
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        no.chain_forward_backward(small, params, x, labels)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    t = float(np.mean(times))
    return dict(value=sample_batch / t, unit=UNIT, cores=host_cores(), kind="oracle",
                sample="store-all step (Algorithm 1) of the same chain on %d of its %d images, float64 numpy, mean of %d timed step(s)"
                       % (sample_batch, spec["batch"], len(times)), seconds_per_step=t, steps=len(times))


def workload_name(spec):
    return "%s: %d units, batch %d of %dx%dx%d %s, plan = peak of Algorithm 6 with the least recomputation among the sets that reach it, schedule = Algorithm 4" % (
        spec["name"], len(spec["units"]), spec["batch"], *spec["input_hwc"], spec["dtype"])


def measure_config(spec, args, rank, world, steps, regions, with_roofline, peaks, sampler=None):
    """All device measurements of one chain.  Returns a dict; `ms_per_step` is the median over `regions` timed
    regions of exactly `steps` steps each (barrier + synchronize on both sides, CUDA events, max over ranks)."""
    import torch
    import torch.distributed as dist
    from paper_2502_12499_b200 import binding as ck

    chain = ck.Chain(spec)
    if not args.no_graph:
        chain.set_graph(True)        # a step whose arguments repeat is recorded once and replayed
    d = chain.sizes()
    shapes = [tuple(int(v) for v in s) for s in chain.shapes()]
    mask_canonical, peak = ck.plan(ck.ALGO_DYNAMIC_N, d)
    # many sets reach Algorithm 6's peak; the step runs the one whose recomputed units are cheapest (unit costs
    # modelled from arithmetic and traffic), and the canonical set of Algorithm 6 is timed beside it
    t1 = time.perf_counter()
    mask, peak_mr, _ = ck.plan_min_recompute(d, chain.unit_costs())
    min_recompute_us = 1e6 * (time.perf_counter() - t1)
    assert peak_mr == peak
    planner_us = {}
    for name, algo in (("algorithm_3", ck.ALGO_STATIC_N3), ("algorithm_5", ck.ALGO_DYNAMIC_N2), ("algorithm_6", ck.ALGO_DYNAMIC_N)):
        runs = []
        for _ in range(3 if len(d) > 200 else 15):
            t1 = time.perf_counter()
            ck.plan(algo, d)
            runs.append(1e6 * (time.perf_counter() - t1))
        planner_us[name] = round(sorted(runs)[len(runs) // 2], 1)
    planner_us["min_recompute"] = round(min_recompute_us, 1)
    store_all = ck.eval(ck.MODEL_STORE_ALL, d, None)

    params_h = wl.make_params(spec, seed=0)
    params, grads, _ = ck.upload_params(chain, params_h)
    del params_h
    param_bytes = sum(t.numel() * t.element_size() for t in params) + sum(t.numel() * t.element_size() for t in grads)
    x_h, labels_h = wl.make_batch(spec, seed=1 + rank)
    tdt = torch.bfloat16 if spec["dtype"] == "bf16" else torch.float32
    x_pinned = torch.from_numpy(x_h).to(tdt).pin_memory()
    labels_pinned = torch.from_numpy(labels_h).pin_memory()
    x_dev, labels_dev = x_pinned.cuda(), labels_pinned.cuda()
    ws_bytes = chain.workspace_bytes()
    ws_plan = chain.workspace_bytes_for(ck.POLICY_DYNAMIC)       # Algorithm 4 needs no buffer for activated copies
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_regions(policy, plan_mask, arena, batch, labels, warm):
        def step():
            return ck.train_step(chain, plan_mask, policy, batch, labels, params, grads, arena, workspace, stream)
        for _ in range(warm):
            rep = step()
        out = []
        for _ in range(regions):
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                rep = step()
            e1.record(stream)
            barrier()
            out.append(max_over_ranks(e0.elapsed_time(e1), world, "cuda"))
        return out, rep

    def timed_regions_staged(policy, plan_mask, arena, batch, labels, warm):
        """End to end with the input copies overlapped: every step's batch goes from pinned host memory through
        ckpt_chain_stage_batch (one copy per step, all inside the timed region), the copy of step k + 1 running on the
        chain's copy stream while step k computes."""
        staging = torch.empty(chain.staging_bytes(), dtype=torch.uint8, device="cuda")

        def run(count):
            nxt = chain.stage_batch(0, batch, labels, staging)
            for k in range(count):
                cur = nxt
                if k + 1 < count:
                    nxt = chain.stage_batch((k + 1) % 2, batch, labels, staging)
                ck.train_step(chain, plan_mask, policy, cur[0], cur[1], params, grads, arena, workspace, stream)
        run(max(warm, 4))
        out = []
        for _ in range(regions):
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run(steps)
            e1.record(stream)
            barrier()
            out.append(max_over_ranks(e0.elapsed_time(e1), world, "cuda"))
        return out

    warm = max(args.warmup, 3)
    arena = torch.empty(peak, dtype=torch.uint8, device="cuda")
    if sampler is not None:
        sampler.start()
    ckpt_ms, rep = timed_regions(ck.POLICY_DYNAMIC, mask, arena, x_dev, labels_dev, warm)
    e2e_ms = timed_regions_staged(ck.POLICY_DYNAMIC, mask, arena, x_pinned, labels_pinned, 3)
    e2e_sync_ms, _ = timed_regions(ck.POLICY_DYNAMIC, mask, arena, x_pinned, labels_pinned, 3)
    canon_ms, rep_canon = timed_regions(ck.POLICY_DYNAMIC, mask_canonical, arena, x_dev, labels_dev, 3)
    clocks = sampler.stop() if sampler is not None else None
    del arena
    arena_all = torch.empty(store_all, dtype=torch.uint8, device="cuda")
    all_ms, rep_all = timed_regions(ck.POLICY_STORE_ALL, None, arena_all, x_dev, labels_dev, warm)
    # Algorithm 1 literally: residual blocks keep their interior tensors as well (a region per block in the workspace)
    kept_ms, ws_kept = None, ws_bytes
    if any(u["kind"] == "bottleneck" for u in spec["units"]):
        chain.set_keep_interiors(True)
        ws_kept = chain.workspace_bytes()
        workspace = None
        torch.cuda.empty_cache()
        workspace = torch.empty(ws_kept, dtype=torch.uint8, device="cuda")
        kept_ms, rep_kept = timed_regions(ck.POLICY_STORE_ALL, None, arena_all, x_dev, labels_dev, warm)
        assert rep_kept["loss"] == rep_all["loss"]
        chain.set_keep_interiors(False)
    del arena_all

    med = lambda v: float(sorted(v)[len(v) // 2])  # noqa: E731
    ms, ms_e2e, ms_all = med(ckpt_ms) / steps, med(e2e_ms) / steps, med(all_ms) / steps
    ms_e2e_sync = med(e2e_sync_ms) / steps
    ms_canon = med(canon_ms) / steps
    ms_kept = med(kept_ms) / steps if kept_ms else None
    flops, _ = conv_flops(spec, mask, shapes)
    gib = 2.0 ** 30
    out = {"workload": workload_name(spec), "n_units": len(spec["units"]), "batch": spec["batch"], "steps": steps,
           "regions_ms": [round(v, 3) for v in ckpt_ms], "ms_per_step": ms,
           "images_per_s": whole_job_images_per_s(spec["batch"], world, 1, ms),
           "e2e_images_per_s": whole_job_images_per_s(spec["batch"], world, 1, ms_e2e), "e2e_ms_per_step": ms_e2e,
           "e2e_path": "pinned host batch -> ckpt_chain_stage_batch (copy of step k+1 under step k) -> ckpt_train_step",
           "e2e_unstaged_images_per_s": whole_job_images_per_s(spec["batch"], world, 1, ms_e2e_sync),
           "h2d_bytes_per_step": int(x_pinned.numel() * x_pinned.element_size() + labels_pinned.numel() * 4), "d2h_bytes_per_step": 12,
           "store_all_ms_per_step": ms_all, "store_all_images_per_s": whole_job_images_per_s(spec["batch"], world, 1, ms_all),
           "recompute_overhead_pct": 100.0 * (ms / ms_all - 1.0),
           "store_all_note": "residual blocks re-derive their interior tensors in the backward under every schedule, store-all included; "
                             "store_all_keeping_interiors is Algorithm 1 taken literally (every block keeps its interiors in the workspace)",
           "store_all_keeping_interiors": None if ms_kept is None else {
               "ms_per_step": ms_kept, "images_per_s": whole_job_images_per_s(spec["batch"], world, 1, ms_kept),
               "recompute_overhead_pct": 100.0 * (ms / ms_kept - 1.0), "workspace_gib": ws_kept / 2.0 ** 30,
               "total_gib": (store_all + ws_kept + param_bytes) / 2.0 ** 30},
           "recomputed_units": int(rep["recomputed_units"]), "checkpoints": int(mask.sum()),
           "algorithm_6_set": {"ms_per_step": ms_canon, "recomputed_units": int(rep_canon["recomputed_units"]),
                               "checkpoints": int(mask_canonical.sum()), "peak_bytes": int(rep_canon["peak_bytes"]),
                               "recompute_overhead_pct": 100.0 * (ms_canon / ms_all - 1.0)},
           "launches_per_step": int(rep["launches"]), "store_all_launches_per_step": int(rep_all["launches"]),
           "memory_gib": {"arena_plan": peak / gib, "arena_store_all": store_all / gib, "arena_measured": rep["peak_bytes"] / gib,
                          "workspace": ws_plan / gib, "workspace_store_all": ws_bytes / gib, "parameters_and_gradients": param_bytes / gib,
                          "total_plan": (peak + ws_plan + param_bytes) / gib, "total_store_all": (store_all + ws_bytes + param_bytes) / gib},
           "peak_bytes": int(rep["peak_bytes"]), "predicted_bytes": int(peak), "store_all_bytes": int(store_all),
           "planner_us": planner_us, "loss": rep["loss"],
           "step_tflops": flops / (ms * 1e-3) / 1e12, "step_tensor_frac_of_sustained": flops / (ms * 1e-3) / 1e12 / peaks["tflops_sustained"],
           "clocks": clocks}
    assert rep["peak_bytes"] == peak and rep["loss"] == rep_all["loss"]
    del params, grads, workspace, x_dev, chain
    torch.cuda.empty_cache()
    if with_roofline:
        out["roofline"] = kernel_rooflines(spec, peaks)
        torch.cuda.empty_cache()
    return out


def kernel_rooflines(spec, peaks):
    """The step's kernels one at a time on the chain's own layer shapes (CUDA events, buffers rotated beyond the L2,
    >= 20 launches and >= 10 ms per shape): forward, dgrad and wgrad mixes over the chain's convolutions (the fully
    connected layers, HBM-bound matrix-streaming kernels, are listed apart as fc_*) against the measured dense-bf16
    peak (burst: kernels timed in isolation) and, per shape, against whichever of the tensor and HBM roofs bounds it;
    batch norm and 2x2 pooling over every tensor of the chain against the measured copy bandwidth."""
    import bench_ops
    out = {}
    # forward as the forward phase and the recomputation launch it: the convolution with the batch-norm sums of its
    # output in the epilogue, followed by the per-channel finalize (a second, tiny kernel inside the timed call);
    # fwd_plain: without the sums, as a residual block's backward re-derives its interior tensors
    for what, key in (("fwd_stats", "fwd"), ("dgrad", "dgrad"), ("wgrad", "wgrad"), ("fwd", "fwd_plain")):
        mix = bench_ops.conv_mix(what, spec, peaks)
        out["conv_" + key] = {"tflops": mix["tflops"], "frac_of_tensor_peak": mix["frac_of_tensor_peak"], "frac_of_roof": mix["frac_of_roof"],
                              "launches": mix["launches"], "ms": mix["ms"], "flops": mix["flops"], "per_shape": mix["per_shape"]}
    for what in ("fwd", "dgrad", "wgrad"):           # fully connected layers: kernels of their own, bound by the matrix traffic
        mix = bench_ops.conv_mix(what, spec, peaks, layers="fc")
        if mix is not None:
            out["fc_" + what] = {"gbs": sum(r["gbs"] * r["ms"] for r in mix["per_shape"]) / mix["ms"], "frac_of_roof": mix["frac_of_roof"],
                                 "launches": mix["launches"], "ms": mix["ms"], "per_shape": mix["per_shape"]}
    tot_f = sum(out["conv_" + w]["flops"] for w in ("fwd", "dgrad", "wgrad"))
    tot_ms = sum(out["conv_" + w]["ms"] for w in ("fwd", "dgrad", "wgrad"))
    out["conv_all"] = {"tflops": tot_f / tot_ms / 1e9, "frac_of_tensor_peak": tot_f / tot_ms / 1e9 / peaks["tflops_burst"],
                       "frac_of_sustained": tot_f / tot_ms / 1e9 / peaks["tflops_sustained"]}
    out["elementwise"] = bench_ops.elementwise_mix(spec, peaks)
    return out


HEADLINE_STEPS = {2: 30, 3: 20, 4: 8, 5: 6}        # timed steps per region: about a quarter to half a second each


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps per region of the headline workload (default: 30 for the VGG-16 chain)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--config", type=int, default=2, help="headline workload: benchmark configuration 2..5")
    ap.add_argument("--only", action="store_true", help="measure the headline workload only (no `configs` map)")
    ap.add_argument("--regions", type=int, default=3, help="timed regions per measurement; the median is reported")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (debugging only)")
    ap.add_argument("--cpu-batch", type=int, default=2)
    ap.add_argument("--steps-cpu", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-roofline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel of every step from the host")
    ap.add_argument("--split-units", action="store_true",
                    help="finer granularity: conv, batch norm and ReLU as chain units of their own")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    def spec_of(index):
        spec = wl.config(index)
        if args.batch:
            spec = dict(spec, batch=args.batch)
        if args.split_units:
            spec, _ = wl.split_units(spec)
        return spec

    spec = spec_of(args.config)
    steps = args.steps or HEADLINE_STEPS.get(args.config, 10)
    config = {"workload": workload_name(spec),
              "l2": "inputs larger than L2 (every step streams > 1 GB of activations); single kernels rotate over buffer sets beyond the L2",
              "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
              "submission": "launch by launch" if args.no_graph else "CUDA graph replay of the recorded step",
              "timing": "median of %d regions of %d steps" % (args.regions, steps)}

    if args.impl == "reference":
        if rank != 0:
            return
        # the requested step counts, each step a sample of the batch sized so that the run ends within about two minutes
        per_image = 4.5 if args.config == 2 else 2.5
        sample = int(max(1, min(spec["batch"], 120.0 / (per_image * max(1, args.steps + args.warmup)))))
        cpu = run_reference(spec, sample, steps=max(1, args.steps), warmup=max(0, args.warmup))
        config["submission"] = "CPU oracle (float64 numpy), store-all schedule"
        config["timing"] = "mean of %d steps" % cpu["steps"]
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

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")
    peaks = measured_peaks()
    roofs = rank == 0 and world == 1 and not args.no_roofline
    sampler = ClockSampler(local_rank) if rank == 0 else None
    head = measure_config(spec, args, rank, world, steps, args.regions, roofs, peaks, sampler)
    configs = None
    if world == 1 and not args.only and not args.batch and not args.split_units:
        configs = {}
        for index in (2, 3, 4, 5):
            name = wl.config(index)["name"]
            if index == args.config:
                configs[name] = head
            else:
                configs[name] = measure_config(spec_of(index), args, rank, world, HEADLINE_STEPS[index], args.regions, roofs, peaks)

    if rank == 0:
        line = {"metric": METRIC, "value": head["images_per_s"], "unit": UNIT, "n_gpus": world, "steps": steps,
                "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": spec["dtype"], "data": "synthetic", "config": config,
                "e2e": {"value": head["e2e_images_per_s"], "unit": UNIT, "h2d_bytes_per_step": head["h2d_bytes_per_step"],
                        "d2h_bytes_per_step": head["d2h_bytes_per_step"]},
                "gpu_launches": head["launches_per_step"] * steps, "clocks": head["clocks"],
                "peak_bytes": head["peak_bytes"], "predicted_bytes": head["predicted_bytes"], "store_all_bytes": head["store_all_bytes"],
                "peak_gib": head["memory_gib"]["arena_measured"], "workspace_gib": head["memory_gib"]["workspace"],
                "memory_gib": head["memory_gib"], "store_all_ms_per_step": head["store_all_ms_per_step"],
                "recompute_overhead_pct": head["recompute_overhead_pct"], "recomputed_units": head["recomputed_units"],
                "store_all_keeping_interiors": head["store_all_keeping_interiors"], "algorithm_6_set": head["algorithm_6_set"],
                "planner_us": head["planner_us"], "loss": head["loss"], "step_tflops": head["step_tflops"],
                "step_tensor_frac_of_sustained": head["step_tensor_frac_of_sustained"], "peaks": peaks}
        if "roofline" in head:
            line["roofline"] = headline_roofline(head["roofline"], peaks)
        if configs is not None:
            line["configs"] = {k: {kk: vv for kk, vv in v.items() if kk != "clocks"} for k, v in configs.items()}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = run_reference(spec, min(spec["batch"], args.cpu_batch), steps=args.steps_cpu)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def headline_roofline(r, peaks):
    """The contract's roofline object for the dominant kernels of the headline workload: the implicit-GEMM
    convolution-forward kernels (they run in the forward phase, in segment recomputation and, on the transposed
    filter, as dgrad).  achieved = sum of algorithmic FLOPs of the chain's convolution layers / sum of their launch times,
    each launch as the forward phase makes it: with the batch-norm sums in the epilogue and the finalize kernel after it."""
    f = r["conv_fwd"]
    return {"kernel": "tc_conv_tp_kernel / tc_conv_t_kernel (implicit-GEMM conv forward over the chain's layer mix)", "bound": "tensor",
            "achieved": f["tflops"], "peak": peaks["tflops_burst"], "unit": "TFLOP/s", "frac": f["frac_of_tensor_peak"],
            "peak_source": peaks["source"] + " (burst: kernels timed in isolation)", "traffic": None,
            "flops_per_launch": f["flops"] / f["launches"], "ms_per_launch": f["ms"] / f["launches"],
            "conv_fwd": f, "conv_fwd_plain": r["conv_fwd_plain"], "conv_dgrad": r["conv_dgrad"], "conv_wgrad": r["conv_wgrad"], "conv_all": r["conv_all"],
            "fc": {k: v for k, v in r.items() if k.startswith("fc_")}, "elementwise": r["elementwise"]}


if __name__ == "__main__":
    main()
