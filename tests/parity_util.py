"""Unit-by-unit comparison of a store-all GPU step with the oracle, each unit on the GPU's own inputs.

A store-all step (Algorithm 1) leaves d_0 .. d_n in the arena at consecutive offsets, and the gradient tap
(ckpt_chain_set_gradient_tap) leaves r_i = dL/dd_i for i = n .. 1.  With those, every unit can be checked against the
oracle's definition of that unit *locally*: the oracle is handed the tensors the GPU's unit was handed (its stored
input, its incoming gradient) and must reproduce what the GPU's unit produced (its stored output, its weight
gradients, its outgoing gradient).  A wrong hand-over between two units then shows up at that hand-over, and the
comparison is free of the decision flips (ReLU masks, pooling arg-max) that make end-to-end differences of deep
bf16 chains grow from layer to layer.

The executor stores the convolution output of a conv+BN+ReLU unit *before* normalisation as d_i and whoever reads
d_i applies normalisation + ReLU, so the gradient boundary sits half a layer earlier than in the oracle's unit:
r_i is dL/d(conv output).  The helpers below therefore compose the oracle's layer functions (conv2d_fwd/bwd, bn_fwd/
bwd, unit_forward/unit_backward for the other kinds) at that boundary; no arithmetic of their own beyond the ReLU mask.
"""
import numpy as np

from oracle import numeric_oracle as no
from paper_2502_12499_b200 import binding as ck


def max_rel(got, want):
    got = np.asarray(got, dtype=np.float64).reshape(np.shape(want))
    want = np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    if not np.all(np.isfinite(got)):
        return float("inf")
    return float(np.abs(got - want).max() / scale) if scale > 0 else float(np.abs(got).max())


def outlier_fraction(got, want, tol):
    """Fraction of elements further than tol * max|want| from the reference."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64).reshape(want.shape)
    scale = np.abs(want).max()
    return float(np.mean(np.abs(got - want) > tol * scale)) if scale > 0 else float(np.mean(got != 0))


def rel_l2(got, want):
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64).reshape(want.shape)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


class StoredStep:
    """Runs one store-all step with the gradient tap on and gives access to d_i and r_i as float64 arrays."""

    def __init__(self, runner, x, labels):
        import torch
        self.runner = runner
        self.spec = runner.spec
        d = [int(v) for v in runner.d]
        self.d = d
        self.shapes = [tuple(int(v) for v in s) for s in runner.chain.shapes()]
        self.tap = torch.empty(sum(d[1:]), dtype=torch.uint8, device="cuda")
        self.tap.fill_(0xFF)
        runner.chain.set_gradient_tap(self.tap)
        ck.launch_log(True)
        try:
            self.report, self.grads = runner.run(ck.POLICY_STORE_ALL, None, x, labels)
        finally:
            self.kernels = ck.launch_log_read()
            ck.launch_log(False)
            runner.chain.set_gradient_tap(None)
        self.arena = runner.arena
        self.offsets = np.concatenate([[0], np.cumsum(d)]).astype(np.int64)

    def _view(self, buf, off, i):
        import torch
        h, w, c = self.shapes[i]
        b = self.spec["batch"]
        tdt = torch.bfloat16 if self.spec["dtype"] == "bf16" else torch.float32
        es = 2 if self.spec["dtype"] == "bf16" else 4
        t = buf[off: off + b * h * w * c * es].view(tdt).reshape(b, h, w, c)
        return t.float().cpu().numpy().astype(np.float64)

    def stored(self, i):
        """d_i as the executor stored it (for a conv+BN+ReLU unit: the convolution output)."""
        return self._view(self.arena, int(self.offsets[i]), i)

    def gradient(self, i):
        """r_i = dL/d(stored d_i), i = 1 .. n."""
        return self._view(self.tap, int(self.offsets[i] - self.offsets[1]), i)


def _params64(params):
    return [{k: np.asarray(v, dtype=np.float64) for k, v in p.items()} for p in params]


def check_units_locally(step, params, labels, storage):
    """Returns a list of (where, what, error, l2, outliers) for every quantity a unit produces, the oracle being given
    the GPU's own inputs of that unit: error = max|got - want| / max|want|, l2 = relative L2 distance, outliers =
    fraction of elements further than 3e-2 * max|want| from the reference."""
    spec = step.spec
    units = spec["units"]
    n = len(units)
    p64 = _params64(params)
    grads = {}
    for (ui, name, _), g in zip(step.runner.flat, step.grads):
        grads[(ui, name)] = g
    rows = []

    def row(where, what, got, want):
        rows.append((where, what, max_rel(got, want), rel_l2(got, want), outlier_fraction(got, want, 3e-2)))

    def st(a):
        return no.round_bf16(a) if storage == "bf16" else a

    def activated(i, s_i):
        """Oracle's reading of stored d_i: normalisation + ReLU of a conv unit's stored output, else d_i itself."""
        if i >= 1 and units[i - 1]["kind"] == "conv_bn_relu":
            p = p64[i - 1]
            y, cache = no.bn_fwd(s_i, p["gamma"], p["beta"])
            return st(np.maximum(y, 0.0)), cache
        return s_i, None

    def through_pending(i, a_i, cache_i, dx):
        """dL/d(activated d_i) -> dL/d(stored d_i), with the scale/shift gradients of unit i's normalisation."""
        if cache_i is None:
            return dx
        p = p64[i - 1]
        dz, dgamma, dbeta = no.bn_bwd(dx * (a_i > 0), cache_i, p["gamma"])
        row(i, "dgamma", grads[(i - 1, "gamma")], dgamma)
        row(i, "dbeta", grads[(i - 1, "beta")], dbeta)
        return st(dz)

    s_prev = step.stored(0)
    for i in range(1, n + 1):
        unit, p = units[i - 1], p64[i - 1]
        a_prev, cache_prev = activated(i - 1, s_prev)
        s_i = step.stored(i)
        t_i = step.gradient(i)
        if unit["kind"] == "conv_bn_relu":
            want = st(no.conv2d_fwd(a_prev, p["w"], unit["stride"], unit["pad"]))
            row(i, "d_i", s_i, want)
            dx, dw = no.conv2d_bwd(a_prev, p["w"], t_i, unit["stride"], unit["pad"])
            dx = st(dx)
            row(i, "dw", grads[(i - 1, "w")], dw)
        else:
            want, cache = no.unit_forward(unit, p, a_prev, storage)
            row(i, "d_i", s_i, want)
            if unit["kind"] in ("fc", "bottleneck"):
                cache = tuple(cache[:-1]) + (s_i,)      # the final ReLU mask is decided on the stored output
            dx, g = no.unit_backward(unit, p, t_i, cache, storage)
            for name, arr in g.items():
                row(i, "d" + name, grads[(i - 1, name)], arr)
        if i > 1:
            want_t = through_pending(i - 1, a_prev, cache_prev, dx)
            row(i - 1, "r_i", step.gradient(i - 1), want_t)
        s_prev = s_i
    # the loss and r_n
    a_n, cache_n = activated(n, s_prev)
    loss, r = no.loss_and_grad(spec, a_n, labels)
    rows.append((n + 1, "loss", abs(step.report["loss"] - loss) / max(abs(loss), 1e-300), 0.0, 0.0))
    want_t = through_pending(n, a_n, cache_n, st(r))
    row(n, "r_i", step.gradient(n), want_t)
    return rows


def whole_step_errors(step, ref):
    """Per gradient tensor: (unit, name, max relative error, relative L2 distance) against the oracle's whole step."""
    out = []
    for (ui, name, _), g in zip(step.runner.flat, step.grads):
        want = ref["grads"][ui][name]
        out.append((ui + 1, name, max_rel(g, want), rel_l2(g, want)))
    return out


def decision_flips(step, params, ref):
    """Per unit that ends in a ReLU: the fraction of output elements whose ReLU decision differs between the executor's
    stored tensor (a conv unit's stored output read through the oracle's normalisation) and the oracle's whole step."""
    out = []
    p64 = _params64(params)
    for i, unit in enumerate(step.spec["units"], start=1):
        kind = unit["kind"]
        if kind == "conv_bn_relu":
            mine, _ = no.bn_fwd(step.stored(i), p64[i - 1]["gamma"], p64[i - 1]["beta"])
        elif kind == "bottleneck" or (kind == "fc" and unit["relu"]):
            mine = step.stored(i)
        else:
            continue
        out.append((i, float(np.mean((mine > 0) != (ref["d"][i] > 0)))))
    return out
