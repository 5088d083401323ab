"""Numeric oracle: one store-all training step of a layer chain in float64 on the CPU.

TEST INFRASTRUCTURE ONLY.  Plain numpy statement of Algorithm 1 (allocate every d_i, forward by
Eq. (1), backward by Eqs. (2)-(5)) for the layer types the benchmark chains use.  It shares no
code with the CUDA library and must never be imported by it; only ``tests/``, the smoke check and
the benchmark's CPU-baseline leg call it.

The paper leaves f_i abstract, so each layer follows its textbook definition:

* convolution = cross-correlation on NHWC with zero padding and no bias; written as a sum over the
  k x k taps of (shifted input) @ (tap matrix), which is the definition regrouped by tap;
* batch normalisation in training mode: per-channel mean and *biased* variance over N*H*W,
  eps = 1e-5, y = gamma * xhat + beta; its backward is the derivative of exactly that;
* ReLU; max-pool where the first maximum in row-major window order receives the gradient;
  global average pool; fully connected with bias on the NHWC-flattened input;
* losses: sum of all outputs, or softmax cross-entropy averaged over the batch.

``storage="bf16"`` additionally rounds a tensor to bfloat16 (round-to-nearest-even) at each point
where a tensor is written to memory by a low-precision executor: the convolution output, the
unit output, and every activation gradient.  Arithmetic stays float64.  It exists for very deep
chains, where one rounding per stored tensor, not the arithmetic, dominates the difference from
the exact result.  ``storage="exact"`` (default) rounds nothing.

Parity status: pinned by tests/test_oracle_numeric.py - central finite differences of the loss
for every parameter kind, a pure-Python-loop convolution and pool on tiny inputs,
scipy.signal.correlate2d, the zero-gradient property of batch norm under a constant upstream
gradient, and hand-computed softmax values.  The "bf16" storage mode is pinned through its
rounding function (exact bit patterns), the property that exactly the stored tensors are bfloat16
codes, and its distance from the exact mode on a one-unit chain.
"""

import numpy as np

EPS = 1e-5


# ------------------------------------------------------------------------------------------------
# storage rounding
# ------------------------------------------------------------------------------------------------

def round_bf16(a):
    """Nearest-even rounding of float64/float32 values to bfloat16 (via float32), as float64."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    bits = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def _store(a, storage):
    return round_bf16(a) if storage == "bf16" else a


# ------------------------------------------------------------------------------------------------
# layers
# ------------------------------------------------------------------------------------------------

def conv_out_size(h, k, stride, pad):
    return (h + 2 * pad - k) // stride + 1


def conv2d_fwd(x, w, stride, pad):
    n, h, wd, cin = x.shape
    cout, kh, kw, _ = w.shape
    ho = conv_out_size(h, kh, stride, pad)
    wo = conv_out_size(wd, kw, stride, pad)
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, cin), dtype=np.float64)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    z = np.zeros((n, ho, wo, cout), dtype=np.float64)
    for r in range(kh):
        for s in range(kw):
            patch = xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :]
            z += patch @ w[:, r, s, :].T
    return z


def conv2d_bwd(x, w, dz, stride, pad):
    n, h, wd, cin = x.shape
    cout, kh, kw, _ = w.shape
    _, ho, wo, _ = dz.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, cin), dtype=np.float64)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w, dtype=np.float64)
    dz2 = dz.reshape(-1, cout)
    for r in range(kh):
        for s in range(kw):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dw[:, r, s, :] = dz2.T @ xp[sl].reshape(-1, cin)
            dxp[sl] += dz @ w[:, r, s, :]
    return dxp[:, pad:pad + h, pad:pad + wd, :], dw


def bn_fwd(z, gamma, beta):
    mean = z.mean(axis=(0, 1, 2))
    var = ((z - mean) ** 2).mean(axis=(0, 1, 2))        # biased
    inv_std = 1.0 / np.sqrt(var + EPS)
    xhat = (z - mean) * inv_std
    return gamma * xhat + beta, (xhat, inv_std)


def bn_bwd(dy, cache, gamma):
    xhat, inv_std = cache
    m = dy.shape[0] * dy.shape[1] * dy.shape[2]
    dbeta = dy.sum(axis=(0, 1, 2))
    dgamma = (dy * xhat).sum(axis=(0, 1, 2))
    dz = gamma * inv_std * (dy - dbeta / m - xhat * dgamma / m)
    return dz, dgamma, dbeta


def maxpool_fwd(x, k, stride, pad):
    n, h, w, c = x.shape
    ho = conv_out_size(h, k, stride, pad)
    wo = conv_out_size(w, k, stride, pad)
    xp = np.full((n, h + 2 * pad, w + 2 * pad, c), -np.inf)
    xp[:, pad:pad + h, pad:pad + w, :] = x
    y = np.full((n, ho, wo, c), -np.inf)
    arg = np.zeros((n, ho, wo, c), dtype=np.int64)
    for r in range(k):
        for s in range(k):
            patch = xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :]
            better = patch > y                           # strict: the first maximum is kept
            y = np.where(better, patch, y)
            arg = np.where(better, r * k + s, arg)
    return y, arg


def maxpool_bwd(dy, arg, x_shape, k, stride, pad):
    n, h, w, c = x_shape
    _, ho, wo, _ = dy.shape
    dxp = np.zeros((n, h + 2 * pad, w + 2 * pad, c))
    for r in range(k):
        for s in range(k):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dxp[sl] += np.where(arg == r * k + s, dy, 0.0)
    return dxp[:, pad:pad + h, pad:pad + w, :]


def softmax_ce(logits, labels):
    """Mean cross-entropy and its gradient w.r.t. the logits."""
    b = logits.shape[0]
    z = logits.reshape(b, -1)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    loss = -np.log(p[np.arange(b), labels]).mean()
    g = p.copy()
    g[np.arange(b), labels] -= 1.0
    return loss, (g / b).reshape(logits.shape)


# ------------------------------------------------------------------------------------------------
# units: forward returns (output, cache); backward returns (dx, grads dict)
# ------------------------------------------------------------------------------------------------

def _cbr_fwd(x, w, gamma, beta, stride, pad, relu, storage):
    z = _store(conv2d_fwd(x, w, stride, pad), storage)
    y, bn_cache = bn_fwd(z, gamma, beta)
    if relu:
        y = np.maximum(y, 0.0)
    return y, (x, bn_cache)


def _cbr_bwd(dy, y, cache, w, gamma, stride, pad, relu, storage):
    x, bn_cache = cache
    if relu:
        dy = dy * (y > 0)
    dz, dgamma, dbeta = bn_bwd(dy, bn_cache, gamma)
    dz = _store(dz, storage)
    dx, dw = conv2d_bwd(x, w, dz, stride, pad)
    return dx, dw, dgamma, dbeta


def unit_forward(unit, p, x, storage="exact"):
    kind = unit["kind"]
    if kind == "conv_bn_relu":
        y, c = _cbr_fwd(x, p["w"], p["gamma"], p["beta"], unit["stride"], unit["pad"], True, storage)
        y = _store(y, storage)
        return y, (c, y)
    if kind == "conv":                                   # finer granularity (Section 5.4): the three
        return _store(conv2d_fwd(x, p["w"], unit["stride"], unit["pad"]), storage), x
    if kind == "bn":                                     # steps of a conv unit as chain units of their own
        y, c = bn_fwd(x, p["gamma"], p["beta"])
        return _store(y, storage), c
    if kind == "relu":
        y = np.maximum(x, 0.0)
        return y, y
    if kind == "maxpool":
        y, arg = maxpool_fwd(x, unit["k"], unit["stride"], unit["pad"])
        return y, (arg, x.shape)
    if kind == "avgpool":
        return x.mean(axis=(1, 2), keepdims=True), x.shape
    if kind == "fc":
        b = x.shape[0]
        y = x.reshape(b, -1) @ p["w"].T + p["b"]
        if unit["relu"]:
            y = np.maximum(y, 0.0)
        y = _store(y.reshape(b, 1, 1, -1), storage)
        return y, (x, y)
    if kind == "bottleneck":
        st = unit["stride"]
        a, ca = _cbr_fwd(x, p["w1"], p["g1"], p["b1"], 1, 0, True, storage)
        a = _store(a, storage)
        b2, cb = _cbr_fwd(a, p["w2"], p["g2"], p["b2"], st, 1, True, storage)
        b2 = _store(b2, storage)
        c3, cc = _cbr_fwd(b2, p["w3"], p["g3"], p["b3"], 1, 0, False, storage)
        if unit["project"]:
            sc, cs = _cbr_fwd(x, p["wp"], p["gp"], p["bp"], st, 0, False, storage)
        else:
            sc, cs = x, None
        y = _store(np.maximum(c3 + sc, 0.0), storage)
        return y, (ca, a, cb, b2, cc, cs, y)
    raise ValueError(kind)


def unit_backward(unit, p, dy, cache, storage="exact"):
    kind = unit["kind"]
    if kind == "conv_bn_relu":
        c, y = cache
        dx, dw, dg, db = _cbr_bwd(dy, y, c, p["w"], p["gamma"], unit["stride"], unit["pad"], True, storage)
        return _store(dx, storage), {"w": dw, "gamma": dg, "beta": db}
    if kind == "conv":
        dx, dw = conv2d_bwd(cache, p["w"], dy, unit["stride"], unit["pad"])
        return _store(dx, storage), {"w": dw}
    if kind == "bn":
        dx, dgamma, dbeta = bn_bwd(dy, cache, p["gamma"])
        return _store(dx, storage), {"gamma": dgamma, "beta": dbeta}
    if kind == "relu":
        return dy * (cache > 0), {}
    if kind == "maxpool":
        arg, xs = cache
        return maxpool_bwd(dy, arg, xs, unit["k"], unit["stride"], unit["pad"]), {}
    if kind == "avgpool":
        n, h, w, c = cache
        return _store(np.broadcast_to(dy / (h * w), (n, h, w, c)).copy(), storage), {}
    if kind == "fc":
        x, y = cache
        b = x.shape[0]
        g = dy.reshape(b, -1)
        if unit["relu"]:
            g = g * (y.reshape(b, -1) > 0)
        dw = g.T @ x.reshape(b, -1)
        dbias = g.sum(axis=0)
        dx = (g @ p["w"]).reshape(x.shape)
        return _store(dx, storage), {"w": dw, "b": dbias}
    if kind == "bottleneck":
        ca, a, cb, b2, cc, cs, y = cache
        st = unit["stride"]
        g = dy * (y > 0)
        grads = {}
        if unit["project"]:
            dxs, grads["wp"], grads["gp"], grads["bp"] = _cbr_bwd(g, None, cs, p["wp"], p["gp"], st, 0, False, storage)
        else:
            dxs = g
        db2, grads["w3"], grads["g3"], grads["b3"] = _cbr_bwd(g, None, cc, p["w3"], p["g3"], 1, 0, False, storage)
        db2 = _store(db2, storage)
        da, grads["w2"], grads["g2"], grads["b2"] = _cbr_bwd(db2, b2, cb, p["w2"], p["g2"], st, 1, True, storage)
        da = _store(da, storage)
        dx, grads["w1"], grads["g1"], grads["b1"] = _cbr_bwd(da, a, ca, p["w1"], p["g1"], 1, 0, True, storage)
        return _store(dx + dxs, storage), grads
    raise ValueError(kind)


# ------------------------------------------------------------------------------------------------
# the whole step (Algorithm 1)
# ------------------------------------------------------------------------------------------------

def loss_and_grad(chain, d_n, labels):
    if chain["loss"] == "sum":
        return float(d_n.sum()), np.ones_like(d_n)
    if chain["loss"] == "softmax_ce":
        return softmax_ce(d_n, labels)
    raise ValueError(chain["loss"])


def chain_forward(chain, params, x, storage="exact"):
    """Forward phase: returns the list d_0..d_n and the per-unit caches."""
    params = [{k: np.asarray(v, dtype=np.float64) for k, v in p.items()} for p in params]
    d = [np.asarray(x, dtype=np.float64)]
    caches = []
    for unit, p in zip(chain["units"], params):
        y, c = unit_forward(unit, p, d[-1], storage)
        d.append(y)
        caches.append(c)
    return d, caches, params


def chain_forward_backward(chain, params, x, labels=None, storage="exact"):
    """One store-all step.  Returns dict(loss, grads=[{name: array}], d=[d_0..d_n])."""
    d, caches, params = chain_forward(chain, params, x, storage)
    loss, r = loss_and_grad(chain, d[-1], labels)
    r = _store(r, storage)
    grads = [None] * len(chain["units"])
    for i in range(len(chain["units"]) - 1, -1, -1):      # units are 1-based in the paper
        r, grads[i] = unit_backward(chain["units"][i], params[i], r, caches[i], storage)
    return dict(loss=loss, grads=grads, d=d, input_grad=r)


def sgd_update(params, grads, lr, storage="exact"):
    """Last line of the backward loop of Algorithm 1, "update w_i with g_i", read as plain gradient descent:
    w_i <- w_i - lr * g_i for every parameter of every unit.  With storage="bf16" the matrices (names starting with
    "w"), which a low-precision executor keeps in bfloat16, are rounded after the update."""
    out = []
    for p, g in zip(params, grads):
        q = {}
        for name, w in p.items():
            new = np.asarray(w, dtype=np.float64) - lr * np.asarray(g[name], dtype=np.float64)
            q[name] = _store(new, storage) if name.startswith("w") else new
        out.append(q)
    return out


def output_shapes(chain):
    """(H, W, C) of d_0..d_n by running shapes through the layer definitions."""
    h, w, c = chain["input_hwc"]
    out = [(h, w, c)]
    for u in chain["units"]:
        k = u["kind"]
        if k in ("conv_bn_relu", "conv"):
            h, w, c = conv_out_size(h, u["k"], u["stride"], u["pad"]), conv_out_size(w, u["k"], u["stride"], u["pad"]), u["cout"]
        elif k == "maxpool":
            h, w = conv_out_size(h, u["k"], u["stride"], u["pad"]), conv_out_size(w, u["k"], u["stride"], u["pad"])
        elif k == "avgpool":
            h, w = 1, 1
        elif k == "fc":
            h, w, c = 1, 1, u["cout"]
        elif k == "bottleneck":
            h, w, c = conv_out_size(h, 3, u["stride"], 1), conv_out_size(w, 3, u["stride"], 1), u["cout"]
        out.append((h, w, c))
    return out
