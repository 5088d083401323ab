"""Seeded synthetic workloads: chain descriptions and input arrays.

This module only *describes* chains (plain dicts) and draws random arrays.  It contains none of the
training-step or planner arithmetic, and is the one module that both the test oracle and the CUDA
binding's callers use, so that both sides see exactly the same arrays.

A chain is ``dict(units=[...], input_hwc=(H, W, C), batch=B, dtype="f32"|"bf16",
loss="sum"|"softmax_ce", name=...)``.  Unit dicts:

* ``{"kind": "conv_bn_relu", "cin", "cout", "k", "stride", "pad"}`` - convolution without bias,
  training-mode batch normalisation, ReLU; parameters ``w [cout,k,k,cin]``, ``gamma``, ``beta``.
* ``{"kind": "conv", ...}``, ``{"kind": "bn", "cin", "cout"}``, ``{"kind": "relu"}`` - the three steps of a
  conv_bn_relu unit as chain units of their own (finer granularity).
* ``{"kind": "maxpool", "k", "stride", "pad"}``
* ``{"kind": "avgpool"}`` - global average over H and W.
* ``{"kind": "fc", "cin", "cout", "relu"}`` - fully connected with bias on the NHWC-flattened input;
  parameters ``w [cout,cin]``, ``b``.
* ``{"kind": "bottleneck", "cin", "mid", "cout", "stride", "project"}`` - ResNet v1.5 bottleneck
  (1x1, 3x3 carrying the stride, 1x1, each followed by batch norm; optional 1x1 projection
  shortcut; ReLU after the residual add); parameters ``w1,g1,b1,w2,g2,b2,w3,g3,b3[,wp,gp,bp]``.

Activations are NHWC.  Arrays are float32 numpy; for ``dtype == "bf16"`` every value is first
rounded to the nearest bfloat16 so that a bf16 copy of it is exact.
"""

import numpy as np

PARAM_NAMES = {
    "conv_bn_relu": ["w", "gamma", "beta"],
    "maxpool": [],
    "avgpool": [],
    "fc": ["w", "b"],
    "conv": ["w"],
    "bn": ["gamma", "beta"],
    "relu": [],
    "bottleneck": ["w1", "g1", "b1", "w2", "g2", "b2", "w3", "g3", "b3", "wp", "gp", "bp"],
}


def to_bf16_representable(a):
    """Round float32 values to the nearest-even bfloat16, returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    rounded = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(a.shape)


# ------------------------------------------------------------------------------------------------
# chain builders
# ------------------------------------------------------------------------------------------------

def conv_unit(cin, cout, k=3, stride=1, pad=1):
    return {"kind": "conv_bn_relu", "cin": cin, "cout": cout, "k": k, "stride": stride, "pad": pad}


def plain_chain(n, channels, in_channels, hw, batch, dtype, loss="sum", name=None):
    """n units of 3x3 conv (stride 1, pad 1) + BN + ReLU."""
    units = []
    c = in_channels
    for _ in range(n):
        units.append(conv_unit(c, channels))
        c = channels
    return dict(units=units, input_hwc=(hw[0], hw[1], in_channels), batch=batch, dtype=dtype,
                loss=loss, name=name or "plain%d" % n)


def vgg16_chain(batch, hw=(224, 224), dtype="bf16", widths=(64, 128, 256, 512, 512),
                fc_width=4096, classes=1000, in_channels=3, name="vgg16"):
    """13 conv units in five stages (2,2,3,3,3), a 2x2 max-pool after each stage, three FC units."""
    units = []
    c = in_channels
    h, w = hw
    for stage, reps in enumerate((2, 2, 3, 3, 3)):
        for _ in range(reps):
            units.append(conv_unit(c, widths[stage]))
            c = widths[stage]
        units.append({"kind": "maxpool", "k": 2, "stride": 2, "pad": 0})
        h, w = h // 2, w // 2
    flat = h * w * c
    units.append({"kind": "fc", "cin": flat, "cout": fc_width, "relu": True})
    units.append({"kind": "fc", "cin": fc_width, "cout": fc_width, "relu": True})
    units.append({"kind": "fc", "cin": fc_width, "cout": classes, "relu": False})
    return dict(units=units, input_hwc=(hw[0], hw[1], in_channels), batch=batch, dtype=dtype,
                loss="softmax_ce", name=name)


def resnet_chain(blocks, batch, hw=(224, 224), dtype="bf16", base=64, classes=1000,
                 in_channels=3, name="resnet"):
    """Stem (7x7 s2 conv unit, 3x3 s2 max-pool), bottleneck stages, global avg-pool, FC."""
    units = [conv_unit(in_channels, base, k=7, stride=2, pad=3),
             {"kind": "maxpool", "k": 3, "stride": 2, "pad": 1}]
    cin = base
    for stage, reps in enumerate(blocks):
        mid = base * (2 ** stage)
        cout = 4 * mid
        for r in range(reps):
            stride = 2 if (r == 0 and stage > 0) else 1
            units.append({"kind": "bottleneck", "cin": cin, "mid": mid, "cout": cout,
                          "stride": stride, "project": r == 0})
            cin = cout
    units.append({"kind": "avgpool"})
    units.append({"kind": "fc", "cin": cin, "cout": classes, "relu": False})
    return dict(units=units, input_hwc=(hw[0], hw[1], in_channels), batch=batch, dtype=dtype,
                loss="softmax_ce", name=name)


def split_units(chain):
    """Finer granularity (Section 5.4): every conv+BN+ReLU unit becomes three chain units - convolution,
    batch normalisation, ReLU - each with an output of its own that the planner may keep or drop.
    Returns the new chain and, per new unit, (index of the original unit, names of the parameters it takes)."""
    units, origin = [], []
    for ui, u in enumerate(chain["units"]):
        if u["kind"] == "conv_bn_relu":
            units.append({"kind": "conv", "cin": u["cin"], "cout": u["cout"], "k": u["k"], "stride": u["stride"], "pad": u["pad"]})
            units.append({"kind": "bn", "cin": u["cout"], "cout": u["cout"]})
            units.append({"kind": "relu"})
            origin += [(ui, ["w"]), (ui, ["gamma", "beta"]), (ui, [])]
        else:
            units.append(dict(u))
            origin.append((ui, PARAM_NAMES[u["kind"]]))
    fine = dict(chain)
    fine["units"] = units
    fine["name"] = chain.get("name", "chain") + "_fine"
    return fine, origin


def split_params(origin, params):
    """Parameters of the original chain re-filed under the units of the split chain."""
    return [{name: params[ui][name] for name in names if name in params[ui]} for ui, names in origin]


def config(index):
    """The five benchmark configurations (index 1..5)."""
    if index == 1:
        return plain_chain(8, 16, 3, (32, 32), 4, "f32", "sum", name="cfg1_plain8_f32")
    if index == 2:
        return vgg16_chain(64, name="cfg2_vgg16_b64")
    if index == 3:
        return resnet_chain((3, 4, 6, 3), 128, name="cfg3_resnet50_b128")
    if index == 4:
        return resnet_chain((3, 8, 36, 3), 256, name="cfg4_resnet152_b256")
    if index == 5:
        return plain_chain(1000, 64, 64, (56, 56), 32, "bf16", "sum",
                           name="cfg5_plain1000_b32")
    raise ValueError("config index must be 1..5")


# ------------------------------------------------------------------------------------------------
# seeded arrays
# ------------------------------------------------------------------------------------------------

def param_shapes(unit):
    """Parameter name -> shape for one unit (no spatial information needed)."""
    k = unit["kind"]
    if k == "conv_bn_relu":
        return {"w": (unit["cout"], unit["k"], unit["k"], unit["cin"]),
                "gamma": (unit["cout"],), "beta": (unit["cout"],)}
    if k == "conv":
        return {"w": (unit["cout"], unit["k"], unit["k"], unit["cin"])}
    if k == "bn":
        return {"gamma": (unit["cout"],), "beta": (unit["cout"],)}
    if k == "fc":
        return {"w": (unit["cout"], unit["cin"]), "b": (unit["cout"],)}
    if k == "bottleneck":
        s = {"w1": (unit["mid"], 1, 1, unit["cin"]), "g1": (unit["mid"],), "b1": (unit["mid"],),
             "w2": (unit["mid"], 3, 3, unit["mid"]), "g2": (unit["mid"],), "b2": (unit["mid"],),
             "w3": (unit["cout"], 1, 1, unit["mid"]), "g3": (unit["cout"],), "b3": (unit["cout"],)}
        if unit["project"]:
            s.update({"wp": (unit["cout"], 1, 1, unit["cin"]),
                      "gp": (unit["cout"],), "bp": (unit["cout"],)})
        return s
    return {}


def make_params(chain, seed=0, bn_affine="standard"):
    """He-normal matrices (std = sqrt(2/fan_in)); BN scale 1 / shift 0 ("standard") or a random
    scale in [0.5, 1.5] and shift ~ N(0, 0.2) ("random", used by parity tests so that a misplaced
    gamma or beta changes the result); FC bias ~ N(0, 0.1) under "random", else 0.
    Returns a list (one dict per unit)."""
    rng = np.random.default_rng(seed)
    low_precision = chain["dtype"] == "bf16"
    out = []
    for unit in chain["units"]:
        p = {}
        for name, shape in param_shapes(unit).items():
            if name.startswith("w"):
                fan_in = int(np.prod(shape[1:]))
                a = rng.standard_normal(shape).astype(np.float32) * np.float32(np.sqrt(2.0 / fan_in))
                if low_precision:
                    a = to_bf16_representable(a)
            elif name.startswith("g"):
                a = (np.ones(shape, np.float32) if bn_affine == "standard"
                     else rng.uniform(0.5, 1.5, shape).astype(np.float32))
            else:
                a = (np.zeros(shape, np.float32) if bn_affine == "standard"
                     else (rng.standard_normal(shape) * (0.1 if name == "b" and unit["kind"] == "fc" else 0.2)).astype(np.float32))
            p[name] = np.ascontiguousarray(a)
        out.append(p)
    return out


def make_batch(chain, seed=1, classes=None):
    """Input x ~ N(0,1) in NHWC and uniform integer labels."""
    rng = np.random.default_rng(seed)
    h, w, c = chain["input_hwc"]
    x = rng.standard_normal((chain["batch"], h, w, c)).astype(np.float32)
    if chain["dtype"] == "bf16":
        x = to_bf16_representable(x)
    if classes is None:
        classes = 1000
        for unit in reversed(chain["units"]):
            if unit["kind"] == "fc":
                classes = unit["cout"]
                break
    labels = rng.integers(0, classes, size=(chain["batch"],)).astype(np.int32)
    return x, labels
