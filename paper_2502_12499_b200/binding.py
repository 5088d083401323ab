"""ctypes binding of libckpt_b200.so: argument marshalling only.

Every function here has the name of the C entry point it wraps (minus the ``ckpt_`` prefix) and
does no arithmetic of its own.  torch is used only to own device memory and streams.  If the shared
library is missing, loading fails with an error: there is no fallback path.
"""

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libckpt_b200.so")

ALGO_STATIC_N3, ALGO_DYNAMIC_N2, ALGO_DYNAMIC_N, ALGO_SQRT_N = 0, 1, 2, 3
MODEL_STATIC, MODEL_DYNAMIC, MODEL_STORE_ALL = 0, 1, 2
POLICY_STORE_ALL, POLICY_STATIC, POLICY_DYNAMIC = 0, 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1
LOSS_SUM, LOSS_SOFTMAX_CE = 0, 1
UNIT_KINDS = {"conv_bn_relu": 0, "maxpool": 1, "fc": 2, "avgpool": 3, "bottleneck": 4, "conv": 5, "bn": 6, "relu": 7}
ERROR_NAMES = {-1: "E_NULL", -2: "E_BAD_N", -3: "E_BAD_SIZE", -4: "E_OVERFLOW", -5: "E_BAD_PLAN",
               -6: "E_BAD_ARG", -7: "E_ARENA_OOM", -8: "E_WORKSPACE", -9: "E_CUDA",
               -10: "E_DEVICE_TIMEOUT", -11: "E_UNSUPPORTED", -12: "E_NO_DEVICE"}


class CkptError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("%s (%d): %s" % (ERROR_NAMES.get(code, "?"), code, message))
        self.code = code


class UnitDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("c_in", C.c_int32), ("c_out", C.c_int32), ("k", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32), ("mid", C.c_int32), ("flags", C.c_int32)]


class ConvShape(C.Structure):
    _fields_ = [("n", C.c_int32), ("h", C.c_int32), ("w", C.c_int32), ("c_in", C.c_int32),
                ("c_out", C.c_int32), ("k", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32)]


class StepReport(C.Structure):
    _fields_ = [("peak_bytes", C.c_int64), ("extent_bytes", C.c_int64), ("predicted_bytes", C.c_int64),
                ("workspace_bytes", C.c_int64), ("launches", C.c_int64), ("recomputed_units", C.c_int64),
                ("loss", C.c_double), ("device_status", C.c_int32), ("replayed", C.c_int32)]


_lib = None


def lib():
    """The loaded shared library (built by ``paper_2502_12499_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libckpt_b200.so is not built: run `python -m paper_2502_12499_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        _lib = C.CDLL(LIB_PATH)
        _lib.ckpt_last_error.restype = C.c_char_p
    return _lib


def _check(rc):
    if rc != 0:
        raise CkptError(rc, lib().ckpt_last_error().decode())


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _ptr(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _dev(t):
    """Raw address of a torch tensor (or None)."""
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(stream if isinstance(stream, int) else stream.cuda_stream)


# ------------------------------------------------------------------------------------------------
# host planners
# ------------------------------------------------------------------------------------------------

def plan(algo, d):
    """ckpt_plan: returns (is_ckpt uint8[n+1], peak_bytes)."""
    d = _i64(d)
    n = len(d) - 1
    mask = np.zeros(max(n + 1, 1), dtype=np.uint8)
    peak = C.c_int64(0)
    _check(lib().ckpt_plan(C.c_int(algo), C.c_int64(n), _ptr(d, C.c_int64), _ptr(mask, C.c_uint8), C.byref(peak)))
    return mask, peak.value


def plan_counted(algo, d):
    """ckpt_plan_counted: returns (is_ckpt, peak_bytes, work)."""
    d = _i64(d)
    n = len(d) - 1
    mask = np.zeros(max(n + 1, 1), dtype=np.uint8)
    peak, work = C.c_int64(0), C.c_int64(0)
    _check(lib().ckpt_plan_counted(C.c_int(algo), C.c_int64(n), _ptr(d, C.c_int64), _ptr(mask, C.c_uint8),
                                   C.byref(peak), C.byref(work)))
    return mask, peak.value, work.value


def eval(model, d, is_ckpt):  # noqa: A001 - named after ckpt_eval
    d = _i64(d)
    n = len(d) - 1
    peak = C.c_int64(0)
    mask_p = None
    if is_ckpt is not None:
        mask = np.ascontiguousarray(is_ckpt, dtype=np.uint8)
        mask_p = _ptr(mask, C.c_uint8)
    _check(lib().ckpt_eval(C.c_int(model), C.c_int64(n), _ptr(d, C.c_int64), mask_p, C.byref(peak)))
    return peak.value


def plan_min_recompute(d, cost, budget=0):
    """ckpt_plan_min_recompute: (is_ckpt mask, peak bytes, recomputation cost) of a set with the least recomputation
    cost among those whose Eq. (memory) value is at most ``budget`` (0: the optimum of Algorithms 5/6)."""
    d = np.ascontiguousarray(d, dtype=np.int64)
    cost = np.ascontiguousarray(cost, dtype=np.int64)
    if cost.shape != d.shape:
        raise ValueError("cost needs one entry per tensor d_0..d_n")
    n = d.size - 1
    mask = np.zeros(n + 1, dtype=np.uint8)
    peak, rec = C.c_int64(0), C.c_int64(0)
    _check(lib().ckpt_plan_min_recompute(C.c_int64(n), _ptr(d, C.c_int64), _ptr(cost, C.c_int64), C.c_int64(int(budget)),
                                         _ptr(mask, C.c_uint8), C.byref(peak), C.byref(rec)))
    return mask, peak.value, rec.value


def plan_sizes(algo, kept, live, grad, incoming=False):
    """ckpt_plan_sizes: returns (is_ckpt uint8[n+1], peak_bytes)."""
    kept, live, grad = _i64(kept), _i64(live), _i64(grad)
    n = len(kept) - 1
    mask = np.zeros(max(n + 1, 1), dtype=np.uint8)
    peak = C.c_int64(0)
    _check(lib().ckpt_plan_sizes(C.c_int(algo), C.c_int64(n), _ptr(kept, C.c_int64), _ptr(live, C.c_int64), _ptr(grad, C.c_int64),
                                 C.c_int(1 if incoming else 0), _ptr(mask, C.c_uint8), C.byref(peak)))
    return mask, peak.value


def eval_sizes(kept, live, grad, is_ckpt, incoming=False):
    kept, live, grad = _i64(kept), _i64(live), _i64(grad)
    n = len(kept) - 1
    mask = np.ascontiguousarray(is_ckpt, dtype=np.uint8)
    peak = C.c_int64(0)
    _check(lib().ckpt_eval_sizes(C.c_int64(n), _ptr(kept, C.c_int64), _ptr(live, C.c_int64), _ptr(grad, C.c_int64),
                                 C.c_int(1 if incoming else 0), _ptr(mask, C.c_uint8), C.byref(peak)))
    return peak.value


def arena_dry_run(policy, d, is_ckpt):
    """ckpt_arena_dry_run: returns dict(events=int64[k,4], high_water, extent)."""
    d = _i64(d)
    n = len(d) - 1
    mask_p = None
    if is_ckpt is not None:
        mask = np.ascontiguousarray(is_ckpt, dtype=np.uint8)
        mask_p = _ptr(mask, C.c_uint8)
    cap = 8 * (n + 2) + 16
    ev = np.zeros((cap, 4), dtype=np.int64)
    n_ev, hw, ext = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    _check(lib().ckpt_arena_dry_run(C.c_int(policy), C.c_int64(n), _ptr(d, C.c_int64), mask_p, _ptr(ev, C.c_int64),
                                    C.c_int64(cap), C.byref(n_ev), C.byref(hw), C.byref(ext)))
    return dict(events=ev[: n_ev.value].copy(), high_water=hw.value, extent=ext.value)


def arena_stage_trace(policy, d, is_ckpt):
    """ckpt_arena_stage_trace: int64[2n+2], arena bytes at the end of every training phase index."""
    d = _i64(d)
    n = len(d) - 1
    mask_p = None
    if is_ckpt is not None:
        mask = np.ascontiguousarray(is_ckpt, dtype=np.uint8)
        mask_p = _ptr(mask, C.c_uint8)
    trace = np.zeros(2 * n + 2, dtype=np.int64)
    _check(lib().ckpt_arena_stage_trace(C.c_int(policy), C.c_int64(n), _ptr(d, C.c_int64), mask_p, _ptr(trace, C.c_int64)))
    return trace


def mask_from_set(n, checkpoints):
    m = np.zeros(n + 1, dtype=np.uint8)
    m[list(checkpoints)] = 1
    return m


# ------------------------------------------------------------------------------------------------
# chain
# ------------------------------------------------------------------------------------------------

class Chain:
    """ckpt_chain_*: owns the opaque handle."""

    def __init__(self, chain):
        units = chain["units"]
        arr = (UnitDesc * len(units))()
        for i, u in enumerate(units):
            kind = UNIT_KINDS[u["kind"]]
            flags = (1 if u.get("relu") else 0) | (2 if u.get("project") else 0)
            arr[i] = UnitDesc(kind, u.get("cin", 0), u.get("cout", 0), u.get("k", 0), u.get("stride", 1),
                              u.get("pad", 0), u.get("mid", 0), flags)
        h, w, c = chain["input_hwc"]
        self.dtype = DTYPE_BF16 if chain["dtype"] == "bf16" else DTYPE_F32
        self.loss = LOSS_SOFTMAX_CE if chain["loss"] == "softmax_ce" else LOSS_SUM
        self.n = len(units)
        self.batch = chain["batch"]
        self.spec = chain
        self._h = C.c_void_p(0)
        _check(lib().ckpt_chain_create(arr, C.c_int64(self.n), C.c_int64(self.batch), C.c_int32(h), C.c_int32(w),
                                       C.c_int32(c), C.c_int(self.dtype), C.c_int(self.loss), C.byref(self._h)))

    def __del__(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().ckpt_chain_destroy(self._h)
            self._h = C.c_void_p(0)

    def sizes(self):
        d = np.zeros(self.n + 1, dtype=np.int64)
        _check(lib().ckpt_chain_sizes(self._h, _ptr(d, C.c_int64), None))
        return d

    def shapes(self):
        d = np.zeros(self.n + 1, dtype=np.int64)
        s = np.zeros((self.n + 1, 3), dtype=np.int32)
        _check(lib().ckpt_chain_sizes(self._h, _ptr(d, C.c_int64), _ptr(s, C.c_int32)))
        return s

    def num_params(self):
        c = C.c_int64(0)
        _check(lib().ckpt_chain_num_params(self._h, C.byref(c)))
        return c.value

    def param_info(self, p):
        unit, elems, dt = C.c_int64(0), C.c_int64(0), C.c_int32(0)
        _check(lib().ckpt_chain_param_info(self._h, C.c_int64(p), C.byref(unit), C.byref(elems), C.byref(dt)))
        return unit.value, elems.value, dt.value

    def workspace_bytes(self):
        b = C.c_int64(0)
        _check(lib().ckpt_chain_workspace_bytes(self._h, C.byref(b)))
        return b.value

    def workspace_bytes_for(self, policy):
        """ckpt_chain_workspace_bytes_for: the workspace one schedule needs (Algorithm 4's is shorter)."""
        b = C.c_int64(0)
        _check(lib().ckpt_chain_workspace_bytes_for(self._h, C.c_int(policy), C.byref(b)))
        return b.value

    def set_keep_interiors(self, enable):
        """ckpt_chain_set_keep_interiors: store-all steps keep every residual block's interior tensors."""
        _check(lib().ckpt_chain_set_keep_interiors(self._h, C.c_int(1 if enable else 0)))

    def set_impl(self, impl):
        _check(lib().ckpt_chain_set_impl(self._h, C.c_int(impl)))

    def set_gradient_tap(self, tap):
        """ckpt_chain_set_gradient_tap: a device uint8 tensor of at least d_1 + .. + d_n bytes, or None."""
        nbytes = 0 if tap is None else tap.numel() * tap.element_size()
        _check(lib().ckpt_chain_set_gradient_tap(self._h, _dev(tap), C.c_int64(nbytes)))

    def set_sgd(self, learning_rate):
        """ckpt_chain_set_sgd: steps also apply w <- w - learning_rate * g to every parameter (0 switches it off)."""
        _check(lib().ckpt_chain_set_sgd(self._h, C.c_double(learning_rate)))

    def set_selftest(self, wait_runs_out):
        _check(lib().ckpt_chain_set_selftest(self._h, C.c_int(1 if wait_runs_out else 0)))

    def set_graph(self, enable):
        """ckpt_chain_set_graph: record the launch sequence of a repeated step once and replay it."""
        _check(lib().ckpt_chain_set_graph(self._h, C.c_int(1 if enable else 0)))

    def unit_costs(self):
        """ckpt_chain_unit_costs: modelled forward time of every unit in nanoseconds (entry 0 is 0)."""
        out = np.zeros(self.n + 1, dtype=np.int64)
        _check(lib().ckpt_chain_unit_costs(self._h, _ptr(out, C.c_int64)))
        return out

    def staging_bytes(self):
        """ckpt_chain_staging_bytes: size of the two-slot staging buffer of ckpt_chain_stage_batch."""
        b = C.c_int64(0)
        _check(lib().ckpt_chain_staging_bytes(self._h, C.byref(b)))
        return b.value

    def stage_batch(self, slot, batch, labels, staging):
        """ckpt_chain_stage_batch: starts the copy of a host batch (torch tensor or numpy array in the chain's storage
        layout) and its labels into a slot of the device tensor ``staging``; returns the device addresses (ints; the
        second is None without labels) to hand to train_step as ``batch`` and ``labels``."""
        def addr(a):
            if a is None:
                return C.c_void_p(0)
            return C.c_void_p(a.ctypes.data if isinstance(a, np.ndarray) else a.data_ptr())
        b_dev, l_dev = C.c_void_p(0), C.c_void_p(0)
        _check(lib().ckpt_chain_stage_batch(self._h, C.c_int(slot), addr(batch), addr(labels), _dev(staging),
                                            C.c_int64(staging.numel() * staging.element_size()), C.byref(b_dev), C.byref(l_dev)))
        return b_dev.value, l_dev.value


def flatten_params(chain_spec, params):
    """List of (unit index, name, array) in the library's parameter order."""
    from .workloads import PARAM_NAMES
    out = []
    for ui, (unit, p) in enumerate(zip(chain_spec["units"], params)):
        for name in PARAM_NAMES[unit["kind"]]:
            if name in p:
                out.append((ui, name, p[name]))
    return out


def upload_params(chain, params, device="cuda"):
    """Host arrays -> device tensors in each parameter's storage dtype, plus zeroed f32 gradients."""
    import torch
    flat = flatten_params(chain.spec, params)
    assert len(flat) == chain.num_params()
    tensors, grads = [], []
    for p, (_, _, arr) in enumerate(flat):
        _, elems, dt = chain.param_info(p)
        assert elems == arr.size, (p, elems, arr.shape)
        t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(device)
        tensors.append(t.to(torch.bfloat16).contiguous() if dt == DTYPE_BF16 else t.contiguous())
        grads.append(torch.zeros(arr.shape, dtype=torch.float32, device=device))
    return tensors, grads, flat


def train_step(chain, is_ckpt, policy, batch, labels, params, grads, arena, workspace, stream=None):
    """ckpt_train_step.  ``batch``/``labels``: torch tensors (device, or pinned/pageable host), numpy arrays already
    in the chain's storage layout, or the device addresses Chain.stage_batch returned; everything else: device torch
    tensors."""
    n_p = chain.num_params()
    p_arr = (C.c_void_p * n_p)(*[t.data_ptr() for t in params])
    g_arr = (C.c_void_p * n_p)(*[t.data_ptr() for t in grads])
    mask_p = None
    if is_ckpt is not None:
        mask = np.ascontiguousarray(is_ckpt, dtype=np.uint8)
        mask_p = _ptr(mask, C.c_uint8)

    def addr(a):
        if a is None:
            return C.c_void_p(0)
        if isinstance(a, int):                  # a device address from Chain.stage_batch
            return C.c_void_p(a)
        if isinstance(a, np.ndarray):
            return C.c_void_p(a.ctypes.data)
        return C.c_void_p(a.data_ptr())

    rep = StepReport()
    rc = lib().ckpt_train_step(chain._h, mask_p, C.c_int(policy), addr(batch), addr(labels), p_arr, g_arr,
                               _dev(arena), C.c_int64(arena.numel() * arena.element_size()), _dev(workspace),
                               C.c_int64(workspace.numel() * workspace.element_size()), _stream(stream), C.byref(rep))
    _check(rc)
    return {name: getattr(rep, name) for name, _ in StepReport._fields_}


# ------------------------------------------------------------------------------------------------
# launch log, status of the single operations
# ------------------------------------------------------------------------------------------------

def launch_log(enable):
    _check(lib().ckpt_launch_log(C.c_int(1 if enable else 0)))


def launch_log_read():
    """ckpt_launch_log_read: {kernel name: launches}."""
    need = C.c_int64(0)
    _check(lib().ckpt_launch_log_read(None, C.c_int64(0), C.byref(need)))
    buf = C.create_string_buffer(need.value)
    _check(lib().ckpt_launch_log_read(buf, C.c_int64(need.value), C.byref(need)))
    out = {}
    for line in buf.value.decode().splitlines():
        count, name = line.split("\t", 1)
        out[name] = int(count)
    return out


def op_status():
    """ckpt_op_status: raises CkptError(E_DEVICE_TIMEOUT) when a bounded wait of a single operation gave up."""
    status = C.c_int32(0)
    rc = lib().ckpt_op_status(C.byref(status))
    if rc != 0:
        err = CkptError(rc, lib().ckpt_last_error().decode())
        err.status = status.value
        raise err
    return status.value


def selftest_bounded_wait(limit_cycles, stream=None):
    _check(lib().ckpt_selftest_bounded_wait(C.c_int64(limit_cycles), _stream(stream)))


# ------------------------------------------------------------------------------------------------
# single operations
# ------------------------------------------------------------------------------------------------

def conv2d_scratch_bytes(shape, dtype):
    b = C.c_int64(0)
    _check(lib().ckpt_conv2d_scratch_bytes(C.byref(shape), C.c_int(dtype), C.byref(b)))
    return b.value


def _scratch_args(scratch):
    if scratch is None:
        return C.c_void_p(0), C.c_int64(0)
    return _dev(scratch), C.c_int64(scratch.numel() * scratch.element_size())


def conv2d_forward(shape, dtype, impl, x, w, z, scratch=None, stream=None):
    sp, sb = _scratch_args(scratch)
    _check(lib().ckpt_conv2d_forward(C.byref(shape), C.c_int(dtype), C.c_int(impl), _dev(x), _dev(w), _dev(z), sp, sb, _stream(stream)))


def conv2d_bn_statistics(shape, dtype, x, w, z, gamma, beta, stats, scratch, stream=None):
    """ckpt_conv2d_bn_statistics; returns True when the sums were gathered in the convolution's epilogue."""
    sp, sb = _scratch_args(scratch)
    fused = C.c_int32(0)
    _check(lib().ckpt_conv2d_bn_statistics(C.byref(shape), C.c_int(dtype), _dev(x), _dev(w), _dev(z), _dev(gamma), _dev(beta),
                                           _dev(stats), sp, sb, C.byref(fused), _stream(stream)))
    return bool(fused.value)


def conv2d_dgrad(shape, dtype, impl, dz, w, dx, scratch=None, stream=None):
    sp, sb = _scratch_args(scratch)
    _check(lib().ckpt_conv2d_dgrad(C.byref(shape), C.c_int(dtype), C.c_int(impl), _dev(dz), _dev(w), _dev(dx), sp, sb, _stream(stream)))


def conv2d_wgrad(shape, dtype, impl, dz, x, dw, scratch=None, stream=None):
    sp, sb = _scratch_args(scratch)
    _check(lib().ckpt_conv2d_wgrad(C.byref(shape), C.c_int(dtype), C.c_int(impl), _dev(dz), _dev(x), _dev(dw), sp, sb, _stream(stream)))


def bn_scratch_bytes(rows, c):
    b = C.c_int64(0)
    _check(lib().ckpt_bn_scratch_bytes(C.c_int64(rows), C.c_int32(c), C.byref(b)))
    return b.value


def bn_relu_forward(dtype, rows, c, z, gamma, beta, relu, y, stats, scratch, stream=None):
    _check(lib().ckpt_bn_relu_forward(C.c_int(dtype), C.c_int64(rows), C.c_int32(c), _dev(z), _dev(gamma), _dev(beta),
                                      C.c_int(relu), _dev(y), _dev(stats), _dev(scratch), _stream(stream)))


def bn_relu_forward_noalloc(dtype, rows, c, z, gamma, beta, relu, y, stats, stream=None):
    """ckpt_bn_relu_forward_noalloc: same arguments as bn_relu_forward minus the scratch buffer."""
    _check(lib().ckpt_bn_relu_forward_noalloc(C.c_int(dtype), C.c_int64(rows), C.c_int32(c), _dev(z), _dev(gamma), _dev(beta),
                                              C.c_int(relu), _dev(y), _dev(stats), _stream(stream)))


def bn_relu_backward(dtype, rows, c, dy, z, gamma, stats, relu, dz, dgamma, dbeta, scratch, stream=None):
    _check(lib().ckpt_bn_relu_backward(C.c_int(dtype), C.c_int64(rows), C.c_int32(c), _dev(dy), _dev(z), _dev(gamma),
                                       _dev(stats), C.c_int(relu), _dev(dz), _dev(dgamma), _dev(dbeta), _dev(scratch),
                                       _stream(stream)))


def maxpool_forward(dtype, n, h, w, c, k, stride, pad, x, y, stream=None):
    _check(lib().ckpt_maxpool_forward(C.c_int(dtype), n, h, w, c, k, stride, pad, _dev(x), _dev(y), _stream(stream)))


def maxpool_backward_scratch_bytes(dtype, n, h, w, c, k, stride, pad):
    b = C.c_int64(0)
    _check(lib().ckpt_maxpool_backward_scratch_bytes(C.c_int(dtype), n, h, w, c, k, stride, pad, C.byref(b)))
    return b.value


def maxpool_backward(dtype, n, h, w, c, k, stride, pad, x, dy, dx, scratch=None, stream=None):
    sp, sb = _scratch_args(scratch)
    _check(lib().ckpt_maxpool_backward(C.c_int(dtype), n, h, w, c, k, stride, pad, _dev(x), _dev(dy), _dev(dx), sp, sb, _stream(stream)))


def softmax_ce(dtype, batch, classes, logits, labels, loss, dlogits, stream=None):
    _check(lib().ckpt_softmax_ce(C.c_int(dtype), batch, classes, _dev(logits), _dev(labels), _dev(loss), _dev(dlogits), _stream(stream)))
