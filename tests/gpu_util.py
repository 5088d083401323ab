"""Helpers shared by the GPU parity tests (marshalling only)."""
import numpy as np

from paper_2502_12499_b200 import binding as ck


def torch_dtype(dtype):
    import torch
    return torch.bfloat16 if dtype == ck.DTYPE_BF16 else torch.float32


def to_dev(a, dtype):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch_dtype(dtype)).contiguous()


def to_host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def max_rel_err(got, want):
    """max |got - want| / max |want| over one tensor (the tolerance metric of the parity tests)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    if scale == 0:
        return float(np.abs(got).max())
    return float(np.abs(got - want).max() / scale)


class StepRunner:
    """Owns the device buffers of one chain and runs ckpt_train_step on them."""

    def __init__(self, spec, params, impl=0):
        import torch
        self.spec = spec
        self.chain = ck.Chain(spec)
        if impl:
            self.chain.set_impl(impl)
        self.d = self.chain.sizes()
        self.n = self.chain.n
        self.params, self.grads, self.flat = ck.upload_params(self.chain, params)
        self.workspace = torch.empty(self.chain.workspace_bytes(), dtype=torch.uint8, device="cuda")
        self.arena = None

    def run(self, policy, mask, x, labels, arena_bytes=None):
        import torch
        model = {ck.POLICY_STORE_ALL: ck.MODEL_STORE_ALL, ck.POLICY_STATIC: ck.MODEL_STATIC,
                 ck.POLICY_DYNAMIC: ck.MODEL_DYNAMIC}[policy]
        need = ck.eval(model, self.d, mask)
        if arena_bytes is None:
            arena_bytes = need                      # exactly the predicted peak: one byte less fails
        if self.arena is None or self.arena.numel() != arena_bytes:
            self.arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
        self.arena.fill_(0xFF)                      # NaN pattern: stale data must never be read
        for g in self.grads:
            g.fill_(float("nan"))
        xb = to_dev(x, self.chain.dtype)
        lab = None if labels is None else torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).cuda()
        rep = ck.train_step(self.chain, mask, policy, xb, lab, self.params, self.grads, self.arena, self.workspace)
        torch.cuda.synchronize()
        rep["need"] = need
        return rep, [g.detach().cpu().numpy().copy() for g in self.grads]
