"""The allocation-free batch-norm entry point (collected last on purpose: a run that stops at the
first failure has then already gone through every other test).

ckpt_bn_relu_forward_noalloc serves callers that cannot give the library a scratch buffer because
they are not allowed to allocate device memory where they call it (code inside a framework that owns
all device memory, loops that cannot afford cudaMalloc's device-wide synchronisation).  Its partial
sums go into an array that is part of the library image, shared by all calls.  The test drives it
through the C ABI twice in a row on different inputs and compares each result with the ordinary
entry point, which gets its scratch from the caller; the second call would expose anything stale
left in the shared array by the first."""
import numpy as np
import pytest

from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import max_rel_err, to_dev, to_host

pytestmark = pytest.mark.gpu
TIGHT = {ck.DTYPE_F32: 2e-5, ck.DTYPE_BF16: 6e-3}       # same bounds as tests/test_gpu_ops.py


@pytest.mark.parametrize("dtype", [ck.DTYPE_F32, ck.DTYPE_BF16])
def test_noalloc_matches_ordinary_entry_point_twice(dtype):
    import torch
    rng = np.random.default_rng(99)
    # The first call on a device looks up the built-in array (and, with lazy module loading, makes
    # the driver load the module that contains it): do it before watching the free-memory counter.
    warm = torch.zeros(8, 8, device="cuda").to(torch.bfloat16 if dtype == ck.DTYPE_BF16 else torch.float32)
    ones = torch.ones(8, device="cuda")
    ck.bn_relu_forward_noalloc(dtype, 8, 8, warm, ones, ones, 0, torch.empty_like(warm), torch.empty(32, device="cuda"))
    torch.cuda.synchronize()
    # first a large, wide case that fills much of the shared array, then a small one
    for rows, c, relu in ((20000, 512, 1), (333, 24, 0)):
        z = (rng.standard_normal((rows, c)) * 1.5 + 0.3).astype(np.float32)
        if dtype == ck.DTYPE_BF16:
            z = wl.to_bf16_representable(z)
        gamma = rng.uniform(0.5, 1.5, c).astype(np.float32)
        beta = (rng.standard_normal(c) * 0.3).astype(np.float32)
        zd = to_dev(z, dtype)
        gd, bd = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
        y_ref, y_new = torch.empty_like(zd), torch.empty_like(zd)
        st_ref = torch.empty(4 * c, device="cuda", dtype=torch.float32)
        st_new = torch.full((4 * c,), float("nan"), device="cuda", dtype=torch.float32)
        scratch = torch.empty(ck.bn_scratch_bytes(rows, c), dtype=torch.uint8, device="cuda")
        ck.bn_relu_forward(dtype, rows, c, zd, gd, bd, relu, y_ref, st_ref, scratch)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # device-wide: sees any cudaMalloc, whoever makes it
        ck.bn_relu_forward_noalloc(dtype, rows, c, zd, gd, bd, relu, y_new, st_new)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free_before
        assert max_rel_err(to_host(st_new), to_host(st_ref)) <= 1e-6
        assert max_rel_err(to_host(y_new), to_host(y_ref)) <= TIGHT[dtype]


def test_noalloc_rejects_more_channels_than_the_built_in_array_holds():
    import torch
    c = 513
    z = torch.zeros(8, c, device="cuda")
    g = torch.ones(c, device="cuda")
    st = torch.empty(4 * c, device="cuda")
    with pytest.raises(ck.CkptError) as e:
        ck.bn_relu_forward_noalloc(ck.DTYPE_F32, 8, c, z, g, g, 0, z, st)
    assert e.value.code == -11 and "512" in str(e.value)
