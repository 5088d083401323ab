"""The failure path of the bounded device waits, driven to its limit without a fault: a wait whose producer never
arrives gives up after a short limit, the kernel records a status code and returns, the host call reports
CKPT_E_DEVICE_TIMEOUT, and the context stays usable."""
import numpy as np
import pytest

from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import StepRunner

pytestmark = pytest.mark.gpu


def test_single_operation_status_word():
    import torch
    assert ck.op_status() == 0
    ck.selftest_bounded_wait(200000)              # about 0.1 ms of spinning, then the wait gives up
    with pytest.raises(ck.CkptError) as e:
        ck.op_status()
    assert e.value.code == -10 and e.value.status == 9001
    assert ck.op_status() == 0                    # reading cleared the word
    # the context is intact: an ordinary tensor-core operation runs and leaves the word at 0
    shape = ck.ConvShape(2, 16, 16, 64, 128, 3, 1, 1)
    x = torch.randn(2, 16, 16, 64, device="cuda").bfloat16()
    w = torch.randn(128, 3, 3, 64, device="cuda").bfloat16()
    z = torch.empty(2, 16, 16, 128, device="cuda", dtype=torch.bfloat16)
    scratch = torch.empty(max(256, ck.conv2d_scratch_bytes(shape, ck.DTYPE_BF16)), dtype=torch.uint8, device="cuda")
    ck.conv2d_forward(shape, ck.DTYPE_BF16, 2, x, w, z, scratch)
    assert ck.op_status() == 0
    ref = torch.nn.functional.conv2d(x.float().permute(0, 3, 1, 2), w.float().permute(0, 3, 1, 2), padding=1).permute(0, 2, 3, 1)
    assert float((z.float() - ref).abs().max()) <= 6e-3 * float(ref.abs().max())


@pytest.mark.parametrize("graph", [False, True])
def test_train_step_reports_a_wait_that_ran_out(graph):
    spec = wl.plain_chain(3, 64, 64, (12, 12), 4, "bf16", "sum", name="status_chain")
    params = wl.make_params(spec, seed=0)
    x, _ = wl.make_batch(spec, seed=1)
    runner = StepRunner(spec, params)
    mask = ck.mask_from_set(runner.n, [0, 2, runner.n])
    rep0, g0 = runner.run(ck.POLICY_DYNAMIC, mask, x, None)
    assert rep0["device_status"] == 0
    if graph:
        runner.chain.set_graph(True)
    runner.chain.set_selftest(True)
    for _ in range(3 if graph else 1):            # plain step, recorded step, replayed step
        with pytest.raises(ck.CkptError) as e:
            runner.run(ck.POLICY_DYNAMIC, mask, x, None)
        assert e.value.code == -10
    runner.chain.set_selftest(False)
    for _ in range(3 if graph else 1):
        rep, g = runner.run(ck.POLICY_DYNAMIC, mask, x, None)
        assert rep["device_status"] == 0 and rep["loss"] == rep0["loss"]
        for a, b in zip(g, g0):
            assert np.array_equal(a, b)
