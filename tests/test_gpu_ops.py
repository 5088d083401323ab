"""GPU parity of the single operations against the float64 oracle, through the C ABI.

Tolerances (max |err| / max |ref| per tensor): 1e-3 for float32 storage (plain FMA arithmetic, no
TF32), 3e-2 for bfloat16 storage with float32 accumulation.  Inputs handed to both sides are
already rounded to the storage type, so the only differences are accumulation order and the final
rounding of each output element."""
import numpy as np
import pytest

from oracle import numeric_oracle as no
from paper_2502_12499_b200 import binding as ck
from paper_2502_12499_b200 import workloads as wl
from tests.gpu_util import max_rel_err, to_dev, to_host

pytestmark = pytest.mark.gpu
TOL = {ck.DTYPE_F32: 1e-3, ck.DTYPE_BF16: 3e-2}


@pytest.fixture(autouse=True)
def no_device_timeout():
    """Every operation of a test must leave the library's device status word at zero: a bounded wait that gave up inside
    a kernel would otherwise look like a numeric error (or pass, on a tensor the test does not read)."""
    yield
    assert ck.op_status() == 0

# pure rounding of one bf16 output is 2^-9 relative; anything above a few of those is a bug
TIGHT = {ck.DTYPE_F32: 2e-5, ck.DTYPE_BF16: 6e-3}

CONV_CASES = [
    # n, h, w, cin, cout, k, stride, pad
    (2, 9, 7, 3, 5, 3, 1, 1),        # ragged everything, tiny channels
    (4, 32, 32, 3, 16, 3, 1, 1),     # first layer of the 8-unit chain
    (4, 32, 32, 16, 16, 3, 1, 1),
    (3, 17, 13, 24, 40, 3, 2, 1),    # stride 2
    (2, 14, 14, 64, 96, 1, 1, 0),    # 1x1
    (2, 15, 15, 32, 64, 1, 2, 0),    # 1x1 stride 2 (projection shortcut)
    (2, 23, 19, 3, 16, 7, 2, 3),     # stem-like
    (3, 28, 28, 64, 64, 3, 1, 1),    # several 64-wide tiles with a tail
    (5, 1, 1, 200, 70, 1, 1, 0),     # fully connected as a 1x1 convolution
    (3, 21, 18, 3, 64, 3, 1, 1),     # first-layer kernels (3 input channels, 64 outputs)
    (2, 40, 40, 3, 128, 3, 1, 1),
]


TC_CASES = [
    # n, h, w, cin, cout, k, pad: shapes served by the tensor-core kernels (stride 1, channels % 64 == 0)
    (2, 16, 16, 64, 64, 3, 1),       # one pixel tile per image pair
    (3, 13, 19, 64, 128, 3, 1),      # ragged in every spatial dimension and in the batch
    (4, 28, 28, 128, 256, 3, 1),     # two channel blocks, 256-wide output tile
    (2, 14, 14, 192, 64, 3, 1),      # three channel blocks
    (8, 7, 7, 64, 320, 1, 0),        # 1x1, output channels not a multiple of 128
    (5, 30, 30, 128, 64, 1, 0),
    (64, 1, 1, 512, 192, 1, 0),      # fully connected shape
    (48, 1, 1, 256, 1000, 1, 0),     # classifier: output channels not a multiple of 64
    (64, 1, 1, 2048, 320, 1, 0),     # wide fully connected layer: matrix on M, batch on N, split reduction
    (5, 1, 1, 1024, 1000, 1, 0),     # the same with a ragged batch and a ragged last tile of output features
    (200, 1, 1, 4096, 128, 1, 0),    # batch wider than one 128-column accumulator chunk
    (2, 56, 56, 64, 64, 3, 1),
    (2, 16, 16, 128, 128, 3, 1),     # halo-patch kernel, one tile per CTA
    (2, 28, 24, 128, 256, 3, 1),     # halo-patch kernel, 14-row tiles, 256-wide output tile
    (2, 32, 16, 192, 64, 3, 1),      # halo-patch kernel, three channel blocks, 64-wide output tile
    (2, 112, 112, 128, 128, 3, 1),   # halo-patch kernel, several tiles per persistent CTA
    # role-swapped kernel corner cases: a single partial pixel tile, three output-channel tiles, 64 outputs without pairs
    (1, 5, 7, 128, 128, 3, 1),
    (2, 9, 11, 192, 384, 1, 0),
    (3, 10, 6, 256, 64, 3, 1),
    (1, 515, 510, 64, 64, 3, 1),     # pixel pairs, one image, odd height
    (4, 48, 104, 128, 256, 3, 1),    # halo-patch strips 24 rows high, two output-channel tiles
    # pixel-pair form of 64-channel outputs (large tensors only): forward 64 -> 64 and 128 -> 64, dgrad into 64 channels
    (5, 232, 228, 64, 64, 3, 1),     # ragged tiles in every dimension, pairs across tile borders
    (3, 300, 296, 128, 64, 3, 1),    # two reduction blocks per term
    (3, 300, 296, 64, 128, 3, 1),    # its dgrad: 128 reduction channels, filter widened from the forward filter
    # stride 2 (8th field): strided operand boxes forward and in wgrad, one stride-1 sum per parity class in dgrad
    (2, 28, 28, 128, 128, 3, 1, 2),  # first 3x3 of a residual stage
    (3, 15, 13, 64, 192, 3, 1, 2),   # odd sizes: ragged parity classes
    (2, 56, 56, 256, 128, 1, 0, 2),  # projection shortcut: three of four input classes get a zero gradient
    (3, 9, 11, 64, 64, 1, 0, 2),
]


def rounded(a, dtype):
    a = a.astype(np.float32)
    return wl.to_bf16_representable(a) if dtype == ck.DTYPE_BF16 else a


@pytest.mark.parametrize("dtype", [ck.DTYPE_F32, ck.DTYPE_BF16])
@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_cuda_core_kernels(case, dtype):
    import torch
    n, h, w, cin, cout, k, stride, pad = case
    rng = np.random.default_rng(hash(case) % 2 ** 31)
    x = rounded(rng.standard_normal((n, h, w, cin)), dtype)
    wt = rounded(rng.standard_normal((cout, k, k, cin)) / np.sqrt(k * k * cin), dtype)
    z_ref = no.conv2d_fwd(x.astype(np.float64), wt.astype(np.float64), stride, pad)
    dz = rounded(rng.standard_normal(z_ref.shape), dtype)
    dx_ref, dw_ref = no.conv2d_bwd(x.astype(np.float64), wt.astype(np.float64), dz.astype(np.float64), stride, pad)

    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    xd, wd, dzd = to_dev(x, dtype), to_dev(wt, dtype), to_dev(dz, dtype)
    z = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
    dx = torch.full(x.shape, float("nan"), device="cuda").to(xd.dtype)
    dw = torch.full(wt.shape, float("nan"), device="cuda", dtype=torch.float32)
    sb = ck.conv2d_scratch_bytes(shape, dtype)
    scratch = torch.empty(max(sb, 256), dtype=torch.uint8, device="cuda")
    ck.conv2d_forward(shape, dtype, 1, xd, wd, z, scratch)
    ck.conv2d_dgrad(shape, dtype, 1, dzd, wd, dx, scratch)
    ck.conv2d_wgrad(shape, dtype, 1, dzd, xd, dw, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(z), z_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dx), dx_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dw), dw_ref) <= 2e-5        # gradients are float32 in both modes
    assert TIGHT[dtype] <= TOL[dtype]


@pytest.mark.parametrize("case", TC_CASES)
def test_conv_tensor_core_kernels(case):
    """tcgen05 forward / dgrad / wgrad against the float64 oracle, and bit-reproducible."""
    import torch
    dtype = ck.DTYPE_BF16
    n, h, w, cin, cout, k, pad = case[:7]
    stride = case[7] if len(case) > 7 else 1
    rng = np.random.default_rng(hash(case) % 2 ** 31)
    x = rounded(rng.standard_normal((n, h, w, cin)), dtype)
    wt = rounded(rng.standard_normal((cout, k, k, cin)) / np.sqrt(k * k * cin), dtype)
    z_ref = no.conv2d_fwd(x.astype(np.float64), wt.astype(np.float64), stride, pad)
    dz = rounded(rng.standard_normal(z_ref.shape), dtype)
    dx_ref, dw_ref = no.conv2d_bwd(x.astype(np.float64), wt.astype(np.float64), dz.astype(np.float64), stride, pad)
    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    xd, wd, dzd = to_dev(x, dtype), to_dev(wt, dtype), to_dev(dz, dtype)
    scratch = torch.empty(max(ck.conv2d_scratch_bytes(shape, dtype), 256), dtype=torch.uint8, device="cuda")
    results = []
    for rep in range(2):
        z = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
        dx = torch.full(x.shape, float("nan"), device="cuda").to(xd.dtype)
        dw = torch.full(wt.shape, float("nan"), device="cuda", dtype=torch.float32)
        ck.conv2d_forward(shape, dtype, 2, xd, wd, z, scratch)
        ck.conv2d_dgrad(shape, dtype, 2, dzd, wd, dx, scratch)
        ck.conv2d_wgrad(shape, dtype, 2, dzd, xd, dw, scratch)
        torch.cuda.synchronize()
        results.append((z, dx, dw))
    z, dx, dw = results[0]
    assert max_rel_err(to_host(z), z_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dx), dx_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dw), dw_ref) <= 2e-5
    for a, b in zip(results[0], results[1]):
        assert torch.equal(a, b)
    # and the CUDA-core kernels agree with them to rounding
    z2 = torch.empty_like(z)
    ck.conv2d_forward(shape, dtype, 1, xd, wd, z2, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(z2), to_host(z)) <= TIGHT[dtype]


@pytest.mark.parametrize("n,h,w,cout", [(3, 21, 18, 64), (2, 40, 40, 128), (5, 32, 32, 64), (1, 5, 3, 64), (7, 96, 80, 64)])
def test_first_layer_kernels(n, h, w, cout):
    """3 input channels, bf16, automatic kernel choice: tensor-core forward on thread-gathered operand tiles
    (checked against the CUDA-core kernel too), unfolded tensor-core wgrad."""
    import torch
    dtype = ck.DTYPE_BF16
    rng = np.random.default_rng(n * h + cout)
    x = rounded(rng.standard_normal((n, h, w, 3)), dtype)
    wt = rounded(rng.standard_normal((cout, 3, 3, 3)) / np.sqrt(27), dtype)
    z_ref = no.conv2d_fwd(x.astype(np.float64), wt.astype(np.float64), 1, 1)
    dz = rounded(rng.standard_normal(z_ref.shape), dtype)
    _, dw_ref = no.conv2d_bwd(x.astype(np.float64), wt.astype(np.float64), dz.astype(np.float64), 1, 1)
    shape = ck.ConvShape(n, h, w, 3, cout, 3, 1, 1)
    xd, wd, dzd = to_dev(x, dtype), to_dev(wt, dtype), to_dev(dz, dtype)
    scratch = torch.empty(max(ck.conv2d_scratch_bytes(shape, dtype), 256), dtype=torch.uint8, device="cuda")
    z = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
    dw = torch.full(wt.shape, float("nan"), device="cuda", dtype=torch.float32)
    dw2 = torch.empty_like(dw)
    ck.conv2d_forward(shape, dtype, 0, xd, wd, z, scratch)
    ck.conv2d_wgrad(shape, dtype, 0, dzd, xd, dw, scratch)
    ck.conv2d_wgrad(shape, dtype, 0, dzd, xd, dw2, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(z), z_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dw), dw_ref) <= 2e-5
    assert torch.equal(dw, dw2)
    z1 = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
    ck.conv2d_forward(shape, dtype, 1, xd, wd, z1, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(z1), z_ref) <= TIGHT[dtype]
    assert not torch.isnan(z.float()).any()


@pytest.mark.parametrize("n,h,w,cout", [(2, 23, 19, 64), (3, 64, 64, 64), (1, 224, 224, 64), (2, 30, 37, 128), (1, 7, 520, 64),
                                        (40, 32, 32, 64)])
def test_stem_kernels(n, h, w, cout):
    """7x7 stride-2 padding-3 convolution on 3 input channels, bf16, automatic kernel choice: the stem kernels that
    gather their operand tiles from staged input rows (forward and wgrad), against the oracle and the CUDA-core
    kernels.  Odd widths (rows that start on an odd element), rows of several 128-pixel pieces, more tiles than CTAs."""
    import torch
    dtype = ck.DTYPE_BF16
    rng = np.random.default_rng(n * h + w + cout)
    x = rounded(rng.standard_normal((n, h, w, 3)), dtype)
    wt = rounded(rng.standard_normal((cout, 7, 7, 3)) / np.sqrt(147), dtype)
    z_ref = no.conv2d_fwd(x.astype(np.float64), wt.astype(np.float64), 2, 3)
    dz = rounded(rng.standard_normal(z_ref.shape), dtype)
    _, dw_ref = no.conv2d_bwd(x.astype(np.float64), wt.astype(np.float64), dz.astype(np.float64), 2, 3)
    shape = ck.ConvShape(n, h, w, 3, cout, 7, 2, 3)
    xd, wd, dzd = to_dev(x, dtype), to_dev(wt, dtype), to_dev(dz, dtype)
    scratch = torch.empty(max(ck.conv2d_scratch_bytes(shape, dtype), 256), dtype=torch.uint8, device="cuda")
    outs = []
    ck.launch_log(True)
    try:
        for rep in range(2):
            z = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
            dw = torch.full(wt.shape, float("nan"), device="cuda", dtype=torch.float32)
            scratch.fill_(0xFF)
            ck.conv2d_forward(shape, dtype, 0, xd, wd, z, scratch)
            scratch.fill_(0xFF)
            ck.conv2d_wgrad(shape, dtype, 0, dzd, xd, dw, scratch)
            torch.cuda.synchronize()
            outs.append((z, dw))
    finally:
        kernels = ck.launch_log_read()
        ck.launch_log(False)
    assert kernels.get("tc_conv_stem_kernel") == 2 and kernels.get("tc_wgrad_stem_kernel") == 2, kernels
    assert ck.op_status() == 0
    z, dw = outs[0]
    assert max_rel_err(to_host(z), z_ref) <= TIGHT[dtype]
    assert max_rel_err(to_host(dw), dw_ref) <= 2e-5
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    z1 = torch.empty_like(z)
    ck.conv2d_forward(shape, dtype, 1, xd, wd, z1, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(z1), z_ref) <= TIGHT[dtype]


@pytest.mark.parametrize("case,expect_fused", [
    ((8, 56, 56, 64, 64, 3, 1), True),        # 64-channel persistent kernel, two tiles for some CTAs
    ((5, 232, 228, 64, 64, 3, 1), True),      # pixel-pair form: sums of the two pixels of a pair in separate partial rows
    ((3, 13, 19, 64, 128, 3, 1), True),       # ragged tiles: rows outside the image must not count
    ((2, 112, 112, 128, 128, 3, 1), True),    # halo-patch kernel, 128-wide output tile
    ((4, 56, 56, 128, 256, 3, 1), True),      # halo-patch kernel, 256-wide output tile
    ((2, 14, 14, 192, 64, 3, 1), True),       # generic tensor-core kernel: one partial row pair per pixel tile
    ((5, 30, 30, 128, 320, 1, 0), False),     # 1x1 with a short reduction: separate statistics kernel
    ((5, 30, 30, 1024, 320, 1, 0), True),     # 1x1, long reduction, several pixel tiles, 64-wide output tiles
    ((3, 21, 18, 3, 64, 3, 1), True),         # first-layer kernel, ragged last tile
    ((9, 96, 80, 3, 128, 3, 1), True),        # first-layer kernel, several tiles per CTA, two channel blocks
    ((2, 9, 9, 16, 24, 3, 1), False),         # CUDA-core kernel + separate statistics kernel
    ((3, 50, 46, 3, 64, 7, 3, 2), True),      # stem kernel: several tiles per CTA, short output rows
    ((2, 300, 290, 3, 128, 7, 3, 2), True),   # stem kernel: output rows of two 128-pixel pieces, two channel blocks
])
def test_conv_bn_statistics(case, expect_fused):
    """Convolution + batch statistics of its stored output (gathered in the epilogue of the persistent
    tensor-core kernels) against the oracle's convolution, bf16 rounding and batch norm."""
    import torch
    dtype = ck.DTYPE_BF16
    n, h, w, cin, cout, k, pad = case[:7]
    stride = case[7] if len(case) > 7 else 1
    rng = np.random.default_rng(sum(case))
    x = rounded(rng.standard_normal((n, h, w, cin)) + 0.3, dtype)
    wt = rounded(rng.standard_normal((cout, k, k, cin)) / np.sqrt(k * k * cin), dtype)
    gamma = rng.uniform(0.5, 1.5, cout).astype(np.float32)
    beta = (rng.standard_normal(cout) * 0.3).astype(np.float32)
    z_ref = no.round_bf16(no.conv2d_fwd(x.astype(np.float64), wt.astype(np.float64), stride, pad))
    y_ref, (xhat, inv_std) = no.bn_fwd(z_ref, gamma.astype(np.float64), beta.astype(np.float64))
    mean_ref = z_ref.mean(axis=(0, 1, 2))
    shape = ck.ConvShape(n, h, w, cin, cout, k, stride, pad)
    rows = int(np.prod(z_ref.shape[:3]))
    xd, wd = to_dev(x, dtype), to_dev(wt, dtype)
    gd, bd = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    scratch = torch.empty(max(ck.conv2d_scratch_bytes(shape, dtype), ck.bn_scratch_bytes(rows, cout)), dtype=torch.uint8, device="cuda")
    outs = []
    for rep in range(2):
        z = torch.full(z_ref.shape, float("nan"), device="cuda").to(xd.dtype)
        stats = torch.full((4 * cout,), float("nan"), device="cuda")
        scratch.fill_(0xFF)
        fused = ck.conv2d_bn_statistics(shape, dtype, xd, wd, z, gd, bd, stats, scratch)
        torch.cuda.synchronize()
        assert fused == expect_fused
        outs.append((z, stats))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    z, stats = outs[0]
    st = to_host(stats).astype(np.float64)
    mean, inv, scale, shift = st[:cout], st[cout:2 * cout], st[2 * cout:3 * cout], st[3 * cout:]
    assert max_rel_err(to_host(z), z_ref) <= TIGHT[dtype]
    std_ref = 1.0 / inv_std
    assert np.abs(mean - mean_ref).max() <= 2e-3 * std_ref.max()
    assert max_rel_err(inv, inv_std) <= 5e-4
    assert max_rel_err(scale, gamma * inv_std) <= 5e-4
    assert np.abs(shift - (beta - mean_ref * gamma * inv_std)).max() <= 3e-3
    # the normalised tensor that a consumer of (z, stats) would see
    y = to_host(z).astype(np.float64) * scale + shift
    assert max_rel_err(y, y_ref) <= 1e-2
    # the stand-alone statistics kernel on the same stored tensor agrees to accumulation order
    stats2 = torch.empty_like(stats)
    y2 = torch.empty_like(z)
    ck.bn_relu_forward(dtype, rows, cout, z, gd, bd, 0, y2, stats2, scratch)
    torch.cuda.synchronize()
    assert max_rel_err(to_host(stats2[cout:2 * cout]), inv) <= 1e-5
    assert np.abs(to_host(stats2[:cout]) - mean).max() <= 1e-5 * max(1.0, np.abs(mean).max())


@pytest.mark.parametrize("dtype", [ck.DTYPE_F32, ck.DTYPE_BF16])
@pytest.mark.parametrize("rows,c,relu", [(37, 3, 1), (4096, 16, 1), (5000, 64, 1), (777, 40, 0), (64, 1000, 0), (3001, 24, 1)])
def test_batchnorm_relu(rows, c, relu, dtype):
    import torch
    rng = np.random.default_rng(rows * 7 + c)
    z = rounded(rng.standard_normal((1, 1, rows, c)) * 2 + 0.5, dtype)
    gamma = rng.uniform(0.5, 1.5, c).astype(np.float32)
    beta = (rng.standard_normal(c) * 0.3).astype(np.float32)
    dy = rounded(rng.standard_normal(z.shape), dtype)
    y_ref, cache = no.bn_fwd(z.astype(np.float64), gamma.astype(np.float64), beta.astype(np.float64))
    if relu:
        y_ref = np.maximum(y_ref, 0)
    g_ref = dy.astype(np.float64) * ((y_ref > 0) if relu else 1.0)
    dz_ref, dgamma_ref, dbeta_ref = no.bn_bwd(g_ref, cache, gamma.astype(np.float64))

    zd, dyd = to_dev(z, dtype), to_dev(dy, dtype)
    gd, bd = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    y = torch.empty_like(zd)
    stats = torch.empty(4 * c, device="cuda", dtype=torch.float32)
    scratch = torch.empty(ck.bn_scratch_bytes(rows, c), dtype=torch.uint8, device="cuda")
    ck.bn_relu_forward(dtype, rows, c, zd, gd, bd, relu, y, stats, scratch)
    dz = torch.empty_like(zd)
    dgamma = torch.empty(c, device="cuda"); dbeta = torch.empty(c, device="cuda")
    ck.bn_relu_backward(dtype, rows, c, dyd, zd, gd, stats, relu, dz, dgamma, dbeta, scratch)
    torch.cuda.synchronize()
    xhat, inv_std = cache
    assert max_rel_err(to_host(stats[c:2 * c]), inv_std) <= 1e-5
    assert max_rel_err(to_host(y), y_ref) <= TIGHT[dtype]
    # elements whose forward output rounds to exactly zero in bf16 may flip the mask; none here
    assert max_rel_err(to_host(dbeta), dbeta_ref) <= 1e-4
    assert max_rel_err(to_host(dgamma), dgamma_ref) <= 1e-4
    assert max_rel_err(to_host(dz), dz_ref) <= TIGHT[dtype]
    # in-place variant (dz aliases dy) gives the same bits
    ck.bn_relu_backward(dtype, rows, c, dyd, zd, gd, stats, relu, dyd, dgamma, dbeta, scratch)
    torch.cuda.synchronize()
    assert torch.equal(dyd, dz)


@pytest.mark.parametrize("dtype", [ck.DTYPE_F32, ck.DTYPE_BF16])
@pytest.mark.parametrize("n,h,w,c,k,stride,pad", [(2, 8, 6, 5, 2, 2, 0), (3, 13, 11, 8, 3, 2, 1), (2, 32, 32, 16, 2, 2, 0),
                                                 (2, 20, 18, 64, 3, 2, 1), (2, 9, 9, 6, 3, 2, 1), (2, 11, 14, 16, 3, 1, 1)])
def test_maxpool(n, h, w, c, k, stride, pad, dtype):
    import torch
    rng = np.random.default_rng(h * w)
    x = rng.integers(-3, 4, size=(n, h, w, c)).astype(np.float32)          # many exact ties
    y_ref, arg = no.maxpool_fwd(x.astype(np.float64), k, stride, pad)
    dy = rounded(rng.standard_normal(y_ref.shape), dtype)
    dx_ref = no.maxpool_bwd(dy.astype(np.float64), arg, x.shape, k, stride, pad)
    xd, dyd = to_dev(x, dtype), to_dev(dy, dtype)
    y = torch.empty(y_ref.shape, device="cuda").to(xd.dtype)
    dx = torch.empty_like(xd)
    ck.maxpool_forward(dtype, n, h, w, c, k, stride, pad, xd, y)
    ck.maxpool_backward(dtype, n, h, w, c, k, stride, pad, xd, dyd, dx)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(y), y_ref)
    assert max_rel_err(to_host(dx), dx_ref) <= TIGHT[dtype]
    # with scratch the general backward records the arg-max positions first and gathers from them: same result
    sb = ck.maxpool_backward_scratch_bytes(dtype, n, h, w, c, k, stride, pad)
    if sb > 0:
        scratch = torch.full((sb,), 0xEE, dtype=torch.uint8, device="cuda")
        dx2 = torch.full_like(xd, float("nan"))
        ck.maxpool_backward(dtype, n, h, w, c, k, stride, pad, xd, dyd, dx2, scratch)
        torch.cuda.synchronize()
        assert torch.equal(dx2, dx)


@pytest.mark.parametrize("dtype", [ck.DTYPE_F32, ck.DTYPE_BF16])
def test_softmax_cross_entropy(dtype):
    import torch
    rng = np.random.default_rng(5)
    logits = rounded(rng.standard_normal((64, 1, 1, 1000)) * 3, dtype)
    labels = rng.integers(0, 1000, 64).astype(np.int32)
    loss_ref, g_ref = no.softmax_ce(logits.astype(np.float64), labels)
    ld = to_dev(logits, dtype)
    lab = torch.from_numpy(labels).cuda()
    loss = torch.zeros(1, device="cuda")
    g = torch.empty_like(ld)
    ck.softmax_ce(dtype, 64, 1000, ld, lab, loss, g)
    torch.cuda.synchronize()
    assert abs(loss.item() - loss_ref) <= 1e-5 * abs(loss_ref)
    assert max_rel_err(to_host(g), g_ref) <= TIGHT[dtype]
