"""Per-kernel GPU parity on identical inputs: every convolution mode and BN+ReLU forward/backward, in fp32 and in
bf16 storage, through the layer-level C entry points, against the oracle's layer routines.

fp32: 1e-4 max relative error (1 % floor).  bf16: 2e-2 normalised max-abs against the oracle with the same
storage rounding; the observed error is one bf16 ulp (4e-3) on the few elements where the fp32 sum lands on the
other side of a rounding boundary.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from parity import max_rel_err, norm_max_abs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def m():
    import paper_2107_00961_b200 as mod
    mod.lib()
    return mod


def rnd(seed, *shape, bf16=False):
    x = synth.standard_normal(seed, int(np.prod(shape))).astype(np.float32).reshape(shape)
    return synth.round_to_bf16(x) if bf16 else x


def dev(x, bf16):
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


# (N, H, W, C, K, ksz, stride): the shapes of the CIFAR ResNet-110 and of the bottleneck nets at small batch,
# strided and projection layers, 3-channel stems, and ragged extents that end inside a tile
SHAPES = [
    (4, 32, 32, 16, 16, 3, 1), (4, 16, 16, 32, 32, 3, 1), (6, 8, 8, 64, 64, 3, 1),
    (4, 32, 32, 16, 32, 3, 2), (4, 16, 16, 32, 64, 3, 2), (4, 32, 32, 16, 32, 1, 2),
    (2, 32, 32, 64, 256, 1, 1), (2, 32, 32, 256, 64, 1, 1), (2, 16, 16, 128, 128, 3, 2),
    (3, 8, 8, 256, 256, 3, 1), (4, 32, 32, 3, 16, 3, 1), (2, 36, 36, 3, 64, 7, 2),
    (3, 10, 6, 24, 40, 3, 1), (5, 7, 7, 72, 40, 3, 2), (2, 14, 14, 64, 64, 3, 1), (1, 28, 28, 128, 128, 3, 1),
    (3, 13, 9, 40, 24, 1, 1),
    # wide layers of the bottleneck nets: several 64-channel slabs, several column tiles, 4x4 maps, strided projections
    (2, 4, 4, 512, 512, 3, 1), (2, 16, 16, 256, 512, 1, 2), (2, 8, 8, 1024, 256, 1, 1), (2, 8, 8, 256, 1024, 1, 1),
    (2, 8, 8, 256, 256, 3, 2), (3, 6, 10, 136, 72, 3, 1), (2, 9, 7, 64, 128, 1, 2),
    # maps of 2x2 and 1x1 positions (the last stage of a deep net on a small input)
    (5, 2, 2, 128, 128, 3, 1), (5, 4, 4, 128, 256, 3, 2), (6, 1, 1, 128, 128, 3, 1), (5, 2, 2, 128, 256, 1, 2),
]


@pytest.mark.parametrize("shape", SHAPES)
# backend: 0 automatic choice, 1 CUDA cores only, 2 tcgen05 where the shape allows, 3 warp-level MMA where it allows
@pytest.mark.parametrize("dtype,backend", [("f32", 1), ("bf16", 1), ("bf16", 0), ("bf16", 2), ("bf16", 3)])
def test_conv_modes(m, shape, dtype, backend):
    N, H, W, C, K, k, s = shape
    bf = dtype == "bf16"
    q = 1 if bf else 0
    a, w = rnd(1, N, H, W, C, bf16=bf), rnd(2, K, k, k, C, bf16=bf) * np.float32(0.25)
    if bf:
        w = synth.round_to_bf16(w)
    y_ref = oracle.conv_fwd(a, w, s, quant=q)
    P, Q = y_ref.shape[1:3]
    add_y, dy, add_a = rnd(3, N, P, Q, K, bf16=bf), rnd(4, N, P, Q, K, bf16=bf), rnd(5, N, H, W, C, bf16=bf)
    geom = (N, H, W, C, K, k, s)
    err = (lambda x, r: norm_max_abs(x, r)) if bf else (lambda x, r: max_rel_err(x, r))
    tol = 2e-2 if bf else 1e-4
    # forward, plain and with the fused residual add and scale
    y, used = m.resist_conv2d(0, dev(a, bf), dev(w, bf), geom, backend=backend)
    assert err(y.float().cpu().numpy(), y_ref) < tol
    y2, _ = m.resist_conv2d(0, dev(a, bf), dev(w, bf), geom, add=dev(add_y, bf), scale=0.5, backend=backend)
    assert err(y2.float().cpu().numpy(), oracle.conv_fwd(a, w, s, add=add_y, quant=q, scale=0.5)) < tol
    # dgrad, plain and with the fused add
    da, _ = m.resist_conv2d(1, dev(dy, bf), dev(w, bf), geom, backend=backend)
    assert err(da.float().cpu().numpy(), oracle.conv_dgrad(dy, w, (H, W), s, quant=q)) < tol
    da2, _ = m.resist_conv2d(1, dev(dy, bf), dev(w, bf), geom, add=dev(add_a, bf), backend=backend)
    assert err(da2.float().cpu().numpy(), oracle.conv_dgrad(dy, w, (H, W), s, add=add_a, quant=q)) < tol
    # wgrad (fp32 output in both modes)
    dw, _ = m.resist_conv2d(2, dev(a, bf), dev(dy, bf), geom, backend=backend)
    assert max_rel_err(dw.cpu().numpy(), oracle.conv_wgrad(dy, a, k, s)) < (2e-3 if bf else 1e-4)
    if backend == 1:
        assert not used           # RESIST_CONV_CUDA_CORES really keeps the tensor cores out
    if backend == 2:
        assert used in (0, 1)
    if backend == 3:
        assert used in (0, 2)


@pytest.mark.parametrize("m_rows,C", [(4096, 16), (1000, 32), (517, 64), (300, 24), (64, 256), (50, 2048), (9000, 8)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bn_relu_forward_backward(m, m_rows, C, dtype):
    bf = dtype == "bf16"
    q = 1 if bf else 0
    x = rnd(11, m_rows, C, bf16=bf) * np.float32(1.7) + rnd(12, C)[None, :]          # per-channel offsets: mean != 0
    if bf:
        x = synth.round_to_bf16(x)
    g, b = (1 + 0.2 * rnd(13, C)).astype(np.float32), (0.3 * rnd(14, C)).astype(np.float32)
    rm, rv = rnd(15, C), (np.abs(rnd(16, C)) + 0.5).astype(np.float32)
    da, add = rnd(17, m_rows, C, bf16=bf), rnd(18, m_rows, C, bf16=bf)
    rm_ref, rv_ref = rm.copy(), rv.copy()
    a_ref, mean, invstd = oracle.bn_relu_fwd(x, g, b, rm_ref, rv_ref, quant=q)
    dx_ref, dg_ref, db_ref = oracle.bn_relu_bwd(da, x, g, b, mean, invstd, add=add, quant=q)
    dg_, db_, drm, drv = (torch.from_numpy(v).cuda() for v in (g, b, rm, rv))
    a, stat = m.resist_bn_relu_forward(dev(x, bf), dg_, db_, drm, drv)
    dx, dg, db = m.resist_bn_relu_backward(dev(x, bf), dev(da, bf), dg_, db_, stat, add=dev(add, bf))
    err = norm_max_abs if bf else max_rel_err
    tol = 2e-2 if bf else 1e-4
    assert err(a.float().cpu().numpy(), a_ref) < tol
    assert max_rel_err(stat[:C].cpu().numpy(), mean) < 5e-5 and max_rel_err(stat[C:2 * C].cpu().numpy(), invstd) < 5e-5
    assert max_rel_err(drm.cpu().numpy(), rm_ref) < 1e-5 and max_rel_err(drv.cpu().numpy(), rv_ref) < 1e-5
    assert err(dx.float().cpu().numpy(), dx_ref) < tol
    assert max_rel_err(dg.cpu().numpy(), dg_ref) < (1e-3 if bf else 1e-4)
    assert max_rel_err(db.cpu().numpy(), db_ref) < (1e-3 if bf else 1e-4)


def test_bn_statistics_survive_a_large_mean(m):
    # mean 1000, std 1: sums of x^2 would lose the variance entirely in fp32; the shifted sums do not
    x = (rnd(21, 2048, 16) + np.float32(1000.0)).astype(np.float32)
    g, b = np.ones(16, np.float32), np.zeros(16, np.float32)
    _, mean, invstd = oracle.bn_relu_fwd(x, g, b)
    a, stat = m.resist_bn_relu_forward(dev(x, False), torch.from_numpy(g).cuda(), torch.from_numpy(b).cuda())
    assert max_rel_err(stat[16:32].cpu().numpy(), invstd) < 1e-4
