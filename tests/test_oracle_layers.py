"""Pins for the oracle's layer routines (CPU only).

Each routine is checked against something other than itself: a library routine (numpy matmul,
scipy correlate, torch.nn.functional in fp64 with autograd), an adjoint identity, a closed form,
or central finite differences.  A dropped term, a wrong sign, a transposed operand or an
off-by-one in the padding fails at least one of them.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F
from scipy.signal import correlate2d

import oracle

RNG = np.random.default_rng(20210700961)


def rnd(*shape):
    return RNG.standard_normal(shape)


def t_conv(a, w, stride):
    """torch's conv2d on NHWC / KRSC arrays (library routine)."""
    k = w.shape[1]
    y = F.conv2d(torch.from_numpy(a).permute(0, 3, 1, 2), torch.from_numpy(w).permute(0, 3, 1, 2),
                 stride=stride, padding=(k - 1) // 2)
    return y.permute(0, 2, 3, 1).contiguous().numpy()


@pytest.mark.parametrize("k,stride,H,W", [(3, 1, 6, 5), (3, 2, 8, 8), (3, 2, 7, 9), (1, 1, 4, 4), (1, 2, 8, 6),
                                          (1, 2, 7, 7), (7, 2, 16, 16), (7, 2, 15, 13)])
def test_conv_fwd_matches_library(k, stride, H, W):
    a, w = rnd(2, H, W, 3), rnd(4, k, k, 3)
    np.testing.assert_allclose(oracle.conv_fwd(a, w, stride), t_conv(a, w, stride), rtol=1e-12, atol=1e-12)


def test_conv_1x1_is_matmul():
    a, w = rnd(3, 5, 4, 6), rnd(7, 1, 1, 6)
    y = oracle.conv_fwd(a, w, 1)
    np.testing.assert_allclose(y.reshape(-1, 7), a.reshape(-1, 6) @ w.reshape(7, 6).T, rtol=1e-12, atol=1e-12)


def test_conv_single_channel_is_scipy_correlate():
    a, w = rnd(1, 9, 7, 1), rnd(1, 3, 3, 1)
    ref = correlate2d(a[0, :, :, 0], w[0, :, :, 0], mode="same", boundary="fill", fillvalue=0.0)
    np.testing.assert_allclose(oracle.conv_fwd(a, w, 1)[0, :, :, 0], ref, rtol=1e-12, atol=1e-12)


def test_conv_add_and_scale():
    a, w, add = rnd(2, 4, 4, 3), rnd(5, 3, 3, 3), rnd(2, 4, 4, 5)
    y = oracle.conv_fwd(a, w, 1, add=add, scale=0.25)
    np.testing.assert_allclose(y, 0.25 * t_conv(a, w, 1) + add, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("k,stride,H,W", [(3, 1, 6, 5), (3, 2, 8, 8), (3, 2, 7, 9), (1, 2, 8, 6), (1, 2, 7, 7),
                                          (1, 1, 3, 3), (7, 2, 12, 12)])
def test_dgrad_wgrad_match_autograd(k, stride, H, W):
    a = torch.from_numpy(rnd(2, H, W, 3)).requires_grad_()
    w = torch.from_numpy(rnd(4, k, k, 3)).requires_grad_()
    y = F.conv2d(a.permute(0, 3, 1, 2), w.permute(0, 3, 1, 2), stride=stride, padding=(k - 1) // 2).permute(0, 2, 3, 1)
    dy = rnd(*y.shape)
    y.backward(torch.from_numpy(dy))
    da = oracle.conv_dgrad(dy, w.detach().numpy(), (H, W), stride)
    dw = oracle.conv_wgrad(dy, a.detach().numpy(), k, stride)
    np.testing.assert_allclose(da, a.grad.numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dw, w.grad.numpy(), rtol=1e-11, atol=1e-11)


def test_conv_adjoint_identities():
    # <conv(a; w), dy> = <a, dgrad(dy; w)> = <w, wgrad(dy, a)>
    a, w = rnd(2, 7, 6, 3), rnd(5, 3, 3, 3)
    y = oracle.conv_fwd(a, w, 2)
    dy = rnd(*y.shape)
    lhs = np.sum(y * dy)
    assert abs(lhs - np.sum(a * oracle.conv_dgrad(dy, w, (7, 6), 2))) < 1e-10 * abs(lhs) + 1e-10
    assert abs(lhs - np.sum(w * oracle.conv_wgrad(dy, a, 3, 2))) < 1e-10 * abs(lhs) + 1e-10


def test_dgrad_add_term():
    a, w = rnd(1, 4, 4, 2), rnd(3, 3, 3, 2)
    dy, add = rnd(1, 4, 4, 3), rnd(1, 4, 4, 2)
    np.testing.assert_allclose(oracle.conv_dgrad(dy, w, (4, 4), 1, add=add),
                               oracle.conv_dgrad(dy, w, (4, 4), 1) + add, rtol=1e-13, atol=1e-13)


def test_bn_relu_fwd_matches_library_and_running_stats():
    x, g, b = rnd(4, 3, 5, 6), rnd(6), rnd(6)
    rm, rv = rnd(6), np.abs(rnd(6)) + 0.5
    trm, trv = torch.from_numpy(rm.copy()), torch.from_numpy(rv.copy())
    ref = F.relu(F.batch_norm(torch.from_numpy(x).permute(0, 3, 1, 2), trm, trv, torch.from_numpy(g),
                              torch.from_numpy(b), training=True, momentum=0.1, eps=1e-5)).permute(0, 2, 3, 1)
    a, mean, invstd = oracle.bn_relu_fwd(x, g, b, rm, rv)
    np.testing.assert_allclose(a, ref.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(rm, trm.numpy(), rtol=1e-12)       # running mean: 0.9*old + 0.1*batch mean
    np.testing.assert_allclose(rv, trv.numpy(), rtol=1e-12)       # running var uses the unbiased estimate
    np.testing.assert_allclose(mean, x.reshape(-1, 6).mean(0), rtol=1e-12)
    np.testing.assert_allclose(invstd, 1 / np.sqrt(x.reshape(-1, 6).var(0) + 1e-5), rtol=1e-12)


def test_bn_of_constant_map_is_relu_beta_with_zero_input_gradient():
    x = np.full((2, 3, 3, 4), 1.7)
    g, b = rnd(4), np.array([0.3, -0.2, 1.0, 0.0])
    a, mean, invstd = oracle.bn_relu_fwd(x, g, b)
    np.testing.assert_allclose(a, np.broadcast_to(np.maximum(b, 0), x.shape), atol=1e-12)
    dx, dg, db = oracle.bn_relu_bwd(rnd(2, 3, 3, 4), x, g, b, mean, invstd)
    # gradient w.r.t. a constant input vanishes up to the eps-regularised scale: sum over the batch is 0
    np.testing.assert_allclose(dx.reshape(-1, 4).sum(0), 0, atol=1e-9)


def test_bn_relu_bwd_matches_autograd():
    x = torch.from_numpy(rnd(3, 4, 2, 5)).requires_grad_()
    g = torch.from_numpy(rnd(5)).requires_grad_()
    b = torch.from_numpy(rnd(5)).requires_grad_()
    y = F.relu(F.batch_norm(x.permute(0, 3, 1, 2), None, None, g, b, training=True, eps=1e-5)).permute(0, 2, 3, 1)
    da, add = rnd(*y.shape), rnd(*y.shape)
    y.backward(torch.from_numpy(da))
    _, mean, invstd = oracle.bn_relu_fwd(x.detach().numpy(), g.detach().numpy(), b.detach().numpy())
    dx, dg, db = oracle.bn_relu_bwd(da, x.detach().numpy(), g.detach().numpy(), b.detach().numpy(), mean, invstd, add=add)
    np.testing.assert_allclose(dx - add, x.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dg, g.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(db, b.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_maxpool_matches_library_and_routes_to_first_maximum():
    x = rnd(2, 7, 8, 3)
    y, arg = oracle.maxpool_fwd(x)
    ref = F.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(y, ref)
    # ties: an all-zero map (common after ReLU).  Brute force: the first in-bounds window cell, row-major.
    z = np.zeros((1, 4, 4, 1))
    _, arg = oracle.maxpool_fwd(z)
    expect = np.array([[0, 1], [4, 5]])     # windows start at (-1,-1): first valid cell is (max(0,2p-1), max(0,2q-1))
    np.testing.assert_array_equal(arg[0, :, :, 0], expect)
    dx = oracle.maxpool_bwd(np.ones((1, 2, 2, 1)), arg, (4, 4))
    assert dx.sum() == 4 and dx[0, 0, 0, 0] == 1 and dx[0, 0, 1, 0] == 1 and dx[0, 1, 0, 0] == 1 and dx[0, 1, 1, 0] == 1
    # negative inputs: padding must never win
    n = -np.abs(rnd(1, 5, 5, 2)) - 1.0
    y, _ = oracle.maxpool_fwd(n)
    assert (y < 0).all()


def test_bf16_storage_rounding_is_nearest_even():
    # quant=1 output of a 1x1 identity conv = bf16(x); compare with torch's conversion (library routine)
    x = rnd(1, 8, 8, 4).astype(np.float32)
    w = np.eye(4, dtype=np.float32).reshape(4, 1, 1, 4)
    y = oracle.conv_fwd(x, w, 1, quant=1)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(y, ref)


def _bf16(x):
    """nearest-even bf16 rounding by the library routine (torch), back in fp32"""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def test_bf16_storage_rounding_points_of_the_layer_routines():
    """quant=1 rounds what a layer STORES (Q15: activations and activation gradients are bf16, every sum is wider) and nothing
    else: each layer's quant=1 output must be the bf16 rounding of its quant=0 output, element by element, and the statistics
    a layer returns (mean, 1/std, dgamma, dbeta, running statistics) must not be rounded at all."""
    a, w = _bf16(rnd(2, 6, 5, 8)), _bf16(rnd(16, 3, 3, 8) * 0.25)
    add = _bf16(rnd(2, 6, 5, 16))
    for stride in (1, 2):
        sub = np.ascontiguousarray(add[:, ::stride, ::stride])        # a residual of the output's shape
        y0 = oracle.conv_fwd(a, w, stride, add=sub, scale=0.5)
        y1 = oracle.conv_fwd(a, w, stride, add=sub, scale=0.5, quant=1)
        np.testing.assert_array_equal(y1, _bf16(y0))
        dy = _bf16(rnd(*y0.shape))
        adda = _bf16(rnd(*a.shape))
        np.testing.assert_array_equal(oracle.conv_dgrad(dy, w, a.shape[1:3], stride, add=adda, quant=1),
                                      _bf16(oracle.conv_dgrad(dy, w, a.shape[1:3], stride, add=adda)))
    x = _bf16(rnd(60, 8) * 1.5 + rnd(8)[None, :])
    g, b = (1 + 0.2 * rnd(8)).astype(np.float32), (0.3 * rnd(8)).astype(np.float32)
    rm0, rv0, rm1, rv1 = np.zeros(8, np.float32), np.ones(8, np.float32), np.zeros(8, np.float32), np.ones(8, np.float32)
    a0, mean0, istd0 = oracle.bn_relu_fwd(x, g, b, rm0, rv0)
    a1, mean1, istd1 = oracle.bn_relu_fwd(x, g, b, rm1, rv1, quant=1)
    np.testing.assert_array_equal(a1, _bf16(a0))
    for u, v in ((mean0, mean1), (istd0, istd1), (rm0, rm1), (rv0, rv1)):
        np.testing.assert_array_equal(u, v)
    da, skip = _bf16(rnd(60, 8)), _bf16(rnd(60, 8))
    dx0, dg0, db0 = oracle.bn_relu_bwd(da, x, g, b, mean0, istd0, add=skip)
    dx1, dg1, db1 = oracle.bn_relu_bwd(da, x, g, b, mean0, istd0, add=skip, quant=1)
    np.testing.assert_array_equal(dx1, _bf16(dx0))
    np.testing.assert_array_equal(dg0, dg1)
    np.testing.assert_array_equal(db0, db1)
