"""GPU parity of the launches the local step really makes for a convolution and the BN+ReLU that consumes its output
(Sec. 2.1: BN -> ReLU -> conv, so every convolution's output feeds a BN), element by element against the oracle's layer
routines composed in the same order, with the same bf16 storage rounding, on identical inputs.

Forward: y = conv(a, w) (+ residual), a_out = relu(bn(y)): narrow layers run the BN inside the warp-MMA convolution's
launch, wide ones take the statistics from the per-tile sums of the tcgen05 epilogue.  Backward: da = dgrad(dy, w),
dx = BN+ReLU backward with da as the output gradient (+ skip gradient).
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


def rnd(seed, *shape):
    return synth.round_to_bf16(synth.standard_normal(seed, int(np.prod(shape))).astype(np.float32).reshape(shape))


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda().to(torch.bfloat16)


def fdev(x):
    return torch.from_numpy(np.ascontiguousarray(x.astype(np.float32))).cuda()


# (N, H, W, C, K, ksz, stride, family): 16/32/64 channels on the warp-MMA family (BN inside the launch, several pieces per
# CTA, stride 1 and 2), wider layers on tcgen05 (several slabs and column tiles, 3x3 and 1x1, stride 2, ragged tails)
PAIRS = [
    (24, 32, 32, 16, 16, 3, 1, 2), (24, 16, 16, 32, 32, 3, 1, 2), (40, 8, 8, 64, 64, 3, 1, 2), (16, 32, 32, 16, 32, 3, 2, 2),
    (16, 16, 16, 32, 64, 3, 2, 2), (12, 16, 16, 64, 64, 1, 1, 0),
    (6, 16, 16, 128, 128, 3, 1, 1), (4, 32, 32, 64, 256, 1, 1, 1), (4, 32, 32, 256, 64, 1, 1, 1), (6, 16, 16, 128, 128, 3, 2, 1),
    (5, 8, 8, 256, 512, 1, 1, 1), (3, 9, 7, 128, 256, 3, 1, 1), (4, 16, 16, 256, 512, 1, 2, 1),
]


@pytest.mark.parametrize("pair", PAIRS)
@pytest.mark.parametrize("with_add", [False, True])
def test_conv_then_bn_relu_forward(m, pair, with_add):
    N, H, W, C, K, k, s, family = pair
    a, w = rnd(1, N, H, W, C), synth.round_to_bf16(rnd(2, K, k, k, C) * np.float32(0.25))
    y_shape = oracle.conv_fwd(a[:1], w, s, quant=1).shape
    add = rnd(3, N, y_shape[1], y_shape[2], K) if with_add else None
    g, b = (1 + 0.2 * rnd(13, K)).astype(np.float32), (0.3 * rnd(14, K)).astype(np.float32)
    rm, rv = rnd(15, K).astype(np.float32), (np.abs(rnd(16, K)) + 0.5).astype(np.float32)
    y_ref = oracle.conv_fwd(a, w, s, add=add, quant=1)
    rm_ref, rv_ref = rm.copy(), rv.copy()
    a_ref, mean, invstd = oracle.bn_relu_fwd(y_ref.reshape(-1, K), g, b, rm_ref, rv_ref, quant=1)
    drm, drv = fdev(rm), fdev(rv)
    y, a_out, stat, used = m.resist_conv2d_bn_relu(0, dev(a), dev(w), (N, H, W, C, K, k, s), fdev(g), fdev(b),
                                                    add=dev(add) if with_add else None, run_mean=drm, run_var=drv)
    assert family == 0 or used == family          # family 0: whichever tensor-core family takes the pair
    assert norm_max_abs(y.float().cpu().numpy(), y_ref) < 2e-2
    # The two sides' y differ by one bf16 ulp in a few elements (fp32 sums that land on either side of a rounding boundary), which
    # moves a channel's mean by ulp / m per element: the mean is held to 2e-4 standard deviations (what the normalised value sees;
    # a convolution output's mean is near zero, so an error relative to the mean itself says nothing).  One such element at 3 sigma
    # moves the variance by 2 * 3 sigma * (0.004 * 3 sigma) / m = 0.07 sigma^2 / m: 4e-4 at the smallest m here (189 rows), so
    # 1/std and the running variance are held to 1e-3 relative.
    assert float(np.abs((stat[:K].cpu().numpy() - mean) * invstd).max()) < 2e-4
    assert max_rel_err(stat[K:2 * K].cpu().numpy(), invstd) < 1e-3
    assert float(np.abs(drm.cpu().numpy() - rm_ref).max()) < 1e-4 and max_rel_err(drv.cpu().numpy(), rv_ref) < 1e-3
    assert norm_max_abs(a_out.float().cpu().numpy().reshape(-1, K), a_ref) < 2e-2


@pytest.mark.parametrize("pair", PAIRS)
@pytest.mark.parametrize("with_add", [False, True])
def test_dgrad_then_bn_relu_backward(m, pair, with_add):
    N, H, W, C, K, k, s, family = pair
    if family == 1 and k == 1 and s == 2:
        pytest.skip("the step never pairs a strided projection's dgrad with a BN (its gradient joins conv1's)")
    w = synth.round_to_bf16(rnd(2, K, k, k, C) * np.float32(0.25))
    P, Q = oracle.conv_fwd(rnd(1, 1, H, W, C), w, s, quant=1).shape[1:3]
    dy = rnd(4, N, P, Q, K)
    x = synth.round_to_bf16(rnd(5, N, H, W, C) * np.float32(1.7) + rnd(6, C)[None, None, None, :])
    skip = rnd(7, N, H, W, C) if with_add else None
    g, b = (1 + 0.2 * rnd(13, C)).astype(np.float32), (0.3 * rnd(14, C)).astype(np.float32)
    _, mean, invstd = oracle.bn_relu_fwd(x.reshape(-1, C), g, b, quant=1)
    da_ref = oracle.conv_dgrad(dy, w, (H, W), s, quant=1)
    dx_ref, dg_ref, db_ref = oracle.bn_relu_bwd(da_ref.reshape(-1, C), x.reshape(-1, C), g, b, mean, invstd,
                                                add=skip.reshape(-1, C) if with_add else None, quant=1)
    stat = torch.zeros(4 * C, dtype=torch.float32, device="cuda")
    stat[:C] = fdev(mean)
    stat[C:2 * C] = fdev(invstd)
    da, dx, dg, db, used = m.resist_conv2d_bn_relu(1, dev(dy), dev(w), (N, H, W, C, K, k, s), fdev(g), fdev(b), stat=stat, x=dev(x),
                                                   bn_add=dev(skip) if with_add else None)
    assert family == 0 or used == family          # family 0: whichever tensor-core family takes the pair
    assert norm_max_abs(da.float().cpu().numpy(), da_ref) < 2e-2
    assert norm_max_abs(dx.float().cpu().numpy().reshape(-1, C), dx_ref) < 2e-2
    # sums over all rows of da values that differ by a bf16 ulp (0.4 %) where the two sides round differently: 1e-2 of the largest entry
    assert norm_max_abs(dg.cpu().numpy(), dg_ref) < 1e-2 and norm_max_abs(db.cpu().numpy(), db_ref) < 1e-2
