"""Pins for the CPU oracle's per-layer primitives (Section 2, Eq. 3-5 per layer type): brute force on tiny
inputs, closed forms, invariants, central finite differences and a library routine.  No GPU."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ddg_oracle as orc

RNG = np.random.default_rng(7)


def golden():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                vals[line[0]] = float(line[1])
    return vals


def brute_conv(x, w, stride):
    B, Ci, H, W = x.shape
    Co = w.shape[0]
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    y = np.zeros((B, Co, Ho, Wo))
    for n, co, ho, wo, ci, ky, kx in itertools.product(range(B), range(Co), range(Ho), range(Wo), range(Ci),
                                                       range(3), range(3)):
        hi, wi = stride * ho + ky - 1, stride * wo + kx - 1
        if 0 <= hi < H and 0 <= wi < W:
            y[n, co, ho, wo] += w[co, ci, ky, kx] * x[n, ci, hi, wi]
    return y


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", [(2, 3, 5, 5, 4), (1, 2, 4, 6, 3), (2, 1, 1, 1, 2)])
def test_conv_forward_brute_force(shape, stride):
    B, Ci, H, W, Co = shape
    x, w = RNG.standard_normal((B, Ci, H, W)), RNG.standard_normal((Co, Ci, 3, 3))
    np.testing.assert_allclose(orc.conv3x3_forward(x, w, stride), brute_conv(x, w, stride), rtol=1e-12, atol=1e-12)


def test_conv_identity_kernel_and_stride_subsampling():
    x = RNG.standard_normal((2, 3, 6, 6))
    w = np.zeros((3, 3, 3, 3))
    for c in range(3):
        w[c, c, 1, 1] = 1.0
    np.testing.assert_array_equal(orc.conv3x3_forward(x, w, 1), x)
    w = RNG.standard_normal((4, 3, 3, 3))
    np.testing.assert_allclose(orc.conv3x3_forward(x, w, 2), orc.conv3x3_forward(x, w, 1)[:, :, ::2, ::2], rtol=1e-13)
    # a one-sided kernel tells cross-correlation from convolution: tap (ky=0,kx=1) reads the row above
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 1] = 1.0
    x1 = RNG.standard_normal((1, 1, 4, 4))
    y = orc.conv3x3_forward(x1, w, 1)
    np.testing.assert_array_equal(y[0, 0, 1:], x1[0, 0, :-1])
    np.testing.assert_array_equal(y[0, 0, 0], 0)


@pytest.mark.parametrize("stride", [1, 2])
def test_conv_matches_library(stride):
    x, w = RNG.standard_normal((3, 5, 9, 7)), RNG.standard_normal((6, 5, 3, 3))
    dy_shape = orc.conv3x3_forward(x, w, stride).shape
    dy = RNG.standard_normal(dy_shape)
    xt, wt = torch.tensor(x, requires_grad=True), torch.tensor(w, requires_grad=True)
    yt = F.conv2d(xt, wt, None, stride, 1)
    yt.backward(torch.tensor(dy))
    np.testing.assert_allclose(orc.conv3x3_forward(x, w, stride), yt.detach().numpy(), rtol=1e-11, atol=1e-12)
    dx, dw = orc.conv3x3_backward(x, w, dy, stride)
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(dw, wt.grad.numpy(), rtol=1e-11, atol=1e-12)


def fd_grad(f, a, h=1e-6):
    g = np.zeros_like(a)
    it = np.nditer(a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = a[i]
        a[i] = old + h; fp = f()
        a[i] = old - h; fm = f()
        a[i] = old
        g[i] = (fp - fm) / (2 * h)
    return g


def rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


@pytest.mark.parametrize("stride", [1, 2])
def test_conv_backward_finite_differences(stride):
    x, w = RNG.standard_normal((2, 3, 5, 5)), RNG.standard_normal((4, 3, 3, 3))
    r = RNG.standard_normal(orc.conv3x3_forward(x, w, stride).shape)
    f = lambda: float((orc.conv3x3_forward(x, w, stride) * r).sum())
    dx, dw = orc.conv3x3_backward(x, w, r, stride)
    assert rel(dx, fd_grad(f, x)) < 1e-6
    assert rel(dw, fd_grad(f, w)) < 1e-6


def test_fc_finite_differences_and_library():
    x, W, b = RNG.standard_normal((4, 5)), RNG.standard_normal((3, 5)), RNG.standard_normal(3)
    r = RNG.standard_normal((4, 3))
    np.testing.assert_allclose(orc.fc_forward(x, W, b), x @ W.T + b, rtol=1e-13)
    f = lambda: float((orc.fc_forward(x, W, b) * r).sum())
    dx, dW, db = orc.fc_backward(x, W, r)
    assert rel(dx, fd_grad(f, x)) < 1e-6 and rel(dW, fd_grad(f, W)) < 1e-6 and rel(db, fd_grad(f, b)) < 1e-6
    np.testing.assert_allclose(dW, r.T @ x, rtol=1e-13)   # a transposed operand would fail here


def test_softmax_ce_closed_forms():
    g = golden()
    for C, key in ((10, "ce_zero_logits_10"), (100, "ce_zero_logits_100")):
        y = RNG.integers(0, C, size=6).astype(np.int32)
        loss, dz = orc.softmax_ce(np.zeros((6, C)), y)
        assert abs(loss - g[key]) < 1e-14 and abs(loss - math.log(C)) < 1e-14
        expect = np.full((6, C), 1.0 / C)
        expect[np.arange(6), y] -= 1.0
        np.testing.assert_allclose(dz, expect / 6, rtol=1e-14)
    z = RNG.standard_normal((5, 7)) * 3
    y = RNG.integers(0, 7, size=5).astype(np.int32)
    loss, dz = orc.softmax_ce(z, y)
    np.testing.assert_allclose(dz.sum(axis=1), 0, atol=1e-15)
    assert abs(loss - float(F.cross_entropy(torch.tensor(z), torch.tensor(y).long()))) < 1e-13
    assert rel(dz, fd_grad(lambda: orc.softmax_ce(z, y)[0], z)) < 1e-7
    # shift invariance and large logits (stability)
    assert abs(orc.softmax_ce(z + 1000.0, y)[0] - loss) < 1e-9


def test_bn_forward_invariants_and_library():
    x = RNG.standard_normal((4, 3, 5, 5)) * 2 + 1
    gamma, beta = RNG.standard_normal(3), RNG.standard_normal(3)
    y, mean, invstd = orc.bn_forward(x, gamma, beta)
    np.testing.assert_allclose(y.mean(axis=(0, 2, 3)), beta, atol=1e-13)
    var = x.var(axis=(0, 2, 3))  # biased
    np.testing.assert_allclose(y.var(axis=(0, 2, 3)), gamma ** 2 * var / (var + 1e-5), rtol=1e-12)
    np.testing.assert_allclose(mean, x.mean(axis=(0, 2, 3)), rtol=1e-13)
    np.testing.assert_allclose(invstd, 1 / np.sqrt(var + 1e-5), rtol=1e-13)
    yt = F.batch_norm(torch.tensor(x), None, None, torch.tensor(gamma), torch.tensor(beta), True, 0.0, 1e-5)
    np.testing.assert_allclose(y, yt.numpy(), rtol=1e-11, atol=1e-12)


def test_bn_backward_invariants_fd_and_library():
    x = RNG.standard_normal((3, 2, 4, 4))
    gamma, beta = RNG.standard_normal(2) + 1.5, RNG.standard_normal(2)
    dy = RNG.standard_normal(x.shape)
    y, mean, invstd = orc.bn_forward(x, gamma, beta)
    dx, dg, db = orc.bn_backward(x, mean, invstd, gamma, dy)
    xhat = (x - mean[None, :, None, None]) * invstd[None, :, None, None]
    np.testing.assert_allclose(dx.sum(axis=(0, 2, 3)), 0, atol=1e-12)
    # sum(dx * xhat) vanishes as eps -> 0; for finite eps it equals gamma*invstd*dgamma * eps*invstd^2 exactly
    np.testing.assert_allclose((dx * xhat).sum(axis=(0, 2, 3)), gamma * invstd * dg * 1e-5 * invstd ** 2,
                               rtol=1e-8, atol=1e-13)
    f = lambda: float((orc.bn_forward(x, gamma, beta)[0] * dy).sum())
    assert rel(dx, fd_grad(f, x)) < 1e-6 and rel(dg, fd_grad(f, gamma)) < 1e-6 and rel(db, fd_grad(f, beta)) < 1e-6
    xt, gt, bt = (torch.tensor(a, requires_grad=True) for a in (x, gamma, beta))
    F.batch_norm(xt, None, None, gt, bt, True, 0.0, 1e-5).backward(torch.tensor(dy))
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dg, gt.grad.numpy(), rtol=1e-11)
    np.testing.assert_allclose(db, bt.grad.numpy(), rtol=1e-11)


def test_conv_then_bn_scale_invariance():
    """A conv feeding a batch-stat BN is scale invariant, so <W, dW> = 0 up to eps: pins wgrad and BN-bwd jointly."""
    x, w = RNG.standard_normal((4, 3, 6, 6)), RNG.standard_normal((5, 3, 3, 3))
    gamma, beta = RNG.standard_normal(5), RNG.standard_normal(5)
    r = RNG.standard_normal((4, 5, 6, 6))
    y = orc.conv3x3_forward(x, w, 1)
    _, mean, invstd = orc.bn_forward(y, gamma, beta)
    dy, _, _ = orc.bn_backward(y, mean, invstd, gamma, r)
    _, dw = orc.conv3x3_backward(x, w, dy, 1)
    assert abs((w * dw).sum()) < 1e-4 * np.linalg.norm(w) * np.linalg.norm(dw)


def test_relu_shortcut_avgpool():
    x = np.array([-1.0, 0.0, 2.0])
    y = np.empty(3)
    orc._call("orc_relu_forward", 3, x, y)
    np.testing.assert_array_equal(y, [0, 0, 2])
    dx = np.empty(3)
    orc._call("orc_relu_backward", 3, y, np.ones(3), dx)
    np.testing.assert_array_equal(dx, [0, 0, 1])           # derivative at 0 is 0
    x = RNG.standard_normal((2, 3, 4, 4))
    s = orc.shortcut_forward(x, 6, 2)
    np.testing.assert_array_equal(s[:, :3], x[:, :, ::2, ::2])
    np.testing.assert_array_equal(s[:, 3:], 0)
    np.testing.assert_array_equal(orc.shortcut_forward(x, 3, 1), x)
    dy = RNG.standard_normal((2, 6, 2, 2))
    d = orc.shortcut_backward(dy, 3, 4, 4, 2)
    np.testing.assert_array_equal(d[:, :, ::2, ::2], dy[:, :3])
    d[:, :, ::2, ::2] = 0
    np.testing.assert_array_equal(d, 0)                    # zero at odd positions; padded channels get nothing
    p = orc.avgpool_forward(x)
    np.testing.assert_allclose(p, x.mean(axis=(2, 3)), rtol=1e-14)
    np.testing.assert_allclose(orc.avgpool_backward(p, 4, 4), np.broadcast_to(p[:, :, None, None] / 16, x.shape))


def test_bf16_round_is_nearest_even():
    assert orc.bf16_round(1.0) == 1.0
    assert orc.bf16_round(1.0 + 2 ** -8) == 1.0            # tie -> even (1.0 has an even mantissa)
    assert orc.bf16_round(1.0 + 3 * 2 ** -8) == 1.0 + 2 ** -6   # tie -> even upwards
    assert orc.bf16_round(1.0 + 2 ** -8 + 2 ** -12) == 1.0 + 2 ** -7
    v = torch.randn(1000, dtype=torch.float32)
    ours = np.array([orc.bf16_round(float(a)) for a in v])
    np.testing.assert_array_equal(ours, v.to(torch.bfloat16).to(torch.float64).numpy())


# ---- 1x1 projection (shortcut of a shape-changing residual block) ---------------------------------------------
@pytest.mark.parametrize("stride", [1, 2])
def test_conv1x1_brute_force_center_tap_and_library(stride):
    """Three independent statements of the same operation: explicit loops; the (already pinned) 3x3 convolution with a
    filter that is zero except for its centre tap; the library's conv2d with a 1x1 kernel and no padding."""
    B, Ci, H, W, Co = 2, 3, 5, 6, 4
    x, w = RNG.standard_normal((B, Ci, H, W)), RNG.standard_normal((Co, Ci))
    y = orc.conv1x1_forward(x, w, stride)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    brute = np.zeros((B, Co, Ho, Wo))
    for n, co, ho, wo, ci in itertools.product(range(B), range(Co), range(Ho), range(Wo), range(Ci)):
        brute[n, co, ho, wo] += w[co, ci] * x[n, ci, stride * ho, stride * wo]
    np.testing.assert_allclose(y, brute, rtol=1e-13, atol=1e-13)
    w3 = np.zeros((Co, Ci, 3, 3)); w3[:, :, 1, 1] = w
    np.testing.assert_allclose(y, orc.conv3x3_forward(x, w3, stride), rtol=1e-13, atol=1e-13)
    dy = RNG.standard_normal(y.shape)
    xt, wt = torch.tensor(x, requires_grad=True), torch.tensor(w.reshape(Co, Ci, 1, 1), requires_grad=True)
    yt = F.conv2d(xt, wt, None, stride, 0)
    yt.backward(torch.tensor(dy))
    np.testing.assert_allclose(y, yt.detach().numpy(), rtol=1e-12, atol=1e-13)
    dx, dw = orc.conv1x1_backward(x, w, dy, stride)
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dw, wt.grad.numpy().reshape(Co, Ci), rtol=1e-12, atol=1e-13)
    # the pixels the stride skips receive no gradient; the centre-tap 3x3 backward agrees on both outputs
    if stride == 2:
        assert not dx[:, :, 1::2, :].any() and not dx[:, :, :, 1::2].any()
    dx3, dw3 = orc.conv3x3_backward(x, w3, dy, stride)
    np.testing.assert_allclose(dx, dx3, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dw, dw3[:, :, 1, 1], rtol=1e-12, atol=1e-13)


def test_conv1x1_backward_finite_differences():
    x, w = RNG.standard_normal((2, 3, 4, 4)), RNG.standard_normal((5, 3))
    r = RNG.standard_normal(orc.conv1x1_forward(x, w, 2).shape)
    f = lambda: float(np.sum(orc.conv1x1_forward(x, w, 2) * r))
    dx, dw = orc.conv1x1_backward(x, w, r, 2)
    np.testing.assert_allclose(dx, fd_grad(f, x), rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(dw, fd_grad(f, w), rtol=1e-6, atol=1e-8)
