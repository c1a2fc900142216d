"""Pins for the oracle's comparison layers (no GPU): EvoNorm-S0 (Eq. "en") and range batch-norm
(Eq. "rbn") against the equations written with library routines in float64, torch autograd for the
derived backward passes, hand cases, finite differences and the invariances the equations imply."""
import math

import numpy as np
import pytest
import torch

import oracle


def _inputs(n, B, H, W, C, seed):
    rng = np.random.default_rng(seed)
    x = (1.5 * rng.standard_normal((n, B, H, W, C)) + 0.3).astype(np.float32)
    v = rng.uniform(0.5, 1.5, (n, C)).astype(np.float32)
    g = rng.uniform(0.5, 1.5, (n, C)).astype(np.float32)
    b = rng.uniform(-0.5, 0.5, (n, C)).astype(np.float32)
    dy = rng.standard_normal(x.shape).astype(np.float32)
    return x, v, g, b, dy


def _evonorm_torch(x, v, g, b, groups, eps):
    n, B, H, W, C = x.shape
    xg = x.reshape(n, B, H * W, groups, C // groups)
    var = xg.var(dim=(2, 4), unbiased=False, keepdim=True)
    m = x * torch.sigmoid(v[:, None, None, None, :] * x)
    y = m.reshape(xg.shape) / torch.sqrt(var + eps)
    return y.reshape(x.shape) * g[:, None, None, None, :] + b[:, None, None, None, :]


def test_evonorm_s0_hand_case():
    # one sample, 1x1 map, one group of two channels, v = gamma = 1, beta = 0, eps = 0:
    # x = [1, -1] has mean 0 and variance 1, so y = x * sigmoid(x)
    x = np.array([1.0, -1.0], np.float32).reshape(1, 1, 1, 1, 2)
    one = np.ones((1, 2), np.float32)
    y, mu, var = oracle.evonorm_s0_fwd(x, one, one, 0 * one, 1, 0.0)
    assert mu[0, 0, 0] == 0.0 and var[0, 0, 0] == 1.0
    assert np.allclose(y.ravel(), [1 / (1 + math.exp(-1)), -1 / (1 + math.exp(1))], rtol=1e-15)


@pytest.mark.parametrize("shape,groups", [((2, 3, 4, 5, 8), 2), ((1, 2, 3, 3, 12), 3), ((1, 1, 1, 1, 4), 1)])
def test_evonorm_s0_matches_the_equation_and_autograd(shape, groups):
    x, v, g, b, dy = _inputs(*shape, seed=1)
    eps = 1e-5
    y, mu, var = oracle.evonorm_s0_fwd(x, v, g, b, groups, eps)
    t = lambda a: torch.tensor(a, dtype=torch.float64, requires_grad=True)
    xt, vt, gt, bt = t(x), t(v), t(g), t(b)
    yt = _evonorm_torch(xt, vt, gt, bt, groups, eps)
    assert np.allclose(y, yt.detach().numpy(), rtol=1e-12, atol=1e-13)
    (yt * torch.tensor(dy, dtype=torch.float64)).sum().backward()
    dx, dv, dg, db = oracle.evonorm_s0_bwd(dy, x, v, g, mu, var, groups, eps)      # statistics rounded to fp32
    for got, want in ((dx, xt.grad), (dv, vt.grad), (dg, gt.grad), (db, bt.grad)):
        assert np.allclose(got, want.numpy(), rtol=2e-6, atol=2e-6)


def test_evonorm_s0_scale_invariance_and_shift_sensitivity():
    # eps = 0: x -> a*x with v -> v/a leaves y unchanged (numerator and standard deviation both scale by a)
    x, v, g, b, _ = _inputs(1, 2, 3, 3, 8, seed=2)
    y0 = oracle.evonorm_s0_fwd(x, v, g, b, 2, 0.0)[0]
    y1 = oracle.evonorm_s0_fwd(4 * x, v / 4, g, b, 2, 0.0)[0]
    assert np.allclose(y0, y1, rtol=1e-6, atol=1e-7)
    # a constant group has zero variance: D = sqrt(eps)
    xc = np.full((1, 1, 2, 2, 2), 0.5, np.float32)
    one = np.ones((1, 2), np.float32)
    yc = oracle.evonorm_s0_fwd(xc, one, one, 0 * one, 1, 1e-4)[0]
    assert np.allclose(yc, 0.5 / (1 + math.exp(-0.5)) / 1e-2, rtol=1e-12)


def test_evonorm_s0_backward_by_finite_differences():
    x, v, g, b, dy = _inputs(1, 2, 2, 3, 4, seed=3)
    eps, h = 1e-3, 1e-3
    y, mu, var = oracle.evonorm_s0_fwd(x, v, g, b, 2, eps)
    dx, dv, dg, db = oracle.evonorm_s0_bwd(dy, x, v, g, mu, var, 2, eps)
    loss = lambda xx, vv: float((oracle.evonorm_s0_fwd(xx, vv, g, b, 2, eps)[0] * dy).sum())
    for idx in [(0, 0, 0, 0, 0), (0, 1, 1, 2, 3), (0, 0, 1, 1, 2)]:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h; xm[idx] -= h
        fd = (loss(xp, v) - loss(xm, v)) / (float(xp[idx]) - float(xm[idx]))
        assert abs(fd - dx[idx]) < 1e-4 * max(1.0, abs(fd))
    vp, vm = v.copy(), v.copy()
    vp[0, 1] += h; vm[0, 1] -= h
    fd = (loss(x, vp) - loss(x, vm)) / (float(vp[0, 1]) - float(vm[0, 1]))
    assert abs(fd - dv[0, 1]) < 1e-4 * max(1.0, abs(fd))


def _range_bn_torch(x, g, b, eps):
    n, B, H, W, C = x.shape
    mu = x.mean(dim=(1, 2, 3), keepdim=True)
    xc = x - mu
    rng = xc.amax(dim=(1, 2, 3), keepdim=True) - xc.amin(dim=(1, 2, 3), keepdim=True)
    D = rng / math.sqrt(2 * math.log(B)) + eps
    return xc / D * g[:, None, None, None, :] + b[:, None, None, None, :]


def test_range_bn_hand_case():
    # batch of two, one channel, 1x1 map: x = [1, 3] -> mean 2, range 2, C(2) = 1/sqrt(2 ln 2)
    x = np.array([1.0, 3.0], np.float32).reshape(1, 2, 1, 1, 1)
    one = np.ones((1, 1), np.float32)
    y, mu, mn, mx, amn, amx = oracle.range_bn_fwd(x, one, 0 * one, 0.0)
    D = 2.0 / math.sqrt(2 * math.log(2))
    assert mu[0, 0] == 2.0 and mn[0, 0] == 1.0 and mx[0, 0] == 3.0 and amn[0, 0] == 0 and amx[0, 0] == 1
    assert np.allclose(y.ravel(), [-1 / D, 1 / D], rtol=1e-15)
    assert abs(1 / D - 0.588705) < 1e-6


@pytest.mark.parametrize("shape", [(2, 4, 3, 5, 6), (1, 2, 1, 1, 3), (1, 8, 2, 2, 5)])
def test_range_bn_matches_the_equation_and_autograd(shape):
    x, _, g, b, dy = _inputs(*shape, seed=4)
    eps = 1e-5
    y, mu, mn, mx, amn, amx = oracle.range_bn_fwd(x, g, b, eps)
    t = lambda a: torch.tensor(a, dtype=torch.float64, requires_grad=True)
    xt, gt, bt = t(x), t(g), t(b)
    yt = _range_bn_torch(xt, gt, bt, eps)
    assert np.allclose(y, yt.detach().numpy(), rtol=1e-12, atol=1e-13)
    (yt * torch.tensor(dy, dtype=torch.float64)).sum().backward()       # extrema are unique in random data
    dx, dg, db = oracle.range_bn_bwd(dy, x, g, mu, mn, mx, amn, amx, eps)
    for got, want in ((dx, xt.grad), (dg, gt.grad), (db, bt.grad)):
        assert np.allclose(got, want.numpy(), rtol=2e-6, atol=2e-6)


def test_range_bn_invariances():
    x, _, g, b, dy = _inputs(2, 4, 3, 3, 4, seed=5)
    y0, mu, mn, mx, amn, amx = oracle.range_bn_fwd(x, g, b, 0.0)
    # shifting a channel changes nothing; scaling by a > 0 changes nothing when eps = 0
    assert np.allclose(oracle.range_bn_fwd(x + 2.0, g, b, 0.0)[0], y0, rtol=1e-5, atol=1e-6)
    assert np.allclose(oracle.range_bn_fwd(3 * x, g, b, 0.0)[0], y0, rtol=1e-5, atol=1e-6)
    dx, dg, db = oracle.range_bn_bwd(dy, x, g, mu, mn, mx, amn, amx, 0.0)
    # hence the input gradient is orthogonal to the constant and to x itself, per node and channel
    assert np.abs(dx.sum(axis=(1, 2, 3))).max() < 1e-9
    assert np.abs((dx * x).sum(axis=(1, 2, 3))).max() < 1e-5
    # ties: the lowest position takes the extremum
    xt = np.zeros((1, 3, 1, 2, 1), np.float32); xt[0, 1, 0, 1, 0] = 1; xt[0, 2, 0, 0, 0] = 1
    _, _, _, _, amn, amx = oracle.range_bn_fwd(xt, np.ones((1, 1), np.float32), np.zeros((1, 1), np.float32), 0.0)
    assert amn[0, 0] == 0 and amx[0, 0] == 3
