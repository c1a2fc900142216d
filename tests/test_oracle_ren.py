"""Pins for the oracle's Range-EvoNorm (no GPU)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _params(n, C, rng=None):
    if rng is None:
        return (np.ones((n, C), np.float32), np.ones((n, C), np.float32),
                np.zeros((n, C), np.float32))
    return (rng.uniform(0.5, 1.5, (n, C)).astype(np.float32),
            rng.uniform(0.5, 1.5, (n, C)).astype(np.float32),
            rng.uniform(-0.5, 0.5, (n, C)).astype(np.float32))


def test_constant_table():
    # C(c/g) is observable as y = x*hs(x)/(C*range): one positive and one zero element
    for line in open(os.path.join(GOLD, "range_evonorm_constants.txt")):
        if line.startswith("#") or not line.strip():
            continue
        cpg, cst = line.split()
        cpg = int(cpg); cst = float(cst)
        x = np.zeros((1, 1, 1, 1, cpg), np.float32)
        x[..., 0] = 4.0                          # hs(4) = 1, range = 4
        v, g, b = _params(1, cpg)
        y = oracle.range_evonorm_fwd(x, v, g, b, groups=1, eps=0.0, precision="f64")[0]
        assert abs(1.0 / y[0, 0, 0, 0, 0] - cst) < 1e-6


@pytest.mark.parametrize("precision,tol", [("f64", 2e-6), ("f32", 3e-6)])
def test_hand_cases(precision, tol):
    for line in open(os.path.join(GOLD, "range_evonorm_hand_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        cpg, xs, ys = line.split("|")
        x = np.array(xs.split(), np.float32).reshape(1, 1, 1, 1, -1)
        want = np.array(ys.split(), np.float64)
        v, g, b = _params(1, int(cpg))
        y, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, 1, 0.0, precision)
        assert np.allclose(y.ravel(), want, atol=tol, rtol=0)
        assert mn.ravel()[0] == x.min() and mx.ravel()[0] == x.max()
        assert amn.ravel()[0] == x.argmin() and amx.ravel()[0] == x.argmax()


def _closed_form(x, v, g, b, groups, eps):
    """Vectorised restatement with a true quotient (the equation as printed)."""
    n, B, H, W, C = x.shape
    cpg = C // groups
    xg = x.astype(np.float64).reshape(n, B, H * W, groups, cpg)
    rng = xg.max(axis=(2, 4), keepdims=True) - xg.min(axis=(2, 4), keepdims=True)
    D = rng / np.sqrt(2 * np.log(cpg)) + eps
    vv = v.astype(np.float64).reshape(n, 1, 1, groups, cpg)
    gg = g.astype(np.float64).reshape(n, 1, 1, groups, cpg)
    bb = b.astype(np.float64).reshape(n, 1, 1, groups, cpg)
    hs = np.clip((vv * xg + 3) / 6, 0, 1)
    return (xg * hs / D * gg + bb).reshape(x.shape)


@pytest.mark.parametrize("C,groups", [(8, 4), (16, 2), (6, 1), (4, 2)])
def test_fwd_matches_equation(C, groups):
    rng = np.random.default_rng(C)
    x = (3 * rng.standard_normal((2, 3, 4, 5, C))).astype(np.float32)
    v, g, b = _params(2, C, rng)
    y64 = oracle.range_evonorm_fwd(x, v, g, b, groups, 1e-5, "f64")[0]
    y32 = oracle.range_evonorm_fwd(x, v, g, b, groups, 1e-5, "f32")[0]
    ref = _closed_form(x, v, g, b, groups, 1e-5)
    assert np.allclose(y64, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(y32, ref, rtol=1e-5, atol=1e-6)


def test_scale_property():
    # x -> a*x with v -> v/a leaves y unchanged when eps = 0 (a a power of two: exact in fp32)
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 2, 3, 3, 8)).astype(np.float32)
    v, g, b = _params(1, 8, rng)
    y1 = oracle.range_evonorm_fwd(x, v, g, b, 2, 0.0, "f64")[0]
    y2 = oracle.range_evonorm_fwd(4 * x, v / 4, g, b, 2, 0.0, "f64")[0]
    assert np.allclose(y1, y2, rtol=1e-13, atol=1e-13)


def test_groups_and_samples_are_independent():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 2, 3, 3, 8)).astype(np.float32)
    v, g, b = _params(2, 8, rng)
    y = oracle.range_evonorm_fwd(x, v, g, b, 2, 1e-5)[0]
    x2 = x.copy(); x2[0, 0, :, :, 4:] *= 10.0        # disturb group 1 of sample (0,0)
    y2 = oracle.range_evonorm_fwd(x2, v, g, b, 2, 1e-5)[0]
    assert np.array_equal(y[0, 0, :, :, :4], y2[0, 0, :, :, :4])
    assert np.array_equal(y[0, 1], y2[0, 1]) and np.array_equal(y[1], y2[1])
    assert not np.array_equal(y[0, 0, :, :, 4:], y2[0, 0, :, :, 4:])


def test_first_index_wins_on_ties():
    x = np.zeros((1, 1, 2, 2, 2), np.float32)
    x[0, 0, 0, 1, 0] = 2.0; x[0, 0, 1, 1, 1] = 2.0          # two maxima
    x[0, 0, 0, 0, 1] = -1.0; x[0, 0, 1, 0, 0] = -1.0        # two minima
    v, g, b = _params(1, 2)
    _, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, 1, 0.0)
    assert amx.ravel()[0] == (0 * 2 + 1) * 2 + 0 and amn.ravel()[0] == 1
    assert mx.ravel()[0] == 2.0 and mn.ravel()[0] == -1.0


def _loss(x, v, g, b, dy, groups, eps):
    return float((_closed_form(x, v, g, b, groups, eps) * dy).sum())


def test_bwd_finite_differences():
    rng = np.random.default_rng(2)
    n, B, H, W, C, groups, eps = 2, 2, 3, 3, 8, 2, 1e-3
    x = rng.uniform(-2.5, 2.5, (n, B, H, W, C)).astype(np.float32)
    v = rng.uniform(0.3, 0.9, (n, C)).astype(np.float32)      # |v*x| < 2.25: off the kinks
    g = rng.uniform(0.5, 1.5, (n, C)).astype(np.float32)
    b = rng.uniform(-0.5, 0.5, (n, C)).astype(np.float32)
    dy = rng.standard_normal(x.shape).astype(np.float32)
    _, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, groups, eps)
    dx, dv, dg, db = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, groups, eps, "f64")
    h = 2.0 ** -10   # exactly representable steps keep the fp32 inputs exact
    probes = list(np.ndindex(x.shape))
    rng.shuffle(probes)
    # always include the extrema, where the range term lives
    ext = []
    for nn in range(n):
        for bb in range(B):
            for gg in range(groups):
                for a in (amn, amx):
                    ext.append((nn, bb) + tuple(np.unravel_index(a[nn, bb, gg], (H, W, C))))
    for idx in ext + probes[:60]:
        xp = x.copy(); xm = x.copy()
        xp[idx] += h; xm[idx] -= h
        fd = (_loss(xp, v, g, b, dy, groups, eps) - _loss(xm, v, g, b, dy, groups, eps)) / (2 * h)
        assert abs(fd - dx[idx]) < 1e-5 * max(1.0, abs(fd)), idx
    for name, arr, grad in (("v", v, dv), ("g", g, dg), ("b", b, db)):
        for idx in np.ndindex(arr.shape):
            ap = arr.copy(); am = arr.copy()
            ap[idx] += h; am[idx] -= h
            args_p = dict(v=v, g=g, b=b); args_m = dict(v=v, g=g, b=b)
            args_p[name] = ap; args_m[name] = am
            fd = (_loss(x, args_p["v"], args_p["g"], args_p["b"], dy, groups, eps) -
                  _loss(x, args_m["v"], args_m["g"], args_m["b"], dy, groups, eps)) / (2 * h)
            assert abs(fd - grad[idx]) < 1e-5 * max(1.0, abs(fd)), (name, idx)


def test_bwd_kink_and_saturation_rules():
    # outside (-3,3) the hard sigmoid is flat: dx = t*hs/D there (hs = 1 above, 0 below);
    # exactly at u = +-3 the derivative is taken as 0.
    x = np.array([3.0, -3.0, 5.0, -4.0, 1.0, 0.0, 2.0, -1.0], np.float32).reshape(1, 1, 1, 1, 8)
    v, g, b = _params(1, 8)
    dy = np.ones_like(x)
    _, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, 1, 0.0)
    dx, dv, dg, db = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, 1, 0.0, "f64")
    D = 9.0 / np.sqrt(2 * np.log(8))
    xd = x.ravel().astype(np.float64)
    m = xd * np.clip((xd + 3) / 6, 0, 1)
    S = m.sum()
    coef = S / np.sqrt(2 * np.log(8)) / D ** 2
    want = np.array([1 / D, 0.0, 1 / D - coef, 0.0 + coef,
                     (4 / 6 + 1 / 6) / D, 0.5 / D, (5 / 6 + 2 / 6) / D, (2 / 6 - 1 / 6) / D])
    assert np.allclose(dx.ravel(), want, rtol=1e-12, atol=1e-14)
    assert np.allclose(db.ravel(), 1.0) and np.allclose(dg.ravel(), m / D, rtol=1e-12)


def test_bwd_range_terms_cancel_and_constant_group():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 2, 4, 4, 4)).astype(np.float32)
    v, g, b = _params(1, 4, rng)
    dy = rng.standard_normal(x.shape).astype(np.float32)
    _, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, 1, 1e-5)
    dx, *_ = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, 1, 1e-5, "f64")
    # local part alone, recomputed: everything except the two extremum corrections
    D = (mx - mn).astype(np.float64) / np.sqrt(2 * np.log(4)) + 1e-5
    u = v[:, None, None, None, :].astype(np.float64) * x
    hs = np.clip((u + 3) / 6, 0, 1); hp = ((u > -3) & (u < 3)) / 6.0
    local = dy * g[:, None, None, None, :].astype(np.float64) * (hs + u * hp) / D.reshape(1, 2, 1, 1, 1)
    diff = (dx - local).reshape(2, -1)
    assert np.allclose(diff.sum(axis=1), 0, atol=1e-12)             # the two terms cancel
    assert np.all((np.abs(diff) > 1e-12).sum(axis=1) == 2)
    # constant group: argmax == argmin, no range term at all, finite with eps > 0
    xc = np.full((1, 1, 2, 2, 4), 0.5, np.float32)
    _, mn, mx, amn, amx = oracle.range_evonorm_fwd(xc, v, g, b, 1, 1e-2)
    assert amn.ravel()[0] == amx.ravel()[0] == 0
    dxc, *_ = oracle.range_evonorm_bwd(np.ones_like(xc), xc, v, g, mn, mx, amn, amx, 1, 1e-2, "f64")
    uc = v.astype(np.float64) * 0.5
    assert np.allclose(dxc[0, 0, 0, 0], g * (np.clip((uc + 3) / 6, 0, 1) + uc / 6) / 1e-2, rtol=1e-6)


def test_f32_variant_tracks_f64():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 4, 8, 8, 16)).astype(np.float32)
    v, g, b = _params(2, 16, rng)
    dy = rng.standard_normal(x.shape).astype(np.float32)
    st = oracle.range_evonorm_fwd(x, v, g, b, 2, 1e-5, "f32")[1:]
    a = oracle.range_evonorm_bwd(dy, x, v, g, *st, 2, 1e-5, "f32")
    c = oracle.range_evonorm_bwd(dy, x, v, g, *st, 2, 1e-5, "f64")
    for p, q in zip(a, c):
        assert p.dtype == np.float32 and q.dtype == np.float64
        assert np.allclose(p, q, rtol=1e-5, atol=1e-6)
