"""Pins for the oracle's integer contractions (no GPU)."""
import itertools

import numpy as np
import pytest

import oracle


def _rand_s8(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


def test_all_ones_closed_form():
    # 3x3, pad 1, all-ones operands: 9*Cin inside, 6*Cin on edges, 4*Cin at corners
    Cin, Cout = 5, 3
    A = np.ones((1, 2, 6, 7, Cin), np.int8)
    W = np.ones((1, Cout, 3, 3, Cin), np.int8)
    acc, ovf = oracle.qconv_fwd(A, W, stride=1, pad=1)
    assert ovf == 0 and acc.shape == (1, 2, 6, 7, Cout)
    assert np.all(acc[:, :, 1:-1, 1:-1] == 9 * Cin)
    assert np.all(acc[:, :, 0, 1:-1] == 6 * Cin) and np.all(acc[:, :, 1:-1, -1] == 6 * Cin)
    for h, w in itertools.product((0, -1), (0, -1)):
        assert np.all(acc[:, :, h, w] == 4 * Cin)


def test_delta_kernel_is_a_shift():
    rng = np.random.default_rng(0)
    A = _rand_s8(rng, (2, 2, 5, 6, 4))
    for (r, s) in [(1, 1), (0, 2), (2, 0)]:
        W = np.zeros((2, 4, 3, 3, 4), np.int8)
        for c in range(4):
            W[:, c, r, s, c] = 1          # out[oh,ow,c] = A[oh+r-1, ow+s-1, c]
        acc, _ = oracle.qconv_fwd(A, W, 1, 1)
        Ap = np.pad(A.astype(np.int32), ((0, 0), (0, 0), (1, 1), (1, 1), (0, 0)))
        assert np.array_equal(acc, Ap[:, :, r:r + 5, s:s + 6, :])


def test_1x1_conv_is_a_matmul():
    # R=S=1, pad 0: per node Y = A_flat @ W^T, a library matrix product
    rng = np.random.default_rng(1)
    A = _rand_s8(rng, (3, 2, 4, 5, 7))
    W = _rand_s8(rng, (3, 6, 1, 1, 7))
    acc, _ = oracle.qconv_fwd(A, W, 1, 0)
    for n in range(3):
        ref = A[n].reshape(-1, 7).astype(np.int64) @ W[n].reshape(6, 7).astype(np.int64).T
        assert np.array_equal(acc[n].reshape(-1, 6), ref)
    # linear layer = H=W=1
    X = _rand_s8(rng, (2, 9, 1, 1, 11))
    Wl = _rand_s8(rng, (2, 4, 1, 1, 11))
    acc, _ = oracle.qconv_fwd(X, Wl, 1, 0)
    E = _rand_s8(rng, (2, 9, 1, 1, 4))
    dX, _ = oracle.qconv_bwd_data(E, Wl, 1, 1, 1, 0)
    dW, _ = oracle.qconv_bwd_weight(E, X, 1, 1, 1, 0)
    for n in range(2):
        x = X[n].reshape(9, 11).astype(np.int64); w = Wl[n].reshape(4, 11).astype(np.int64)
        e = E[n].reshape(9, 4).astype(np.int64)
        assert np.array_equal(acc[n].reshape(9, 4), x @ w.T)
        assert np.array_equal(dX[n].reshape(9, 11), e @ w)
        assert np.array_equal(dW[n].reshape(4, 11), e.T @ x)


def _fwd_via_padding(A, W, stride, pad):
    """Independent restatement: explicit zero padding + strided window slices + einsum."""
    n, B, H, Wd, Cin = A.shape
    _, Cout, R, S, _ = W.shape
    Ho = (H + 2 * pad - R) // stride + 1
    Wo = (Wd + 2 * pad - S) // stride + 1
    Ap = np.pad(A.astype(np.int64), ((0, 0), (0, 0), (pad, pad), (pad, pad), (0, 0)))
    out = np.zeros((n, B, Ho, Wo, Cout), np.int64)
    for r in range(R):
        for s in range(S):
            win = Ap[:, :, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :]
            out += np.einsum("nbhwc,nkc->nbhwk", win, W[:, :, r, s, :].astype(np.int64))
    return out


@pytest.mark.parametrize("H,W,Cin,Cout,R,S,stride,pad", [
    (5, 6, 3, 4, 3, 3, 1, 1),
    (8, 8, 4, 5, 3, 3, 2, 1),
    (7, 5, 2, 3, 3, 3, 2, 1),
    (6, 6, 3, 2, 1, 1, 2, 0),
    (4, 4, 2, 2, 3, 3, 1, 0),
    (5, 5, 1, 1, 5, 5, 1, 2),
])
def test_fwd_against_padded_window_sum(H, W, Cin, Cout, R, S, stride, pad):
    rng = np.random.default_rng(7)
    A = _rand_s8(rng, (2, 2, H, W, Cin))
    Wq = _rand_s8(rng, (2, Cout, R, S, Cin))
    acc, ovf = oracle.qconv_fwd(A, Wq, stride, pad)
    assert ovf == 0
    assert np.array_equal(acc, _fwd_via_padding(A, Wq, stride, pad))


@pytest.mark.parametrize("H,W,Cin,Cout,R,S,stride,pad", [
    (5, 6, 3, 4, 3, 3, 1, 1),
    (8, 8, 4, 5, 3, 3, 2, 1),
    (7, 5, 2, 3, 3, 3, 2, 1),
    (6, 6, 3, 2, 1, 1, 2, 0),
    (4, 4, 2, 2, 3, 3, 1, 0),
])
def test_adjoint_identities_exact(H, W, Cin, Cout, R, S, stride, pad):
    # <fwd(A,W), E> = <A, bwd_data(E,W)> = <W, bwd_weight(E,A)> exactly in int64:
    # pins both backward contractions to the forward one.
    rng = np.random.default_rng(11)
    A = _rand_s8(rng, (2, 3, H, W, Cin))
    Wq = _rand_s8(rng, (2, Cout, R, S, Cin))
    Y, _ = oracle.qconv_fwd(A, Wq, stride, pad)
    E = _rand_s8(rng, Y.shape)
    dA, o1 = oracle.qconv_bwd_data(E, Wq, H, W, stride, pad)
    dW, o2 = oracle.qconv_bwd_weight(E, A, R, S, stride, pad)
    assert o1 == 0 and o2 == 0
    for n in range(2):
        lhs = int((Y[n].astype(np.int64) * E[n]).sum())
        assert lhs == int((dA[n].astype(np.int64) * A[n]).sum())
        assert lhs == int((dW[n].astype(np.int64) * Wq[n]).sum())


def test_bwd_by_unit_probes():
    # The adjoint identity fixes the bilinear form; unit probes fix every entry:
    # dA[p] = <fwd(e_p, W), E>, dW[k] = <fwd(A, e_k), E> on a tiny shape.
    rng = np.random.default_rng(5)
    H, W, Cin, Cout, stride, pad = 4, 3, 2, 2, 2, 1
    A = _rand_s8(rng, (1, 1, H, W, Cin))
    Wq = _rand_s8(rng, (1, Cout, 3, 3, Cin))
    Y, _ = oracle.qconv_fwd(A, Wq, stride, pad)
    E = _rand_s8(rng, Y.shape)
    dA, _ = oracle.qconv_bwd_data(E, Wq, H, W, stride, pad)
    dW, _ = oracle.qconv_bwd_weight(E, A, 3, 3, stride, pad)
    for idx in np.ndindex(A.shape):
        probe = np.zeros(A.shape, np.int8); probe[idx] = 1
        y, _ = oracle.qconv_fwd(probe, Wq, stride, pad)
        assert dA[idx] == int((y.astype(np.int64) * E).sum())
    for idx in np.ndindex(Wq.shape):
        probe = np.zeros(Wq.shape, np.int8); probe[idx] = 1
        y, _ = oracle.qconv_fwd(A, probe, stride, pad)
        assert dW[idx] == int((y.astype(np.int64) * E).sum())


def test_nodes_are_independent():
    rng = np.random.default_rng(3)
    A = _rand_s8(rng, (3, 2, 4, 4, 3)); Wq = _rand_s8(rng, (3, 2, 3, 3, 3))
    full, _ = oracle.qconv_fwd(A, Wq, 1, 1)
    for n in range(3):
        one, _ = oracle.qconv_fwd(A[n:n + 1], Wq[n:n + 1], 1, 1)
        assert np.array_equal(full[n:n + 1], one)


def test_overflow_is_counted_and_wraps():
    K = 140000     # 127*127*K > 2^31
    A = np.full((1, 1, 1, 1, K), 127, np.int8)
    Wq = np.full((1, 1, 1, 1, K), 127, np.int8)
    acc, ovf = oracle.qconv_fwd(A, Wq, 1, 0)
    assert ovf == 1
    assert int(acc.ravel()[0]) == ((127 * 127 * K + 2 ** 31) % 2 ** 32) - 2 ** 31


def test_dequant_acc():
    acc = np.array([[[3, -5]], [[7, 11]]], np.int32)          # [nodes=2, 1, C=2]
    s1 = np.array([0.5, 0.25], np.float32); s2 = np.array([0.125, 2.0], np.float32)
    y = oracle.dequant_acc(acc, s1, s2)
    assert np.array_equal(y, np.array([[[3 * 0.0625, -5 * 0.0625]], [[3.5, 5.5]]], np.float32))
    b = np.array([[1.0, -1.0], [0.5, 0.0]], np.float32)
    yb = oracle.dequant_acc(acc, s1, s2, b)
    assert np.array_equal(yb, y + b[:, None, :])


# ---- affine (zero-point) operands (Section 3 names the scheme; taps outside the image are real zeros) ----
def _affine_case(seed, n=2, B=2, H=5, W=6, Cin=3, Cout=4, R=3, S=3):
    rng = np.random.default_rng(seed)
    A = rng.integers(0, 256, (n, B, H, W, Cin), dtype=np.uint8)
    Wq = rng.integers(0, 256, (n, Cout, R, S, Cin), dtype=np.uint8)
    zA = rng.integers(0, 256, n).astype(np.int32)
    zW = rng.integers(0, 256, n).astype(np.int32)
    return A, zA, Wq, zW


def test_affine_zero_zero_points_is_the_plain_product():
    # with both zero points 0 and codes below 128 the affine product is the signed one
    rng = np.random.default_rng(1)
    A = rng.integers(0, 128, (2, 2, 6, 5, 4), dtype=np.uint8)
    Wq = rng.integers(0, 128, (2, 3, 3, 3, 4), dtype=np.uint8)
    z = np.zeros(2, np.int32)
    acc, ovf = oracle.qconv_fwd_affine(A, z, Wq, z, stride=1, pad=1)
    ref, _ = oracle.qconv_fwd(A.astype(np.int8), Wq.astype(np.int8), stride=1, pad=1)
    assert ovf == 0 and np.array_equal(acc, ref)


def test_affine_constant_input_at_the_zero_point_gives_zero():
    A, zA, Wq, zW = _affine_case(2)
    for i in range(A.shape[0]):
        A[i] = zA[i]                        # real 0 everywhere, borders included
    acc, _ = oracle.qconv_fwd_affine(A, zA, Wq, zW, stride=1, pad=1)
    assert not acc.any()
    for i in range(Wq.shape[0]):            # and a weight tensor of real zeros
        Wq[i] = zW[i]
    A2 = _affine_case(3)[0]
    acc, _ = oracle.qconv_fwd_affine(A2, zA, Wq, zW, stride=2, pad=1)
    assert not acc.any()


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (1, 0, 1), (1, 2, 5)])
def test_affine_equals_real_domain_correlation(stride, pad, R):
    # dequantize, zero-pad the REAL tensor, correlate with numpy in float64: a library routine on the meaning
    A, zA, Wq, zW = _affine_case(4, H=7, W=6, R=R, S=R)
    sA, sW = 0.013, 0.21
    acc, ovf = oracle.qconv_fwd_affine(A, zA, Wq, zW, stride=stride, pad=pad)
    assert ovf == 0
    n, B, H, W, Cin = A.shape
    Cout = Wq.shape[1]
    Ho, Wo = acc.shape[2], acc.shape[3]
    for i in range(n):
        a = sA * (A[i].astype(np.float64) - zA[i])
        w = sW * (Wq[i].astype(np.float64) - zW[i])
        ap = np.pad(a, ((0, 0), (pad, pad), (pad, pad), (0, 0)))
        win = np.lib.stride_tricks.sliding_window_view(ap, (R, R), axis=(1, 2))[:, ::stride, ::stride]   # b,oh,ow,ci,r,s
        ref = np.einsum("bhwcrs,orsc->bhwo", win[:, :Ho, :Wo], w)
        np.testing.assert_allclose(sA * sW * acc[i].astype(np.float64), ref, rtol=1e-12, atol=1e-9)


def test_affine_expansion_identity():
    # sum (qa - zA)(qw - zW) = sum qa qw - zW sum qa - zA sum qw + (#terms) zA zW over the taps inside the image:
    # each term evaluated with the zero-point-free oracle on helper tensors
    A, zA, Wq, zW = _affine_case(5, Cin=2, Cout=3)
    acc, _ = oracle.qconv_fwd_affine(A, zA, Wq, zW, stride=1, pad=1)
    z0 = np.zeros(A.shape[0], np.int32)
    raw, _ = oracle.qconv_fwd_affine(A, z0, Wq, z0, stride=1, pad=1)
    ones_w = np.ones_like(Wq)
    ones_a = np.ones_like(A)
    ra, _ = oracle.qconv_fwd_affine(A, z0, ones_w, z0, stride=1, pad=1)        # sum of qa over the valid taps
    rw, _ = oracle.qconv_fwd_affine(ones_a, z0, Wq, z0, stride=1, pad=1)       # sum of qw over the valid taps
    cnt, _ = oracle.qconv_fwd_affine(ones_a, z0, ones_w, z0, stride=1, pad=1)  # number of terms
    zA_, zW_ = zA[:, None, None, None, None].astype(np.int64), zW[:, None, None, None, None].astype(np.int64)
    ref = raw.astype(np.int64) - zW_ * ra - zA_ * rw + cnt * zA_ * zW_
    assert np.array_equal(acc.astype(np.int64), ref)
    assert cnt[0, 0, 0, 0, 0] == 4 * 2 and cnt[0, 0, 2, 2, 0] == 9 * 2         # corner and interior term counts


# ---- affine backward products: pinned to the (already pinned) affine forward product and to its meaning ----
@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (1, 0, 1), (1, 2, 5), (2, 0, 2)])
def test_affine_backward_products_are_the_adjoints_of_the_forward_product(stride, pad, R):
    # <fwd(A, W), E'> = <A', bwd_data(E, W)> = <W', bwd_weight(E, A)> exactly in int64, primes = code - zero point:
    # a dropped tap, a wrong border rule or a transposed index in either backward product breaks one of the two
    A, zA, Wq, zW = _affine_case(11 + R, H=7, W=6, R=R, S=R)
    n, B, H, W, Cin = A.shape
    fwd, ovf = oracle.qconv_fwd_affine(A, zA, Wq, zW, stride=stride, pad=pad)
    assert ovf == 0
    rng = np.random.default_rng(stride * 10 + R)
    E = rng.integers(0, 256, fwd.shape, dtype=np.uint8)
    zE = rng.integers(0, 256, n).astype(np.int32)
    dA, o1 = oracle.qconv_bwd_data_affine(E, zE, Wq, zW, H, W, stride=stride, pad=pad)
    dW, o2 = oracle.qconv_bwd_weight_affine(E, zE, A, zA, R, R, stride=stride, pad=pad)
    assert o1 == 0 and o2 == 0
    c = lambda q, z: q.astype(np.int64) - z.reshape((-1,) + (1,) * (q.ndim - 1))
    for i in range(n):
        lhs = int((fwd[i].astype(np.int64) * c(E, zE)[i]).sum())
        assert lhs == int((c(A, zA)[i] * dA[i]).sum())
        assert lhs == int((c(Wq, zW)[i] * dW[i]).sum())


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1)])
def test_affine_backward_products_equal_real_domain_gradients(stride, pad):
    # the real-valued layer y = conv(a, w) with zero padding: dL/da and dL/dw for upstream gradient e, computed
    # in float64 by probing the bilinear form with numpy (a library routine on the meaning of the codes)
    A, zA, Wq, zW = _affine_case(21, n=1, B=2, H=5, W=4, Cin=2, Cout=3)
    n, B, H, W, Cin = A.shape
    Cout, R = Wq.shape[1], Wq.shape[2]
    rng = np.random.default_rng(5)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    E = rng.integers(0, 256, (n, B, Ho, Wo, Cout), dtype=np.uint8)
    zE = np.array([97], np.int32)
    a = A[0].astype(np.float64) - zA[0]
    w = Wq[0].astype(np.float64) - zW[0]
    e = E[0].astype(np.float64) - zE[0]

    def fwd_real(a_, w_):
        ap = np.pad(a_, ((0, 0), (pad, pad), (pad, pad), (0, 0)))
        win = np.lib.stride_tricks.sliding_window_view(ap, (R, R), axis=(1, 2))[:, ::stride, ::stride]
        return np.einsum("bhwcrs,orsc->bhwo", win[:, :Ho, :Wo], w_)
    # gradients of <fwd_real(a, w), e> by unit probes (the form is linear in a and in w)
    da = np.zeros_like(a); dw = np.zeros_like(w)
    for idx in np.ndindex(a.shape):
        u = np.zeros_like(a); u[idx] = 1.0
        da[idx] = (fwd_real(u, w) * e).sum()
    for idx in np.ndindex(w.shape):
        u = np.zeros_like(w); u[idx] = 1.0
        dw[idx] = (fwd_real(a, u) * e).sum()
    dA, _ = oracle.qconv_bwd_data_affine(E, zE, Wq, zW, H, W, stride=stride, pad=pad)
    dW, _ = oracle.qconv_bwd_weight_affine(E, zE, A, zA, R, R, stride=stride, pad=pad)
    assert np.array_equal(dA[0].astype(np.float64), da)
    assert np.array_equal(dW[0].astype(np.float64), dw)


def test_affine_backward_with_zero_zero_points_is_the_plain_product():
    rng = np.random.default_rng(31)
    E = rng.integers(0, 128, (2, 2, 6, 5, 3), dtype=np.uint8)
    Wq = rng.integers(0, 128, (2, 3, 3, 3, 4), dtype=np.uint8)
    A = rng.integers(0, 128, (2, 2, 6, 5, 4), dtype=np.uint8)
    z = np.zeros(2, np.int32)
    dA, _ = oracle.qconv_bwd_data_affine(E, z, Wq, z, 6, 5, stride=1, pad=1)
    ref, _ = oracle.qconv_bwd_data(E.astype(np.int8), Wq.astype(np.int8), 6, 5, stride=1, pad=1)
    assert np.array_equal(dA, ref)
    dW, _ = oracle.qconv_bwd_weight_affine(E, z, A, z, 3, 3, stride=1, pad=1)
    ref, _ = oracle.qconv_bwd_weight(E.astype(np.int8), A.astype(np.int8), 3, 3, stride=1, pad=1)
    assert np.array_equal(dW, ref)


def test_affine_backward_of_a_real_zero_gradient_is_zero():
    A, zA, Wq, zW = _affine_case(41)
    n = A.shape[0]
    zE = np.array([200, 3], np.int32)
    E = np.empty((n, 2, 5, 6, 4), np.uint8)
    for i in range(n):
        E[i] = zE[i]
    dA, _ = oracle.qconv_bwd_data_affine(E, zE, Wq, zW, 5, 6, stride=1, pad=1)
    dW, _ = oracle.qconv_bwd_weight_affine(E, zE, A, zA, 3, 3, stride=1, pad=1)
    assert not dA.any() and not dW.any()
