"""CPU oracle for the 8-bit decentralized training step (arXiv 2111.09389).

TEST INFRASTRUCTURE ONLY.  Thin numpy wrappers over oracle/lpdt_oracle.c, a
plain C restatement of what the method computes.  Nothing in the product
imports this package; only the tests, the smoke check and the CPU-baseline leg
of the benchmark do.  It shares no code with the CUDA library.

Layouts: activations [nodes][B][H][W][C], weights [nodes][Cout][R][S][Cin],
per-node scales [nodes], flat parameters [nodes][d].
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None

_i64 = C.c_longlong
_P = C.c_void_p


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
    return _lib


def _p(a):
    return a.ctypes.data_as(_P)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def num_threads():
    return int(lib().orc_num_threads())


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def quantize_sym_s8(x, rounding=0, seed=0, ctr_offset=0):
    """x: [nodes, ...] fp32 -> (q int8 same shape, scale [nodes])."""
    x = _c(x, np.float32)
    nodes = x.shape[0]
    n = x.size // nodes if nodes else 0
    q = np.zeros(x.shape, np.int8)
    scale = np.zeros(nodes, np.float32)
    lib().orc_quantize_sym_s8(_p(x), C.c_int(nodes), _i64(n), C.c_int(rounding),
                              C.c_uint64(seed), C.c_uint32(ctr_offset), _p(q), _p(scale))
    return q, scale


def quantize_affine_u8(x):
    x = _c(x, np.float32)
    nodes = x.shape[0]
    n = x.size // nodes if nodes else 0
    q = np.zeros(x.shape, np.uint8)
    scale = np.zeros(nodes, np.float32)
    zp = np.zeros(nodes, np.int32)
    lib().orc_quantize_affine_u8(_p(x), C.c_int(nodes), _i64(n), _p(q), _p(scale), _p(zp))
    return q, scale, zp


def dequantize(q, scale, zero_point=None):
    nodes = q.shape[0]
    n = q.size // nodes if nodes else 0
    y = np.zeros(q.shape, np.float32)
    scale = _c(scale, np.float32)
    if zero_point is None:
        q = _c(q, np.int8)
        lib().orc_dequantize_s8(_p(q), C.c_int(nodes), _i64(n), _p(scale), _p(y))
    else:
        q = _c(q, np.uint8)
        zp = _c(zero_point, np.int32)
        lib().orc_dequantize_u8(_p(q), C.c_int(nodes), _i64(n), _p(scale), _p(zp), _p(y))
    return y


def _out_hw(H, W, R, S, stride, pad):
    return (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1


def qconv_fwd(A, Wq, stride=1, pad=1):
    """A int8 [n,B,H,W,Cin], Wq int8 [n,Cout,R,S,Cin] -> (acc int32 [n,B,Ho,Wo,Cout], overflow)."""
    A = _c(A, np.int8)
    Wq = _c(Wq, np.int8)
    n, B, H, W, Cin = A.shape
    _, Cout, R, S, _ = Wq.shape
    Ho, Wo = _out_hw(H, W, R, S, stride, pad)
    acc = np.zeros((n, B, Ho, Wo, Cout), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_fwd(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(A), _p(Wq), _p(acc),
                        C.byref(ovf))
    return acc, ovf.value


def qconv_fwd_affine(A, zA, Wq, zW, stride=1, pad=1):
    """A uint8 [n,B,H,W,Cin], Wq uint8 [n,Cout,R,S,Cin], zero points int32 [n] ->
    (acc int32 [n,B,Ho,Wo,Cout] of (qa - zA)(qw - zW) over the taps inside the image, overflow)."""
    A = _c(A, np.uint8)
    Wq = _c(Wq, np.uint8)
    zA = _c(zA, np.int32)
    zW = _c(zW, np.int32)
    n, B, H, W, Cin = A.shape
    _, Cout, R, S, _ = Wq.shape
    assert zA.shape == (n,) and zW.shape == (n,)
    Ho, Wo = _out_hw(H, W, R, S, stride, pad)
    acc = np.zeros((n, B, Ho, Wo, Cout), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_fwd_affine(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(A), _p(zA), _p(Wq), _p(zW),
                               _p(acc), C.byref(ovf))
    return acc, ovf.value


def qconv_bwd_data(E, Wq, H, W, stride=1, pad=1):
    """E int8 [n,B,Ho,Wo,Cout], Wq int8 [n,Cout,R,S,Cin] -> (dA int32 [n,B,H,W,Cin], overflow)."""
    E = _c(E, np.int8)
    Wq = _c(Wq, np.int8)
    n, B, Ho, Wo, Cout = E.shape
    _, _, R, S, Cin = Wq.shape
    assert (Ho, Wo) == _out_hw(H, W, R, S, stride, pad)
    dA = np.zeros((n, B, H, W, Cin), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_bwd_data(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(E), _p(Wq), _p(dA),
                             C.byref(ovf))
    return dA, ovf.value


def qconv_bwd_weight(E, A, R, S, stride=1, pad=1):
    """E int8 [n,B,Ho,Wo,Cout], A int8 [n,B,H,W,Cin] -> (dW int32 [n,Cout,R,S,Cin], overflow)."""
    E = _c(E, np.int8)
    A = _c(A, np.int8)
    n, B, Ho, Wo, Cout = E.shape
    _, _, H, W, Cin = A.shape
    assert (Ho, Wo) == _out_hw(H, W, R, S, stride, pad)
    dW = np.zeros((n, Cout, R, S, Cin), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_bwd_weight(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(E), _p(A), _p(dW),
                               C.byref(ovf))
    return dW, ovf.value


def qconv_bwd_data_affine(E, zE, Wq, zW, H, W, stride=1, pad=1):
    """E uint8 [n,B,Ho,Wo,Cout], Wq uint8 [n,Cout,R,S,Cin], zero points int32 [n] ->
    (dA int32 [n,B,H,W,Cin] of (qe - zE)(qw - zW) over the taps that exist, overflow)."""
    E = _c(E, np.uint8)
    Wq = _c(Wq, np.uint8)
    zE = _c(zE, np.int32)
    zW = _c(zW, np.int32)
    n, B, Ho, Wo, Cout = E.shape
    _, _, R, S, Cin = Wq.shape
    assert (Ho, Wo) == _out_hw(H, W, R, S, stride, pad) and zE.shape == (n,) and zW.shape == (n,)
    dA = np.zeros((n, B, H, W, Cin), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_bwd_data_affine(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(E), _p(zE), _p(Wq), _p(zW),
                                    _p(dA), C.byref(ovf))
    return dA, ovf.value


def qconv_bwd_weight_affine(E, zE, A, zA, R, S, stride=1, pad=1):
    """E uint8 [n,B,Ho,Wo,Cout], A uint8 [n,B,H,W,Cin], zero points int32 [n] ->
    (dW int32 [n,Cout,R,S,Cin] of (qe - zE)(qa - zA) over the taps inside the image, overflow)."""
    E = _c(E, np.uint8)
    A = _c(A, np.uint8)
    zE = _c(zE, np.int32)
    zA = _c(zA, np.int32)
    n, B, Ho, Wo, Cout = E.shape
    _, _, H, W, Cin = A.shape
    assert (Ho, Wo) == _out_hw(H, W, R, S, stride, pad) and zE.shape == (n,) and zA.shape == (n,)
    dW = np.zeros((n, Cout, R, S, Cin), np.int32)
    ovf = _i64(0)
    lib().orc_qconv_bwd_weight_affine(n, B, H, W, Cin, Cout, R, S, stride, pad, _p(E), _p(zE), _p(A), _p(zA),
                                      _p(dW), C.byref(ovf))
    return dW, ovf.value


def dequant_acc(acc, s1, s2, bias=None):
    """y = float(acc) * (s1*s2) (+ bias over the last axis); per-node scales."""
    acc = _c(acc, np.int32)
    nodes = acc.shape[0]
    n = acc.size // nodes if nodes else 0
    Cc = acc.shape[-1]
    s1 = _c(s1, np.float32)
    s2 = _c(s2, np.float32)
    y = np.zeros(acc.shape, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    lib().orc_dequant_acc(_p(acc), C.c_int(nodes), _i64(n), C.c_int(Cc), _p(s1), _p(s2),
                          _p(b) if b is not None else None, _p(y))
    return y


def _real(precision):
    if precision == "f32":
        return np.float32, "_f32"
    if precision == "f64":
        return np.float64, "_f64"
    raise ValueError(precision)


def range_evonorm_fwd(x, v, gamma, beta, groups, eps, precision="f64"):
    """x fp32 [n,B,H,W,C]; v/gamma/beta fp32 [n,C].
    Returns (y, gmin, gmax, argmin, argmax); stats are [n,B,groups]."""
    dt, suf = _real(precision)
    x = _c(x, np.float32)
    n, B, H, W, Cc = x.shape
    v = _c(v, np.float32); gamma = _c(gamma, np.float32); beta = _c(beta, np.float32)
    y = np.zeros(x.shape, dt)
    gmin = np.zeros((n, B, groups), np.float32)
    gmax = np.zeros((n, B, groups), np.float32)
    amin = np.zeros((n, B, groups), np.int32)
    amax = np.zeros((n, B, groups), np.int32)
    getattr(lib(), "orc_ren_fwd" + suf)(n, B, H, W, Cc, groups, C.c_double(eps), _p(x), _p(v),
                                         _p(gamma), _p(beta), _p(y), _p(gmin), _p(gmax),
                                         _p(amin), _p(amax))
    return y, gmin, gmax, amin, amax


def range_evonorm_bwd(dy, x, v, gamma, gmin, gmax, argmin, argmax, groups, eps, precision="f64"):
    """Returns (dx [n,B,H,W,C], dv, dgamma, dbeta [n,C])."""
    dt, suf = _real(precision)
    x = _c(x, np.float32); dy = _c(dy, np.float32)
    n, B, H, W, Cc = x.shape
    v = _c(v, np.float32); gamma = _c(gamma, np.float32)
    gmin = _c(gmin, np.float32); gmax = _c(gmax, np.float32)
    argmin = _c(argmin, np.int32); argmax = _c(argmax, np.int32)
    dx = np.zeros(x.shape, dt)
    dv = np.zeros((n, Cc), dt); dg = np.zeros((n, Cc), dt); db = np.zeros((n, Cc), dt)
    getattr(lib(), "orc_ren_bwd" + suf)(n, B, H, W, Cc, groups, C.c_double(eps), _p(dy), _p(x),
                                         _p(v), _p(gamma), _p(gmin), _p(gmax), _p(argmin),
                                         _p(argmax), _p(dx), _p(dv), _p(dg), _p(db))
    return dx, dv, dg, db


def evonorm_s0_fwd(x, v, gamma, beta, groups, eps):
    """EvoNorm-S0 in double.  Returns (y, gmean, gvar); statistics are [n,B,groups]."""
    x = _c(x, np.float32)
    n, B, H, W, Cc = x.shape
    v = _c(v, np.float32); gamma = _c(gamma, np.float32); beta = _c(beta, np.float32)
    y = np.zeros(x.shape, np.float64)
    gmean = np.zeros((n, B, groups), np.float64); gvar = np.zeros((n, B, groups), np.float64)
    lib().orc_evonorm_s0_fwd(n, B, H, W, Cc, groups, C.c_double(eps), _p(x), _p(v), _p(gamma), _p(beta), _p(y),
                             _p(gmean), _p(gvar))
    return y, gmean, gvar


def evonorm_s0_bwd(dy, x, v, gamma, gmean, gvar, groups, eps):
    """gmean, gvar: the stored fp32 statistics.  Returns (dx, dv, dgamma, dbeta) in double."""
    x = _c(x, np.float32); dy = _c(dy, np.float32)
    n, B, H, W, Cc = x.shape
    v = _c(v, np.float32); gamma = _c(gamma, np.float32)
    gmean = _c(gmean, np.float32); gvar = _c(gvar, np.float32)
    dx = np.zeros(x.shape, np.float64)
    dv = np.zeros((n, Cc), np.float64); dg = np.zeros((n, Cc), np.float64); db = np.zeros((n, Cc), np.float64)
    lib().orc_evonorm_s0_bwd(n, B, H, W, Cc, groups, C.c_double(eps), _p(dy), _p(x), _p(v), _p(gamma), _p(gmean),
                             _p(gvar), _p(dx), _p(dv), _p(dg), _p(db))
    return dx, dv, dg, db


def range_bn_fwd(x, gamma, beta, eps):
    """Range batch-norm in double.  Returns (y, cmean, cmin, cmax, argmin, argmax); statistics are [n,C]."""
    x = _c(x, np.float32)
    n, B, H, W, Cc = x.shape
    gamma = _c(gamma, np.float32); beta = _c(beta, np.float32)
    y = np.zeros(x.shape, np.float64)
    cmean = np.zeros((n, Cc), np.float64)
    cmin = np.zeros((n, Cc), np.float32); cmax = np.zeros((n, Cc), np.float32)
    amin = np.zeros((n, Cc), np.int32); amax = np.zeros((n, Cc), np.int32)
    lib().orc_range_bn_fwd(n, B, H, W, Cc, C.c_double(eps), _p(x), _p(gamma), _p(beta), _p(y), _p(cmean), _p(cmin),
                           _p(cmax), _p(amin), _p(amax))
    return y, cmean, cmin, cmax, amin, amax


def range_bn_bwd(dy, x, gamma, cmean, cmin, cmax, argmin, argmax, eps):
    """cmean: the stored fp32 mean.  Returns (dx, dgamma, dbeta) in double."""
    x = _c(x, np.float32); dy = _c(dy, np.float32)
    n, B, H, W, Cc = x.shape
    gamma = _c(gamma, np.float32); cmean = _c(cmean, np.float32)
    cmin = _c(cmin, np.float32); cmax = _c(cmax, np.float32)
    argmin = _c(argmin, np.int32); argmax = _c(argmax, np.int32)
    dx = np.zeros(x.shape, np.float64)
    dg = np.zeros((n, Cc), np.float64); db = np.zeros((n, Cc), np.float64)
    lib().orc_range_bn_bwd(n, B, H, W, Cc, C.c_double(eps), _p(dy), _p(x), _p(gamma), _p(cmean), _p(cmin), _p(cmax),
                           _p(argmin), _p(argmax), _p(dx), _p(dg), _p(db))
    return dx, dg, db


def gossip_mix(x_half, x_hat, Wmix, gamma, seg_offsets=None, seg_k=None):
    """x_half, x_hat fp32 [n,d]; Wmix [n,n].  Returns (x_out, x_hat_new, q)."""
    x_half = _c(x_half, np.float32)
    x_hat = np.array(x_hat, dtype=np.float32, order="C", copy=True)
    n, d = x_half.shape
    Wm = _c(Wmix, np.float32)
    if seg_offsets is None:
        seg_offsets = [0, d]
        seg_k = [d]
    so = _c(seg_offsets, np.int64)
    sk = _c(seg_k, np.int64)
    x_out = np.zeros((n, d), np.float32)
    q = np.zeros((n, d), np.float32)
    lib().orc_gossip_mix(C.c_int(n), _i64(d), _p(x_half), _p(x_hat), _p(x_out), _p(Wm),
                         C.c_float(gamma), C.c_int(len(sk)), _p(so), _p(sk), _p(q))
    return x_out, x_hat, q


def gossip_mix_q8(x_half, x_hat, Wmix, gamma, seg_offsets=None, seg_k=None):
    """Gossip step with 8-bit messages.  Returns (x_out, x_hat_new, q, codes int8 [n,d], scales fp32 [n,n_seg])."""
    x_half = _c(x_half, np.float32)
    x_hat = np.array(x_hat, dtype=np.float32, order="C", copy=True)
    n, d = x_half.shape
    Wm = _c(Wmix, np.float32)
    if seg_offsets is None:
        seg_offsets = [0, d]
        seg_k = [d]
    so = _c(seg_offsets, np.int64)
    sk = _c(seg_k, np.int64)
    x_out = np.zeros((n, d), np.float32)
    q = np.zeros((n, d), np.float32)
    codes = np.zeros((n, d), np.int8)
    scales = np.zeros((n, len(sk)), np.float32)
    lib().orc_gossip_mix_q8(C.c_int(n), _i64(d), _p(x_half), _p(x_hat), _p(x_out), _p(Wm),
                            C.c_float(gamma), C.c_int(len(sk)), _p(so), _p(sk), _p(q), _p(codes), _p(scales))
    return x_out, x_hat, q, codes, scales


def deepsqueeze_mix(x_half, delta, Wmix, eta, seg_offsets=None, seg_k=None, bits=32):
    """Deep-Squeeze gossip step.  Returns (x_out, delta_new, c, scales fp32 [n,n_seg])."""
    x_half = _c(x_half, np.float32)
    delta = np.array(delta, dtype=np.float32, order="C", copy=True)
    n, d = x_half.shape
    Wm = _c(Wmix, np.float32)
    if seg_offsets is None:
        seg_offsets = [0, d]
        seg_k = [d]
    so = _c(seg_offsets, np.int64)
    sk = _c(seg_k, np.int64)
    x_out = np.zeros((n, d), np.float32)
    c = np.zeros((n, d), np.float32)
    scales = np.zeros((n, len(sk)), np.float32)
    lib().orc_deepsqueeze_mix(C.c_int(n), _i64(d), _p(x_half), _p(delta), _p(x_out), _p(Wm), C.c_float(eta),
                              C.c_int(len(sk)), _p(so), _p(sk), C.c_int(bits), _p(c), _p(scales))
    return x_out, delta, c, scales


def pushsum_debias(x, u, Wmix, eta):
    """x fp32 [n,d], u fp32 [n].  Returns (u_new [n], z [n,d])."""
    x = _c(x, np.float32); u = _c(u, np.float32); Wm = _c(Wmix, np.float32)
    n, d = x.shape
    u_new = np.zeros(n, np.float32)
    z = np.zeros((n, d), np.float32)
    lib().orc_pushsum_debias(C.c_int(n), _i64(d), _p(x), _p(u), _p(Wm), C.c_float(eta), _p(u_new), _p(z))
    return u_new, z


def sgd_update(x, g, lr):
    x = _c(x, np.float32); g = _c(g, np.float32)
    out = np.zeros(x.shape, np.float32)
    lib().orc_sgd_update(_i64(x.size), _p(x), _p(g), C.c_float(lr), _p(out))
    return out


def residual_add(r, a, stride=1, ch_off=0):
    r = _c(r, np.float32); a = _c(a, np.float32)
    n, B, H, W, Ca = a.shape
    Cc = r.shape[-1]
    y = np.zeros(r.shape, np.float32)
    lib().orc_residual_add(n, B, H, W, Ca, Cc, stride, ch_off, _p(r), _p(a), _p(y))
    return y


def residual_add_bwd(dy, g_main, stride=1, ch_off=0):
    dy = _c(dy, np.float32); g_main = _c(g_main, np.float32)
    n, B, H, W, Ca = g_main.shape
    Cc = dy.shape[-1]
    da = np.zeros(g_main.shape, np.float32)
    lib().orc_residual_add_bwd(n, B, H, W, Ca, Cc, stride, ch_off, _p(dy), _p(g_main), _p(da))
    return da


def avgpool(x):
    x = _c(x, np.float32)
    n, B, H, W, Cc = x.shape
    y = np.zeros((n, B, Cc), np.float32)
    lib().orc_avgpool(n, B, H * W, Cc, _p(x), _p(y))
    return y


def avgpool_bwd(dy, H, W):
    dy = _c(dy, np.float32)
    n, B, Cc = dy.shape
    dx = np.zeros((n, B, H, W, Cc), np.float32)
    lib().orc_avgpool_bwd(n, B, H * W, Cc, _p(dy), _p(dx))
    return dx


def maxpool2x2(x):
    x = _c(x, np.float32)
    n, B, H, W, Cc = x.shape
    y = np.zeros((n, B, H // 2, W // 2, Cc), np.float32)
    idx = np.zeros(y.shape, np.int8)
    lib().orc_maxpool2x2(n, B, H, W, Cc, _p(x), _p(y), _p(idx))
    return y, idx


def maxpool2x2_bwd(dy, idx, H, W):
    dy = _c(dy, np.float32); idx = _c(idx, np.int8)
    n, B, _, _, Cc = dy.shape
    dx = np.zeros((n, B, H, W, Cc), np.float32)
    lib().orc_maxpool2x2_bwd(n, B, H, W, Cc, _p(dy), _p(idx), _p(dx))
    return dx


def softmax_ce(logits, labels):
    logits = _c(logits, np.float32); labels = _c(labels, np.int32)
    n, B, K = logits.shape
    loss = np.zeros(n, np.float32)
    dz = np.zeros(logits.shape, np.float32)
    lib().orc_softmax_ce(n, B, K, _p(logits), _p(labels), _p(loss), _p(dz))
    return loss, dz


def colsum(x):
    x = _c(x, np.float32)
    n, B, Cc = x.shape
    out = np.zeros((n, Cc), np.float32)
    lib().orc_colsum(n, B, Cc, _p(x), _p(out))
    return out
