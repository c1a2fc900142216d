"""Python binding of the lpdt C ABI: argument marshalling only.

Every function has the name of the C entry point it calls (include/lpdt.h),
takes torch CUDA tensors as device memory, and launches on torch's current
stream.  No arithmetic happens here.
"""
import ctypes as C

import torch

from ._lib import ConvDesc, lib


# Entry points that enqueue kernels (wrapped for the optional call log and per-call timing).
LAUNCHING = {"lpdt_quantize", "lpdt_quantize_with_range", "lpdt_quantize_static", "lpdt_quantize_batch", "lpdt_dequantize", "lpdt_qconv_fwd", "lpdt_qconv_fwd_affine", "lpdt_qconv_bwd_data_affine", "lpdt_qconv_bwd_weight_affine", "lpdt_qconv_bwd_data", "lpdt_qconv_bwd_weight", "lpdt_range_evonorm_fwd", "lpdt_range_evonorm_bwd", "lpdt_range_evonorm_fwd_q8", "lpdt_range_evonorm_bwd_q8", "lpdt_range_evonorm_bwd_params", "lpdt_range_evonorm_bwd_params_batch", "lpdt_dequantize_acc_batch", "lpdt_gossip_mix", "lpdt_gossip_mix_q8", "lpdt_deepsqueeze_mix", "lpdt_pushsum_debias", "lpdt_sgd_gossip_mix", "lpdt_evonorm_s0_fwd", "lpdt_evonorm_s0_bwd", "lpdt_range_bn_fwd", "lpdt_range_bn_bwd", "lpdt_sgd_update", "lpdt_residual_add", "lpdt_residual_add_bwd", "lpdt_avgpool", "lpdt_avgpool_bwd", "lpdt_maxpool2x2", "lpdt_maxpool2x2_bwd", "lpdt_softmax_ce", "lpdt_colsum", "lpdt_selftest_bounded_wait"}
# Kernel launches are counted inside the library (lpdt_launch_count); replays of a captured CUDA graph launch
# the recorded kernels again without passing through the library, so TrainStep.replay adds them here.
_REPLAYED = 0


def lpdt_launch_count():
    """Kernels enqueued by this thread through the library, plus those of graph replays."""
    return int(lib().lpdt_launch_count()) + _REPLAYED


def add_replayed_launches(n):
    global _REPLAYED
    _REPLAYED += int(n)

# Optional per-entry-point timing: {name: [(start_event, end_event), ...]} when TIMED holds names.
TIMED = set()
TIMINGS = {}


class LpdtError(RuntimeError):
    def __init__(self, fn, code):
        self.code = code
        super().__init__(f"{fn} failed: {lib().lpdt_status_string(code).decode()} ({code})")


def _check(fn, code):
    if code != 0:
        raise LpdtError(fn, code)


def timed(name):
    """Context manager: brackets the enclosed call with CUDA events on the current
    stream when `name` is in TIMED (used by the benchmark for the dominant kernel)."""
    return _Timed(name)


class _Timed:
    def __init__(self, name):
        self.on = name in TIMED
        self.name = name

    def __enter__(self):
        if self.on:
            self.a = torch.cuda.Event(enable_timing=True)
            self.b = torch.cuda.Event(enable_timing=True)
            self.a.record()

    def __exit__(self, *exc):
        if self.on:
            self.b.record()
            TIMINGS.setdefault(self.name, []).append((self.a, self.b))
        return False


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda, "device tensor expected"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _ws(ws):
    return (_ptr(ws), 0 if ws is None else ws.numel() * ws.element_size())


def lpdt_version():
    return lib().lpdt_version().decode()


def lpdt_last_kernel():
    return lib().lpdt_last_kernel().decode()


def conv_desc(nodes, B, H, W, Cin, Cout, R=3, S=3, stride=1, pad=1):
    return ConvDesc(nodes, B, H, W, Cin, Cout, R, S, stride, pad)


def lpdt_quantize_workspace_size(nodes):
    return lib().lpdt_quantize_workspace_size(nodes)


def lpdt_quantize(x, nodes, n_per_node, x_node_stride, q, scale, ws, mode=0, rounding=0, seed=0,
                  ctr_offset=0, zero_point=None):
    p, nb = _ws(ws)
    _check("lpdt_quantize", lib().lpdt_quantize(_ptr(x), nodes, n_per_node, x_node_stride, mode, rounding,
                                                seed, ctr_offset, _ptr(q), _ptr(scale), _ptr(zero_point),
                                                p, nb, _stream()))


def lpdt_quantize_with_range(x, nodes, n_per_node, x_node_stride, amax, q, scale, rounding=0, seed=0, ctr_offset=0):
    _check("lpdt_quantize_with_range", lib().lpdt_quantize_with_range(
        _ptr(x), nodes, n_per_node, x_node_stride, _ptr(amax), rounding, seed, ctr_offset, _ptr(q), _ptr(scale),
        _stream()))


def lpdt_fill_zero(t):
    _check("lpdt_fill_zero", lib().lpdt_fill_zero(_ptr(t), t.numel() * t.element_size(), _stream()))


def lpdt_check_status(dev_status):
    """Waits for the current stream and returns the status word (0 = ok); raises nothing."""
    return int(lib().lpdt_check_status(_ptr(dev_status), _stream()))


def lpdt_selftest_bounded_wait(limit_ns, dev_status, returned=None):
    _check("lpdt_selftest_bounded_wait", lib().lpdt_selftest_bounded_wait(int(limit_ns), _ptr(dev_status),
                                                                          _ptr(returned), _stream()))


def lpdt_message_bytes(d, seg_offsets, seg_k, value_bits=32, index_bits=32):
    """Bytes one node sends to each neighbour per gossip step (host arithmetic in the library)."""
    ns = len(seg_k)
    so = (C.c_int64 * (ns + 1))(*[int(v) for v in seg_offsets])
    sk = (C.c_int64 * ns)(*[int(v) for v in seg_k])
    return int(lib().lpdt_message_bytes(int(d), ns, C.addressof(so), C.addressof(sk), value_bits, index_bits))


def lpdt_quantize_batch_workspace_size(nodes, n_tensors):
    return lib().lpdt_quantize_batch_workspace_size(nodes, n_tensors)


def lpdt_quantize_batch(params, nodes, row_stride, src_offsets, sizes, dst_offsets, q, scales, ws):
    """src_offsets / sizes / dst_offsets: host sequences of Python ints (one entry per tensor)."""
    n = len(sizes)
    so = (C.c_int64 * n)(*[int(v) for v in src_offsets])
    sz = (C.c_int64 * n)(*[int(v) for v in sizes])
    do = (C.c_int64 * n)(*[int(v) for v in dst_offsets])
    p, nb = _ws(ws)
    _check("lpdt_quantize_batch", lib().lpdt_quantize_batch(_ptr(params), nodes, row_stride, n, C.addressof(so),
                                                            C.addressof(sz), C.addressof(do), _ptr(q), _ptr(scales),
                                                            p, nb, _stream()))


def lpdt_quantize_static(x, nodes, n_per_node, x_node_stride, q, scale, mode=0, rounding=0, seed=0,
                         ctr_offset=0, zero_point=None):
    """lpdt_quantize for callers without device scratch: the range words live inside the
    library.  At most 1024 nodes; calls that may overlap on the GPU must be ordered."""
    _check("lpdt_quantize_static", lib().lpdt_quantize_static(
        _ptr(x), nodes, n_per_node, x_node_stride, mode, rounding, seed, ctr_offset, _ptr(q), _ptr(scale),
        _ptr(zero_point), _stream()))


def lpdt_dequantize(q, nodes, n_per_node, scale, y, y_node_stride=None, zero_point=None):
    ys = n_per_node if y_node_stride is None else y_node_stride
    _check("lpdt_dequantize", lib().lpdt_dequantize(_ptr(q), nodes, n_per_node, _ptr(scale),
                                                    _ptr(zero_point), _ptr(y), ys, _stream()))


def lpdt_qconv_workspace_size(desc, which):
    return lib().lpdt_qconv_workspace_size(C.byref(desc), which)


def lpdt_qconv_fwd(desc, A, sA, Wq, sW, Y=None, Yacc=None, bias=None, bias_node_stride=0, ws=None,
                   dev_status=None):
    p, nb = _ws(ws)
    _check("lpdt_qconv_fwd", lib().lpdt_qconv_fwd(C.byref(desc), _ptr(A), _ptr(sA), _ptr(Wq), _ptr(sW),
                                                  _ptr(bias), bias_node_stride, _ptr(Y), _ptr(Yacc), p, nb,
                                                  _ptr(dev_status), _stream()))


def lpdt_qconv_fwd_affine_workspace_size(desc):
    return lib().lpdt_qconv_fwd_affine_workspace_size(C.byref(desc))


def lpdt_qconv_fwd_affine(desc, A, sA, zA, Wq, sW, zW, Y=None, Yacc=None, bias=None, bias_node_stride=0, ws=None,
                          dev_status=None):
    """Forward contraction on unsigned codes with per-node zero points (A, Wq uint8; zA, zW int32)."""
    p, nb = _ws(ws)
    _check("lpdt_qconv_fwd_affine", lib().lpdt_qconv_fwd_affine(
        C.byref(desc), _ptr(A), _ptr(sA), _ptr(zA), _ptr(Wq), _ptr(sW), _ptr(zW), _ptr(bias), bias_node_stride,
        _ptr(Y), _ptr(Yacc), p, nb, _ptr(dev_status), _stream()))


def lpdt_qconv_bwd_data_affine_workspace_size(desc):
    return lib().lpdt_qconv_bwd_data_affine_workspace_size(C.byref(desc))


def lpdt_qconv_bwd_data_affine(desc, E, sE, zE, Wq, sW, zW, dA=None, dAacc=None, ws=None, dev_status=None):
    """Backward-data contraction on unsigned codes with per-node zero points (E, Wq uint8; zE, zW int32)."""
    p, nb = _ws(ws)
    _check("lpdt_qconv_bwd_data_affine", lib().lpdt_qconv_bwd_data_affine(
        C.byref(desc), _ptr(E), _ptr(sE), _ptr(zE), _ptr(Wq), _ptr(sW), _ptr(zW), _ptr(dA), _ptr(dAacc), p, nb,
        _ptr(dev_status), _stream()))


def lpdt_qconv_bwd_weight_affine_workspace_size(desc):
    return lib().lpdt_qconv_bwd_weight_affine_workspace_size(C.byref(desc))


def lpdt_qconv_bwd_weight_affine(desc, E, sE, zE, A, sA, zA, dW=None, dw_node_stride=0, dWacc=None, ws=None,
                                 dev_status=None):
    """Backward-weight contraction on unsigned codes with per-node zero points (E, A uint8; zE, zA int32)."""
    p, nb = _ws(ws)
    _check("lpdt_qconv_bwd_weight_affine", lib().lpdt_qconv_bwd_weight_affine(
        C.byref(desc), _ptr(E), _ptr(sE), _ptr(zE), _ptr(A), _ptr(sA), _ptr(zA), _ptr(dW), dw_node_stride,
        _ptr(dWacc), p, nb, _ptr(dev_status), _stream()))


def lpdt_qconv_bwd_data(desc, E, sE, Wq, sW, dA=None, dAacc=None, ws=None, dev_status=None, addend=None):
    p, nb = _ws(ws)
    _check("lpdt_qconv_bwd_data", lib().lpdt_qconv_bwd_data(C.byref(desc), _ptr(E), _ptr(sE), _ptr(Wq),
                                                            _ptr(sW), _ptr(dA), _ptr(dAacc), _ptr(addend), p, nb,
                                                            _ptr(dev_status), _stream()))


def lpdt_qconv_bwd_weight(desc, E, sE, A, sA, dW=None, dw_node_stride=0, dWacc=None, ws=None,
                          dev_status=None):
    p, nb = _ws(ws)
    _check("lpdt_qconv_bwd_weight", lib().lpdt_qconv_bwd_weight(C.byref(desc), _ptr(E), _ptr(sE), _ptr(A),
                                                                _ptr(sA), _ptr(dW), dw_node_stride,
                                                                _ptr(dWacc), p, nb, _ptr(dev_status),
                                                                _stream()))


def lpdt_range_evonorm_fwd(nodes, B, H, W, Cc, groups, eps, x, v, gamma, beta, param_node_stride, y,
                           gmin, gmax, argmin, argmax, amax_out=None, res=None):
    _check("lpdt_range_evonorm_fwd", lib().lpdt_range_evonorm_fwd(
        nodes, B, H, W, Cc, groups, eps, _ptr(x), _ptr(v), _ptr(gamma), _ptr(beta), param_node_stride,
        _ptr(y), _ptr(gmin), _ptr(gmax), _ptr(argmin), _ptr(argmax), _ptr(amax_out), _ptr(res), _stream()))


def lpdt_range_evonorm_q8_ctl_size(nodes):
    return lib().lpdt_range_evonorm_q8_ctl_size(nodes)


def lpdt_range_evonorm_fwd_q8_fits(B, H, W, Cc, groups):
    return lib().lpdt_range_evonorm_fwd_q8_fits(B, H, W, Cc, groups)


def lpdt_range_evonorm_fwd_q8(nodes, B, H, W, Cc, groups, eps, x, v, gamma, beta, param_node_stride, y,
                              gmin, gmax, argmin, argmax, q, scale, ctl, amax_out=None, res=None, dev_status=None):
    c, cb = _ws(ctl)
    _check("lpdt_range_evonorm_fwd_q8", lib().lpdt_range_evonorm_fwd_q8(
        nodes, B, H, W, Cc, groups, eps, _ptr(x), _ptr(v), _ptr(gamma), _ptr(beta), param_node_stride,
        _ptr(y), _ptr(gmin), _ptr(gmax), _ptr(argmin), _ptr(argmax), _ptr(amax_out), _ptr(res), _ptr(q), _ptr(scale),
        c, cb, _ptr(dev_status), _stream()))


def lpdt_range_evonorm_bwd_q8_fits(B, H, W, Cc, groups):
    return lib().lpdt_range_evonorm_bwd_q8_fits(B, H, W, Cc, groups)


def lpdt_range_evonorm_bwd_q8(nodes, B, H, W, Cc, groups, eps, dy, x, v, gamma, param_node_stride, gmin,
                              gmax, argmin, argmax, q, scale, dv, dgamma, dbeta, grad_node_stride, ws, ctl,
                              amax_out=None, dev_status=None):
    p, nb = _ws(ws)
    c, cb = _ws(ctl)
    _check("lpdt_range_evonorm_bwd_q8", lib().lpdt_range_evonorm_bwd_q8(
        nodes, B, H, W, Cc, groups, eps, _ptr(dy), _ptr(x), _ptr(v), _ptr(gamma), param_node_stride,
        _ptr(gmin), _ptr(gmax), _ptr(argmin), _ptr(argmax), _ptr(q), _ptr(scale), _ptr(dv), _ptr(dgamma), _ptr(dbeta),
        grad_node_stride, _ptr(amax_out), p, nb, c, cb, _ptr(dev_status), _stream()))


def lpdt_range_evonorm_bwd_workspace_size(nodes, B, Cc):
    return lib().lpdt_range_evonorm_bwd_workspace_size(nodes, B, Cc)


def lpdt_range_evonorm_bwd(nodes, B, H, W, Cc, groups, eps, dy, x, v, gamma, param_node_stride, gmin,
                           gmax, argmin, argmax, dx, dv, dgamma, dbeta, grad_node_stride, ws, amax_out=None):
    p, nb = _ws(ws)
    _check("lpdt_range_evonorm_bwd", lib().lpdt_range_evonorm_bwd(
        nodes, B, H, W, Cc, groups, eps, _ptr(dy), _ptr(x), _ptr(v), _ptr(gamma), param_node_stride,
        _ptr(gmin), _ptr(gmax), _ptr(argmin), _ptr(argmax), _ptr(dx), _ptr(dv), _ptr(dgamma), _ptr(dbeta),
        grad_node_stride, _ptr(amax_out), p, nb, _stream()))


def lpdt_evonorm_s0_fwd(nodes, B, H, W, Cc, groups, eps, x, v, gamma, beta, param_node_stride, y, gmean, gvar):
    _check("lpdt_evonorm_s0_fwd", lib().lpdt_evonorm_s0_fwd(
        nodes, B, H, W, Cc, groups, eps, _ptr(x), _ptr(v), _ptr(gamma), _ptr(beta), param_node_stride, _ptr(y),
        _ptr(gmean), _ptr(gvar), _stream()))


def lpdt_evonorm_s0_bwd_workspace_size(nodes, B, Cc):
    return lib().lpdt_evonorm_s0_bwd_workspace_size(nodes, B, Cc)


def lpdt_evonorm_s0_bwd(nodes, B, H, W, Cc, groups, eps, dy, x, v, gamma, param_node_stride, gmean, gvar, dx, dv,
                        dgamma, dbeta, grad_node_stride, ws):
    p, nb = _ws(ws)
    _check("lpdt_evonorm_s0_bwd", lib().lpdt_evonorm_s0_bwd(
        nodes, B, H, W, Cc, groups, eps, _ptr(dy), _ptr(x), _ptr(v), _ptr(gamma), param_node_stride, _ptr(gmean),
        _ptr(gvar), _ptr(dx), _ptr(dv), _ptr(dgamma), _ptr(dbeta), grad_node_stride, p, nb, _stream()))


def lpdt_range_bn_workspace_size(nodes, Cc):
    return lib().lpdt_range_bn_workspace_size(nodes, Cc)


def lpdt_range_bn_fwd(nodes, B, H, W, Cc, eps, x, gamma, beta, param_node_stride, y, cmean, cmin, cmax, argmin, argmax,
                      ws):
    p, nb = _ws(ws)
    _check("lpdt_range_bn_fwd", lib().lpdt_range_bn_fwd(
        nodes, B, H, W, Cc, eps, _ptr(x), _ptr(gamma), _ptr(beta), param_node_stride, _ptr(y), _ptr(cmean), _ptr(cmin),
        _ptr(cmax), _ptr(argmin), _ptr(argmax), p, nb, _stream()))


def lpdt_range_bn_bwd(nodes, B, H, W, Cc, eps, dy, x, gamma, param_node_stride, cmean, cmin, cmax, argmin, argmax, dx,
                      dgamma, dbeta, grad_node_stride, ws):
    p, nb = _ws(ws)
    _check("lpdt_range_bn_bwd", lib().lpdt_range_bn_bwd(
        nodes, B, H, W, Cc, eps, _ptr(dy), _ptr(x), _ptr(gamma), param_node_stride, _ptr(cmean), _ptr(cmin), _ptr(cmax),
        _ptr(argmin), _ptr(argmax), _ptr(dx), _ptr(dgamma), _ptr(dbeta), grad_node_stride, p, nb, _stream()))


def lpdt_range_evonorm_bwd_params(nodes, B, Cc, ws, dv, dgamma, dbeta, grad_node_stride):
    """Second half of a backward call made with dv = dgamma = dbeta = None: adds the partial sums in ws."""
    p, nb = _ws(ws)
    _check("lpdt_range_evonorm_bwd_params", lib().lpdt_range_evonorm_bwd_params(
        nodes, B, Cc, p, nb, _ptr(dv), _ptr(dgamma), _ptr(dbeta), grad_node_stride, _stream()))


def lpdt_range_evonorm_bwd_params_batch(nodes, B, channels, workspaces, grad_offsets, grads, grad_node_stride):
    """channels / grad_offsets: host sequences of ints; workspaces: the layers' partial-sum tensors."""
    n = len(channels)
    cc = (C.c_int32 * n)(*[int(v) for v in channels])
    wp = (C.c_void_p * n)(*[_ptr(w) for w in workspaces])
    go = (C.c_int64 * n)(*[int(v) for v in grad_offsets])
    _check("lpdt_range_evonorm_bwd_params_batch", lib().lpdt_range_evonorm_bwd_params_batch(
        nodes, B, n, C.addressof(cc), C.addressof(wp), C.addressof(go), _ptr(grads), grad_node_stride, _stream()))


def lpdt_dequantize_acc_batch(acc, nodes, acc_offsets, sizes, out_offsets, s1, s2, out, out_node_stride):
    """acc_offsets / sizes / out_offsets: host sequences of ints; s1 / s2: sequences of per-node scale tensors,
    one pair per tensor."""
    n = len(sizes)
    af = (C.c_int64 * n)(*[int(v) for v in acc_offsets])
    sz = (C.c_int64 * n)(*[int(v) for v in sizes])
    of = (C.c_int64 * n)(*[int(v) for v in out_offsets])
    p1 = (C.c_void_p * n)(*[_ptr(t) for t in s1])
    p2 = (C.c_void_p * n)(*[_ptr(t) for t in s2])
    _check("lpdt_dequantize_acc_batch", lib().lpdt_dequantize_acc_batch(
        _ptr(acc), nodes, n, C.addressof(af), C.addressof(sz), C.addressof(of), C.addressof(p1), C.addressof(p2),
        _ptr(out), out_node_stride, _stream()))


def lpdt_gossip_mix_workspace_size(nodes, d, n_segments):
    return lib().lpdt_gossip_mix_workspace_size(nodes, d, n_segments)


def lpdt_gossip_mix(nodes, d, x_half, x_hat, x_out, Wmix, gamma, seg_offsets, seg_k, ws, dev_status=None):
    """seg_offsets / seg_k: host sequences of Python ints."""
    ns = len(seg_k)
    so = (C.c_int64 * (ns + 1))(*[int(v) for v in seg_offsets])
    sk = (C.c_int64 * ns)(*[int(v) for v in seg_k])
    p, nb = _ws(ws)
    _check("lpdt_gossip_mix", lib().lpdt_gossip_mix(nodes, d, _ptr(x_half), _ptr(x_hat), _ptr(x_out),
                                                    _ptr(Wmix), gamma, ns, C.addressof(so), C.addressof(sk),
                                                    p, nb, _ptr(dev_status), _stream()))


def lpdt_gossip_mix_q8(nodes, d, x_half, x_hat, x_out, Wmix, gamma, seg_offsets, seg_k, msg_scale, ws,
                       dev_status=None):
    """Gossip step with 8-bit messages; msg_scale fp32 [nodes][len(seg_k)] receives the steps sent."""
    ns = len(seg_k)
    so = (C.c_int64 * (ns + 1))(*[int(v) for v in seg_offsets])
    sk = (C.c_int64 * ns)(*[int(v) for v in seg_k])
    p, nb = _ws(ws)
    _check("lpdt_gossip_mix_q8", lib().lpdt_gossip_mix_q8(nodes, d, _ptr(x_half), _ptr(x_hat), _ptr(x_out),
                                                          _ptr(Wmix), gamma, ns, C.addressof(so), C.addressof(sk),
                                                          _ptr(msg_scale), p, nb, _ptr(dev_status), _stream()))


def lpdt_deepsqueeze_mix(nodes, d, x_half, delta, x_out, Wmix, eta, seg_offsets, seg_k, ws, message_bits=32,
                         msg_scale=None, dev_status=None):
    """Deep-Squeeze gossip step; delta [nodes][d] is the error buffer (in/out)."""
    ns = len(seg_k)
    so = (C.c_int64 * (ns + 1))(*[int(v) for v in seg_offsets])
    sk = (C.c_int64 * ns)(*[int(v) for v in seg_k])
    p, nb = _ws(ws)
    _check("lpdt_deepsqueeze_mix", lib().lpdt_deepsqueeze_mix(nodes, d, _ptr(x_half), _ptr(delta), _ptr(x_out),
                                                              _ptr(Wmix), eta, ns, C.addressof(so), C.addressof(sk),
                                                              message_bits, _ptr(msg_scale), p, nb, _ptr(dev_status),
                                                              _stream()))


def lpdt_sgd_gossip_mix(nodes, d, x, g, lr, x_half, x_hat, x_out, Wmix, gamma):
    """SGD half-step + uncompressed gossip step in one launch."""
    _check("lpdt_sgd_gossip_mix", lib().lpdt_sgd_gossip_mix(nodes, d, _ptr(x), _ptr(g), lr, _ptr(x_half), _ptr(x_hat),
                                                            _ptr(x_out), _ptr(Wmix), gamma, _stream()))


def lpdt_pushsum_debias(nodes, d, x, u, Wmix, eta, u_new, z):
    """Push-sum bias-weight update and de-biased model z = x / u_new."""
    _check("lpdt_pushsum_debias", lib().lpdt_pushsum_debias(nodes, d, _ptr(x), _ptr(u), _ptr(Wmix), eta, _ptr(u_new),
                                                            _ptr(z), _stream()))


def lpdt_sgd_update(n, x, g, lr, out):
    _check("lpdt_sgd_update", lib().lpdt_sgd_update(n, _ptr(x), _ptr(g), lr, _ptr(out), _stream()))


def lpdt_residual_add(nodes, B, H, W, Ca, Cc, stride, ch_off, r, a, y, amax_out=None):
    _check("lpdt_residual_add", lib().lpdt_residual_add(nodes, B, H, W, Ca, Cc, stride, ch_off, _ptr(r),
                                                        _ptr(a), _ptr(y), _ptr(amax_out), _stream()))


def lpdt_residual_add_bwd(nodes, B, H, W, Ca, Cc, stride, ch_off, dy, g_main, da):
    _check("lpdt_residual_add_bwd", lib().lpdt_residual_add_bwd(nodes, B, H, W, Ca, Cc, stride, ch_off,
                                                                _ptr(dy), _ptr(g_main), _ptr(da), _stream()))


def lpdt_avgpool(nodes, B, HW, Cc, x, y):
    _check("lpdt_avgpool", lib().lpdt_avgpool(nodes, B, HW, Cc, _ptr(x), _ptr(y), _stream()))


def lpdt_avgpool_bwd(nodes, B, HW, Cc, dy, dx):
    _check("lpdt_avgpool_bwd", lib().lpdt_avgpool_bwd(nodes, B, HW, Cc, _ptr(dy), _ptr(dx), _stream()))


def lpdt_maxpool2x2(nodes, B, H, W, Cc, x, y, idx):
    _check("lpdt_maxpool2x2", lib().lpdt_maxpool2x2(nodes, B, H, W, Cc, _ptr(x), _ptr(y), _ptr(idx), _stream()))


def lpdt_maxpool2x2_bwd(nodes, B, H, W, Cc, dy, idx, dx):
    _check("lpdt_maxpool2x2_bwd", lib().lpdt_maxpool2x2_bwd(nodes, B, H, W, Cc, _ptr(dy), _ptr(idx), _ptr(dx),
                                                            _stream()))


def lpdt_softmax_ce(nodes, B, K, logits, labels, loss, dlogits, dev_status=None):
    _check("lpdt_softmax_ce", lib().lpdt_softmax_ce(nodes, B, K, _ptr(logits), _ptr(labels), _ptr(loss),
                                                    _ptr(dlogits), _ptr(dev_status), _stream()))


def lpdt_colsum(nodes, B, Cc, x, out, out_node_stride):
    _check("lpdt_colsum", lib().lpdt_colsum(nodes, B, Cc, _ptr(x), _ptr(out), out_node_stride, _stream()))


# Optional call log: while RECORD is a list, every entry-point call appends (name, function, args, kwargs,
# contraction kernel launched or "", node group).  The logged calls can be re-issued later on the same buffers, which is
# how the benchmark times one kind of call of a whole step in isolation.
RECORD = None
GROUP = 0          # node group whose calls are being issued (set by TrainStep; logged with every call)


def _with_timing(fn):
    name = fn.__name__

    def call(*a, **kw):
        if RECORD is not None:
            r = fn(*a, **kw)
            RECORD.append((name, fn, a, kw, lpdt_last_kernel() if name.startswith("lpdt_qconv") else "", GROUP))
            return r
        if name in TIMED:
            with timed(name):
                return fn(*a, **kw)
        return fn(*a, **kw)

    call.__name__ = name
    call.__doc__ = fn.__doc__
    return call


for _n in [n for n in list(globals()) if n in LAUNCHING or n == "lpdt_fill_zero"]:
    globals()[_n] = _with_timing(globals()[_n])
del _n
