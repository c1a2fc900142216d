"""One full 8-bit training step of every simulated node, composed from the
oracle's primitives.  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The step follows Algorithm 1 / Algorithm 3 and Section 3 "Low Precision
Training" of arXiv 2111.09389:
  forward : every conv/linear quantizes its input activation and its weights
            to 8 bit (one range per tensor per node), runs the integer
            contraction and dequantizes; Range-EvoNorm follows in fp32.
  backward: the incoming layer gradient is quantized to 8 bit once per layer
            and feeds both adjoint contractions (layer gradient for the
            previous layer, weight gradient); weight gradients stay fp32
            ("gradient bifurcation"); the quantizer's derivative is taken as
            the identity (straight-through).
  update  : x_half = x - lr*g ; compress x_half - x_hat ; update x_hat ; mix.

Values that feed a quantizer are computed in the kernels' precision: fixed
sequences of fp32 operations with double-accumulated reductions.
"""
import numpy as np

import oracle as orc


def _view(params, off, shape):
    n = int(np.prod(shape))
    return np.ascontiguousarray(params[:, off:off + n]).reshape((params.shape[0],) + tuple(shape))


def forward_backward(ops, params, x, labels=None, dy=None, eps=1e-5, grad_rounding=0, seed=0,
                     quantize_wgrad=False, input_grad=False, keep=None):
    """Returns (grads [N,d] fp32, loss [N] or None, extras dict).

    keep: optional dict that receives intermediate tensors by name for tests."""
    nodes, B = x.shape[0], x.shape[1]
    d = params.shape[1]
    grads = np.zeros((nodes, d), np.float32)
    tape = []
    saved = []
    cur = np.ascontiguousarray(x, np.float32)
    for li, op in enumerate(ops):
        kind = op["op"]
        if kind in ("conv", "linear"):
            if kind == "linear":
                R = S = 1; stride = 1; pad = 0
                cur = cur.reshape(nodes, B, 1, 1, op["cin"])
            else:
                R, S, stride, pad = op["R"], op["S"], op["stride"], op["pad"]
            Wf = _view(params, op["w_off"], (op["cout"], R, S, op["cin"]))
            qA, sA = orc.quantize_sym_s8(cur)
            qW, sW = orc.quantize_sym_s8(Wf)
            acc, ovf = orc.qconv_fwd(qA, qW, stride, pad)
            assert ovf == 0
            bias = params[:, op["b_off"]:op["b_off"] + op["cout"]] if kind == "linear" else None
            tape.append((qA, sA, qW, sW, cur.shape))
            cur = orc.dequant_acc(acc, sA, sW, bias)
            if keep is not None:
                keep[f"acc{li}"] = acc
        elif kind == "ren":
            C = op["C"]
            v = params[:, op["p_off"]:op["p_off"] + C]
            g = params[:, op["p_off"] + C:op["p_off"] + 2 * C]
            b = params[:, op["p_off"] + 2 * C:op["p_off"] + 3 * C]
            y, mn, mx, amn, amx = orc.range_evonorm_fwd(cur, v, g, b, op["groups"], eps, "f32")
            tape.append((cur, mn, mx, amn, amx))
            cur = y
        elif kind == "save":
            saved.append(cur)
            tape.append(None)
        elif kind == "add":
            a = saved.pop()
            cur = orc.residual_add(cur, a, op["stride"], op["ch_off"])
            tape.append(None)
        elif kind == "maxpool":
            y, idx = orc.maxpool2x2(cur)
            tape.append((idx, cur.shape))
            cur = y
        elif kind == "avgpool":
            tape.append(cur.shape)
            cur = orc.avgpool(cur).reshape(nodes, B, 1, 1, op["C"])
        else:
            raise ValueError(kind)
        if keep is not None:
            keep[f"out{li}"] = cur

    loss = None
    if dy is None:
        logits = cur.reshape(nodes, B, -1)
        loss, g = orc.softmax_ce(logits, labels)
        g = g.reshape(cur.shape)
    else:
        g = np.ascontiguousarray(dy, np.float32)

    sc_grads = []
    ctr = 0
    for li in range(len(ops) - 1, -1, -1):
        op = ops[li]
        kind = op["op"]
        t = tape[li]
        if kind in ("conv", "linear"):
            qA, sA, qW, sW, in_shape = t
            if kind == "linear":
                R = S = 1; stride = 1; pad = 0
                g = g.reshape(nodes, B, 1, 1, op["cout"])
                grads[:, op["b_off"]:op["b_off"] + op["cout"]] = orc.colsum(g.reshape(nodes, B, -1))
            else:
                R, S, stride, pad = op["R"], op["S"], op["stride"], op["pad"]
            E, sE = orc.quantize_sym_s8(g, grad_rounding, seed, ctr)
            ctr += 1
            if keep is not None:
                keep[f"E{li}"] = E
            dWacc, ovf = orc.qconv_bwd_weight(E, qA, R, S, stride, pad)
            assert ovf == 0
            dW = orc.dequant_acc(dWacc, sE, sA)
            if quantize_wgrad:
                qg, sg = orc.quantize_sym_s8(dW)
                dW = orc.dequantize(qg, sg)
            n = op["cout"] * R * S * op["cin"]
            grads[:, op["w_off"]:op["w_off"] + n] = dW.reshape(nodes, n)
            if li > 0 or input_grad:
                dAacc, ovf = orc.qconv_bwd_data(E, qW, in_shape[2], in_shape[3], stride, pad)
                assert ovf == 0
                g = orc.dequant_acc(dAacc, sE, sW)
            else:
                g = None
        elif kind == "ren":
            C = op["C"]
            xin, mn, mx, amn, amx = t
            v = params[:, op["p_off"]:op["p_off"] + C]
            gam = params[:, op["p_off"] + C:op["p_off"] + 2 * C]
            dx, dv, dg, db = orc.range_evonorm_bwd(g, xin, v, gam, mn, mx, amn, amx,
                                                   op["groups"], eps, "f32")
            grads[:, op["p_off"]:op["p_off"] + C] = dv
            grads[:, op["p_off"] + C:op["p_off"] + 2 * C] = dg
            grads[:, op["p_off"] + 2 * C:op["p_off"] + 3 * C] = db
            g = dx
        elif kind == "add":
            sc_grads.append(g)
        elif kind == "save":
            add_op = next(o for o in ops[li:] if o["op"] == "add")
            g = orc.residual_add_bwd(sc_grads.pop(), g, add_op["stride"], add_op["ch_off"])
        elif kind == "maxpool":
            idx, shp = t
            g = orc.maxpool2x2_bwd(g, idx, shp[2], shp[3])
        elif kind == "avgpool":
            shp = t
            g = orc.avgpool_bwd(g.reshape(nodes, B, -1), shp[2], shp[3])
        if keep is not None and g is not None:
            keep[f"grad_in{li}"] = g
    return grads, loss, dict(input_grad=g)


def train_step(wl, grad_rounding=0, seed=0, quantize_wgrad=False, keep=None, message_bits=32):
    """Whole step on a workload dict (see the workloads module); message_bits = 8 sends the gossip
    messages as 8-bit codes.  Returns dict(grads, loss, x_half, x_hat, x, q)."""
    grads, loss, extra = forward_backward(
        wl["ops"], wl["params"], wl["x"], wl.get("labels"), wl.get("dy"), wl["ren_eps"],
        grad_rounding, seed, quantize_wgrad, input_grad=("dy" in wl), keep=keep)
    x_half = orc.sgd_update(wl["params"], grads, wl["lr"])
    if message_bits == 8:
        x, x_hat, q, _, _ = orc.gossip_mix_q8(x_half, wl["x_hat"], wl["Wmix"], wl["gamma"],
                                              wl["seg_offsets"], wl["seg_k"])
    else:
        x, x_hat, q = orc.gossip_mix(x_half, wl["x_hat"], wl["Wmix"], wl["gamma"],
                                     wl["seg_offsets"], wl["seg_k"])
    return dict(grads=grads, loss=loss, x_half=x_half, x_hat=x_hat, x=x, q=q,
                input_grad=extra["input_grad"])
