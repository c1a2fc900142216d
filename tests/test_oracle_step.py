"""Pins for the oracle's whole-step composition (no GPU): the 8-bit step must
track an unquantized fp64 autograd model of the same network closely, and the
parameter bookkeeping must match the paper's parameter counts."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import step as ostep
from paper_2111_09389_b200 import workloads as wlmod


def test_parameter_counts_match_paper():
    # Table "baseline": ResNet-20 has 0.27 M parameters
    ops, d = wlmod.resnet20_ops()
    assert d == 270410 and round(d / 1e6, 2) == 0.27
    assert sum(1 for o in ops if o["op"] == "conv") == 19
    # forward MACs per image, Conv/Linear rows of the operation-count table
    assert wlmod.conv_macs(ops, 1) == 442368 + 14155776 + 2 * 12976128 + 640
    ops, d = wlmod.vgg11_ops()
    assert sum(1 for o in ops if o["op"] == "conv") == 8
    assert abs(d / 1e6 - 9.23) < 0.01


def _torch_ren(x, v, g, b, groups, eps):
    # x: [B,H,W,C] double
    B, H, W, C = x.shape
    cpg = C // groups
    xg = x.reshape(B, H * W, groups, cpg)
    rng = xg.amax(dim=(1, 3), keepdim=True) - xg.amin(dim=(1, 3), keepdim=True)
    D = rng / np.sqrt(2 * np.log(cpg)) + eps
    hs = torch.clamp((v.reshape(1, 1, groups, cpg) * xg + 3) / 6, 0, 1)
    y = xg * hs / D * g.reshape(1, 1, groups, cpg) + b.reshape(1, 1, groups, cpg)
    return y.reshape(B, H, W, C)


def _torch_model(ops, p, x, labels=None, dy=None, eps=1e-5):
    """Unquantized fp64 model of one node; p: flat parameter tensor requiring grad."""
    cur = x
    saved = []
    for op in ops:
        k = op["op"]
        if k == "conv":
            n = op["cout"] * op["R"] * op["S"] * op["cin"]
            w = p[op["w_off"]:op["w_off"] + n].reshape(op["cout"], op["R"], op["S"], op["cin"])
            cur = F.conv2d(cur.permute(0, 3, 1, 2), w.permute(0, 3, 1, 2), stride=op["stride"],
                           padding=op["pad"]).permute(0, 2, 3, 1)
        elif k == "ren":
            C = op["C"]; o = op["p_off"]
            cur = _torch_ren(cur, p[o:o + C], p[o + C:o + 2 * C], p[o + 2 * C:o + 3 * C],
                             op["groups"], eps)
        elif k == "save":
            saved.append(cur)
        elif k == "add":
            a = saved.pop()[:, ::op["stride"], ::op["stride"], :]
            lo = op["ch_off"]; hi = op["C"] - op["Ca"] - lo
            cur = cur + F.pad(a, (lo, hi))
        elif k == "maxpool":
            cur = F.max_pool2d(cur.permute(0, 3, 1, 2), 2).permute(0, 2, 3, 1)
        elif k == "avgpool":
            cur = cur.mean(dim=(1, 2), keepdim=True)
        elif k == "linear":
            w = p[op["w_off"]:op["w_off"] + op["cout"] * op["cin"]].reshape(op["cout"], op["cin"])
            cur = cur.reshape(cur.shape[0], -1) @ w.T + p[op["b_off"]:op["b_off"] + op["cout"]]
    if dy is not None:
        return (cur * dy).sum()
    return F.cross_entropy(cur, labels)


def _cos(a, b):
    a = a.ravel().astype(np.float64); b = b.ravel().astype(np.float64)
    return float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b) + 1e-300))


def test_conv16_step_tracks_float_model():
    wl = wlmod.make_workload("conv16")
    out = ostep.train_step(wl)
    for n in range(wl["nodes"]):
        p = torch.tensor(wl["params"][n], dtype=torch.float64, requires_grad=True)
        xin = torch.tensor(wl["x"][n], dtype=torch.float64, requires_grad=True)
        L = _torch_model(wl["ops"], p, xin, dy=torch.tensor(wl["dy"][n], dtype=torch.float64))
        L.backward()
        gref = p.grad.numpy()
        op = wl["ops"][0]
        nw = 16 * 9 * 16
        assert _cos(out["grads"][n, :nw], gref[:nw]) > 0.995              # weight gradient
        assert _cos(out["grads"][n, nw:], gref[nw:]) > 0.995              # v, gamma, beta
        assert _cos(out["input_grad"][n], xin.grad.numpy()) > 0.995       # layer gradient
        rel = np.linalg.norm(out["grads"][n] - gref) / np.linalg.norm(gref)
        assert rel < 0.1
    # update and gossip are composed from the step's own gradient
    assert np.array_equal(out["x_half"], oracle.sgd_update(wl["params"], out["grads"], wl["lr"]))
    assert np.array_equal(out["x_hat"], out["x_half"])                     # dense, x_hat was 0
    assert np.allclose(out["x"], wl["Wmix"].astype(np.float64) @ out["x_half"], atol=1e-6)


def test_conv16_weight_gradient_quantization_option():
    wl = wlmod.make_workload("conv16", nodes=1, batch=2)
    a = ostep.train_step(wl)
    b = ostep.train_step(wl, quantize_wgrad=True)
    nw = 16 * 9 * 16
    ga, gb = a["grads"][0, :nw], b["grads"][0, :nw]
    step = np.abs(ga).max() / 127
    assert np.all(np.abs(ga - gb) <= 0.5 * step * (1 + 1e-5)) and not np.array_equal(ga, gb)
    assert np.array_equal(a["grads"][0, nw:], b["grads"][0, nw:])


@pytest.mark.parametrize("name", ["resnet20", "vgg11"])
def test_network_step_tracks_float_model(name):
    wl = wlmod.make_workload(name, nodes=2, batch=4)
    out = ostep.train_step(wl)
    assert out["loss"].shape == (2,)
    for n in range(2):
        p = torch.tensor(wl["params"][n], dtype=torch.float64, requires_grad=True)
        L = _torch_model(wl["ops"], p, torch.tensor(wl["x"][n], dtype=torch.float64),
                         labels=torch.tensor(wl["labels"][n], dtype=torch.long))
        L.backward()
        assert abs(float(L.detach()) - float(out["loss"][n])) < 0.05 * max(1.0, float(L.detach()))
        gref = p.grad.numpy()
        # 8-bit noise accumulates over ~20 layers; direction must still agree per tensor
        last = [o for o in wl["ops"] if o["op"] == "linear"][0]
        sl = slice(last["w_off"], last["w_off"] + last["cin"] * last["cout"])
        assert _cos(out["grads"][n, sl], gref[sl]) > 0.98
        first = wl["ops"][0]
        sl = slice(0, first["cout"] * 9 * first["cin"])
        assert _cos(out["grads"][n, sl], gref[sl]) > 0.8
        assert _cos(out["grads"][n], gref) > 0.9


def test_layerwise_topk_segments_tile_the_parameters():
    """Layer-wise top-K: one segment per conv/linear layer, tiling the flat parameter vector; the oracle
    step keeps exactly seg_k entries of every (node, segment)."""
    wl = wlmod.make_workload("resnet20_topk_layerwise", nodes=3, batch=2)
    off, k = wl["seg_offsets"], wl["seg_k"]
    assert off[0] == 0 and off[-1] == wl["d"] and (np.diff(off) > 0).all() and len(k) == 20
    starts = [op["w_off"] for op in wl["ops"] if op["op"] in ("conv", "linear")]
    assert list(off[:-1]) == starts
    ref = ostep.train_step(wl)
    for s in range(len(k)):
        for i in range(3):
            assert np.count_nonzero(ref["q"][i][off[s]:off[s + 1]]) == k[s]
    assert np.array_equal(ref["x_hat"], (wl["x_hat"] + ref["q"]).astype(np.float32))
