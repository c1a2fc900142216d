"""GPU parity: every lpdt entry point against the CPU oracle on the same seeded
inputs, through the C ABI.  Integer results bit-exact; fp32 results within
1e-5 relative / 1e-6 absolute."""
import numpy as np
import pytest
import torch

import oracle
from paper_2111_09389_b200 import api, workloads as wlmod

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, want, rtol=RTOL, atol=ATOL):
    got = got.cpu().numpy() if isinstance(got, torch.Tensor) else got
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got.astype(np.float64) - want)
    ok = err <= atol + rtol * np.abs(want)
    assert ok.all(), f"{(~ok).sum()} of {ok.size} outside tolerance, worst {err.max():.3e}"


def ws_bytes(n):
    return torch.empty(max(int(n), 256), dtype=torch.uint8, device="cuda")


# ------------------------------------------------------------------ quantizer
@pytest.mark.parametrize("nodes,n", [(1, 1), (3, 7), (4, 4096), (2, 100003), (16, 98304), (1, 1 << 22)])
@pytest.mark.parametrize("rounding", [0, 1])
def test_quantize_sym(nodes, n, rounding):
    rng = np.random.default_rng(n + rounding)
    x = (rng.standard_normal((nodes, n)) * rng.uniform(0.01, 100, (nodes, 1))).astype(np.float32)
    q_ref, s_ref = oracle.quantize_sym_s8(x, rounding, seed=(9 << 32) | 77, ctr_offset=3)
    xd = dev(x)
    q = torch.empty(nodes, n, dtype=torch.int8, device="cuda")
    s = torch.empty(nodes, dtype=torch.float32, device="cuda")
    ws = ws_bytes(api.lpdt_quantize_workspace_size(nodes))
    api.lpdt_quantize(xd, nodes, n, n, q, s, ws, mode=0, rounding=rounding, seed=(9 << 32) | 77, ctr_offset=3)
    assert np.array_equal(s.cpu().numpy(), s_ref)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    y = torch.empty(nodes, n, dtype=torch.float32, device="cuda")
    api.lpdt_dequantize(q, nodes, n, s, y)
    assert np.array_equal(y.cpu().numpy(), oracle.dequantize(q_ref, s_ref))


def test_quantize_strided_rows_zero_tensor_and_ties():
    # rows inside a wider flat vector (odd stride -> scalar path), an all-zero node, exact ties
    rng = np.random.default_rng(0)
    nodes, n, stride = 3, 432, 1001
    flat = rng.standard_normal((nodes, stride)).astype(np.float32)
    flat[1, 5:5 + n] = 0.0
    flat[2, 5:5 + n] = np.round(flat[2, 5:5 + n] * 4) / 8      # many .5 ties once scaled
    flat[2, 5] = 127.0 / 2
    q_ref, s_ref = oracle.quantize_sym_s8(flat[:, 5:5 + n])
    fd = dev(flat)
    q = torch.empty(nodes, n, dtype=torch.int8, device="cuda")
    s = torch.empty(nodes, dtype=torch.float32, device="cuda")
    api.lpdt_quantize(fd[:, 5:], nodes, n, stride, q, s, ws_bytes(256))
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)
    assert s_ref[1] == 1.0 and not q_ref[1].any()


@pytest.mark.parametrize("nodes,n", [(2, 1001), (3, 65536)])
def test_quantize_affine(nodes, n):
    rng = np.random.default_rng(n)
    x = rng.uniform(-1, 3, (nodes, n)).astype(np.float32)
    x[-1] = np.abs(x[-1]) + 0.5                                  # one-sided node
    q_ref, s_ref, z_ref = oracle.quantize_affine_u8(x)
    q = torch.empty(nodes, n, dtype=torch.int8, device="cuda")
    s = torch.empty(nodes, dtype=torch.float32, device="cuda")
    zp = torch.empty(nodes, dtype=torch.int32, device="cuda")
    api.lpdt_quantize(dev(x), nodes, n, n, q, s, ws_bytes(256), mode=1, zero_point=zp)
    assert np.array_equal(q.cpu().numpy().view(np.uint8), q_ref)
    assert np.array_equal(s.cpu().numpy(), s_ref) and np.array_equal(zp.cpu().numpy(), z_ref)
    y = torch.empty(nodes, n, dtype=torch.float32, device="cuda")
    api.lpdt_dequantize(q, nodes, n, s, y, zero_point=zp)
    assert np.array_equal(y.cpu().numpy(), oracle.dequantize(q_ref, s_ref, z_ref))


def test_quantize_batch_matches_per_tensor_calls():
    rng = np.random.default_rng(11)
    nodes, d = 5, 20011
    params = (rng.standard_normal((nodes, d)) * rng.uniform(0.01, 3, (nodes, 1))).astype(np.float32)
    src = [0, 432, 433, 5000, 15003]; size = [432, 1, 2304, 9216, 5008]
    params[2, 432] = 0.0                                   # an all-zero single-element tensor on one node
    dst, off = [], 0
    for n in size:
        dst.append(off); off += (nodes * n + 255) // 256 * 256
    q = torch.full((off,), 99, dtype=torch.int8, device="cuda")
    sc = torch.zeros(len(size), nodes, device="cuda")
    ws = ws_bytes(api.lpdt_quantize_batch_workspace_size(nodes, len(size)))
    api.lpdt_quantize_batch(dev(params), nodes, d, src, size, dst, q, sc, ws)
    qh, sh = q.cpu().numpy(), sc.cpu().numpy()
    for t, (o, n, do) in enumerate(zip(src, size, dst)):
        q_ref, s_ref = oracle.quantize_sym_s8(params[:, o:o + n])
        assert np.array_equal(sh[t], s_ref)
        assert np.array_equal(qh[do:do + nodes * n].reshape(nodes, n), q_ref)
    assert sh[1, 2] == 1.0


def test_quantize_argument_errors():
    x = torch.zeros(8, device="cuda")
    q = torch.zeros(8, dtype=torch.int8, device="cuda")
    s = torch.zeros(1, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_quantize(x, 1, 8, 8, q, s, None)
    assert e.value.code == 3
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_quantize(None, 1, 8, 8, q, s, ws_bytes(256))
    assert e.value.code == 1
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_quantize(x, 1, 8, 8, q, s, ws_bytes(256), mode=1)     # affine without zero_point
    assert e.value.code == 1
    api.lpdt_quantize(x, 0, 8, 8, q, s, None)                          # empty: no-op


# ------------------------------------------------------------------ contractions
CONV_CASES = [
    # nodes, B, H, W, Cin, Cout, R, S, stride, pad
    (4, 8, 16, 16, 16, 16, 3, 3, 1, 1),      # the single-layer workload
    (2, 3, 32, 32, 3, 16, 3, 3, 1, 1),       # first layer of the networks
    (2, 2, 16, 16, 16, 32, 3, 3, 2, 1),      # strided stage transition
    (1, 2, 9, 7, 5, 6, 3, 3, 1, 1),          # ragged everything
    (2, 4, 8, 8, 64, 64, 3, 3, 1, 1),
    (1, 1, 12, 12, 32, 48, 1, 1, 1, 0),      # 1x1
    (3, 32, 1, 1, 64, 10, 1, 1, 1, 0),       # classifier
    (1, 5, 4, 4, 8, 8, 3, 3, 1, 0),          # no padding
    (1, 2, 40, 24, 128, 64, 3, 3, 1, 1),
    (2, 3, 32, 32, 32, 64, 3, 3, 2, 1),      # strided, tensor-core path
    (1, 2, 15, 13, 16, 16, 3, 3, 2, 1),      # strided with odd image sizes
    (1, 2, 16, 16, 32, 32, 1, 1, 2, 0),      # strided 1x1: three of four input parities get no tap
    (1, 1, 56, 56, 64, 64, 3, 3, 1, 1),      # image width that no power-of-two tile divides
    (1, 3, 7, 7, 16, 32, 5, 5, 1, 2),        # 5x5 filter
    (2, 40, 1, 1, 256, 128, 1, 1, 1, 0),     # linear layer on the tensor-core path
    (1, 130, 1, 1, 512, 272, 1, 1, 1, 0),    # linear: ragged row tile, two N tiles (272 = 16*17)
    (1, 1, 4, 4, 512, 512, 3, 3, 1, 1),      # wide channels on a tiny map
    (3, 5, 32, 32, 16, 16, 3, 3, 1, 1),      # 16-channel halo-tile path, several nodes per CTA range
    (2, 3, 19, 13, 16, 48, 3, 3, 1, 1),      # halo path: ragged image, 16 -> 48 channels
    (2, 2, 20, 20, 48, 16, 3, 3, 1, 1),      # halo path on the backward-data side (Cout = 16)
    (1, 2, 17, 9, 16, 16, 5, 4, 1, 2),       # halo path: 5x4 filter (even tap count), asymmetric padding effect
    (1, 2, 12, 12, 16, 32, 1, 1, 1, 0),      # halo path with a single tap
    (2, 2, 10, 10, 16, 16, 3, 3, 1, 0),      # halo path without padding
    (2, 3, 16, 16, 32, 32, 3, 3, 1, 1),      # halo path with two 16-channel chunks
    (2, 5, 8, 8, 64, 64, 3, 3, 1, 1),        # halo path: 8x8 maps (half of each tile is outside the image)
    (1, 2, 13, 11, 96, 32, 3, 3, 1, 1),      # halo path: 6 chunks forward, 2 chunks backward
    (1, 2, 9, 20, 128, 128, 3, 3, 1, 1),     # halo path at its channel limit
]


def _conv_inputs(case, seed=0):
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    rng = np.random.default_rng(seed)
    A = wlmod.random_s8(rng, (nodes, B, H, W, Cin))
    Wq = wlmod.random_s8(rng, (nodes, Cout, R, S, Cin))
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    E = wlmod.random_s8(rng, (nodes, B, Ho, Wo, Cout))
    s1 = rng.uniform(0.001, 0.1, nodes).astype(np.float32)
    s2 = rng.uniform(0.001, 0.1, nodes).astype(np.float32)
    return A, Wq, E, s1, s2


@pytest.mark.parametrize("case", CONV_CASES)
def test_qconv_fwd_affine(case):
    """Zero-point operands (Section 3's scheme) on every forward shape: int32 sums bit-exact, fp32 as dequant_acc."""
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    rng = np.random.default_rng(77)
    A = rng.integers(0, 256, (nodes, B, H, W, Cin), dtype=np.uint8)
    Wq = rng.integers(0, 256, (nodes, Cout, R, S, Cin), dtype=np.uint8)
    zA = rng.integers(0, 256, nodes).astype(np.int32)
    zW = rng.integers(0, 256, nodes).astype(np.int32)
    zA[0], zW[0] = 255, 0                                   # extreme zero points on one node
    s1 = rng.uniform(0.001, 0.1, nodes).astype(np.float32)
    s2 = rng.uniform(0.001, 0.1, nodes).astype(np.float32)
    acc_ref, ovf = oracle.qconv_fwd_affine(A, zA, Wq, zW, stride, pad)
    assert ovf == 0
    desc = api.conv_desc(*case)
    ws = ws_bytes(api.lpdt_qconv_fwd_affine_workspace_size(desc))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bias = rng.standard_normal((nodes, Cout)).astype(np.float32)
    Y = torch.empty(acc_ref.shape, dtype=torch.float32, device="cuda")
    Yacc = torch.empty(acc_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd_affine(desc, dev(A), dev(s1), dev(zA), dev(Wq), dev(s2), dev(zW), Y=Y, Yacc=Yacc,
                              bias=dev(bias), bias_node_stride=Cout, ws=ws, dev_status=status)
    assert int(status.item()) == 0
    assert np.array_equal(Yacc.cpu().numpy(), acc_ref)
    assert np.array_equal(Y.cpu().numpy(), oracle.dequant_acc(acc_ref, s1, s2, bias))


@pytest.mark.parametrize("case", CONV_CASES)
def test_qconv_bwd_affine(case):
    """Both backward products on zero-point operands, every shape: int32 sums bit-exact, fp32 as dequant_acc;
    the weight gradient also into a strided destination."""
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    rng = np.random.default_rng(78)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    A = rng.integers(0, 256, (nodes, B, H, W, Cin), dtype=np.uint8)
    Wq = rng.integers(0, 256, (nodes, Cout, R, S, Cin), dtype=np.uint8)
    E = rng.integers(0, 256, (nodes, B, Ho, Wo, Cout), dtype=np.uint8)
    zA, zW, zE = (rng.integers(0, 256, nodes).astype(np.int32) for _ in range(3))
    zE[0], zW[0], zA[0] = 255, 0, 255                       # extreme zero points on one node
    sA, sW, sE = (rng.uniform(0.001, 0.1, nodes).astype(np.float32) for _ in range(3))
    dA_ref, o1 = oracle.qconv_bwd_data_affine(E, zE, Wq, zW, H, W, stride, pad)
    dW_ref, o2 = oracle.qconv_bwd_weight_affine(E, zE, A, zA, R, S, stride, pad)
    assert o1 == 0 and o2 == 0
    desc = api.conv_desc(*case)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Ed, Wd, Ad = dev(E), dev(Wq), dev(A)
    dA = torch.empty(dA_ref.shape, dtype=torch.float32, device="cuda")
    dAacc = torch.empty(dA_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_bwd_data_affine(desc, Ed, dev(sE), dev(zE), Wd, dev(sW), dev(zW), dA=dA, dAacc=dAacc,
                                   ws=ws_bytes(api.lpdt_qconv_bwd_data_affine_workspace_size(desc)), dev_status=status)
    assert np.array_equal(dAacc.cpu().numpy(), dA_ref)
    assert np.array_equal(dA.cpu().numpy(), oracle.dequant_acc(dA_ref, sE, sW))
    wn = Cout * R * S * Cin
    stride_w = wn + 12
    dW = torch.zeros(nodes, stride_w, dtype=torch.float32, device="cuda")
    dWacc = torch.empty(dW_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_bwd_weight_affine(desc, Ed, dev(sE), dev(zE), Ad, dev(sA), dev(zA), dW=dW, dw_node_stride=stride_w,
                                     dWacc=dWacc, ws=ws_bytes(api.lpdt_qconv_bwd_weight_affine_workspace_size(desc)),
                                     dev_status=status)
    assert int(status.item()) == 0
    assert np.array_equal(dWacc.cpu().numpy(), dW_ref)
    assert np.array_equal(dW[:, :wn].cpu().numpy(), oracle.dequant_acc(dW_ref, sE, sA).reshape(nodes, wn))
    assert not dW[:, wn:].any()


def test_qconv_fwd_affine_matches_quantizer_output():
    # end to end with lpdt_quantize's affine mode: real 0 maps to the zero point, so a zero-padded real
    # convolution of the dequantized tensors equals scale * acc
    nodes, B, H, W, Cin, Cout = 2, 2, 10, 9, 16, 32
    rng = np.random.default_rng(5)
    x = rng.standard_normal((nodes, B, H, W, Cin)).astype(np.float32) + 0.7
    w = rng.standard_normal((nodes, Cout, 3, 3, Cin)).astype(np.float32) * 0.1
    qx, sx, zx = oracle.quantize_affine_u8(x.reshape(nodes, -1))
    qw, sw, zw = oracle.quantize_affine_u8(w.reshape(nodes, -1))
    A, Wq = qx.reshape(x.shape), qw.reshape(w.shape)
    acc_ref, _ = oracle.qconv_fwd_affine(A, zx, Wq, zw, 1, 1)
    desc = api.conv_desc(nodes, B, H, W, Cin, Cout, 3, 3, 1, 1)
    Yacc = torch.empty(acc_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd_affine(desc, dev(A), dev(sx), dev(zx.astype(np.int32)), dev(Wq), dev(sw), dev(zw.astype(np.int32)),
                              Yacc=Yacc, ws=ws_bytes(api.lpdt_qconv_fwd_affine_workspace_size(desc)))
    assert np.array_equal(Yacc.cpu().numpy(), acc_ref)


def test_qconv_fwd_affine_errors():
    desc = api.conv_desc(1, 1, 4, 4, 16, 16)
    A = torch.zeros(1, 1, 4, 4, 16, dtype=torch.uint8, device="cuda")
    Wq = torch.zeros(1, 16, 3, 3, 16, dtype=torch.uint8, device="cuda")
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    Yacc = torch.zeros(1, 1, 4, 4, 16, dtype=torch.int32, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_qconv_fwd_affine(desc, A, None, z, Wq, None, z, Yacc=Yacc, ws=ws_bytes(256))
    assert e.value.code == 3                                 # workspace too small
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_qconv_fwd_affine(desc, A, None, None, Wq, None, z, Yacc=Yacc,
                                  ws=ws_bytes(api.lpdt_qconv_fwd_affine_workspace_size(desc)))
    assert e.value.code == 1                                 # zero points missing


@pytest.mark.parametrize("case", CONV_CASES)
def test_qconv_all_three(case):
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    A, Wq, E, s1, s2 = _conv_inputs(case)
    desc = api.conv_desc(*case)
    ws = ws_bytes(max(api.lpdt_qconv_workspace_size(desc, w) for w in (0, 1, 2)))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Ad, Wd, Ed, s1d, s2d = dev(A), dev(Wq), dev(E), dev(s1), dev(s2)
    # forward, with bias living in a strided parameter vector
    acc_ref, ovf = oracle.qconv_fwd(A, Wq, stride, pad)
    assert ovf == 0
    bias = np.random.default_rng(1).standard_normal((nodes, Cout + 3)).astype(np.float32)
    Y = torch.empty(acc_ref.shape, dtype=torch.float32, device="cuda")
    Yacc = torch.empty(acc_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd(desc, Ad, s1d, Wd, s2d, Y=Y, Yacc=Yacc, bias=dev(bias)[:, 3:], bias_node_stride=Cout + 3,
                       ws=ws, dev_status=status)
    assert np.array_equal(Yacc.cpu().numpy(), acc_ref)
    assert np.array_equal(Y.cpu().numpy(), oracle.dequant_acc(acc_ref, s1, s2, bias[:, 3:]))
    # fp32-only output (the path the training step takes; results may leave through bulk tensor stores):
    # same values, every element written, nothing written outside the tensor
    def guarded(shape):
        n = int(np.prod(shape))
        buf = torch.full((n + 2048,), float("nan"), dtype=torch.float32, device="cuda")
        return buf, buf[1024:1024 + n].view(*shape)
    buf, Y2 = guarded(acc_ref.shape)
    api.lpdt_qconv_fwd(desc, Ad, s1d, Wd, s2d, Y=Y2, bias=dev(bias)[:, 3:], bias_node_stride=Cout + 3, ws=ws,
                       dev_status=status)
    assert torch.equal(Y2, Y) and bool(buf[:1024].isnan().all()) and bool(buf[-1024:].isnan().all())
    # backward data
    dA_ref, _ = oracle.qconv_bwd_data(E, Wq, H, W, stride, pad)
    dA = torch.empty(dA_ref.shape, dtype=torch.float32, device="cuda")
    dAacc = torch.empty(dA_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_bwd_data(desc, Ed, s1d, Wd, s2d, dA=dA, dAacc=dAacc, ws=ws, dev_status=status)
    assert np.array_equal(dAacc.cpu().numpy(), dA_ref)
    assert np.array_equal(dA.cpu().numpy(), oracle.dequant_acc(dA_ref, s1, s2))
    buf, dA2 = guarded(dA_ref.shape)
    api.lpdt_qconv_bwd_data(desc, Ed, s1d, Wd, s2d, dA=dA2, ws=ws, dev_status=status)
    assert torch.equal(dA2, dA) and bool(buf[:1024].isnan().all()) and bool(buf[-1024:].isnan().all())
    # fused shortcut gradient: dA = dequantized sums + addend, one more fp32 addition (= the oracle's residual adjoint)
    addend = np.random.default_rng(2).standard_normal(dA_ref.shape).astype(np.float32)
    buf, dA3 = guarded(dA_ref.shape)
    api.lpdt_qconv_bwd_data(desc, Ed, s1d, Wd, s2d, dA=dA3, ws=ws, dev_status=status, addend=dev(addend))
    want = oracle.residual_add_bwd(addend, oracle.dequant_acc(dA_ref, s1, s2))
    assert np.array_equal(dA3.cpu().numpy(), want) and bool(buf[:1024].isnan().all()) and bool(buf[-1024:].isnan().all())
    dA4 = torch.empty_like(dA); dAacc4 = torch.empty_like(dAacc)
    api.lpdt_qconv_bwd_data(desc, Ed, s1d, Wd, s2d, dA=dA4, dAacc=dAacc4, ws=ws, dev_status=status, addend=dev(addend))
    assert torch.equal(dA4, dA3) and torch.equal(dAacc4, dAacc)
    # backward weight, into a strided gradient vector
    dW_ref, _ = oracle.qconv_bwd_weight(E, A, R, S, stride, pad)
    wn = Cout * R * S * Cin
    dW = torch.zeros(nodes, wn + 5, dtype=torch.float32, device="cuda")
    dWacc = torch.empty(dW_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_bwd_weight(desc, Ed, s1d, Ad, s2d, dW=dW[:, 5:], dw_node_stride=wn + 5, dWacc=dWacc, ws=ws,
                              dev_status=status)
    assert np.array_equal(dWacc.cpu().numpy(), dW_ref)
    assert np.array_equal(dW[:, 5:].cpu().numpy(), oracle.dequant_acc(dW_ref, s1, s2).reshape(nodes, wn))
    assert float(dW[:, :5].abs().max()) == 0.0
    # fp32-only outputs (workspace accumulators) give the same values
    dW2 = torch.zeros(nodes, wn, dtype=torch.float32, device="cuda")
    api.lpdt_qconv_bwd_weight(desc, Ed, s1d, Ad, s2d, dW=dW2, dw_node_stride=wn, ws=ws, dev_status=status)
    assert torch.equal(dW2, dW[:, 5:])
    assert int(status.item()) == 0


def test_qconv_extreme_values_and_errors():
    # all operands at +-127: the largest accumulators the shape can produce
    case = (1, 2, 6, 6, 16, 16, 3, 3, 1, 1)
    A = np.full((1, 2, 6, 6, 16), 127, np.int8); Wq = np.full((1, 16, 3, 3, 16), -127, np.int8)
    desc = api.conv_desc(*case)
    acc_ref, _ = oracle.qconv_fwd(A, Wq, 1, 1)
    Yacc = torch.empty(acc_ref.shape, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd(desc, dev(A), None, dev(Wq), None, Yacc=Yacc, ws=ws_bytes(256))
    assert np.array_equal(Yacc.cpu().numpy(), acc_ref) and acc_ref.min() == -127 * 127 * 144
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_qconv_fwd(desc, dev(A), None, dev(Wq), None, ws=ws_bytes(256))      # no output
    assert e.value.code == 1
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_qconv_bwd_data(desc, dev(A), None, dev(Wq), None, dAacc=Yacc, ws=None)
    assert e.value.code == 3
    bad = api.conv_desc(1, 1, 2, 2, 4, 4, 5, 5, 1, 0)                                 # kernel larger than image
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_qconv_fwd(bad, dev(A), None, dev(Wq), None, Yacc=Yacc, ws=ws_bytes(256))
    assert e.value.code == 1


# ------------------------------------------------------------------ Range-EvoNorm
REN_CASES = [(4, 8, 16, 16, 16, 4), (2, 3, 32, 32, 16, 2), (2, 2, 8, 8, 64, 8), (1, 3, 5, 7, 6, 3),
             (1, 2, 4, 4, 12, 1), (2, 2, 32, 32, 64, 8), (1, 2, 2, 2, 512, 64), (1, 1, 1, 1, 8, 2),
             # samples split over a cluster: ragged pixel counts, odd column counts, large samples
             (1, 3, 7, 9, 24, 3), (1, 2, 15, 15, 32, 4), (2, 1, 9, 9, 16, 2), (1, 2, 31, 33, 64, 16), (1, 1, 40, 40, 64, 8),
             (2, 40, 16, 16, 32, 4)]


def _ren_inputs(case, seed=0, ties=False):
    nodes, B, H, W, C, groups = case
    rng = np.random.default_rng(seed)
    x = (2 * rng.standard_normal((nodes, B, H, W, C))).astype(np.float32)
    if ties:
        x = np.round(x * 2) / 2                # 8-bit-like grid: many tied extrema, hits u = +-3 exactly
    pad = 7
    P = rng.uniform(0.5, 1.5, (nodes, 3 * C + pad)).astype(np.float32)
    P[:, 2 * C:3 * C] -= 1.0
    if ties:
        P[:, :C] = 1.0
    dy = rng.standard_normal(x.shape).astype(np.float32)
    return x, P, dy


@pytest.mark.parametrize("case", REN_CASES)
@pytest.mark.parametrize("ties", [False, True])
def test_range_evonorm_fwd_bwd(case, ties):
    nodes, B, H, W, C, groups = case
    x, P, dy = _ren_inputs(case, ties=ties)
    eps = 1e-5
    v, g, b = P[:, :C], P[:, C:2 * C], P[:, 2 * C:3 * C]
    y32, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, groups, eps, "f32")
    y64 = oracle.range_evonorm_fwd(x, v, g, b, groups, eps, "f64")[0]
    xd, Pd = dev(x), dev(P)
    stride = P.shape[1]
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    i = lambda *s: torch.empty(*s, dtype=torch.int32, device="cuda")
    y, gmin, gmax, amin_, amax_ = f(*x.shape), f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
    api.lpdt_range_evonorm_fwd(nodes, B, H, W, C, groups, eps, xd, Pd, Pd[:, C:], Pd[:, 2 * C:], stride, y, gmin, gmax,
                               amin_, amax_)
    assert np.array_equal(gmin.cpu().numpy(), mn) and np.array_equal(gmax.cpu().numpy(), mx)
    assert np.array_equal(amin_.cpu().numpy(), amn) and np.array_equal(amax_.cpu().numpy(), amx)
    assert np.array_equal(y.cpu().numpy(), y32)            # same fp32 operation sequence: bit-equal
    close(y, y64)
    dx32, dv32, dg32, db32 = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, groups, eps, "f32")
    dx64, dv64, dg64, db64 = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, groups, eps, "f64")
    G = torch.zeros(nodes, stride, dtype=torch.float32, device="cuda")
    dx = f(*x.shape)
    ws = ws_bytes(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, C))
    api.lpdt_range_evonorm_bwd(nodes, B, H, W, C, groups, eps, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_, amax_,
                               dx, G, G[:, C:], G[:, 2 * C:], stride, ws)
    close(dx, dx32, 1e-6, 1e-7)
    close(dx, dx64)
    # two-call form: dx first, the parameter-gradient sums later from the partial sums in the workspace
    G2 = torch.zeros_like(G); dx2 = f(*x.shape)
    api.lpdt_range_evonorm_bwd(nodes, B, H, W, C, groups, eps, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_, amax_,
                               dx2, None, None, None, stride, ws)
    api.lpdt_range_evonorm_bwd_params(nodes, B, C, ws, G2, G2[:, C:], G2[:, 2 * C:], stride)
    assert torch.equal(dx2, dx) and torch.equal(G2, G)
    # parameter-gradient sums at the stated bar (1e-5 relative + 1e-6 absolute, no scaling): the kernel adds
    # the same fp32 terms as the oracle's fp32 instantiation into double accumulators, so it sits within
    # double rounding noise of that one, and within the bar of the all-double evaluation
    Gh = G.cpu().numpy()
    for got, w32, w64 in ((Gh[:, :C], dv32, dv64), (Gh[:, C:2 * C], dg32, dg64), (Gh[:, 2 * C:3 * C], db32, db64)):
        close(got, w32, 1e-6, 1e-7)
        close(got, w64, RTOL, ATOL)
    assert not Gh[:, 3 * C:].any()


@pytest.mark.parametrize("case", REN_CASES)
def test_range_evonorm_fwd_fused_shortcut(case):
    """y = RangeEvoNorm(x) + res in one launch: one more fp32 addition on the bit-equal norm output; the
    per-node max|y| it reports is that of the sum."""
    nodes, B, H, W, C, groups = case
    x, P, _ = _ren_inputs(case, seed=3)
    v, g, b = P[:, :C], P[:, C:2 * C], P[:, 2 * C:3 * C]
    res = np.random.default_rng(11).standard_normal(x.shape).astype(np.float32)
    y32, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, groups, 1e-5, "f32")
    want = oracle.residual_add(res, y32)
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    i = lambda *s: torch.empty(*s, dtype=torch.int32, device="cuda")
    Pd = dev(P)
    y, gmin, gmax, amin_, amax_ = f(*x.shape), f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
    rng_out = torch.zeros(nodes, device="cuda")
    api.lpdt_range_evonorm_fwd(nodes, B, H, W, C, groups, 1e-5, dev(x), Pd, Pd[:, C:], Pd[:, 2 * C:], P.shape[1], y, gmin,
                               gmax, amin_, amax_, amax_out=rng_out, res=dev(res))
    assert np.array_equal(y.cpu().numpy(), want)
    assert np.array_equal(amin_.cpu().numpy(), amn) and np.array_equal(amax_.cpu().numpy(), amx)
    assert np.array_equal(gmin.cpu().numpy(), mn) and np.array_equal(gmax.cpu().numpy(), mx)
    assert np.array_equal(rng_out.cpu().numpy(), np.abs(want).reshape(nodes, -1).max(1))


def test_fused_ranges_feed_the_quantizer_exactly():
    # the producers' per-node max|x| must equal the range pass bit for bit, so that
    # lpdt_quantize_with_range gives the same codes as lpdt_quantize
    case = (3, 4, 16, 16, 16, 2)
    nodes, B, H, W, C, groups = case
    x, P, dy = _ren_inputs(case, seed=5, ties=True)
    v, g, b = P[:, :C], P[:, C:2 * C], P[:, 2 * C:3 * C]
    y32, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, groups, 1e-5, "f32")
    dx32 = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, groups, 1e-5, "f32")[0]
    xd, Pd = dev(x), dev(P)
    stride = P.shape[1]
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    i = lambda *s: torch.empty(*s, dtype=torch.int32, device="cuda")
    ranges = torch.zeros(3, nodes, device="cuda")
    y, gmin, gmax, amin_, amax_ = f(*x.shape), f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
    api.lpdt_range_evonorm_fwd(nodes, B, H, W, C, groups, 1e-5, xd, Pd, Pd[:, C:], Pd[:, 2 * C:], stride, y, gmin, gmax,
                               amin_, amax_, amax_out=ranges[0])
    G = torch.zeros(nodes, stride, device="cuda")
    dx = f(*x.shape)
    ws = ws_bytes(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, C))
    api.lpdt_range_evonorm_bwd(nodes, B, H, W, C, groups, 1e-5, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_, amax_,
                               dx, G, G[:, C:], G[:, 2 * C:], stride, ws, amax_out=ranges[1])
    r = f(*x.shape)
    api.lpdt_residual_add(nodes, B, H, W, C, C, 1, 0, y, dx, r, amax_out=ranges[2])
    rh = ranges.cpu().numpy()
    assert np.array_equal(rh[0], np.abs(y32).reshape(nodes, -1).max(1))
    assert np.array_equal(rh[1], np.abs(dx.cpu().numpy()).reshape(nodes, -1).max(1))
    assert np.array_equal(rh[2], np.abs(r.cpu().numpy()).reshape(nodes, -1).max(1))
    n = B * H * W * C
    for t, row, rounding in ((y, 0, 0), (dx, 1, 1), (r, 2, 0)):
        q1 = torch.empty(nodes, n, dtype=torch.int8, device="cuda"); s1 = f(nodes)
        q2 = torch.empty(nodes, n, dtype=torch.int8, device="cuda"); s2 = f(nodes)
        api.lpdt_quantize(t, nodes, n, n, q1, s1, ws_bytes(256), rounding=rounding, seed=5, ctr_offset=1)
        api.lpdt_quantize_with_range(t, nodes, n, n, ranges[row], q2, s2, rounding=rounding, seed=5, ctr_offset=1)
        assert torch.equal(q1, q2) and torch.equal(s1, s2)


# cases whose sample fits one CTA's shared memory: one to 40 samples per node, ragged pixel counts, 2 to 128
# vector columns
REN_Q8_CASES = [(4, 8, 16, 16, 16, 4), (2, 3, 32, 32, 16, 2), (2, 2, 8, 8, 64, 8), (1, 2, 4, 4, 12, 1), (2, 2, 16, 16, 64, 8),
                (1, 2, 2, 2, 512, 64), (1, 1, 1, 1, 8, 2), (1, 3, 7, 9, 24, 3), (1, 2, 15, 17, 64, 16), (2, 40, 16, 16, 32, 4),
                (3, 32, 32, 32, 16, 2), (2, 32, 8, 8, 64, 8), (1, 5, 3, 3, 256, 8)]


def _ren_q8_check(case, ties, with_res, keep_y):
    nodes, B, H, W, C, groups = case
    x, P, dy = _ren_inputs(case, seed=21, ties=ties)
    eps = 1e-5
    v, g, b = P[:, :C], P[:, C:2 * C], P[:, 2 * C:3 * C]
    res = np.random.default_rng(5).standard_normal(x.shape).astype(np.float32) if with_res else None
    y32, mn, mx, amn, amx = oracle.range_evonorm_fwd(x, v, g, b, groups, eps, "f32")
    want_y = oracle.residual_add(res, y32) if with_res else y32
    n = B * H * W * C
    q_ref, s_ref = oracle.quantize_sym_s8(want_y.reshape(nodes, n))
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    i = lambda *s: torch.empty(*s, dtype=torch.int32, device="cuda")
    xd, Pd, stride = dev(x), dev(P), P.shape[1]
    assert api.lpdt_range_evonorm_fwd_q8_fits(B, H, W, C, groups) == 1
    assert api.lpdt_range_evonorm_bwd_q8_fits(B, H, W, C, groups) == 1
    ctl = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(nodes), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.full(x.shape, float("nan"), dtype=torch.float32, device="cuda") if keep_y else None
    gmin, gmax, amin_, amax_ = f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
    q = torch.full((nodes, n), 99, dtype=torch.int8, device="cuda")
    sc = f(nodes)
    rng_out = torch.full((nodes,), -1.0, device="cuda")
    api.lpdt_range_evonorm_fwd_q8(nodes, B, H, W, C, groups, eps, xd, Pd, Pd[:, C:], Pd[:, 2 * C:], stride, y, gmin, gmax,
                                  amin_, amax_, q, sc, ctl, amax_out=rng_out, res=None if res is None else dev(res),
                                  dev_status=status)
    assert not ctl.any() and int(status.item()) == 0           # the control block is left clean
    assert np.array_equal(gmin.cpu().numpy(), mn) and np.array_equal(gmax.cpu().numpy(), mx)
    assert np.array_equal(amin_.cpu().numpy(), amn) and np.array_equal(amax_.cpu().numpy(), amx)
    if keep_y:
        assert np.array_equal(y.cpu().numpy(), want_y)
    assert np.array_equal(rng_out.cpu().numpy(), np.abs(want_y).reshape(nodes, -1).max(1))
    assert np.array_equal(sc.cpu().numpy(), s_ref)
    assert np.array_equal(q.cpu().numpy(), q_ref)            # the oracle's norm followed by the oracle's quantizer
    # backward: the codes of dx.  dx itself matches the oracle to 1e-6 relative, not bit for bit, so the codes are
    # pinned two ways: they equal the ORACLE's quantizer applied to the dx the plain backward call writes (same
    # arithmetic inside the fused kernel), and dequantized they sit within half a step of the oracle's dx
    dx32 = oracle.range_evonorm_bwd(dy, x, v, g, mn, mx, amn, amx, groups, eps, "f32")[0]
    dx = f(*x.shape)
    ws = ws_bytes(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, C))
    G = torch.zeros(nodes, stride, device="cuda")
    api.lpdt_range_evonorm_bwd(nodes, B, H, W, C, groups, eps, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_, amax_,
                               dx, G, G[:, C:], G[:, 2 * C:], stride, ws)
    qe_ref, se_ref = oracle.quantize_sym_s8(dx.cpu().numpy().reshape(nodes, n))
    E = torch.full((nodes, n), 99, dtype=torch.int8, device="cuda")
    sE = f(nodes)
    G2 = torch.zeros_like(G)
    ws2 = ws_bytes(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, C))
    rng2 = torch.full((nodes,), -1.0, device="cuda")
    api.lpdt_range_evonorm_bwd_q8(nodes, B, H, W, C, groups, eps, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_,
                                  amax_, E, sE, G2, G2[:, C:], G2[:, 2 * C:], stride, ws2, ctl, amax_out=rng2,
                                  dev_status=status)
    assert not ctl.any() and int(status.item()) == 0
    assert np.array_equal(sE.cpu().numpy(), se_ref)
    assert np.array_equal(E.cpu().numpy(), qe_ref)
    assert torch.equal(G2, G)
    assert np.array_equal(rng2.cpu().numpy(), np.abs(dx.cpu().numpy()).reshape(nodes, -1).max(1))
    deq = E.cpu().numpy().astype(np.float64) * se_ref[:, None].astype(np.float64)
    err = np.abs(deq - dx32.reshape(nodes, n).astype(np.float64))
    bar = 0.5 * se_ref[:, None].astype(np.float64) * (1 + 1e-5) + 1e-6 * np.abs(dx32.reshape(nodes, n)) + 1e-7
    assert (err <= bar).all()
    # deferred parameter sums: same partial sums in the workspace
    G3 = torch.zeros_like(G)
    api.lpdt_range_evonorm_bwd_q8(nodes, B, H, W, C, groups, eps, dev(dy), xd, Pd, Pd[:, C:], stride, gmin, gmax, amin_,
                                  amax_, E, sE, None, None, None, stride, ws2, ctl, dev_status=status)
    api.lpdt_range_evonorm_bwd_params(nodes, B, C, ws2, G3, G3[:, C:], G3[:, 2 * C:], stride)
    assert torch.equal(G3, G) and np.array_equal(E.cpu().numpy(), qe_ref)
    assert not ctl.any() and int(status.item()) == 0


@pytest.mark.parametrize("case", REN_Q8_CASES)
@pytest.mark.parametrize("ties", [False, True])
def test_range_evonorm_q8(case, ties):
    """Range-EvoNorm with the requantize step inside: codes, scales, statistics and parameter gradients equal
    those of the norm call followed by the quantizer."""
    _ren_q8_check(case, ties, with_res=False, keep_y=False)
    _ren_q8_check(case, ties, with_res=True, keep_y=True)


@pytest.mark.parametrize("env", [{"LPDT_REN_Q8_THREADS": "128"}, {"LPDT_REN_Q8_THREADS": "256", "LPDT_REN_Q8_DEPTH": "4"},
                                 {"LPDT_REN_Q8_THREADS": "384"}])
def test_range_evonorm_q8_on_every_launch_shape(env):
    """The same cases in child processes with the CTA size and ring depth forced."""
    import os, subprocess, sys
    if os.environ.get("LPDT_CHILD") == "1":
        pytest.skip("already inside a child run")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    child_env = dict(os.environ, LPDT_CHILD="1", **env)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_ops.py"), "-m", "gpu",
                        "-q", "-x", "-k", "test_range_evonorm_q8 and not launch_shape and not reports"], env=child_env,
                       cwd=root, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and " passed" in r.stdout, r.stdout[-3000:] + r.stderr[-2000:]


def test_range_evonorm_q8_reports_shapes_that_do_not_fit():
    # a sample of 32x32x64 fp32 is 256 KB: beyond one CTA's shared memory
    assert api.lpdt_range_evonorm_fwd_q8_fits(32, 32, 32, 64, 8) == 0
    assert api.lpdt_range_evonorm_bwd_q8_fits(32, 32, 32, 64, 8) == 0
    assert api.lpdt_range_evonorm_fwd_q8_fits(4, 4, 4, 6, 3) == 0          # 2 channels per group: no 4-wide columns
    # more samples per node than half the CTAs the device can hold at once: the meeting could starve
    assert api.lpdt_range_evonorm_bwd_q8_fits(4096, 32, 32, 16, 2) == 0
    t = torch.zeros(2 * 32 * 32 * 64, device="cuda"); ti = torch.zeros(256, dtype=torch.int32, device="cuda")
    q = torch.zeros(2 * 32 * 32 * 64, dtype=torch.int8, device="cuda")
    ctl = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(1), dtype=torch.uint8, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_range_evonorm_fwd_q8(1, 2, 32, 32, 64, 8, 1e-5, t, t, t, t, 64, None, t, t, ti, ti, q, t, ctl)
    assert e.value.code == 2
    with pytest.raises(api.LpdtError) as e:      # no control block
        api.lpdt_range_evonorm_fwd_q8(1, 2, 8, 8, 64, 8, 1e-5, t, t, t, t, 64, None, t, t, ti, ti, q, t, None)
    assert e.value.code == 3


def test_range_evonorm_q8_with_a_control_block_that_was_not_cleared():
    """The control block must be zero at launch.  When its ticket counter is not, the tickets name no sample of
    the call: every CTA records LPDT_ERR_INVALID_ARG and returns without touching the tensors (no out-of-range
    access), and the context stays usable."""
    nodes, B, H, W, C, groups = 2, 4, 8, 8, 16, 2
    x, P, dy = _ren_inputs((nodes, B, H, W, C, groups), seed=2)
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    i = lambda *s: torch.empty(*s, dtype=torch.int32, device="cuda")
    Pd, stride = dev(P), P.shape[1]
    n = B * H * W * C
    ctl = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(nodes) // 4, dtype=torch.int32, device="cuda")
    ctl[3 * nodes] = nodes * B                         # the ticket counter of a call that never finished
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q = torch.full((nodes, n), 77, dtype=torch.int8, device="cuda")
    sc = torch.full((nodes,), -1.0, device="cuda")
    gmin, gmax, amin_, amax_ = f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
    api.lpdt_range_evonorm_fwd_q8(nodes, B, H, W, C, groups, 1e-5, dev(x), Pd, Pd[:, C:], Pd[:, 2 * C:], stride, None, gmin,
                                  gmax, amin_, amax_, q, sc, ctl.view(torch.uint8), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1                     # LPDT_ERR_INVALID_ARG
    assert (q == 77).all() and (sc == -1.0).all()
    # cleared, the same buffers serve a correct call
    ctl.zero_(); status.zero_()
    api.lpdt_range_evonorm_fwd_q8(nodes, B, H, W, C, groups, 1e-5, dev(x), Pd, Pd[:, C:], Pd[:, 2 * C:], stride, None, gmin,
                                  gmax, amin_, amax_, q, sc, ctl.view(torch.uint8), dev_status=status)
    v, g, b = P[:, :C], P[:, C:2 * C], P[:, 2 * C:3 * C]
    y32 = oracle.range_evonorm_fwd(x, v, g, b, groups, 1e-5, "f32")[0]
    q_ref, s_ref = oracle.quantize_sym_s8(y32.reshape(nodes, n))
    assert int(status.item()) == 0 and not ctl.any()
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(sc.cpu().numpy(), s_ref)


def test_range_evonorm_errors():
    t = torch.zeros(64, device="cuda"); ti = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(api.LpdtError) as e:      # one channel per group: the constant is infinite
        api.lpdt_range_evonorm_fwd(1, 1, 2, 2, 4, 4, 1e-5, t, t, t, t, 4, t, t, t, ti, ti)
    assert e.value.code == 1
    with pytest.raises(api.LpdtError) as e:      # groups must divide C
        api.lpdt_range_evonorm_fwd(1, 1, 2, 2, 6, 4, 1e-5, t, t, t, t, 6, t, t, t, ti, ti)
    assert e.value.code == 1


# ------------------------------------------------------------------ gossip
def _gossip_case(nodes, d, seed, heavy=False):
    rng = np.random.default_rng(seed)
    xh = rng.standard_normal((nodes, d)).astype(np.float32)
    resid = rng.standard_normal((nodes, d)) * (np.where(rng.random((nodes, d)) < 0.05, 1.0, 0.01) if heavy else 1.0)
    xhat = (xh - resid).astype(np.float32)
    return xh, xhat


@pytest.mark.parametrize("nodes,d,segs", [
    (4, 2736, None), (16, 10007, None), (8, 50000, [(0, 50000, 500)]), (40, 27041, [(0, 27041, 270)]),
    (5, 3000, [(0, 1000, 10), (1000, 1001, 1), (1001, 3000, 1999)]), (3, 1000, [(0, 1000, 0)]),
    (1, 777, [(0, 777, 5)]), (64, 300, [(0, 300, 3)]),
    # long segments: selection spread over several CTAs (with short and trivial ones beside them)
    (3, 100000, [(0, 100000, 1000)]), (2, 200000, [(0, 40000, 39999), (40000, 41000, 7), (41000, 200000, 1)]),
    (2, 70001, [(0, 33000, 0), (33000, 70001, 37001)]),
    # parameter counts that are even but not multiples of 4 (8-byte accesses), segments starting at odd offsets
    (4, 2738, None), (8, 270410, None), (6, 100002, [(0, 33333, 300), (33333, 100002, 700)]),
])
def test_gossip_mix(nodes, d, segs):
    xh, xhat = _gossip_case(nodes, d, d, heavy=True)
    W = wlmod.ring_matrix(nodes) if nodes >= 3 else np.full((nodes, nodes), 1.0 / nodes, np.float32)
    so = [0, d] if segs is None else [s[0] for s in segs] + [d]
    sk = [d] if segs is None else [s[2] for s in segs]
    gamma = 1.0 if segs is None else 0.3
    x_ref, xhat_ref, q_ref = oracle.gossip_mix(xh, xhat, W, gamma, so, sk)
    xhd, xhatd = dev(xh), dev(xhat)
    xo = torch.empty_like(xhd)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, len(sk)))
    api.lpdt_gossip_mix(nodes, d, xhd, xhatd, xo, dev(W), gamma, so, sk, ws)
    assert np.array_equal(xhatd.cpu().numpy(), xhat_ref)          # selection + update: bit-exact
    close(xo, x_ref)
    # second call on the updated state (error feedback carried over)
    x_ref2, xhat_ref2, _ = oracle.gossip_mix(x_ref, xhat_ref, W, gamma, so, sk)
    xo2 = torch.empty_like(xhd)
    api.lpdt_gossip_mix(nodes, d, dev(x_ref), xhatd, xo2, dev(W), gamma, so, sk, ws)
    assert np.array_equal(xhatd.cpu().numpy(), xhat_ref2)
    close(xo2, x_ref2)


def test_gossip_topk_with_massive_ties_and_alias():
    # magnitudes from a 4-value set: the tie cut decides almost every pick
    nodes, d, k = 6, 9000, 1234
    rng = np.random.default_rng(5)
    xh = rng.choice(np.array([-2, -1, 1, 2, 0.5, -0.5], np.float32), size=(nodes, d))
    xhat = np.zeros((nodes, d), np.float32)
    W = wlmod.ring_matrix(nodes)
    x_ref, xhat_ref, q_ref = oracle.gossip_mix(xh, xhat, W, 0.5, [0, d], [k])
    assert all(np.count_nonzero(q_ref[i]) == k for i in range(nodes))
    xhd, xhatd = dev(xh), dev(xhat)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, 1))
    api.lpdt_gossip_mix(nodes, d, xhd, xhatd, xhd, dev(W), 0.5, [0, d], [k], ws)   # x_out aliases x_half
    assert np.array_equal(xhatd.cpu().numpy(), xhat_ref)
    close(xhd, x_ref)


def test_gossip_topk_ties_across_chunks():
    # a long segment whose threshold value repeats thousands of times: the tie cut falls inside
    # one of many chunks, in the first one, or in the last one, depending on k
    nodes, d = 3, 90001
    rng = np.random.default_rng(11)
    xh = rng.choice(np.array([-2, -1, 1, 2, 0.5, -0.5], np.float32), size=(nodes, d))
    xh[0, :200] = 1.0; xh[0, 200:] = 0.25            # node 0: every tie of value 1 sits in the first chunk
    xh[2, :-50] = 0.125; xh[2, -50:] = -3.0           # node 2: threshold ties reach into the last chunk
    W = wlmod.ring_matrix(nodes)
    for k in (150, 20000, 60000, 89990):
        xhat = np.zeros((nodes, d), np.float32)
        x_ref, xhat_ref, q_ref = oracle.gossip_mix(xh, xhat, W, 0.5, [0, d], [k])
        assert all(np.count_nonzero(q_ref[i]) == k for i in range(nodes))
        xhd, xhatd = dev(xh), dev(xhat)
        xo = torch.empty_like(xhd)
        ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, 1))
        api.lpdt_gossip_mix(nodes, d, xhd, xhatd, xo, dev(W), 0.5, [0, d], [k], ws)
        assert np.array_equal(xhatd.cpu().numpy(), xhat_ref), k
        close(xo, x_ref)


def test_gossip_topk_candidate_list_with_planted_ties():
    """Long segments of distinct magnitudes (the candidate-list path) with the threshold value planted a few
    hundred times at scattered positions, so that only the ties at the lowest positions are kept; a second
    segment of constant magnitude overflows its list and takes the whole-segment path in the same call."""
    nodes, d1, d2, k1 = 3, 300000, 40000, 3000
    d = d1 + d2
    rng = np.random.default_rng(21)
    xh = rng.standard_normal((nodes, d)).astype(np.float32)
    for i in range(nodes):
        mags = np.sort(np.abs(xh[i, :d1]))[::-1]
        v = mags[k1 - 100]                                    # inside the top k1
        pos = rng.choice(d1, size=400, replace=False)
        xh[i, pos] = v * rng.choice(np.array([-1.0, 1.0], np.float32), size=400)
    xh[:, d1:] = 0.75
    xh[1, d1:] = 0.0                                          # all-zero differences
    xhat = np.zeros((nodes, d), np.float32)
    W = wlmod.ring_matrix(nodes)
    so, sk = [0, d1, d], [k1, 12345]
    x_ref, xhat_ref, q_ref = oracle.gossip_mix(xh, xhat, W, 0.4, so, sk)
    assert all(np.count_nonzero(q_ref[i][:d1]) == k1 for i in range(nodes))
    xhd, xhatd = dev(xh), dev(xhat)
    xo = torch.empty_like(xhd)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, 2))
    api.lpdt_gossip_mix(nodes, d, xhd, xhatd, xo, dev(W), 0.4, so, sk, ws)
    assert np.array_equal(xhatd.cpu().numpy(), xhat_ref)
    close(xo, x_ref)


@pytest.mark.parametrize("nodes,d,segs", [
    (4, 2736, None), (16, 10007, None), (8, 50000, [(0, 50000, 500)]),
    (5, 3000, [(0, 1000, 10), (1000, 1001, 1), (1001, 3000, 1999)]), (3, 1000, [(0, 1000, 0)]),
    (3, 100000, [(0, 100000, 1000)]), (2, 200000, [(0, 40000, 39999), (40000, 41000, 7), (41000, 200000, 1)]),
])
def test_gossip_mix_q8(nodes, d, segs):
    """8-bit messages: public copies (hence the codes sent) bit-exact, mixed parameters within the fp32 bar,
    transmitted steps equal; two steps in a row so that the rounding error is fed back."""
    xh, xhat = _gossip_case(nodes, d, d, heavy=True)
    W = wlmod.ring_matrix(nodes) if nodes >= 3 else np.full((nodes, nodes), 1.0 / nodes, np.float32)
    so = [0, d] if segs is None else [s[0] for s in segs] + [d]
    sk = [d] if segs is None else [s[2] for s in segs]
    gamma = 1.0 if segs is None else 0.3
    xhd, xhatd = dev(xh), dev(xhat)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, len(sk)))
    scale = torch.empty(nodes, len(sk), device="cuda")
    x_in, xhat_ref = xh, xhat
    for _ in range(2):
        x_ref, xhat_ref, q_ref, codes_ref, scale_ref = oracle.gossip_mix_q8(x_in, xhat_ref, W, gamma, so, sk)
        xo = torch.empty_like(xhd)
        api.lpdt_gossip_mix_q8(nodes, d, dev(x_in), xhatd, xo, dev(W), gamma, so, sk, scale, ws)
        assert np.array_equal(scale.cpu().numpy(), scale_ref)
        assert np.array_equal(xhatd.cpu().numpy(), xhat_ref)
        close(xo, x_ref)
        x_in = x_ref


@pytest.mark.parametrize("bits", [32, 8])
@pytest.mark.parametrize("nodes,d,segs", [
    (4, 2736, None), (16, 10007, [(0, 10007, 100)]), (8, 50000, [(0, 50000, 500)]),
    (5, 3000, [(0, 1000, 10), (1000, 1001, 1), (1001, 3000, 1999)]), (3, 1000, [(0, 1000, 0)]),
    (3, 100000, [(0, 100000, 1000)]),
])
def test_deepsqueeze_mix(nodes, d, segs, bits):
    """Deep-Squeeze step: error buffer (hence the messages) bit-exact, mixed parameters within the fp32 bar;
    three steps in a row so that the buffer is carried over."""
    rng = np.random.default_rng(nodes * 1000 + d)
    xh = rng.standard_normal((nodes, d)).astype(np.float32)
    delta_ref = np.zeros((nodes, d), np.float32)
    W = wlmod.ring_matrix(nodes) if nodes >= 3 else np.full((nodes, nodes), 1.0 / nodes, np.float32)
    so = [0, d] if segs is None else [s[0] for s in segs] + [d]
    sk = [d] if segs is None else [s[2] for s in segs]
    eta = 1.0 if segs is None else 0.3
    deltad = dev(delta_ref)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, len(sk)))
    scale = torch.empty(nodes, len(sk), device="cuda")
    x_in = xh
    for step in range(3):
        x_ref, delta_ref, c_ref, scale_ref = oracle.deepsqueeze_mix(x_in, delta_ref, W, eta, so, sk, bits)
        xo = torch.empty(nodes, d, device="cuda")
        api.lpdt_deepsqueeze_mix(nodes, d, dev(x_in), deltad, xo, dev(W), eta, so, sk, ws, message_bits=bits,
                                 msg_scale=scale if bits == 8 else None)
        if bits == 8:
            assert np.array_equal(scale.cpu().numpy(), scale_ref)
        assert np.array_equal(deltad.cpu().numpy(), delta_ref), step
        close(xo, x_ref)
        x_in = (x_ref - 0.05 * rng.standard_normal((nodes, d))).astype(np.float32)      # a stand-in local update


@pytest.mark.parametrize("nodes,d", [(4, 2736), (16, 10007), (8, 270410), (64, 300), (1, 777), (3, 100002)])
def test_sgd_gossip_mix(nodes, d):
    """Fused half-step + dense mix: x_half and x_hat bit-equal to lpdt_sgd_update / the oracle, x within the fp32 bar;
    also bit-equal to the two separate launches."""
    rng = np.random.default_rng(nodes + d)
    x = rng.standard_normal((nodes, d)).astype(np.float32)
    g = rng.standard_normal((nodes, d)).astype(np.float32)
    xhat = (x - 0.1 * rng.standard_normal((nodes, d))).astype(np.float32)
    W = wlmod.ring_matrix(nodes) if nodes >= 3 else np.full((nodes, nodes), 1.0 / nodes, np.float32)
    xh_ref = oracle.sgd_update(x, g, 0.1)
    x_ref, xhat_ref, _ = oracle.gossip_mix(xh_ref, xhat, W, 0.9, [0, d], [d])
    xhd, xhatd, xo = torch.empty(nodes, d, device="cuda"), dev(xhat), torch.empty(nodes, d, device="cuda")
    api.lpdt_sgd_gossip_mix(nodes, d, dev(x), dev(g), 0.1, xhd, xhatd, xo, dev(W), 0.9)
    assert np.array_equal(xhd.cpu().numpy(), xh_ref) and np.array_equal(xhatd.cpu().numpy(), xhat_ref)
    close(xo, x_ref)
    xh2, xhat2, xo2 = torch.empty(nodes, d, device="cuda"), dev(xhat), torch.empty(nodes, d, device="cuda")
    api.lpdt_sgd_update(nodes * d, dev(x), dev(g), 0.1, xh2)
    api.lpdt_gossip_mix(nodes, d, xh2, xhat2, xo2, dev(W), 0.9, [0, d], [d],
                        ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, 1)))
    assert torch.equal(xo, xo2) and torch.equal(xhatd, xhat2)


def directed_ring_matrix(n, rng):
    """Column-stochastic, not row-stochastic: node j keeps a share and pushes the rest to j+1 and j+2."""
    W = np.zeros((n, n), np.float32)
    for j in range(n):
        w = rng.dirichlet(np.ones(3)).astype(np.float32)
        W[j, j] += w[0]; W[(j + 1) % n, j] += w[1]; W[(j + 2) % n, j] += w[2]
    return W


@pytest.mark.parametrize("nodes,d", [(4, 1), (5, 1001), (16, 40000), (64, 4096), (3, 270410)])
def test_pushsum_debias(nodes, d):
    """Sparse-Push over three steps: Deep-Squeeze mix with a column-stochastic matrix, then the bias
    weights and the de-biased model; bias weights and z bit-exact given the same mixed model."""
    rng = np.random.default_rng(nodes * 7 + d)
    W = directed_ring_matrix(nodes, rng)
    x = rng.standard_normal((nodes, d)).astype(np.float32)
    u_ref = np.ones(nodes, np.float32)
    ud = dev(u_ref)
    for step in range(3):
        u_new_ref, z_ref = oracle.pushsum_debias(x, u_ref, W, 0.8)
        un = torch.empty(nodes, device="cuda"); z = torch.empty(nodes, d, device="cuda")
        api.lpdt_pushsum_debias(nodes, d, dev(x), ud, dev(W), 0.8, un, z)
        assert np.array_equal(un.cpu().numpy(), u_new_ref), step
        assert np.array_equal(z.cpu().numpy(), z_ref), step
        u_ref, ud = u_new_ref, un
        x = (x + 0.1 * rng.standard_normal((nodes, d))).astype(np.float32)
    # in place, and the bias weights alone
    xd = dev(x)
    api.lpdt_pushsum_debias(nodes, d, xd, ud, dev(W), 0.8, un2 := torch.empty(nodes, device="cuda"), xd)
    u3, z3 = oracle.pushsum_debias(x, u_ref, W, 0.8)
    assert np.array_equal(xd.cpu().numpy(), z3) and np.array_equal(un2.cpu().numpy(), u3)
    api.lpdt_pushsum_debias(nodes, 0, None, ud, dev(W), 0.8, un3 := torch.empty(nodes, device="cuda"), None)
    assert np.array_equal(un3.cpu().numpy(), u3)


def test_sparse_push_chain():
    """Supplementary Algorithm 4 end to end on a directed graph: Deep-Squeeze mix (top-10 %) then push-sum
    de-biasing, against the same two oracle calls; total mass sum_i x_i / sum_i u_i is what z tracks."""
    rng = np.random.default_rng(44)
    nodes, d = 8, 5000
    W = directed_ring_matrix(nodes, rng)
    x = rng.standard_normal((nodes, d)).astype(np.float32)
    delta_ref = np.zeros((nodes, d), np.float32); u_ref = np.ones(nodes, np.float32)
    deltad, ud = dev(delta_ref), dev(u_ref)
    ws = ws_bytes(api.lpdt_gossip_mix_workspace_size(nodes, d, 1))
    for step in range(3):
        x_ref, delta_ref, _, _ = oracle.deepsqueeze_mix(x, delta_ref, W, 0.5, [0, d], [d // 10], 32)
        u_ref, z_ref = oracle.pushsum_debias(x_ref, u_ref, W, 0.5)
        xo = torch.empty(nodes, d, device="cuda"); un = torch.empty(nodes, device="cuda"); z = torch.empty_like(xo)
        api.lpdt_deepsqueeze_mix(nodes, d, dev(x), deltad, xo, dev(W), 0.5, [0, d], [d // 10], ws)
        api.lpdt_pushsum_debias(nodes, d, xo, ud, dev(W), 0.5, un, z)
        assert np.array_equal(deltad.cpu().numpy(), delta_ref)
        assert np.array_equal(un.cpu().numpy(), u_ref)
        close(z, z_ref)
        ud = un
        x = (z_ref - 0.05 * rng.standard_normal((nodes, d))).astype(np.float32)


def test_gossip_errors():
    t = torch.zeros(4, 8, device="cuda"); W = torch.zeros(4, 4, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_gossip_mix(4, 8, t, t.clone(), t, W, 1.0, [0, 7], [7], ws_bytes(4096))   # segments don't tile
    assert e.value.code == 1
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_gossip_mix(4, 8, t, t, t, W, 1.0, [0, 8], [8], ws_bytes(4096))           # x_hat aliases x_half
    assert e.value.code == 1
    big = torch.zeros(65, 4, device="cuda")
    with pytest.raises(api.LpdtError) as e:
        api.lpdt_gossip_mix(65, 4, big, big.clone(), big.clone(), torch.zeros(65, 65, device="cuda"), 1.0, [0, 4], [4],
                            ws_bytes(65536))
    assert e.value.code == 2


# ------------------------------------------------------------------ glue
def test_glue_ops():
    rng = np.random.default_rng(8)
    f = lambda *s: torch.empty(*s, dtype=torch.float32, device="cuda")
    x = rng.standard_normal(10007).astype(np.float32); g = rng.standard_normal(10007).astype(np.float32)
    out = f(10007)
    api.lpdt_sgd_update(10007, dev(x), dev(g), 0.1, out)
    assert np.array_equal(out.cpu().numpy(), oracle.sgd_update(x, g, 0.1))
    a = rng.standard_normal((2, 3, 8, 8, 16)).astype(np.float32)
    r = rng.standard_normal((2, 3, 8, 8, 16)).astype(np.float32)
    y = f(*r.shape)
    api.lpdt_residual_add(2, 3, 8, 8, 16, 16, 1, 0, dev(r), dev(a), y)
    assert np.array_equal(y.cpu().numpy(), oracle.residual_add(r, a))
    r2 = rng.standard_normal((2, 3, 4, 4, 32)).astype(np.float32)
    y2 = f(*r2.shape)
    api.lpdt_residual_add(2, 3, 8, 8, 16, 32, 2, 8, dev(r2), dev(a), y2)
    assert np.array_equal(y2.cpu().numpy(), oracle.residual_add(r2, a, 2, 8))
    da = f(*a.shape)
    api.lpdt_residual_add_bwd(2, 3, 8, 8, 16, 32, 2, 8, dev(r2), dev(a), da)
    assert np.array_equal(da.cpu().numpy(), oracle.residual_add_bwd(r2, a, 2, 8))
    p = f(2, 3, 16)
    api.lpdt_avgpool(2, 3, 64, 16, dev(a), p)
    assert np.array_equal(p.cpu().numpy(), oracle.avgpool(a))
    dpx = f(*a.shape)
    api.lpdt_avgpool_bwd(2, 3, 64, 16, p, dpx)
    assert np.array_equal(dpx.cpu().numpy(), oracle.avgpool_bwd(oracle.avgpool(a), 8, 8))
    m_ref, i_ref = oracle.maxpool2x2(a)
    m = f(*m_ref.shape); idx = torch.empty(m_ref.shape, dtype=torch.int8, device="cuda")
    api.lpdt_maxpool2x2(2, 3, 8, 8, 16, dev(a), m, idx)
    assert np.array_equal(m.cpu().numpy(), m_ref) and np.array_equal(idx.cpu().numpy(), i_ref)
    dm = f(*a.shape)
    api.lpdt_maxpool2x2_bwd(2, 3, 8, 8, 16, m, idx, dm)
    assert np.array_equal(dm.cpu().numpy(), oracle.maxpool2x2_bwd(m_ref, i_ref, 8, 8))
    z = (3 * rng.standard_normal((3, 32, 10))).astype(np.float32)
    lab = rng.integers(0, 10, (3, 32)).astype(np.int32)
    loss_ref, dz_ref = oracle.softmax_ce(z, lab)
    loss = f(3); dz = f(3, 32, 10)
    api.lpdt_softmax_ce(3, 32, 10, dev(z), dev(lab), loss, dz)
    close(loss, loss_ref); close(dz, dz_ref, 1e-6, 1e-8)
    cs = torch.zeros(3, 14, device="cuda")
    api.lpdt_colsum(3, 32, 10, dev(z), cs[:, 4:], 14)
    close(cs[:, 4:], oracle.colsum(z), 1e-6, 1e-7)


def test_softmax_ce_label_out_of_range_is_guarded():
    """A label outside [0, K) is never used as an index: the sample adds nothing to the loss, its gradient has
    no one-hot term, the status word reports the bad argument, and the other samples are untouched."""
    rng = np.random.default_rng(5)
    z = (2 * rng.standard_normal((2, 8, 10))).astype(np.float32)
    lab = rng.integers(0, 10, (2, 8)).astype(np.int32)
    bad = lab.copy(); bad[0, 3] = 10; bad[1, 0] = -1; bad[1, 7] = 2 ** 30
    loss_ref, dz_ref = oracle.softmax_ce(z, lab)
    f = lambda *sh: torch.empty(*sh, dtype=torch.float32, device="cuda")
    loss, dz = f(2), f(2, 8, 10)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.lpdt_softmax_ce(2, 8, 10, dev(z), dev(lab), loss, dz, status)
    assert api.lpdt_check_status(status) == 0
    close(loss, loss_ref); close(dz, dz_ref, 1e-6, 1e-8)
    api.lpdt_softmax_ce(2, 8, 10, dev(z), dev(bad), loss, dz, status)
    assert api.lpdt_check_status(status) == 1                      # LPDT_ERR_INVALID_ARG
    # expected values from the oracle on the valid labels: drop the bad samples' loss terms, undo their one-hot
    ok = (bad >= 0) & (bad < 10)
    per_sample = np.stack([[oracle.softmax_ce(z[n:n + 1, b:b + 1], lab[n:n + 1, b:b + 1])[0][0] for b in range(8)]
                           for n in range(2)])
    close(loss, (per_sample * ok).sum(1) / 8)
    dz_want = dz_ref.copy()
    for n, b in zip(*np.nonzero(~ok)):
        dz_want[n, b, lab[n, b]] += 1.0 / 8
    close(dz, dz_want, 1e-6, 1e-7)


def test_qconv_bwd_weight_empty_batch_writes_zeros():
    """B = 0: the gradient of no samples is zero (written, not left stale), as forward and backward-data
    return LPDT_OK for an empty batch."""
    for case in [(2, 0, 8, 8, 16, 16, 3, 3, 1, 1), (1, 0, 4, 4, 3, 5, 3, 3, 1, 1)]:
        desc = api.conv_desc(*case)
        nodes, _, H, W, Cin, Cout = case[:6]
        wn = Cout * 9 * Cin
        E = torch.empty(nodes, 0, H, W, Cout, dtype=torch.int8, device="cuda")
        A = torch.empty(nodes, 0, H, W, Cin, dtype=torch.int8, device="cuda")
        sc = torch.ones(nodes, device="cuda")
        dW = torch.full((nodes, wn), 7.0, device="cuda")
        dWacc = torch.full((nodes, wn), 7, dtype=torch.int32, device="cuda")
        ws = ws_bytes(api.lpdt_qconv_workspace_size(desc, 2))
        api.lpdt_qconv_bwd_weight(desc, E, sc, A, sc, dW=dW, dw_node_stride=wn, dWacc=dWacc, ws=ws)
        torch.cuda.synchronize()
        assert not dW.any() and not dWacc.any()


def test_bounded_wait_runs_out_and_reports():
    """The barrier wait of the tensor-core kernels with a 1 ms limit on a barrier nothing arrives at: the
    kernel returns, the status word holds LPDT_ERR_TIMEOUT, and the context stays usable."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    returned = torch.zeros(1, dtype=torch.int32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    api.lpdt_selftest_bounded_wait(1_000_000, status, returned)
    e1.record()
    assert api.lpdt_check_status(status) == 5                      # LPDT_ERR_TIMEOUT
    assert int(returned.item()) == 2
    ms = e0.elapsed_time(e1)
    assert 0.9 <= ms < 50.0, ms
    with pytest.raises(api.LpdtError):
        api.lpdt_selftest_bounded_wait(10 ** 9, status, returned)  # limits beyond 50 ms are refused on the host
    # the device is still healthy: an ordinary call runs and matches the oracle
    x = np.random.default_rng(0).standard_normal((2, 1000)).astype(np.float32)
    q = torch.empty(2, 1000, dtype=torch.int8, device="cuda"); s = torch.empty(2, device="cuda")
    api.lpdt_quantize(dev(x), 2, 1000, 1000, q, s, ws_bytes(api.lpdt_quantize_workspace_size(2)))
    q_ref, s_ref = oracle.quantize_sym_s8(x)
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)


def test_batched_reductions_equal_the_single_calls():
    """lpdt_range_evonorm_bwd_params_batch and lpdt_dequantize_acc_batch: many layers in one launch, bit-identical
    to the per-layer calls (which the tests above compare with the oracle)."""
    rng = np.random.default_rng(12)
    nodes, B = 3, 5
    layers = [(8, 8, 16, 4), (4, 4, 64, 8), (6, 5, 12, 3)]                   # H, W, C, groups
    stride = sum(3 * c for _, _, c, _ in layers) + 11
    G1 = torch.zeros(nodes, stride, device="cuda"); G2 = torch.zeros_like(G1)
    wss, offs, off = [], [], 3
    for H, W, C, groups in layers:
        x, P, dy = _ren_inputs((nodes, B, H, W, C, groups), seed=C)
        Pd, xd = dev(P), dev(x)
        f = lambda *sh: torch.empty(*sh, dtype=torch.float32, device="cuda")
        i = lambda *sh: torch.empty(*sh, dtype=torch.int32, device="cuda")
        y, gmin, gmax, amn, amx = f(*x.shape), f(nodes, B, groups), f(nodes, B, groups), i(nodes, B, groups), i(nodes, B, groups)
        api.lpdt_range_evonorm_fwd(nodes, B, H, W, C, groups, 1e-5, xd, Pd, Pd[:, C:], Pd[:, 2 * C:], P.shape[1], y, gmin,
                                   gmax, amn, amx)
        ws = ws_bytes(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, C))
        api.lpdt_range_evonorm_bwd(nodes, B, H, W, C, groups, 1e-5, dev(dy), xd, Pd, Pd[:, C:], P.shape[1], gmin, gmax, amn,
                                   amx, f(*x.shape), None, None, None, stride, ws)
        api.lpdt_range_evonorm_bwd_params(nodes, B, C, ws, G1[:, off:], G1[:, off + C:], G1[:, off + 2 * C:], stride)
        wss.append(ws); offs.append(off)
        off += 3 * C
    api.lpdt_range_evonorm_bwd_params_batch(nodes, B, [c for _, _, c, _ in layers], wss, offs, G2, stride)
    assert torch.equal(G1, G2) and G1.abs().sum() > 0
    # int32 sums of three tensors, each a contiguous [nodes][size] block, into one strided fp32 row per node
    sizes, acc_off, out_off = [432, 1000, 7], [0, 64 * 21, 64 * 21 + 64 * 47], [5, 600, 1700]
    acc = torch.from_numpy(rng.integers(-2 ** 31, 2 ** 31 - 1, 64 * 21 + 64 * 47 + 64, dtype=np.int64).astype(np.int32)).cuda()
    s1 = [dev(rng.uniform(0.001, 0.1, nodes).astype(np.float32)) for _ in sizes]
    s2 = [dev(rng.uniform(0.001, 0.1, nodes).astype(np.float32)) for _ in sizes]
    out = torch.zeros(nodes, 1800, device="cuda")
    api.lpdt_dequantize_acc_batch(acc, nodes, acc_off, sizes, out_off, s1, s2, out, 1800)
    want = np.zeros((nodes, 1800), np.float32)
    for t, n in enumerate(sizes):
        a = acc[acc_off[t]:acc_off[t] + nodes * n].cpu().numpy().reshape(nodes, 1, n)
        want[:, out_off[t]:out_off[t] + n] = oracle.dequant_acc(a, s1[t].cpu().numpy(), s2[t].cpu().numpy()).reshape(nodes, n)
    assert np.array_equal(out.cpu().numpy(), want)


@pytest.mark.parametrize("cluster", ["1", "2", "8"])
def test_range_evonorm_cases_on_every_cluster_size(cluster):
    """The forward kernel splits a sample over 1-8 CTAs by a size rule; the cases are re-run in child
    processes with the cluster size forced (capped so that every CTA keeps a thread row)."""
    import os, subprocess, sys
    if os.environ.get("LPDT_CHILD") == "1":
        pytest.skip("already inside a child run")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    child_env = dict(os.environ, LPDT_CHILD="1", LPDT_REN_CLUSTER=cluster)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_ops.py"), "-m", "gpu",
                        "-q", "-x", "-k", "test_range_evonorm_fwd or test_fused_ranges"], env=child_env, cwd=root,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]


@pytest.mark.parametrize("env", [{"LPDT_FORCE_HALO": "1"}, {"LPDT_DISABLE_HALO": "1"}, {"LPDT_DISABLE_TC": "1"},
                                 {"LPDT_AFFINE_SEPARATE": "1"}, {"LPDT_PIX_DIRECT_STORE": "1", "LPDT_DISABLE_HALO": "1"},
                                 {"LPDT_PIX_TWO": "0", "LPDT_DISABLE_HALO": "1"}])
def test_qconv_cases_on_every_kernel_family(env):
    """The kernel choice is made once per process from the environment, so the contraction
    cases are re-run in child processes with the halo kernels forced, with the halo kernels
    off (general tensor-core kernels) and with the tensor-core engine off (CUDA-core kernels)."""
    import os, subprocess, sys
    if os.environ.get("LPDT_CHILD") == "1":
        pytest.skip("already inside a child run")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    child_env = dict(os.environ, LPDT_CHILD="1", **env)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_ops.py"), "-m", "gpu",
                        "-q", "-x", "-k", "test_qconv_all_three or test_qconv_extreme or test_qconv_fwd_affine or test_qconv_bwd_affine"], env=child_env, cwd=root,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
