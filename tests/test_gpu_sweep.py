"""GPU parity of the contraction at the sizes of the roofline sweep: sampled outputs the oracle
recomputes one by one, plus the whole-result checksum identity
    sum_ij C_ij = sum_k (sum_i A_ik)(sum_j B_jk)        (int64, exact)
and its analogues for the two backward products."""
import numpy as np
import pytest
import torch

import oracle
from paper_2111_09389_b200 import api

pytestmark = pytest.mark.gpu


def _rand(shape, seed):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    return torch.randint(-127, 128, shape, generator=g, device="cuda", dtype=torch.int8)


SIZES = (1024, 2048, 4096, 8192)
GEMMS = [(M, N, K) for M in SIZES for N in SIZES for K in SIZES]      # all 64 shapes of the sweep
N_SAMPLED = 64


def _sampled(n, seed):
    """64 distinct indices in [0, n): the first three, the last one, and random ones (first, middle
    and last tiles are all hit)."""
    r = np.random.default_rng(seed).permutation(n)[:N_SAMPLED]
    return np.unique(np.concatenate([r, np.array([0, 1, 2, n - 1]) % n]))


def _check_fp32_paths(desc, A, Wq, E, Y, dA, dW, ws, status):
    """The calls as the benchmark makes them (fp32 results only, scales 1/127): each must equal the
    dequantized int32 result of the raw-accumulator call element for element; the oracle's dequantize
    is the reference on a sample of rows."""
    sc = torch.full((1,), 1.0 / 127, device="cuda")
    Yf = torch.empty(Y.shape, device="cuda"); dAf = torch.empty(dA.shape, device="cuda")
    dWf = torch.empty(1, dW.numel(), device="cuda")
    api.lpdt_qconv_fwd(desc, A, sc, Wq, sc, Y=Yf, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_data(desc, E, sc, Wq, sc, dA=dAf, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_weight(desc, E, sc, A, sc, dW=dWf, dw_node_stride=dWf.shape[1], ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    s_h = sc.cpu().numpy()
    for f, i in ((Yf, Y), (dAf, dA), (dWf, dW)):
        f2, i2 = f.reshape(-1, i.shape[-1]), i.reshape(-1, i.shape[-1])
        rows = torch.from_numpy(_sampled(f2.shape[0], 5)).cuda()
        want = oracle.dequant_acc(i2[rows].cpu().numpy()[None], s_h, s_h)[0]
        assert np.array_equal(f2[rows].cpu().numpy(), want)
        step = max(1, (1 << 26) // f2.shape[1])
        for r in range(0, f2.shape[0], step):                     # whole tensor, in slabs
            assert torch.equal(f2[r:r + step], i2[r:r + step].to(torch.float32) * (sc * sc))


@pytest.mark.parametrize("M,N,K", GEMMS, ids=[f"M{m}N{n}K{k}" for m, n, k in GEMMS])
def test_sweep_gemm_three_passes(M, N, K):
    """Every GEMM shape of the sweep, forward / backward-data / backward-weight: the exact int64 checksum of
    the whole result and 64 full-length rows (columns of the weight gradient) recomputed by the oracle."""
    desc = api.conv_desc(1, M, 1, 1, K, N, 1, 1, 1, 0)
    seed = (M * 31 + N) * 31 + K
    A, Wq, E = _rand((1, M, 1, 1, K), seed), _rand((1, N, 1, 1, K), seed + 1), _rand((1, M, 1, 1, N), seed + 2)
    ws = torch.empty(max(api.lpdt_qconv_workspace_size(desc, w) for w in (0, 1, 2)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = torch.empty(1, M, 1, 1, N, dtype=torch.int32, device="cuda")
    dA = torch.empty(1, M, 1, 1, K, dtype=torch.int32, device="cuda")
    dW = torch.empty(1, N, 1, 1, K, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd(desc, A, None, Wq, None, Yacc=Y, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_data(desc, E, None, Wq, None, dAacc=dA, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_weight(desc, E, None, A, None, dWacc=dW, ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    a64 = lambda t, dim: t.reshape(t.shape[1], t.shape[-1]).sum(dim=dim, dtype=torch.int64)
    # checksums over the whole results
    assert int(Y.sum(dtype=torch.int64)) == int((a64(A, 0) * a64(Wq, 0)).sum())
    assert int(dA.sum(dtype=torch.int64)) == int((a64(E, 0) * a64(Wq, 1)).sum())
    assert int(dW.sum(dtype=torch.int64)) == int((a64(E, 1) * a64(A, 1)).sum())
    rows = _sampled(M, seed)
    rows_d = torch.from_numpy(rows).cuda()
    Wh = Wq.cpu().numpy()
    ref, ovf = oracle.qconv_fwd(A[:, rows_d].cpu().numpy(), Wh, 1, 0)
    assert ovf == 0 and np.array_equal(Y[:, rows_d].cpu().numpy(), ref)
    ref, ovf = oracle.qconv_bwd_data(E[:, rows_d].cpu().numpy(), Wh, 1, 1, 1, 0)
    assert ovf == 0 and np.array_equal(dA[:, rows_d].cpu().numpy(), ref)
    cols = _sampled(N, seed + 7)
    cols_d = torch.from_numpy(cols).cuda()
    ref, ovf = oracle.qconv_bwd_weight(E[..., cols_d].contiguous().cpu().numpy(), A.cpu().numpy(), 1, 1, 1, 0)
    assert ovf == 0 and np.array_equal(dW[:, cols_d].cpu().numpy(), ref)     # dW rows = output channels
    _check_fp32_paths(desc, A, Wq, E, Y, dA, dW, ws, status)


@pytest.mark.parametrize("C", [64, 256, 512])
@pytest.mark.parametrize("HW", [32, 56])
def test_sweep_conv_three_passes(C, HW):
    """Every 3x3 convolution of the sweep at batch 256, three passes: three whole images recomputed by the
    oracle (forward and backward-data), the exact adjoint identities over the whole batch, and a block of
    weight-gradient entries recomputed over all 256 images."""
    batch = 256
    desc = api.conv_desc(1, batch, HW, HW, C, C, 3, 3, 1, 1)
    A, Wq, E = _rand((1, batch, HW, HW, C), 4 + C), _rand((1, C, 3, 3, C), 5 + C), _rand((1, batch, HW, HW, C), 6 + C)
    ws = torch.empty(max(api.lpdt_qconv_workspace_size(desc, w) for w in (0, 1, 2)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = torch.empty(1, batch, HW, HW, C, dtype=torch.int32, device="cuda")
    dA = torch.empty_like(Y)
    dW = torch.empty(1, C, 3, 3, C, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd(desc, A, None, Wq, None, Yacc=Y, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_data(desc, E, None, Wq, None, dAacc=dA, ws=ws, dev_status=status)
    api.lpdt_qconv_bwd_weight(desc, E, None, A, None, dWacc=dW, ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # sampled images, every pixel and channel of them
    imgs = [0, batch // 2 + 1, batch - 1]
    Ah, Wh, Eh = A[:, imgs].cpu().numpy(), Wq.cpu().numpy(), E[:, imgs].cpu().numpy()
    ref, ovf = oracle.qconv_fwd(Ah, Wh, 1, 1)
    assert ovf == 0 and np.array_equal(Y[:, imgs].cpu().numpy(), ref)
    ref, ovf = oracle.qconv_bwd_data(Eh, Wh, HW, HW, 1, 1)
    assert ovf == 0 and np.array_equal(dA[:, imgs].cpu().numpy(), ref)
    # adjoint identity over the whole batch: <fwd(A,W), E> = <W, bwd_weight(E,A)> = <A, bwd_data(E,W)> (int64)
    dot = lambda a, b: sum(int((a[:, i:i + 32].to(torch.int64) * b[:, i:i + 32].to(torch.int64)).sum())
                           for i in range(0, a.shape[1], 32))
    lhs = dot(Y, E)
    assert lhs == int((dW.to(torch.int64) * Wq.to(torch.int64)).sum())
    assert lhs == dot(dA, A)
    # weight-gradient entries recomputed over the full batch by the oracle: 8 output channels (first, last,
    # one per 64-channel tile) x the first and the last 16 input channels x all 9 taps
    co = sorted({0, C - 1, C // 2, C // 2 + 1, 17 % C, C - 18, (C // 4) * 3, 5})
    for c0 in (0, C - 16):
        ref, ovf = oracle.qconv_bwd_weight(np.ascontiguousarray(E[..., co].cpu().numpy()),
                                           A[..., c0:c0 + 16].contiguous().cpu().numpy(), 3, 3, 1, 1)
        assert ovf == 0 and np.array_equal(dW[:, co][..., c0:c0 + 16].cpu().numpy(), ref)
    del Ah, Eh
    _check_fp32_paths(desc, A, Wq, E, Y, dA, dW, ws, status)


@pytest.mark.parametrize("shape", [("gemm", 4096, 4096, 4096), ("conv", 256, 32, 64)])
def test_large_affine_forward(shape):
    """Zero-point operands at sweep sizes: sampled rows / images recomputed by the oracle (modulo 2^32: with
    K up to 4096 the true sums stay inside int32)."""
    g = torch.Generator(device="cuda"); g.manual_seed(9)
    if shape[0] == "gemm":
        _, M, N, K = shape
        case = (1, M, 1, 1, K, N, 1, 1, 1, 0)
    else:
        _, Cc, HW, batch = shape
        case = (1, batch, HW, HW, Cc, Cc, 3, 3, 1, 1)
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    desc = api.conv_desc(*case)
    A = torch.randint(0, 256, (nodes, B, H, W, Cin), generator=g, device="cuda", dtype=torch.uint8)
    Wq = torch.randint(0, 256, (nodes, Cout, R, S, Cin), generator=g, device="cuda", dtype=torch.uint8)
    zA = torch.tensor([133], dtype=torch.int32, device="cuda")
    zW = torch.tensor([121], dtype=torch.int32, device="cuda")
    Y = torch.empty(nodes, B, H, W, Cout, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.lpdt_qconv_fwd_affine_workspace_size(desc), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_fwd_affine(desc, A, None, zA, Wq, None, zW, Yacc=Y, ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = np.unique(np.concatenate([np.arange(2), np.random.default_rng(3).integers(0, B, 4), [B - 1]]))
    ref, ovf = oracle.qconv_fwd_affine(A.cpu().numpy()[:, rows], zA.cpu().numpy(), Wq.cpu().numpy(), zW.cpu().numpy(),
                                       stride, pad)
    assert ovf == 0
    assert np.array_equal(Y.cpu().numpy()[:, rows], ref)


@pytest.mark.parametrize("shape", [("gemm", 2048, 4096, 4096), ("conv", 256, 32, 32)])
def test_large_affine_backward(shape):
    """Zero-point operands at sweep sizes, both backward products: sampled rows / images and a block of
    weight-gradient entries recomputed by the oracle."""
    g = torch.Generator(device="cuda"); g.manual_seed(19)
    if shape[0] == "gemm":
        _, M, N, K = shape
        case = (1, M, 1, 1, K, N, 1, 1, 1, 0)
    else:
        _, Cc, HW, batch = shape
        case = (1, batch, HW, HW, Cc, Cc, 3, 3, 1, 1)
    nodes, B, H, W, Cin, Cout, R, S, stride, pad = case
    desc = api.conv_desc(*case)
    u8 = lambda *sh: torch.randint(0, 256, sh, generator=g, device="cuda", dtype=torch.uint8)
    A, Wq, E = u8(nodes, B, H, W, Cin), u8(nodes, Cout, R, S, Cin), u8(nodes, B, H, W, Cout)
    zA, zW, zE = (torch.tensor([v], dtype=torch.int32, device="cuda") for v in (133, 121, 90))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dA = torch.empty(nodes, B, H, W, Cin, dtype=torch.int32, device="cuda")
    dW = torch.empty(nodes, Cout, R, S, Cin, dtype=torch.int32, device="cuda")
    api.lpdt_qconv_bwd_data_affine(desc, E, None, zE, Wq, None, zW, dAacc=dA, dev_status=status,
                                   ws=torch.empty(api.lpdt_qconv_bwd_data_affine_workspace_size(desc), dtype=torch.uint8, device="cuda"))
    api.lpdt_qconv_bwd_weight_affine(desc, E, None, zE, A, None, zA, dWacc=dW, dev_status=status,
                                     ws=torch.empty(api.lpdt_qconv_bwd_weight_affine_workspace_size(desc), dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = np.unique(np.concatenate([np.arange(2), np.random.default_rng(3).integers(0, B, 4), [B - 1]]))
    ref, _ = oracle.qconv_bwd_data_affine(E.cpu().numpy()[:, rows], zE.cpu().numpy(), Wq.cpu().numpy(), zW.cpu().numpy(),
                                          H, W, stride, pad)
    assert np.array_equal(dA.cpu().numpy()[:, rows], ref)             # the wrapped int32 sums
    co = [0, Cout // 2 + 1, Cout - 1]
    ref, _ = oracle.qconv_bwd_weight_affine(np.ascontiguousarray(E[..., co].cpu().numpy()), zE.cpu().numpy(),
                                            A[..., :16].contiguous().cpu().numpy(), zA.cpu().numpy(), R, S, stride, pad)
    assert np.array_equal(dW[:, co][..., :16].cpu().numpy(), ref)
