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


@pytest.mark.parametrize("M,N,K", [(4096, 8192, 2048), (8192, 8192, 8192), (1024, 1024, 8192)])
def test_large_gemm_three_passes(M, N, K):
    desc = api.conv_desc(1, M, 1, 1, K, N, 1, 1, 1, 0)
    A, Wq, E = _rand((1, M, 1, 1, K), 1), _rand((1, N, 1, 1, K), 2), _rand((1, M, 1, 1, N), 3)
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
    # sampled rows (spanning the first, a middle and the ragged last tile), recomputed by the oracle
    rows = np.unique(np.concatenate([np.arange(3), np.random.default_rng(0).integers(0, M, 10), [M - 1]]))
    Ah, Wh, Eh = A.cpu().numpy(), Wq.cpu().numpy(), E.cpu().numpy()
    ref, _ = oracle.qconv_fwd(Ah[:, rows], Wh, 1, 0)
    assert np.array_equal(Y.cpu().numpy()[:, rows], ref)
    ref, _ = oracle.qconv_bwd_data(Eh[:, rows], Wh, 1, 1, 1, 0)
    assert np.array_equal(dA.cpu().numpy()[:, rows], ref)
    cols = np.unique(np.concatenate([np.arange(2), np.random.default_rng(1).integers(0, N, 6), [N - 1]]))
    ref, _ = oracle.qconv_bwd_weight(np.ascontiguousarray(Eh[..., cols]), Ah, 1, 1, 1, 0)   # dW rows = output channels
    assert np.array_equal(dW.cpu().numpy()[:, cols], ref)


@pytest.mark.parametrize("C,HW,batch", [(64, 56, 256), (256, 32, 256), (512, 32, 64)])
def test_large_conv_three_passes(C, HW, batch):
    desc = api.conv_desc(1, batch, HW, HW, C, C, 3, 3, 1, 1)
    A, Wq, E = _rand((1, batch, HW, HW, C), 4), _rand((1, C, 3, 3, C), 5), _rand((1, batch, HW, HW, C), 6)
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
    ref, _ = oracle.qconv_fwd(Ah, Wh, 1, 1)
    assert np.array_equal(Y[:, imgs].cpu().numpy(), ref)
    ref, _ = oracle.qconv_bwd_data(Eh, Wh, HW, HW, 1, 1)
    assert np.array_equal(dA[:, imgs].cpu().numpy(), ref)
    # adjoint identity over the whole batch: <fwd(A,W), E> = <W, bwd_weight(E,A)> = <A, bwd_data(E,W)> (int64)
    lhs = int((Y.to(torch.int64) * E.to(torch.int64)).sum())
    assert lhs == int((dW.to(torch.int64) * Wq.to(torch.int64)).sum())
    assert lhs == int((dA.to(torch.int64) * A.to(torch.int64)).sum())
    # a few weight-gradient entries recomputed over the full batch by the oracle (one output channel at a time)
    co = [0, C - 1]
    ref, _ = oracle.qconv_bwd_weight(np.ascontiguousarray(E[..., co].cpu().numpy()), A[..., :16].cpu().numpy().copy(), 3, 3, 1, 1)
    assert np.array_equal(dW[:, co][..., :16].cpu().numpy(), ref)


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
