"""Time the int8 contraction alone (forward, backward-data, backward-weight) on
seeded random operands, through the C ABI.

    python -m paper_2111_09389_b200.contraction_sweep gemm M N K [--iters 20]
    python -m paper_2111_09389_b200.contraction_sweep conv C HW BATCH [--nodes 1]
    python -m paper_2111_09389_b200.contraction_sweep sweep           # the large GEMM / conv grid

Operands are iid uniform int8 in [-127, 127]; every shape runs with int32
accumulation and the fused fp32 dequantize.  The optional pass
`fwd_affine` times the forward product on zero-point operands (same operand
bytes; its correction pass re-reads and re-writes the result).  Prints one JSON line per
(shape, pass) with the CUDA-event time, int8 TOPS (2 * MACs / time) and the
HBM bytes the pass must move at least.
"""
import argparse
import json
import sys

import numpy as np
import torch

from . import api, workloads


def _rand_s8(shape, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return torch.randint(-127, 128, shape, generator=g, device="cuda", dtype=torch.int8)


def time_case(nodes, B, H, W, Cin, Cout, R, S, stride, pad, iters=20, warmup=3, passes=("fwd", "bwd_data", "bwd_weight"),
              label=None, graph=False):
    """graph=True records the `iters` calls into one CUDA graph and times its replay, which
    takes the host's launch cost out of calls that run for only a few microseconds."""
    desc = api.conv_desc(nodes, B, H, W, Cin, Cout, R, S, stride, pad)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    A = _rand_s8((nodes, B, H, W, Cin), 1)
    Wq = _rand_s8((nodes, Cout, R, S, Cin), 2)
    E = _rand_s8((nodes, B, Ho, Wo, Cout), 3)
    sc = torch.full((nodes,), 1.0 / 127, device="cuda")
    Y = torch.empty(nodes, B, Ho, Wo, Cout, device="cuda")
    dA = torch.empty(nodes, B, H, W, Cin, device="cuda")
    dW = torch.empty(nodes, Cout * R * S * Cin, device="cuda")
    ws = torch.empty(max(api.lpdt_qconv_workspace_size(desc, w) for w in (0, 1, 2)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    macs = nodes * B * Ho * Wo * Cout * Cin * R * S
    calls = {
        "fwd": (lambda: api.lpdt_qconv_fwd(desc, A, sc, Wq, sc, Y=Y, ws=ws, dev_status=status),
                A.numel() + Wq.numel() + 4 * Y.numel()),
        "bwd_data": (lambda: api.lpdt_qconv_bwd_data(desc, E, sc, Wq, sc, dA=dA, ws=ws, dev_status=status),
                     E.numel() + Wq.numel() + 4 * dA.numel()),
        "bwd_weight": (lambda: api.lpdt_qconv_bwd_weight(desc, E, sc, A, sc, dW=dW, dw_node_stride=dW.shape[1], ws=ws,
                                                         dev_status=status),
                       E.numel() + A.numel() + 4 * dW.numel()),
    }
    if "fwd_affine" in passes:       # zero-point operands: unsigned codes, per-node zero points
        Au, Wu = A.view(torch.uint8), Wq.view(torch.uint8)
        zA = torch.full((nodes,), 131, dtype=torch.int32, device="cuda")
        zW = torch.full((nodes,), 120, dtype=torch.int32, device="cuda")
        wsa = torch.empty(api.lpdt_qconv_fwd_affine_workspace_size(desc), dtype=torch.uint8, device="cuda")
        calls["fwd_affine"] = (lambda: api.lpdt_qconv_fwd_affine(desc, Au, sc, zA, Wu, sc, zW, Y=Y, ws=wsa,
                                                                 dev_status=status),
                               A.numel() + Wq.numel() + 4 * Y.numel())
    out = []
    for name in passes:
        fn, min_bytes = calls[name]
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for _ in range(iters):
                    fn()
            g.replay()
            torch.cuda.synchronize()
            e0.record()
            g.replay()
        else:
            e0.record()
            for _ in range(iters):
                fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        rec = {"shape": label or f"conv n{nodes} b{B} {H}x{W} {Cin}->{Cout} {R}x{S} s{stride}", "pass": name,
               "ms": ms, "tops": 2 * macs / (ms * 1e-3) / 1e12, "macs": macs, "min_hbm_bytes": int(min_bytes),
               "gbs_at_min_bytes": min_bytes / (ms * 1e-3) / 1e9, "dev_status": int(status.item())}
        print(json.dumps(rec), flush=True)
        out.append(rec)
    return out


def gemm(M, N, K, **kw):
    return time_case(1, M, 1, 1, K, N, 1, 1, 1, 0, label=f"gemm M{M} N{N} K{K}", **kw)


def conv(C, HW, batch, nodes=1, **kw):
    return time_case(nodes, batch, HW, HW, C, C, 3, 3, 1, 1, label=f"conv3x3 C{C} {HW}x{HW} batch{batch} nodes{nodes}", **kw)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["gemm", "conv", "sweep"])
    ap.add_argument("dims", nargs="*", type=int)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--nodes", type=int, default=1)
    ap.add_argument("--passes", default="fwd,bwd_data,bwd_weight")
    ap.add_argument("--graph", action="store_true", help="time a CUDA-graph replay of the calls")
    a = ap.parse_args(argv)
    passes = tuple(a.passes.split(","))
    if a.kind == "gemm":
        gemm(*a.dims, iters=a.iters, warmup=a.warmup, passes=passes, graph=a.graph)
    elif a.kind == "conv":
        conv(*a.dims, nodes=a.nodes, iters=a.iters, warmup=a.warmup, passes=passes, graph=a.graph)
    else:
        sizes = (1024, 2048, 4096, 8192)
        for M in sizes:
            for N in sizes:
                for K in sizes:
                    gemm(M, N, K, iters=max(3, a.iters // 4), warmup=2, passes=passes)
        for C in (64, 256, 512):
            for HW in (32, 56):
                conv(C, HW, 256, iters=max(3, a.iters // 4), warmup=2, passes=passes)


if __name__ == "__main__":
    main(sys.argv[1:])
