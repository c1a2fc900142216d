"""Time the int8 contraction alone (forward, backward-data, backward-weight) on
seeded random operands, through the C ABI.

    python -m paper_2111_09389_b200.contraction_sweep gemm M N K [--iters 20]
    python -m paper_2111_09389_b200.contraction_sweep conv C HW BATCH [--nodes 1]
    python -m paper_2111_09389_b200.contraction_sweep sweep           # the large GEMM / conv grid

Operands are iid uniform int8 in [-127, 127]; every shape runs with int32
accumulation and the fused fp32 dequantize.  With --graph (the sweep's default)
the calls are recorded into one CUDA graph and its replay is timed, so that the
host's per-call cost (two tensor-map encodes and the ctypes call, 15-20 us) does
not hide kernels of a few microseconds; consecutive calls then rotate through
enough operand/result sets that the bytes touched between two uses of the same
set exceed the 126 MB L2 (shapes whose own operands exceed it use one set).  The optional pass
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


L2_BYTES = 126 * 1024 * 1024


def time_case(nodes, B, H, W, Cin, Cout, R, S, stride, pad, iters=20, warmup=3, passes=("fwd", "bwd_data", "bwd_weight"),
              label=None, graph=False, quiet=False):
    """graph=True records the `iters` calls into one CUDA graph and times its replay, which
    takes the host's launch cost out of calls that run for only a few microseconds; the calls
    rotate through `nsets` operand sets so that no call finds its operands in L2."""
    desc = api.conv_desc(nodes, B, H, W, Cin, Cout, R, S, stride, pad)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    set_bytes = nodes * (B * H * W * Cin + Cout * R * S * Cin + B * Ho * Wo * Cout) + \
        4 * nodes * min(B * Ho * Wo * Cout, B * H * W * Cin, Cout * R * S * Cin)
    nsets = 1 if not graph else max(1, min(iters, -(-int(1.25 * L2_BYTES) // set_bytes)))
    sets = []
    for i in range(nsets):
        sets.append(dict(A=_rand_s8((nodes, B, H, W, Cin), 1 + 3 * i), Wq=_rand_s8((nodes, Cout, R, S, Cin), 2 + 3 * i),
                         E=_rand_s8((nodes, B, Ho, Wo, Cout), 3 + 3 * i),
                         Y=torch.empty(nodes, B, Ho, Wo, Cout, device="cuda"), dA=torch.empty(nodes, B, H, W, Cin, device="cuda"),
                         dW=torch.empty(nodes, Cout * R * S * Cin, device="cuda")))
    sc = torch.full((nodes,), 1.0 / 127, device="cuda")
    ws = torch.empty(max(api.lpdt_qconv_workspace_size(desc, w) for w in (0, 1, 2)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    macs = nodes * B * Ho * Wo * Cout * Cin * R * S
    t0 = sets[0]
    calls = {
        "fwd": (lambda t: api.lpdt_qconv_fwd(desc, t["A"], sc, t["Wq"], sc, Y=t["Y"], ws=ws, dev_status=status),
                t0["A"].numel() + t0["Wq"].numel() + 4 * t0["Y"].numel()),
        "bwd_data": (lambda t: api.lpdt_qconv_bwd_data(desc, t["E"], sc, t["Wq"], sc, dA=t["dA"], ws=ws, dev_status=status),
                     t0["E"].numel() + t0["Wq"].numel() + 4 * t0["dA"].numel()),
        "bwd_weight": (lambda t: api.lpdt_qconv_bwd_weight(desc, t["E"], sc, t["A"], sc, dW=t["dW"],
                                                           dw_node_stride=t["dW"].shape[1], ws=ws, dev_status=status),
                       t0["E"].numel() + t0["A"].numel() + 4 * t0["dW"].numel()),
    }
    if "fwd_affine" in passes:       # zero-point operands: unsigned codes, per-node zero points
        zA = torch.full((nodes,), 131, dtype=torch.int32, device="cuda")
        zW = torch.full((nodes,), 120, dtype=torch.int32, device="cuda")
        wsa = torch.empty(api.lpdt_qconv_fwd_affine_workspace_size(desc), dtype=torch.uint8, device="cuda")
        calls["fwd_affine"] = (lambda t: api.lpdt_qconv_fwd_affine(desc, t["A"].view(torch.uint8), sc, zA,
                                                                   t["Wq"].view(torch.uint8), sc, zW, Y=t["Y"], ws=wsa,
                                                                   dev_status=status),
                               t0["A"].numel() + t0["Wq"].numel() + 4 * t0["Y"].numel())
    out = []
    for name in passes:
        fn, min_bytes = calls[name]
        for i in range(warmup):
            fn(sets[i % nsets])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(iters):
                    fn(sets[i % nsets])
            g.replay()
            torch.cuda.synchronize()
            e0.record()
            g.replay()
        else:
            e0.record()
            for i in range(iters):
                fn(sets[i % nsets])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        rec = {"shape": label or f"conv n{nodes} b{B} {H}x{W} {Cin}->{Cout} {R}x{S} s{stride}", "pass": name,
               "ms": ms, "tops": 2 * macs / (ms * 1e-3) / 1e12, "macs": macs, "min_hbm_bytes": int(min_bytes),
               "gbs_at_min_bytes": min_bytes / (ms * 1e-3) / 1e9, "dev_status": int(status.item()),
               "timing": f"graph replay of {iters} calls over {nsets} operand sets" if graph else f"{iters} eager calls"}
        if not quiet:
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
    ap.add_argument("--eager", action="store_true", help="sweep: time eager calls instead of a graph replay")
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
                    gemm(M, N, K, iters=a.iters, warmup=2, passes=passes, graph=not a.eager)
        for C in (64, 256, 512):
            for HW in (32, 56):
                conv(C, HW, 256, iters=a.iters, warmup=2, passes=passes, graph=not a.eager)


if __name__ == "__main__":
    main(sys.argv[1:])
