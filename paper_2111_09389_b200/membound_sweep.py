"""Time the memory-bound kernels of the step alone, on tensors much larger than
L2, through the C ABI, and report achieved GB/s on their algorithmic bytes.

    python -m paper_2111_09389_b200.membound_sweep [--iters 20] [--peak-gbs 6547.2] [--only ren_bwd,quantize]

Cases (activation kernels: the VGG-11-shaped workload's first layer, 8 nodes, with
batch 128 so that each fp32 tensor is 268 MB; parameter kernels: 16 nodes with a
32x replicated ResNet-20 parameter vector, 554 MB per array):

  quantize            range pass + scale-and-round: 4 B read twice + 1 B written per element
  quantize_stochastic the same with Philox stochastic rounding
  quantize_with_range range supplied by the producer: 4 B read + 1 B written
  dequantize          1 B read + 4 B written: a write-dominated stream (80 % of its bytes are stores)
  ren_fwd             4 B read + 4 B written (the second read of a sample comes from L2)
  ren_fwd_res         + 4 B shortcut read
  ren_bwd             dy, x read + dx written: 12 B
  evonorm_s0_fwd      comparison layer: 4 B read + 4 B written (second read of a sample from L2)
  evonorm_s0_bwd      dy, x read (twice, the second time from L2) + dx written: 12 B
  range_bn_fwd        statistics pass 4 B + apply pass 4 B read + 4 B written: 12 B (batch statistics: two launches)
  range_bn_bwd        sums pass 8 B + apply pass 4 B read + 4 B written: 16 B
  residual_add        8 B read + 4 B written
  sgd_update          12 B per parameter
  gossip_dense        x_half, x_hat read; x_hat, x written: 16 B per parameter
  gossip_top1pct      + one more pass over x_half and x_hat for the magnitude select: 24 B
  gossip_dense_q8     8-bit messages: + one range pass over x_half and x_hat: 24 B
  gossip_top1pct_q8   range pass + select pass + mix: 32 B

  ren_*_q8_<shape>    Range-EvoNorm with the requantize step inside, on ResNet-20-shaped layers (32 samples per
                      node; enough nodes for 134 MB per fp32 tensor): forward 4 B read + 1 B written, backward
                      8 B read + 1 B written; ren_*_then_quantize_<shape> is the two-call form doing the same
                      job (charged the same bytes, so the two lines compare directly)

One JSON line per case.
"""
import argparse
import json

import torch

from . import api, workloads


def _time(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def cases(nodes=8, B=128, H=32, W=32, Cc=64, d=32 * 270410, gossip_nodes=16):
    """Yield (name, callable, algorithmic bytes per call)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    n = B * H * W * Cc
    tot = nodes * n
    x = torch.randn(nodes, n, generator=g, device="cuda")
    x2 = torch.randn(nodes, n, generator=g, device="cuda")
    y = torch.empty_like(x)
    q = torch.empty(nodes, n, dtype=torch.int8, device="cuda")
    scale = torch.empty(nodes, device="cuda")
    amax = x.abs().amax(dim=1).contiguous()
    ws = torch.empty(api.lpdt_quantize_workspace_size(nodes), dtype=torch.uint8, device="cuda")
    yield ("quantize", lambda: api.lpdt_quantize(x, nodes, n, n, q, scale, ws), tot * 9)
    yield ("quantize_stochastic", lambda: api.lpdt_quantize(x, nodes, n, n, q, scale, ws, rounding=1, seed=3), tot * 9)
    yield ("quantize_with_range", lambda: api.lpdt_quantize_with_range(x, nodes, n, n, amax, q, scale), tot * 5)
    api.lpdt_quantize_with_range(x, nodes, n, n, amax, q, scale)
    yield ("dequantize", lambda: api.lpdt_dequantize(q, nodes, n, scale, y), tot * 5)

    groups = Cc // 8
    v = torch.ones(nodes, Cc, device="cuda")
    gamma = torch.ones(nodes, Cc, device="cuda")
    beta = torch.zeros(nodes, Cc, device="cuda")
    gmin = torch.empty(nodes, B, groups, device="cuda")
    gmax = torch.empty_like(gmin)
    amin_i = torch.empty(nodes, B, groups, dtype=torch.int32, device="cuda")
    amax_i = torch.empty_like(amin_i)
    rng = torch.zeros(nodes, device="cuda")

    def ren_fwd(res=None):
        api.lpdt_range_evonorm_fwd(nodes, B, H, W, Cc, groups, 1e-5, x, v, gamma, beta, Cc, y, gmin, gmax, amin_i,
                                   amax_i, amax_out=rng, res=res)
    yield ("ren_fwd", ren_fwd, tot * 8)
    yield ("ren_fwd_res", lambda: ren_fwd(x2), tot * 12)

    dx = torch.empty_like(x)
    dv, dg, db = (torch.empty(nodes, Cc, device="cuda") for _ in range(3))
    wsb = torch.empty(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, Cc), dtype=torch.uint8, device="cuda")
    ren_fwd()
    yield ("ren_bwd", lambda: api.lpdt_range_evonorm_bwd(nodes, B, H, W, Cc, groups, 1e-5, x2, x, v, gamma, Cc, gmin,
                                                         gmax, amin_i, amax_i, dx, dv, dg, db, Cc, wsb, amax_out=rng),
           tot * 12)
    gm, gv = torch.empty(nodes, B, groups, device="cuda"), torch.empty(nodes, B, groups, device="cuda")
    yield ("evonorm_s0_fwd", lambda: api.lpdt_evonorm_s0_fwd(nodes, B, H, W, Cc, groups, 1e-5, x, v, gamma, beta, Cc, y,
                                                             gm, gv), tot * 8)
    wse = torch.empty(api.lpdt_evonorm_s0_bwd_workspace_size(nodes, B, Cc), dtype=torch.uint8, device="cuda")
    yield ("evonorm_s0_bwd", lambda: api.lpdt_evonorm_s0_bwd(nodes, B, H, W, Cc, groups, 1e-5, x2, x, v, gamma, Cc, gm,
                                                             gv, dx, dv, dg, db, Cc, wse), tot * 12)
    cm, cn, cx = (torch.empty(nodes, Cc, device="cuda") for _ in range(3))
    an, ax = (torch.empty(nodes, Cc, dtype=torch.int32, device="cuda") for _ in range(2))
    wsr = torch.empty(api.lpdt_range_bn_workspace_size(nodes, Cc), dtype=torch.uint8, device="cuda")
    yield ("range_bn_fwd", lambda: api.lpdt_range_bn_fwd(nodes, B, H, W, Cc, 1e-5, x, gamma, beta, Cc, y, cm, cn, cx, an,
                                                         ax, wsr), tot * 12)
    yield ("range_bn_bwd", lambda: api.lpdt_range_bn_bwd(nodes, B, H, W, Cc, 1e-5, x2, x, gamma, Cc, cm, cn, cx, an, ax,
                                                         dx, dg, db, Cc, wsr), tot * 16)
    yield ("residual_add", lambda: api.lpdt_residual_add(nodes, B, H, W, Cc, Cc, 1, 0, x, x2, y, amax_out=rng), tot * 12)
    del x2, dx

    N = gossip_nodes
    xh = torch.randn(N, d, generator=g, device="cuda")
    grad = torch.randn(N, d, generator=g, device="cuda")
    xhat = torch.zeros(N, d, device="cuda")
    xo = torch.empty(N, d, device="cuda")
    yield ("sgd_update", lambda: api.lpdt_sgd_update(N * d, xh, grad, 0.1, xo), N * d * 12)
    Wm = torch.from_numpy(workloads.ring_matrix(N)).float().cuda()
    gws = torch.empty(api.lpdt_gossip_mix_workspace_size(N, d, 1), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    yield ("gossip_dense", lambda: api.lpdt_gossip_mix(N, d, xh, xhat, xo, Wm, 1.0, [0, d], [d], gws, st), N * d * 16)
    # the dense call above left x_hat = x_half; start the compressed cases from lagging public copies again
    # (every call then moves the top 1 % of the remaining differences into x_hat, as consecutive steps do)
    xhat.zero_()
    yield ("gossip_top1pct", lambda: api.lpdt_gossip_mix(N, d, xh, xhat, xo, Wm, 0.1, [0, d], [d // 100], gws, st),
           N * d * 24)
    ms = torch.empty(N, 1, device="cuda")
    yield ("gossip_dense_q8", lambda: api.lpdt_gossip_mix_q8(N, d, xh, xhat, xo, Wm, 1.0, [0, d], [d], ms, gws, st),
           N * d * 24)
    xhat.zero_()
    yield ("gossip_top1pct_q8", lambda: api.lpdt_gossip_mix_q8(N, d, xh, xhat, xo, Wm, 0.1, [0, d], [d // 100], ms, gws,
                                                              st), N * d * 32)


def q8_cases(B=32):
    """Range-EvoNorm handing 8-bit codes on, fused and as two calls, on the three ResNet-20 layer shapes."""
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    for tag, nodes, HW, Cc in (("32x32x16", 64, 32, 16), ("16x16x32", 128, 16, 32), ("8x8x64", 256, 8, 64)):
        n = B * HW * HW * Cc
        tot = nodes * n
        groups = Cc // 8
        x = torch.randn(nodes, n, generator=g, device="cuda")
        dy = torch.randn(nodes, n, generator=g, device="cuda")
        y = torch.empty_like(x)
        q = torch.empty(nodes, n, dtype=torch.int8, device="cuda")
        scale = torch.empty(nodes, device="cuda")
        v = torch.ones(nodes, Cc, device="cuda")
        gamma = torch.ones(nodes, Cc, device="cuda")
        beta = torch.zeros(nodes, Cc, device="cuda")
        gmin = torch.empty(nodes, B, groups, device="cuda")
        gmax = torch.empty_like(gmin)
        amin_i = torch.empty(nodes, B, groups, dtype=torch.int32, device="cuda")
        amax_i = torch.empty_like(amin_i)
        rng = torch.zeros(nodes, device="cuda")
        wsb = torch.empty(api.lpdt_range_evonorm_bwd_workspace_size(nodes, B, Cc), dtype=torch.uint8, device="cuda")
        ctl = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(nodes), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")

        def fwd2():
            api.lpdt_range_evonorm_fwd(nodes, B, HW, HW, Cc, groups, 1e-5, x, v, gamma, beta, Cc, y, gmin, gmax, amin_i,
                                       amax_i, amax_out=rng)
            api.lpdt_quantize_with_range(y, nodes, n, n, rng, q, scale)

        def fwd1():
            api.lpdt_range_evonorm_fwd_q8(nodes, B, HW, HW, Cc, groups, 1e-5, x, v, gamma, beta, Cc, None, gmin, gmax,
                                          amin_i, amax_i, q, scale, ctl, dev_status=status)

        def bwd2():
            api.lpdt_range_evonorm_bwd(nodes, B, HW, HW, Cc, groups, 1e-5, dy, x, v, gamma, Cc, gmin, gmax, amin_i, amax_i,
                                       y, None, None, None, Cc, wsb, amax_out=rng)
            api.lpdt_quantize_with_range(y, nodes, n, n, rng, q, scale)

        def bwd1():
            api.lpdt_range_evonorm_bwd_q8(nodes, B, HW, HW, Cc, groups, 1e-5, dy, x, v, gamma, Cc, gmin, gmax, amin_i,
                                          amax_i, q, scale, None, None, None, Cc, wsb, ctl, dev_status=status)

        yield (f"ren_fwd_then_quantize_{tag}", fwd2, tot * 5)
        if api.lpdt_range_evonorm_fwd_q8_fits(B, HW, HW, Cc, groups):
            yield (f"ren_fwd_q8_{tag}", fwd1, tot * 5)
        yield (f"ren_bwd_then_quantize_{tag}", bwd2, tot * 9)
        if api.lpdt_range_evonorm_bwd_q8_fits(B, HW, HW, Cc, groups):
            yield (f"ren_bwd_q8_{tag}", bwd1, tot * 9)
        del x, dy, y, q


def all_cases():
    yield from cases()
    yield from q8_cases()


def sweep(iters=20, peak_gbs=None, out=print, only=None):
    rows = []
    for name, fn, nbytes in all_cases():
        if only and not any(name == o or (o.endswith("*") and name.startswith(o[:-1])) for o in only):
            continue
        ms = _time(fn, iters)
        row = {"case": name, "ms": ms, "algorithmic_bytes": nbytes, "gbs": nbytes / ms * 1e-6}
        if peak_gbs:
            row["frac_of_hbm_peak"] = row["gbs"] / peak_gbs
        rows.append(row)
        out(json.dumps(row))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--peak-gbs", type=float, default=None, help="HBM copy bandwidth to report fractions against")
    ap.add_argument("--only", default=None, help="comma-separated case names to run (a trailing * matches a prefix)")
    a = ap.parse_args()
    sweep(a.iters, a.peak_gbs, only=a.only.split(",") if a.only else None)


if __name__ == "__main__":
    main()
