#!/usr/bin/env python
"""Benchmark of the whole 8-bit decentralized training step.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload NAME] [--no-extra]

One step = one pass of the whole hot path (quantize, int8 contractions forward /
backward-data / backward-weight, Range-EvoNorm forward/backward, SGD half-step,
top-k compression and gossip mix) over one batch for every simulated node.
Prints ONE JSON line.  The headline workload is the largest single-GPU
configuration: the ResNet-20-shaped network on 40 simulated nodes x batch 32 with
top-1 % compressed gossip.  At one GPU the line also carries, under "extra":

  workloads     every step workload (single conv layer, ResNet-20 x 16 nodes, VGG-11 x 8
                nodes, ResNet-20 x 40 nodes with top-1 %): ms per step, images/s, end to end
  breakdown     the headline step split by entry point / kernel: each kind of call of one
                step replayed alone as a CUDA graph, with its algorithmic bytes
  contractions  the int8 contraction alone on sweep shapes (GEMMs and 3x3 convolutions,
                three passes each): ms, TOPS, fraction of 2 x the measured bf16 peak and of
                the shape's own roofline bound
  membound      the memory-bound kernels alone on tensors beyond L2: GB/s, fraction of the
                measured HBM copy bandwidth

With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the workload on its own GPU ("replicas only": the path has no
inter-GPU exchange); the value is the sum over ranks divided by the slowest
rank's time.
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "int8 train-step images/s (N simulated nodes, 1 B200); int8 TOPS vs dense peak"
UNIT = "images/s"
WORKLOAD_DESC = {
    "conv16": "one 3x3 conv 16->16 + Range-EvoNorm on 16x16 maps, 4 simulated nodes x batch 8, ring gossip",
    "resnet20": "ResNet-20-shaped CIFAR net (Range-EvoNorm), 16 simulated nodes x batch 32, 32x32x3 N(0,1) "
                "inputs, ring gossip, int8 W/A/E with fp32 master weights",
    "vgg11": "VGG-11-shaped CIFAR net (Range-EvoNorm), 8 simulated nodes x batch 32, ring gossip",
    "resnet20_topk": "ResNet-20-shaped CIFAR net (Range-EvoNorm), 40 simulated nodes x batch 32, 32x32x3 N(0,1) "
                     "inputs, int8 W/A/E with fp32 master weights, gossip messages = top-1 % of x - x_hat over the "
                     "flattened parameter vector, error feedback fused into the mix",
    "resnet20_topk_layerwise": "as resnet20_topk with one top-1 % selection per layer (20 segments)",
}
HEADLINE = "resnet20_topk"
STEP_WORKLOADS = ("conv16", "resnet20", "vgg11", "resnet20_topk")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def wait_for_samples(self, n, timeout=3.0):
        t = time.time()
        while self.proc is not None and len(self.rows) < n and time.time() - t < timeout:
            time.sleep(0.01)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm = sorted(int(r[0]) for r in self.rows if len(r) >= 6 and r[0].isdigit())
        mx = [int(r[1]) for r in self.rows if len(r) >= 6 and r[1].isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm), "sm_mhz_min": sm[0] if sm else None}


def dist_setup(n_gpus):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return world, rank, local


def barrier(world, device="cuda"):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if device == "cuda":
        torch.cuda.synchronize()


def max_over_ranks(world, value, device="cuda"):
    """The slowest rank's time: every rank gets the maximum of `value` over the job."""
    import torch
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world, images_per_rank, ms_total, steps):
    """Whole-job images/s of `world` replicas that each ran `steps` steps of `images_per_rank` images in
    `ms_total` milliseconds (the maximum over ranks): weak scaling, no rank shares work with another."""
    return world * images_per_rank / (ms_total / steps * 1e-3)


def rank_seed(rank):
    """Workload seed of a replica: the default recipe on rank 0, a different draw on every other rank."""
    return None if rank == 0 else 1001 + rank


def executed_macs(wl, input_grad):
    """Multiply-accumulates of the contractions one step executes: forward, backward-weight and
    backward-data of every conv/linear layer, without the first layer's backward-data when no
    input gradient is asked for."""
    from paper_2111_09389_b200 import workloads
    images = wl["nodes"] * wl["batch"]
    macs = 3 * workloads.conv_macs(wl["ops"], images)
    if not input_grad:
        first = [op for op in wl["ops"] if op["op"] in ("conv", "linear")][:1]
        macs -= workloads.conv_macs(first, images)
    return macs


# ---------------------------------------------------------------------------------------------------
# Algorithmic bytes of one entry-point call, from its arguments: every input element read once and
# every output element written once, in the width the call handles (int8 codes 1 B, fp32 4 B).
def call_bytes(name, a, kw):
    def numel(t):
        return 0 if t is None else t.numel()
    if name == "lpdt_quantize":                 # range pass + round pass
        return a[1] * a[2] * 9
    if name == "lpdt_quantize_with_range":
        return a[1] * a[2] * 5
    if name == "lpdt_quantize_batch":           # params, nodes, row_stride, src_offsets, sizes, ...
        return a[1] * sum(int(v) for v in a[4]) * 9
    if name == "lpdt_dequantize":
        return a[1] * a[2] * 5
    if name in ("lpdt_qconv_fwd", "lpdt_qconv_bwd_data", "lpdt_qconv_bwd_weight"):
        d = a[0]
        Ho, Wo = (d.H + 2 * d.pad - d.R) // d.stride + 1, (d.W + 2 * d.pad - d.S) // d.stride + 1
        n_in, n_out = d.nodes * d.B * d.H * d.W * d.Cin, d.nodes * d.B * Ho * Wo * d.Cout
        n_w = d.nodes * d.Cout * d.R * d.S * d.Cin
        if name == "lpdt_qconv_fwd":
            return n_in + n_w + 4 * n_out
        if name == "lpdt_qconv_bwd_data":
            return n_out + n_w + 4 * n_in + (4 * n_in if kw.get("addend") is not None else 0)
        return n_out + n_in + 4 * n_w
    if name == "lpdt_range_evonorm_fwd":        # nodes,B,H,W,C,...
        n = a[0] * a[1] * a[2] * a[3] * a[4]
        return n * (12 if kw.get("res") is not None else 8)
    if name == "lpdt_range_evonorm_bwd":
        return a[0] * a[1] * a[2] * a[3] * a[4] * 12
    if name == "lpdt_range_evonorm_fwd_q8":     # x read, codes written (+ fp32 y when kept, + shortcut read)
        n = a[0] * a[1] * a[2] * a[3] * a[4]
        return n * (5 + (4 if a[12] is not None else 0) + (4 if kw.get("res") is not None else 0))
    if name == "lpdt_range_evonorm_bwd_q8":     # dy, x read, codes written
        return a[0] * a[1] * a[2] * a[3] * a[4] * 9
    if name == "lpdt_range_evonorm_bwd_params":
        return a[0] * a[1] * a[2] * 3 * 8
    if name == "lpdt_residual_add":             # nodes,B,H,W,Ca,C,stride,...
        Ho, Wo = (a[2] + a[6] - 1) // a[6], (a[3] + a[6] - 1) // a[6]
        return a[0] * a[1] * Ho * Wo * (8 * a[5] + 4 * a[4])
    if name == "lpdt_residual_add_bwd":
        Ho, Wo = (a[2] + a[6] - 1) // a[6], (a[3] + a[6] - 1) // a[6]
        return a[0] * a[1] * (a[2] * a[3] * a[4] * 8 + Ho * Wo * a[4] * 4)
    if name in ("lpdt_maxpool2x2", "lpdt_maxpool2x2_bwd"):
        n = a[0] * a[1] * a[2] * a[3] * a[4]
        return n * 4 + n // 4 * 5
    if name in ("lpdt_avgpool", "lpdt_avgpool_bwd"):
        return a[0] * a[1] * (a[2] + 1) * a[3] * 4
    if name == "lpdt_softmax_ce":
        return a[0] * a[1] * (a[2] * 8 + 4)
    if name == "lpdt_colsum":
        return a[0] * (a[1] + 1) * a[2] * 4
    if name == "lpdt_sgd_update":
        return a[0] * 12
    if name == "lpdt_sgd_gossip_mix":           # x, g, x_hat read; x_half, x_hat, x written
        return a[0] * a[1] * 24
    if name in ("lpdt_gossip_mix", "lpdt_gossip_mix_q8"):
        # x_half, x_hat read, x_hat, x written (16 B); a compressed segment adds one selection pass over
        # x_half and x_hat (8 B); 8-bit messages add one range pass (8 B)
        nodes, d = a[0], a[1]
        offs, ks = a[7], a[8]
        compressed = sum(int(offs[i + 1]) - int(offs[i]) for i in range(len(ks)) if int(ks[i]) < int(offs[i + 1]) - int(offs[i]))
        return nodes * (d * 16 + compressed * 8 + (d * 8 if name.endswith("q8") else 0))
    if name == "lpdt_fill_zero":
        return a[0].numel() * a[0].element_size()
    return 0


def group_key(rec):
    name, kernel = rec[0], rec[4]
    return f"{name} [{kernel}]" if kernel else name


_REPLAY_STREAMS = {}


def issue(calls):
    """Issue logged calls as the step does: the calls of each node group on a stream of that group, side by
    side between a fork and a join (one group: plainly on the current stream)."""
    import torch
    tags = sorted({c[5] for c in calls})
    if len(tags) <= 1:
        for c in calls:
            c[1](*c[2], **c[3])
        return
    main = torch.cuda.current_stream()
    for t in tags:
        st = _REPLAY_STREAMS.setdefault(t, torch.cuda.Stream())
        st.wait_stream(main)
        with torch.cuda.stream(st):
            for c in calls:
                if c[5] == t:
                    c[1](*c[2], **c[3])
    for t in tags:
        main.wait_stream(_REPLAY_STREAMS[t])


def time_group(calls, reps):
    """Milliseconds per issue of `calls` (logged entry-point calls of one step, in step order; node groups side
    by side as in the step): recorded into one CUDA graph and replayed `reps` times between two events on the
    current stream."""
    import torch
    from paper_2111_09389_b200 import api
    before = api.lpdt_launch_count()
    issue(calls)
    time_group.launches = api.lpdt_launch_count() - before       # kernels one issue of `calls` enqueues
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        issue(calls)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def breakdown(st, reps, peaks):
    """Every kind of call of one step timed alone (see time_group), with its algorithmic bytes."""
    from paper_2111_09389_b200 import api
    log = st.record()
    groups = {}
    for rec in log:
        groups.setdefault(group_key(rec), []).append(rec)
    rows = []
    for key, calls in groups.items():
        ms = time_group(calls, reps)
        nbytes = sum(call_bytes(c[0], c[2], c[3]) for c in calls)
        launches = time_group.launches
        rows.append({"call": key, "calls_per_step": len(calls), "kernel_launches": launches, "ms_per_step": ms,
                     "algorithmic_bytes": int(nbytes), "gbs": nbytes / (ms * 1e-3) / 1e9,
                     "frac_of_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]})
    rows.sort(key=lambda r: -r["ms_per_step"])
    return rows, log


# DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) of the kernel the roofline
# record names, by workload, with the SHA-256 of the kernel sources at the time of the capture: the
# figure is printed only while those sources are unchanged.
KERNEL_SOURCES = {
    "lpdt::ren_bwd_kernel": ("range_evonorm.cu", "common.cuh"),
    "lpdt::ren_fwd_kernel": ("range_evonorm.cu", "common.cuh"),
    "lpdt::ren_fwd_q8_kernel": ("range_evonorm.cu", "common.cuh"),
    "lpdt::ren_bwd_q8_kernel": ("range_evonorm.cu", "common.cuh"),
    "lpdt::tc::conv_halo16_kernel": ("qconv_halo.cu", "tc_common.cuh", "common.cuh"),
    "lpdt::tc::conv_pix_kernel": ("qconv_tc.cu", "tc_common.cuh", "common.cuh"),
    "lpdt::tc::conv_wgrad_kernel": ("qconv_tc.cu", "tc_common.cuh", "common.cuh"),
}
MEASURED_TRAFFIC = {
    ("resnet20_topk", "lpdt::tc::conv_halo16_kernel"): {
        "ratio_to_algorithmic": 53.8 / 104.9, "source_hash": "557c6c824dfa48a1",
        "note": "ncu capture of one forward launch on the 16-channel 32x32 layer shape (40 nodes x batch 32): "
                "dram__bytes_read.sum + dram__bytes_write.sum = 21.1 + 32.7 MB against 104.9 MB algorithmic; scaled to this "
                "step's mean launch by the algorithmic bytes.  Below 1 because part of the fp32 result is still in "
                "the 126 MB L2 when the kernel ends"},
}


def source_hash(kernel):
    files = KERNEL_SOURCES.get(kernel)
    if not files:
        return None
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, "paper_2111_09389_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


# main kernel behind the entry points that are not contractions (contractions report theirs through
# lpdt_last_kernel)
KERNEL_OF = {"lpdt_range_evonorm_fwd": "lpdt::ren_fwd_kernel", "lpdt_range_evonorm_bwd": "lpdt::ren_bwd_kernel",
             "lpdt_range_evonorm_fwd_q8": "lpdt::ren_fwd_q8_kernel", "lpdt_range_evonorm_bwd_q8": "lpdt::ren_bwd_q8_kernel",
             "lpdt_quantize_with_range": "lpdt::quantize_kernel", "lpdt_quantize": "lpdt::range_kernel + lpdt::quantize_kernel",
             "lpdt_gossip_mix": "lpdt::big_sample_kernel + big_collect_kernel + select_and_rows_kernel + gossip_mix_kernel",
             "lpdt_sgd_gossip_mix": "lpdt::sgd_dense_mix_kernel", "lpdt_residual_add": "lpdt::residual_add_v4_kernel",
             "lpdt_residual_add_bwd": "lpdt::residual_add_bwd_v4_kernel", "lpdt_sgd_update": "lpdt::sgd_kernel"}


def kernel_of(rec):
    return rec[4] or KERNEL_OF.get(rec[0], rec[0])


def roofline_record(rows, log, kernel, peaks, workload, reps):
    """Roofline entry of one kernel of the step ("auto" = the kernel with the largest time when its
    launches are replayed alone): algorithmic bytes per launch over the mean launch duration."""
    by_kernel = {}
    for c in log:
        by_kernel.setdefault(kernel_of(c), []).append(c)
    times = {}
    for r in rows:                                     # rows are per (entry point, kernel); sum them per kernel
        k = r["call"].split("[")[1].rstrip("]") if "[" in r["call"] else KERNEL_OF.get(r["call"], r["call"])
        times[k] = times.get(k, 0.0) + r["ms_per_step"]
    if kernel == "auto":
        kernel = max(times, key=times.get)
    if kernel not in by_kernel:
        return None
    calls = by_kernel[kernel]
    ms = time_group(calls, reps)                      # all launches of this kernel in one step, in step order
    nbytes = sum(call_bytes(c[0], c[2], c[3]) for c in calls)
    macs = 0
    for c in calls:
        if c[0].startswith("lpdt_qconv"):
            d = c[2][0]
            Ho, Wo = (d.H + 2 * d.pad - d.R) // d.stride + 1, (d.W + 2 * d.pad - d.S) // d.stride + 1
            macs += d.nodes * d.B * Ho * Wo * d.Cout * d.Cin * d.R * d.S
    gbs = nbytes / (ms * 1e-3) / 1e9
    ranking = sorted(times.items(), key=lambda kv: -kv[1])
    rec = {"kernel": kernel, "entry_points": sorted({c[0] for c in calls}), "bound": "hbm", "achieved": gbs,
           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": None,
           "peak_source": peaks["source"], "launches_per_step": len(calls),
           "mean_launch_us": ms * 1e3 / len(calls), "ms_per_step_in_kernel": ms,
           "algorithmic_bytes_per_step": int(nbytes), "algorithmic_bytes_per_launch": nbytes / len(calls),
           "tops_in_kernel": 2 * macs / (ms * 1e-3) / 1e12 if macs else None,
           "timing": "CUDA events around graph replays of this kernel's launches alone (every layer that uses "
                     "it, step order, operands of the last step), after the timed region",
           "kernels_by_time": [{"kernel": k, "ms_per_step": t} for k, t in ranking[:6]]}
    m = MEASURED_TRAFFIC.get((workload, kernel))
    if m is not None:
        now = source_hash(kernel)
        rec["traffic_source_hash"] = {"captured_at": m["source_hash"], "now": now}
        if now == m["source_hash"]:
            rec["traffic"] = m["ratio_to_algorithmic"] * nbytes / len(calls)
            rec["traffic_note"] = m["note"]
        else:
            rec["traffic_note"] = "kernel sources changed since the DRAM counters were taken: traffic withheld"
    return rec


def run_step_workload(name, rank, world, steps, warmup, graph=True, **step_options):
    """Build one step workload, time `steps` steps (device-resident inputs) and `steps` end-to-end steps."""
    import torch
    from paper_2111_09389_b200 import api, workloads
    from paper_2111_09389_b200.step import TrainStep
    wl = workloads.make_workload(name, seed=rank_seed(rank))
    if not step_options.get("node_groups"):
        step_options["node_groups"] = 2 if wl["nodes"] >= 32 else 1
    st = TrainStep.from_workload(wl, **step_options)
    images = wl["nodes"] * wl["batch"]
    if graph:
        st.capture()
        step = st.replay
    else:
        step = st.run
    for _ in range(warmup):
        step()
    barrier(world)
    launches0 = api.lpdt_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    ms_total = max_over_ranks(world, e0.elapsed_time(e1))
    launches = api.lpdt_launch_count() - launches0
    assert int(st.dev_status.item()) == 0

    # end to end: inputs start in pinned host memory, the loss is read back every step; the upload of the
    # next batch runs on a copy stream while the current step computes, as a training loop would do it
    x_host = torch.from_numpy(wl["x"]).pin_memory()
    lab_host = torch.from_numpy(wl["labels"]).pin_memory() if "labels" in wl else None
    # the loss of every step is copied to pinned host memory inside the timed region; the host waits for it one
    # step late (two buffers), as a loop that logs the loss would, so that the next step is already queued
    loss_host = [torch.empty(wl["nodes"], dtype=torch.float32).pin_memory() for _ in range(2)]
    loss_there = [torch.cuda.Event() for _ in range(2)]
    for _ in range(2):                       # untimed: the staging buffers and the copy stream are created here
        st.upload(x_host, lab_host)
        st.step_from_upload(step)
    torch.cuda.synchronize()
    barrier(world)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    st.upload(x_host, lab_host)
    for i in range(steps):
        st.step_from_upload(step)
        if i + 1 < steps:
            st.upload(x_host, lab_host)
        loss_host[i % 2].copy_(st.loss, non_blocking=True)
        loss_there[i % 2].record()
        if i >= 1:
            loss_there[(i - 1) % 2].synchronize()
    loss_there[(steps - 1) % 2].synchronize()
    t1.record()
    torch.cuda.synchronize()
    barrier(world)
    e2e_ms = max_over_ranks(world, t0.elapsed_time(t1)) / steps
    macs = executed_macs(wl, st.input_grad)
    res = {"ms_per_step": ms_total / steps, "value": job_value(world, images, ms_total, steps),
           "e2e": {"value": world * images / (e2e_ms * 1e-3), "unit": UNIT,
                   "h2d_bytes_per_step": int(x_host.numel() * 4 + (lab_host.numel() * 4 if lab_host is not None else 0)),
                   "d2h_bytes_per_step": int(loss_host[0].numel() * 4)},
           "int8_tops": 2 * macs * world / (ms_total / steps * 1e-3) / 1e12, "macs_per_step": macs,
           "launches": int(launches), "launches_per_step": int(launches) // max(1, steps),
           "nodes": wl["nodes"], "batch_per_node": wl["batch"], "params_per_node": wl["d"],
           "node_groups": st.node_groups, "saved_bytes_per_node": st.saved_bytes_per_node()}
    return res, st, wl


CONTRACTION_CASES = (
    [("gemm", (M, N, K)) for (M, N, K) in ((8192, 8192, 8192), (4096, 4096, 4096), (2048, 2048, 2048),
                                           (8192, 8192, 1024), (1024, 1024, 1024))] +
    [("conv", (C, HW, 256)) for C in (64, 256, 512) for HW in (32, 56)])


def contraction_block(peaks, iters=10):
    """The int8 contraction alone on sweep shapes: CUDA-graph replays over rotating operand sets."""
    import torch
    from paper_2111_09389_b200 import contraction_sweep as cs
    int8_ref = 2 * peaks["bf16_tflops"]              # the recipe's nominal ratio: int8 = 2 x bf16
    out = []
    for kind, dims in CONTRACTION_CASES:
        recs = cs.gemm(*dims, iters=iters, warmup=2, graph=True, quiet=True) if kind == "gemm" else \
            cs.conv(*dims, iters=iters, warmup=2, graph=True, quiet=True)
        for r in recs:
            ai_bound = r["min_hbm_bytes"] and (2 * r["macs"] / r["min_hbm_bytes"]) * peaks["hbm_gbs"] * 1e9 / 1e12
            bound = min(int8_ref, ai_bound)
            out.append({"shape": r["shape"], "pass": r["pass"], "ms": r["ms"], "tops": r["tops"],
                        "frac_of_2x_bf16": r["tops"] / int8_ref, "bound_tops": bound,
                        "bound_kind": "tensor" if bound == int8_ref else "hbm", "frac_of_bound": r["tops"] / bound,
                        "dev_status": r["dev_status"]})
        torch.cuda.empty_cache()
    return {"int8_reference_tops": int8_ref, "reference": "2 x measured bf16 burst (nominal int8:bf16 ratio)",
            "timing": f"CUDA-graph replay of {iters} calls rotating over operand sets larger than L2", "cases": out}


def membound_block(peaks, iters=10):
    import torch
    from paper_2111_09389_b200 import membound_sweep as mb
    rows = mb.sweep(iters, peaks["hbm_gbs"], out=lambda s: None)
    torch.cuda.empty_cache()
    return {"hbm_gbs": peaks["hbm_gbs"], "tensors": "268 MB activations (8 nodes x batch 128 x 32x32x64 fp32), "
            "554 MB parameter arrays (16 nodes x 8.65 M)", "cases": rows}


def run_ours(args):
    import torch
    world, rank, local = dist_setup(args.gpus)
    peaks = measured_peaks()
    sampler = ClockSampler(local)
    sampler.start()
    sampler.wait_for_samples(2)
    head, st, wl = run_step_workload(args.workload, rank, world, args.steps, args.warmup, graph=args.graph,
                                     node_groups=args.node_groups, fuse_requantize=args.fuse_requantize)
    reps = max(args.steps, 5)
    rows, log = breakdown(st, reps, peaks)
    roof = roofline_record(rows, log, args.roofline_kernel, peaks, args.workload, reps)
    clocks = sampler.stop()
    clocks["window"] = "warm-up steps, the timed steps and the per-kernel replays after them"
    step_bytes = sum(r["algorithmic_bytes"] for r in rows)
    out = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "description": WORKLOAD_DESC.get(args.workload, args.workload),
                   "nodes": wl["nodes"], "batch_per_node": wl["batch"], "params_per_node": wl["d"],
                   "parallelism": "replicas only" if world > 1 else "1 GPU, nodes batched",
                   "launch": ("CUDA graph replay of the whole step" if args.graph else "eager launches") +
                             (f", forward/backward of {head['node_groups']} node groups on parallel streams"
                              if head["node_groups"] > 1 else ""),
                   "l2": "activations touched per step exceed L2 (working set of several GB vs 126 MB)"},
        "int8_tops": head["int8_tops"], "macs_per_step": head["macs_per_step"],
        "clocks": clocks, "e2e": head["e2e"], "gpu_launches": head["launches"],
        "roofline": roof,
        "step": {"algorithmic_bytes": int(step_bytes), "gbs": step_bytes / (head["ms_per_step"] * 1e-3) / 1e9,
                 "frac_of_hbm": step_bytes / (head["ms_per_step"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                 "launches_per_step": head["launches_per_step"],
                 "sum_of_isolated_ms": sum(r["ms_per_step"] for r in rows)},
    }
    del st
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.extra:
        extra = {"breakdown": rows, "workloads": {}}
        for name in STEP_WORKLOADS:
            if name == args.workload:
                r = dict(head)
            else:
                r, st2, _ = run_step_workload(name, rank, world, args.steps, args.warmup, graph=args.graph,
                                              node_groups=args.node_groups,
                                              fuse_requantize=args.fuse_requantize)
                del st2
                torch.cuda.empty_cache()
            r["images_per_s"] = r.pop("value")
            extra["workloads"][name] = r
        # what a node keeps between its forward and backward pass when only 8-bit tensors are saved (the norm
        # layers' fp32 inputs are recomputed), beside the default mode's figure under workloads.resnet20
        r, st2, _ = run_step_workload("resnet20", rank, world, args.steps, args.warmup, graph=args.graph,
                                      recompute_norm_input=True)
        del st2
        torch.cuda.empty_cache()
        extra["memory"] = {"workload": "resnet20", "mode": "recompute_norm_input", "ms_per_step": r["ms_per_step"],
                           "images_per_s": r["value"], "saved_bytes_per_node": r["saved_bytes_per_node"],
                           "paper_context": "Table hardware_results: 124.60 MB (fp32) -> 35.43 MB (8-bit) training memory "
                                            "per node for ResNet-20 at batch 32, the paper's own accounting"}
        # the memory-bound block first: the dense contractions after it draw the power limit
        sampler2 = ClockSampler(local)
        sampler2.start()
        extra["membound"] = membound_block(peaks)
        extra["membound"]["clocks"] = sampler2.stop()
        sampler3 = ClockSampler(local)
        sampler3.start()
        extra["contractions"] = contraction_block(peaks)
        extra["contractions"]["clocks"] = sampler3.stop()
        out["extra"] = extra
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args.workload, nodes=args.cpu_nodes)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def cpu_baseline(workload, nodes):
    """The oracle, as it stands, timed on this host on a bounded sample of the workload."""
    from oracle import step as ostep
    import oracle
    from paper_2111_09389_b200 import workloads
    wl = workloads.make_workload(workload, nodes=nodes)
    t = time.perf_counter()
    ostep.train_step(wl)
    dt = time.perf_counter() - t
    return {"value": wl["nodes"] * wl["batch"] / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one step of {nodes} of the workload's nodes x batch {wl['batch']} ({dt:.1f} s)"}


def run_reference(args):
    """Reference arm: the CPU oracle on the host cores, one bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import step as ostep
    import oracle
    from paper_2111_09389_b200 import workloads
    nodes = args.cpu_nodes
    wl = workloads.make_workload(args.workload, nodes=nodes)
    for _ in range(min(args.warmup, 1)):
        ostep.train_step(wl)
    t = time.perf_counter()
    for _ in range(args.steps):
        ostep.train_step(wl)
    dt = (time.perf_counter() - t) / args.steps
    value = nodes * wl["batch"] / dt
    sample = f"each step = one oracle step of {nodes} of the workload's nodes x batch {wl['batch']}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "description": WORKLOAD_DESC.get(args.workload, args.workload),
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--roofline-kernel", default="auto",
                    help="kernel the roofline record is taken on (auto = the one with the most time in the step)")
    ap.add_argument("--node-groups", type=int, default=0,
                    help="split the nodes' forward/backward passes into this many groups on parallel streams "
                         "(0 = two groups from 32 nodes on, else one: measured best per workload)")
    ap.add_argument("--fuse-requantize", action="store_true",
                    help="norm layers write the next convolution's 8-bit codes themselves (A/B timing; slower)")
    ap.add_argument("--cpu-nodes", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", dest="extra", action="store_false",
                    help="skip the other workloads and the contraction / memory-bound blocks")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch every kernel eagerly instead of replaying the captured step")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = min(args.steps, 20)
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
