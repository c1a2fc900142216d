#!/usr/bin/env python
"""Benchmark of the whole 8-bit decentralized training step.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One step = one pass of the whole hot path (quantize, int8 contractions forward /
backward-data / backward-weight, Range-EvoNorm forward/backward, SGD half-step,
gossip mix) over one batch for every simulated node.  Prints ONE JSON line.
With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the workload on its own GPU ("replicas only": the path has no
inter-GPU exchange); the value is the sum over ranks divided by the slowest
rank's time.
"""
import argparse
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
    "resnet20": "ResNet-20-shaped CIFAR net (Range-EvoNorm), 16 simulated nodes x batch 32, 32x32x3 N(0,1) "
                "inputs, ring gossip, int8 W/A/E with fp32 master weights",
}


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
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

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
                "reasons": reasons, "samples": len(sm)}


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


def run_ours(args):
    import numpy as np
    import torch
    from paper_2111_09389_b200 import api, workloads
    from paper_2111_09389_b200.step import TrainStep

    world, rank, local = dist_setup(args.gpus)
    wl = workloads.make_workload(args.workload, seed=rank_seed(rank))
    st = TrainStep.from_workload(wl)
    images = wl["nodes"] * wl["batch"]
    macs_step = 3 * workloads.conv_macs(wl["ops"], images)

    dominant = args.roofline_kernel
    if args.graph:
        st.capture()
        step = st.replay
    else:
        step = st.run
    for _ in range(args.warmup):
        step()
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = api.KERNEL_LAUNCHES
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    ms_total = max_over_ranks(world, e0.elapsed_time(e1))
    launches = api.KERNEL_LAUNCHES - launches0
    assert int(st.dev_status.item()) == 0
    # the dominant entry points.  Contractions: their calls alone, on the operands the step left behind,
    # replayed as a CUDA graph between two events (eager launches would time the host's launch gaps).
    # Other entry points: CUDA events around each eager call of whole steps.
    names = dominant.split(",")
    kernel_ms = {}
    passes = {"lpdt_qconv_fwd": "fwd", "lpdt_qconv_bwd_data": "bwd_data", "lpdt_qconv_bwd_weight": "bwd_weight"}
    if all(n in passes for n in names):
        st.run()
        for n in names:
            kernel_ms[n] = time_contractions(st, (passes[n],), max(args.steps, 5))
    else:
        api.TIMED.update(names)
        api.TIMINGS.clear()
        for _ in range(args.steps):
            st.run()
        torch.cuda.synchronize()
        api.TIMED.difference_update(names)
    clocks = sampler.stop()
    ms_step = ms_total / args.steps
    value = job_value(world, images, ms_total, args.steps)

    # end to end: inputs start in pinned host memory, the loss is read back every step
    x_host = torch.from_numpy(wl["x"]).pin_memory()
    lab_host = torch.from_numpy(wl["labels"]).pin_memory()
    loss_host = torch.empty(wl["nodes"], dtype=torch.float32).pin_memory()
    # every step's batch goes host -> device inside the timed region; the upload of the next batch runs on a copy
    # stream while the current step computes (TrainStep.upload / step_from_upload), as a training loop would do it
    barrier(world)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    st.upload(x_host, lab_host)
    for i in range(args.steps):
        st.step_from_upload(step)
        if i + 1 < args.steps:
            st.upload(x_host, lab_host)
        loss_host.copy_(st.loss, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    t1.record()
    torch.cuda.synchronize()
    barrier(world)
    e2e_ms = max_over_ranks(world, t0.elapsed_time(t1)) / args.steps
    e2e = {"value": world * images / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": int(x_host.numel() * 4 + lab_host.numel() * 4),
           "d2h_bytes_per_step": int(loss_host.numel() * 4)}

    peaks = measured_peaks()
    roof = roofline_sum([roofline_for(n, st, wl, peaks, api, kernel_ms.get(n)) for n in names], peaks)
    roof = attach_traffic(roof, args.workload, dominant)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "description": WORKLOAD_DESC.get(args.workload, args.workload),
                   "nodes": wl["nodes"], "batch_per_node": wl["batch"], "params_per_node": wl["d"],
                   "parallelism": "replicas only" if world > 1 else "1 GPU, nodes batched",
                   "launch": "CUDA graph replay of the whole step" if args.graph else "eager launches",
                   "l2": "activations touched per step exceed L2 (working set of several GB vs 126 MB)"},
        "int8_tops": 2 * macs_step * world / (ms_step * 1e-3) / 1e12,
        "macs_per_step": macs_step,
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roof,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args.workload, nodes=args.cpu_nodes)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


KERNEL_OF = {"lpdt_qconv_fwd": "lpdt::tc::conv_pix_kernel", "lpdt_qconv_bwd_data": "lpdt::tc::conv_pix_kernel",
             "lpdt_qconv_bwd_weight": "lpdt::tc::conv_wgrad_kernel", "lpdt_range_evonorm_fwd": "lpdt::ren_fwd_kernel",
             "lpdt_range_evonorm_bwd": "lpdt::ren_bwd_kernel"}


def roofline_sum(parts, peaks):
    """Merge the per-entry-point records of the calls that launch the same kernel."""
    parts = [p for p in parts if p]
    if not parts:
        return None
    if len(parts) == 1:
        return parts[0]
    ms = sum(p["ms_per_step_in_kernel"] for p in parts)
    by = sum(p["algorithmic_bytes_per_step"] for p in parts)
    gbs = by / (ms * 1e-3) / 1e9
    tops = None
    if all(p["tops_in_kernel"] for p in parts):
        tops = sum(p["tops_in_kernel"] * p["ms_per_step_in_kernel"] for p in parts) / ms
    launches = sum(p["launches_per_step"] for p in parts)
    return {"kernel": parts[0]["kernel"], "entry_points": [p["entry_points"][0] for p in parts], "bound": "hbm",
            "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
            "traffic": None, "peak_source": peaks["source"],
            "launches_timed": sum(p["launches_timed"] for p in parts), "launches_per_step": launches,
            "ms_per_step_in_kernel": ms, "algorithmic_bytes_per_step": by,
            "algorithmic_bytes_per_launch": by / max(1, launches), "tops_in_kernel": tops,
            "timing": parts[0]["timing"]}


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the tensor-core forward / backward-data
# kernels over one step, from the ncu capture summarised in profiles/step_resnet20_launches.md.  Valid
# for that workload and those entry points only, and only while those kernels are unchanged.
MEASURED_TRAFFIC = {("resnet20", "lpdt_qconv_fwd,lpdt_qconv_bwd_data"): {"bytes_per_step": 353.6e6, "launches": 37}}


def attach_traffic(roof, workload, entry_points):
    m = MEASURED_TRAFFIC.get((workload, entry_points))
    if roof is None or m is None:
        return roof
    roof["traffic"] = m["bytes_per_step"] / m["launches"]
    roof["traffic_per_step"] = m["bytes_per_step"]
    roof["traffic_note"] = ("ncu DRAM bytes per launch, mean over the step's 37 tensor-core launches; the fp32 results stay "
                            "in L2 past the kernel's end, so this is below the algorithmic bytes")
    return roof


def time_contractions(st, passes, reps):
    """Milliseconds per step spent in the contraction calls of `passes`: one CUDA graph of those
    calls over every layer, replayed `reps` times between two events on the current stream."""
    import torch
    st.contractions(passes)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        st.contractions(passes)
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


def roofline_for(name, st, wl, peaks, api, graph_ms=None):
    """Roofline entry of the dominant kernel: algorithmic bytes (or ops) per launch,
    summed over the launches of one step, over the event-timed duration."""
    import torch
    pairs = api.TIMINGS.get(name, [])
    if graph_ms is None and not pairs:
        return None
    ms = sum(a.elapsed_time(b) for a, b in pairs)
    N, B = wl["nodes"], wl["batch"]
    calls_per_step = 0
    bytes_step = 0
    ops_step = 0
    for li, op in enumerate(wl["ops"]):
        k = op["op"]
        if name in ("lpdt_range_evonorm_fwd", "lpdt_range_evonorm_bwd") and k == "ren":
            n = N * B * op["H"] * op["W"] * op["C"]
            bytes_step += n * (8 if name.endswith("fwd") else 12)
            calls_per_step += 1
        if name.startswith("lpdt_qconv") and k in ("conv", "linear"):
            if k == "conv":
                Ho = (op["H"] + 2 * op["pad"] - op["R"]) // op["stride"] + 1
                macs = N * B * Ho * Ho * op["cout"] * op["cin"] * op["R"] * op["S"]
                n_in, n_out = N * B * op["H"] * op["W"] * op["cin"], N * B * Ho * Ho * op["cout"]
                n_w = N * op["cout"] * op["R"] * op["S"] * op["cin"]
            else:
                macs = N * B * op["cout"] * op["cin"]
                n_in, n_out, n_w = N * B * op["cin"], N * B * op["cout"], N * op["cout"] * op["cin"]
            if name == "lpdt_qconv_bwd_data" and op is wl["ops"][0]:
                continue
            ops_step += 2 * macs
            if name == "lpdt_qconv_fwd":
                bytes_step += n_in + n_w + 4 * n_out
            elif name == "lpdt_qconv_bwd_data":
                bytes_step += n_out + n_w + 4 * n_in
                if st.buf[li].get("addend") is not None:      # fused shortcut gradient: one more fp32 read
                    bytes_step += 4 * n_in
            else:
                bytes_step += n_out + n_in + 4 * n_w
            calls_per_step += 1
        if name == "lpdt_quantize" and k in ("conv", "linear"):
            pass
    steps = max(1, len(pairs) // max(1, calls_per_step))
    timing = "CUDA events around each call, eager launches of the same steps after the timed region"
    if graph_ms is not None:
        ms, steps = graph_ms, 1
        timing = ("CUDA events around graph replays of these calls alone (every layer, step order, operands "
                  "of the last step) after the timed region")
    sec = ms * 1e-3 / steps
    gbs = bytes_step / sec / 1e9
    return {"kernel": KERNEL_OF.get(name, name), "entry_points": [name],
            "timing": timing,
            "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
            "launches_timed": len(pairs) if graph_ms is None else calls_per_step, "launches_per_step": calls_per_step,
            "ms_per_step_in_kernel": ms / steps,
            "algorithmic_bytes_per_step": bytes_step,
            "tops_in_kernel": ops_step / sec / 1e12 if ops_step else None}


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
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet20")
    ap.add_argument("--roofline-kernel", default="lpdt_qconv_fwd,lpdt_qconv_bwd_data",
                    help="entry point(s), comma separated, whose calls are event-timed for the roofline record")
    ap.add_argument("--cpu-nodes", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
