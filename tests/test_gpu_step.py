"""GPU parity of whole training steps against the oracle's step composition."""
import numpy as np
import pytest
import torch

from oracle import step as ostep
from paper_2111_09389_b200 import workloads as wlmod
from paper_2111_09389_b200.step import TrainStep

pytestmark = pytest.mark.gpu


def close(got, want, rtol=1e-5, atol=1e-6, what=""):
    got = got.cpu().numpy() if isinstance(got, torch.Tensor) else got
    want = np.asarray(want, np.float64)
    err = np.abs(got.astype(np.float64) - want)
    ok = err <= atol + rtol * np.abs(want)
    assert ok.all(), f"{what}: {(~ok).sum()} of {ok.size} outside tolerance, worst {err.max():.3e}"


def _compare(wl, nodes_to_check=None, **kw):
    keep = {}
    ref = ostep.train_step(wl, keep=keep, **kw)
    st = TrainStep.from_workload(wl, **kw)
    st.run()
    torch.cuda.synchronize()
    assert int(st.dev_status.item()) == 0
    # integer paths: every quantized layer gradient and accumulator-derived tensor, bit for bit
    for li, (op, b) in enumerate(zip(wl["ops"], st.buf)):
        if op["op"] in ("conv", "linear"):
            assert np.array_equal(b["E"].cpu().numpy().reshape(keep[f"E{li}"].shape), keep[f"E{li}"]), f"E{li}"
            assert np.array_equal(b["out"].cpu().numpy().reshape(keep[f"out{li}"].shape), keep[f"out{li}"]), f"out{li}"
    if ref["loss"] is not None:
        close(st.loss, ref["loss"], what="loss")
    close(st.grads, ref["grads"], what="grads")
    close(st.x_half, ref["x_half"], what="x_half")
    close(st.x_hat, ref["x_hat"], what="x_hat")
    close(st.x_out, ref["x"], what="x")
    if ref["input_grad"] is not None:
        close(st.input_grad_out, ref["input_grad"], what="input grad")
    return st, ref


def test_conv16_step():
    _compare(wlmod.make_workload("conv16"))


def test_conv16_step_stochastic_and_wgrad_quantized():
    _compare(wlmod.make_workload("conv16"), grad_rounding=1, seed=1234)
    _compare(wlmod.make_workload("conv16", nodes=2, batch=2), quantize_wgrad=True)


def test_resnet20_step_small():
    _compare(wlmod.make_workload("resnet20", nodes=3, batch=4))


def test_resnet20_topk_step_small():
    wl = wlmod.make_workload("resnet20_topk", nodes=5, batch=2)
    st, ref = _compare(wl)
    k = int(wl["seg_k"][0])
    assert all(np.count_nonzero(ref["q"][i]) == k for i in range(5))


def test_resnet20_layerwise_topk_step_small():
    """The paper's layer-wise top-K: one segment per layer (20 for this network), the top 1 % of each kept."""
    wl = wlmod.make_workload("resnet20_topk_layerwise", nodes=5, batch=2)
    assert len(wl["seg_k"]) == 20 and wl["seg_offsets"][-1] == wl["d"]
    st, ref = _compare(wl)
    for s in range(20):
        lo, hi = int(wl["seg_offsets"][s]), int(wl["seg_offsets"][s + 1])
        assert all(np.count_nonzero(ref["q"][i][lo:hi]) == int(wl["seg_k"][s]) for i in range(5))


def test_vgg11_step_small():
    _compare(wlmod.make_workload("vgg11", nodes=2, batch=2))


def test_resnet20_dirichlet_labels():
    _compare(wlmod.make_workload("resnet20", nodes=2, batch=8, dirichlet_alpha=0.1))


def test_graph_replay_matches_eager():
    wl = wlmod.make_workload("resnet20", nodes=2, batch=4)
    a = TrainStep.from_workload(wl)
    a.run()
    b = TrainStep.from_workload(wl)
    b.capture()                 # warm-up run + captured run executed eagerly... state advanced twice
    b.load(wl)                  # restore the inputs, then replay once
    b.replay()
    torch.cuda.synchronize()
    assert torch.equal(a.x_out, b.x_out) and torch.equal(a.x_hat, b.x_hat) and torch.equal(a.grads, b.grads)
    assert b.graph_launches > 100


def test_step_from_upload_matches_loaded_inputs():
    """The host-input pipeline (upload on a copy stream, one batch ahead) feeds the step the same bytes as load():
    two batches in a row, the second uploaded while the first step runs."""
    wl = wlmod.make_workload("resnet20", nodes=2, batch=4)
    wl2 = wlmod.make_workload("resnet20", nodes=2, batch=4, seed=77)
    ref = TrainStep.from_workload(wl)
    ref.run()
    ref.x.copy_(torch.from_numpy(wl2["x"])); ref.labels.copy_(torch.from_numpy(wl2["labels"]))
    ref.params.copy_(ref.x_out)
    ref.run()
    st = TrainStep.from_workload(wl)
    st.x.zero_(); st.labels.zero_()
    pin = lambda a: torch.from_numpy(a).pin_memory()
    st.upload(pin(wl["x"]), pin(wl["labels"]))
    st.step_from_upload()
    st.upload(pin(wl2["x"]), pin(wl2["labels"]))          # overlaps the first step
    st.params.copy_(st.x_out)
    st.step_from_upload()
    torch.cuda.synchronize()
    assert torch.equal(st.x_out, ref.x_out) and torch.equal(st.grads, ref.grads) and torch.equal(st.loss, ref.loss)


def test_resnet20_full_size_step():
    # the benchmark workload at its full size (16 nodes x batch 32): every node's codes, outputs,
    # gradients and the gossip result against the oracle's whole step
    _compare(wlmod.make_workload("resnet20"))


def _subset(wl, sel):
    """The same workload restricted to the nodes in sel (nodes are independent until the gossip step)."""
    sub = dict(wl)
    sub["nodes"] = len(sel)
    for key in ("x", "labels", "dy", "params", "x_hat"):
        if key in wl:
            sub[key] = np.ascontiguousarray(wl[key][sel])
    return sub


def _compare_sampled_nodes(wl, sel, **step_options):
    """Full-size GPU step; the oracle recomputes the sampled nodes' gradients and half-steps, and the mix
    is checked through what holds at any size (top-k count, x_hat update, average preservation)."""
    st = TrainStep.from_workload(wl, **step_options)
    st.run()
    torch.cuda.synchronize()
    assert int(st.dev_status.item()) == 0
    sub = _subset(wl, sel)
    keep = {}
    grads, loss, _ = ostep.forward_backward(sub["ops"], sub["params"], sub["x"], sub.get("labels"), None,
                                            sub["ren_eps"], keep=keep)
    for li, (op, b) in enumerate(zip(wl["ops"], st.buf)):
        if op["op"] in ("conv", "linear"):
            got = b["E"][sel].cpu().numpy()
            assert np.array_equal(got.reshape(keep[f"E{li}"].shape), keep[f"E{li}"]), f"E{li}"
    close(st.loss[sel], loss, what="loss")
    close(st.grads[sel], grads, what="grads")
    import oracle
    close(st.x_half[sel], oracle.sgd_update(sub["params"], grads, wl["lr"]), what="x_half")
    # mix, from the GPU's own x_half (properties only)
    xh = st.x_half.cpu().numpy(); xhat0 = wl["x_hat"]; xhat1 = st.x_hat.cpu().numpy()
    q = xhat1 - xhat0
    delta = xh - xhat0
    for s, k in enumerate(int(v) for v in wl["seg_k"]):
        lo, hi = int(wl["seg_offsets"][s]), int(wl["seg_offsets"][s + 1])
        if k >= hi - lo:
            assert np.array_equal(xhat1[:, lo:hi], xh[:, lo:hi])
            continue
        for i in range(wl["nodes"]):
            nz = np.flatnonzero(q[i, lo:hi])
            assert len(nz) <= k and len(nz) >= k - 8           # exact zeros among the kept deltas are possible
            keptmin = np.abs(delta[i, lo:hi][nz]).min()
            dropped = np.setdiff1d(np.arange(hi - lo), nz)
            assert keptmin >= np.abs(delta[i, lo:hi][dropped]).max()
    assert np.allclose(st.x_out.double().sum(0).cpu().numpy(), xh.astype(np.float64).sum(0),
                       atol=1e-5 * wl["nodes"] * max(1.0, float(np.abs(xh).max())))


def test_vgg11_full_size_sampled_nodes():
    _compare_sampled_nodes(wlmod.make_workload("vgg11"), [0, 5])


def test_resnet20_topk_full_size_sampled_nodes():
    _compare_sampled_nodes(wlmod.make_workload("resnet20_topk"), [0, 17, 39])


def test_resnet20_topk_full_size_in_the_benchmark_configuration():
    # two node groups on parallel streams, as bench.py runs this workload: nodes of both groups sampled
    _compare_sampled_nodes(wlmod.make_workload("resnet20_topk"), [1, 19, 20, 38], node_groups=2)


def test_resnet20_layerwise_topk_full_size_sampled_nodes():
    _compare_sampled_nodes(wlmod.make_workload("resnet20_topk_layerwise"), [3, 22])


def test_resnet20_topk_40_nodes():
    # 40-node ring with top-1% compression of the flattened update (batch reduced to keep the oracle short)
    wl = wlmod.make_workload("resnet20_topk", batch=4)
    st, ref = _compare(wl)
    k = int(wl["seg_k"][0])
    assert all(np.count_nonzero(ref["q"][i]) == k for i in range(wl["nodes"]))
    # doubly-stochastic ring: the node average is preserved by the mix
    assert np.allclose(st.x_out.double().sum(0).cpu().numpy(), st.x_half.double().sum(0).cpu().numpy(),
                       atol=1e-4)


def test_vgg11_8_nodes():
    _compare(wlmod.make_workload("vgg11", batch=4))


@pytest.mark.parametrize("name,kw", [("conv16", {}), ("resnet20_topk", dict(nodes=5, batch=2))])
def test_step_with_8bit_messages(name, kw):
    """Whole step with the gossip messages sent as 8-bit codes.  The op itself is bit-exact on equal inputs
    (test_gossip_mix_q8); here its input x_half carries the step's fp32-vs-fp64 summation differences, which may
    move a difference across a rounding boundary: such entries differ by exactly one code step and must be rare."""
    wl = wlmod.make_workload(name, **kw)
    ref = ostep.train_step(wl, message_bits=8)
    st = TrainStep.from_workload(wl, message_bits=8)
    st.run()
    torch.cuda.synchronize()
    assert int(st.dev_status.item()) == 0
    close(st.x_half, ref["x_half"], what="x_half")
    step = st.msg_scale.cpu().numpy()[:, 0]                     # one segment in these workloads
    for got, want, what in ((st.x_hat, ref["x_hat"], "x_hat"), (st.x_out, ref["x"], "x")):
        err = np.abs(got.cpu().numpy().astype(np.float64) - want)
        tight = err <= 1e-6 + 1e-5 * np.abs(want)
        assert (err <= 1.001 * step[:, None] + 1e-6).all(), what        # never more than one code step (x: a mix of steps)
        assert (~tight).mean() < 2e-3, f"{what}: {(~tight).sum()} entries off by a code step"


@pytest.mark.parametrize("name,nodes,batch", [("resnet20", 3, 4), ("vgg11", 2, 2), ("resnet20_topk", 5, 2)])
def test_step_keeping_only_8bit_tensors_for_backward(name, nodes, batch):
    """recompute_norm_input: the fp32 inputs of the norm layers are not kept per layer but recomputed in the
    backward pass from the saved 8-bit operands.  Same integer sums and the same dequantization, so every
    result of the step is bit-identical to the default mode (which is compared with the oracle above), and
    what a node keeps between the passes shrinks to its 8-bit tensors and the norm statistics."""
    wl = wlmod.make_workload(name, nodes=nodes, batch=batch)
    a = TrainStep.from_workload(wl)
    b = TrainStep.from_workload(wl, recompute_norm_input=True)
    a.run(); b.run()
    torch.cuda.synchronize()
    assert int(b.dev_status.item()) == 0
    for t in ("grads", "x_half", "x_hat", "x_out", "loss"):
        assert torch.equal(getattr(a, t), getattr(b, t)), t
    for li, op in enumerate(wl["ops"]):
        if op["op"] in ("conv", "linear"):
            assert torch.equal(a.buf[li]["E"], b.buf[li]["E"]), f"E{li}"
    ma, mb = a.saved_bytes_per_node(), b.saved_bytes_per_node()
    assert mb["fp32_norm_inputs"] == 0 and ma["fp32_norm_inputs"] > 0
    assert mb["int8_activations"] == ma["int8_activations"] and mb["total"] < ma["total"]


@pytest.mark.parametrize("name,nodes,batch,groups", [("resnet20", 5, 4, 2), ("vgg11", 4, 2, 4), ("resnet20_topk", 6, 2, 3),
                                                     ("conv16", 4, 8, 2)])
def test_step_with_node_groups_on_separate_streams(name, nodes, batch, groups):
    """node_groups: the nodes' forward and backward passes split into groups that run side by side on their own
    streams (uneven group sizes included).  The nodes are independent until the mix, so every result is
    bit-identical to the one-group step; also as a captured CUDA graph."""
    wl = wlmod.make_workload(name, nodes=nodes, batch=batch)
    a = TrainStep.from_workload(wl)
    b = TrainStep.from_workload(wl, node_groups=groups)
    assert len(b.groups) == groups
    a.run(); b.run()
    torch.cuda.synchronize()
    assert int(b.dev_status.item()) == 0
    names = ["grads", "x_half", "x_hat", "x_out"] + (["loss"] if "labels" in wl else [])
    for t in names:
        assert torch.equal(getattr(a, t), getattr(b, t)), t
    for li, op in enumerate(wl["ops"]):
        if op["op"] in ("conv", "linear"):
            assert torch.equal(a.buf[li]["E"], b.buf[li]["E"]), f"E{li}"
    if "dy" in wl:
        assert torch.equal(a.input_grad_out, b.input_grad_out)
    # a second step from the same state, eager against graph replay (capture() runs the step once to warm up)
    b.capture()
    a.params.copy_(a.x_out)
    b.params.copy_(a.params); b.x_hat.copy_(a.x_hat)
    a.run(); b.replay()
    torch.cuda.synchronize()
    for t in names:
        assert torch.equal(getattr(a, t), getattr(b, t)), t


@pytest.mark.parametrize("name,nodes,batch,kw", [("resnet20", 3, 4, {}), ("vgg11", 2, 2, {}), ("resnet20_topk", 5, 2, {}),
                                                 ("resnet20", 4, 32, dict(node_groups=2)),
                                                 ("resnet20", 2, 4, dict(recompute_norm_input=True))])
def test_step_with_requantize_inside_the_norm_layers(name, nodes, batch, kw):
    """fuse_requantize: Range-EvoNorm layers in front of (behind, in the backward pass) a convolution write the
    8-bit codes themselves.  Same codes, so every result equals the default step's bit for bit - eagerly and
    as a graph replay - and the calls that disappear are quantizer launches."""
    wl = wlmod.make_workload(name, nodes=nodes, batch=batch)
    a = TrainStep.from_workload(wl, **kw)
    b = TrainStep.from_workload(wl, fuse_requantize=True, **kw)
    assert any(x.get("q8_fwd") for x in b.buf) and any(x.get("q8_bwd") for x in b.buf)
    la = [c[0] for c in a.record()]
    lb = [c[0] for c in b.record()]
    fused = lb.count("lpdt_range_evonorm_fwd_q8") + lb.count("lpdt_range_evonorm_bwd_q8")
    assert lb.count("lpdt_range_evonorm_fwd_q8") > 0 and lb.count("lpdt_range_evonorm_bwd_q8") > 0
    assert la.count("lpdt_quantize_with_range") - lb.count("lpdt_quantize_with_range") == fused
    a.load(wl); b.load(wl)
    a.run(); b.run()
    torch.cuda.synchronize()
    assert int(b.dev_status.item()) == 0
    names = ["grads", "x_half", "x_hat", "x_out"] + (["loss"] if "labels" in wl else [])
    for t in names:
        assert torch.equal(getattr(a, t), getattr(b, t)), t
    for li, op in enumerate(wl["ops"]):
        if op["op"] in ("conv", "linear"):
            assert torch.equal(a.buf[li]["E"], b.buf[li]["E"]), f"E{li}"
            assert torch.equal(a.buf[li]["qA"], b.buf[li]["qA"]), f"qA{li}"
    b.capture()
    a.params.copy_(a.x_out)
    b.params.copy_(a.params); b.x_hat.copy_(a.x_hat)
    a.run(); b.replay()
    torch.cuda.synchronize()
    assert int(b.dev_status.item()) == 0
    for t in names:
        assert torch.equal(getattr(a, t), getattr(b, t)), t
