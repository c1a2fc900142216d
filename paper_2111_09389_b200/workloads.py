"""Seeded synthetic workloads for the 8-bit decentralized training step.

This module holds data recipes only — tensor shapes, network layer lists,
parameter offsets and random draws — and none of the method's arithmetic, so
that both the CUDA library's callers and the CPU oracle's callers can be fed
the same bits.  It imports neither of them.

The paper's image workloads (CIFAR-10 on ResNet-20 / VGG-11, Section 4) are
replaced by N(0,1) tensors of the same shape: 32x32x3 inputs, batch 32 per
node, ring topologies.

A network is a list of op dicts interpreted front to back (forward) and back to
front (backward):
    conv    : 3x3/1x1 convolution, weights at params[w_off : w_off+Cout*R*S*Cin]
    ren     : Range-EvoNorm; v, gamma, beta at p_off, p_off+C, p_off+2C
    save    : remember the current activation as the shortcut input
    add     : current += shortcut(saved) (stride / channel offset = option-A shortcut)
    maxpool : 2x2, stride 2
    avgpool : global average over H*W
    linear  : fully connected, weights at w_off ([Cout][Cin]), bias at b_off
The loss is softmax cross-entropy on the last op's output unless the workload
supplies an upstream gradient `dy` instead.
"""
import math

import numpy as np

REN_EPS = 1e-5


def ring_matrix(n):
    """Symmetric doubly-stochastic ring: 1/3 on self and on both neighbours."""
    W = np.zeros((n, n), np.float32)
    third = np.float32(1.0 / 3.0)
    for i in range(n):
        for j in (i - 1, i, i + 1):
            W[i, j % n] += third
    return W


class _Net:
    def __init__(self, H, W, C):
        self.ops = []
        self.d = 0
        self.H, self.W, self.C = H, W, C

    def _take(self, n):
        off = self.d
        self.d += n
        return off

    def conv(self, cout, k=3, stride=1, pad=1):
        cin = self.C
        op = dict(op="conv", H=self.H, W=self.W, cin=cin, cout=cout, R=k, S=k, stride=stride,
                  pad=pad, w_off=self._take(cout * k * k * cin))
        self.ops.append(op)
        self.H = (self.H + 2 * pad - k) // stride + 1
        self.W = (self.W + 2 * pad - k) // stride + 1
        self.C = cout
        return self

    def ren(self, cpg=8):
        C = self.C
        self.ops.append(dict(op="ren", H=self.H, W=self.W, C=C, groups=C // cpg,
                             p_off=self._take(3 * C)))
        return self

    def save(self):
        self.ops.append(dict(op="save", H=self.H, W=self.W, C=self.C))
        self._saved = (self.H, self.W, self.C)
        return self

    def add(self):
        H0, W0, C0 = self._saved
        stride = H0 // self.H
        self.ops.append(dict(op="add", H=H0, W=W0, Ca=C0, C=self.C, stride=stride,
                             ch_off=(self.C - C0) // 2))
        return self

    def maxpool(self):
        self.ops.append(dict(op="maxpool", H=self.H, W=self.W, C=self.C))
        self.H //= 2
        self.W //= 2
        return self

    def avgpool(self):
        self.ops.append(dict(op="avgpool", H=self.H, W=self.W, C=self.C))
        self.H = self.W = 1
        return self

    def linear(self, cout):
        cin = self.C * self.H * self.W
        self.ops.append(dict(op="linear", cin=cin, cout=cout, w_off=self._take(cout * cin),
                             b_off=self._take(cout)))
        self.C = cout
        return self


def resnet20_ops():
    """ResNet-20 for 32x32x3 inputs: 3 stages x 3 basic blocks at 16/32/64
    channels, Range-EvoNorm after every convolution, parameter-free shortcuts."""
    net = _Net(32, 32, 3)
    net.conv(16).ren()
    for stage, width in enumerate((16, 32, 64)):
        for block in range(3):
            stride = 2 if (stage > 0 and block == 0) else 1
            net.save()
            net.conv(width, stride=stride).ren()
            net.conv(width).ren()
            net.add()
    net.avgpool().linear(10)
    return net.ops, net.d


def vgg11_ops():
    """VGG-11 for 32x32x3 inputs: widths 64,128,256,256,512,512,512,512 with a
    max-pool after convs 1,2,4,6,8 and a 512->10 classifier."""
    net = _Net(32, 32, 3)
    pool_after = {0, 1, 3, 5, 7}
    for i, width in enumerate((64, 128, 256, 256, 512, 512, 512, 512)):
        net.conv(width).ren()
        if i in pool_after:
            net.maxpool()
    net.avgpool().linear(10)
    return net.ops, net.d


def single_conv_ops(H=16, W=16, cin=16, cout=16, groups=4):
    net = _Net(H, W, cin)
    net.conv(cout).ren(cpg=cout // groups)
    return net.ops, net.d


def conv_macs(ops, batch):
    """Multiply-accumulates of one forward pass over `batch` images (the Conv and
    Linear rows of the paper's operation-count table, forward share)."""
    macs = 0
    for op in ops:
        if op["op"] == "conv":
            Ho = (op["H"] + 2 * op["pad"] - op["R"]) // op["stride"] + 1
            Wo = (op["W"] + 2 * op["pad"] - op["S"]) // op["stride"] + 1
            macs += batch * Ho * Wo * op["cout"] * op["cin"] * op["R"] * op["S"]
        elif op["op"] == "linear":
            macs += batch * op["cout"] * op["cin"]
    return macs


def init_params(ops, d, nodes, rng, node_jitter=0.01):
    """Kaiming-uniform weights (bound sqrt(6/fan_in)), v = gamma = 1, beta = 0,
    zero biases; every node starts from the common draw plus a small per-node
    perturbation of the weights so that the nodes' models differ."""
    base = np.zeros(d, np.float32)
    is_weight = np.zeros(d, bool)
    for op in ops:
        if op["op"] == "conv":
            n = op["cout"] * op["R"] * op["S"] * op["cin"]
            bound = math.sqrt(6.0 / (op["R"] * op["S"] * op["cin"]))
            base[op["w_off"]:op["w_off"] + n] = rng.uniform(-bound, bound, n)
            is_weight[op["w_off"]:op["w_off"] + n] = True
        elif op["op"] == "linear":
            n = op["cout"] * op["cin"]
            bound = math.sqrt(6.0 / op["cin"])
            base[op["w_off"]:op["w_off"] + n] = rng.uniform(-bound, bound, n)
            is_weight[op["w_off"]:op["w_off"] + n] = True
        elif op["op"] == "ren":
            C = op["C"]
            base[op["p_off"]:op["p_off"] + 2 * C] = 1.0
    params = np.tile(base, (nodes, 1))
    jitter = rng.standard_normal((nodes, d)).astype(np.float32) * np.float32(node_jitter)
    params += jitter * is_weight[None, :] * np.abs(base)[None, :]
    return np.ascontiguousarray(params, dtype=np.float32)


def layer_segments(ops, d):
    """Offsets of the per-layer segments of the flat parameter vector: a segment starts at the weights
    of every conv/linear layer and runs to the next layer's weights (so it also holds the norm
    parameters or bias that follow), n_layers + 1 entries."""
    starts = sorted(op["w_off"] for op in ops if op["op"] in ("conv", "linear"))
    assert starts and starts[0] == 0
    return np.array(starts + [d], np.int64)


def make_labels(nodes, batch, classes, rng, dirichlet_alpha=None):
    if dirichlet_alpha is None:
        return rng.integers(0, classes, (nodes, batch)).astype(np.int32)
    out = np.zeros((nodes, batch), np.int32)
    for n in range(nodes):
        p = rng.dirichlet(np.full(classes, dirichlet_alpha))
        out[n] = rng.choice(classes, size=batch, p=p)
    return out


def make_workload(name, nodes=None, batch=None, seed=None, dirichlet_alpha=None):
    """Build one of the named workloads.  Returns a dict with
    ops, d, nodes, batch, x [N,B,H,W,C], labels or dy, params [N,d], x_hat [N,d],
    Wmix [N,N], lr, gamma, seg_offsets, seg_k, ren_eps.

    names: "conv16"       one 3x3 conv 16->16 on 16x16, 4 nodes x batch 8, 4 norm groups
           "resnet20"     16 nodes x batch 32, dense gossip, gamma 1
           "resnet20_topk" 40 nodes x batch 32, top-1% of the flattened update, gamma 0.1
           "resnet20_topk_layerwise" the same with the paper's layer-wise top-K: one segment per
                          conv/linear layer (its weights plus the norm parameters or bias that
                          follow them), the top 1% of each kept
           "vgg11"        8 nodes x batch 32, dense gossip
    """
    defaults = dict(conv16=(4, 8, 0), resnet20=(16, 32, 1001), resnet20_topk=(40, 32, 1003),
                    resnet20_topk_layerwise=(40, 32, 1004), vgg11=(8, 32, 1002))
    dn, db, ds = defaults[name]
    nodes = dn if nodes is None else nodes
    batch = db if batch is None else batch
    seed = ds if seed is None else seed
    rng = np.random.default_rng(seed)
    wl = dict(name=name, nodes=nodes, batch=batch, seed=seed, ren_eps=REN_EPS, lr=0.1, gamma=1.0)
    if name == "conv16":
        ops, d = single_conv_ops()
        wl["x"] = rng.standard_normal((nodes, batch, 16, 16, 16)).astype(np.float32)
        wl["dy"] = rng.standard_normal((nodes, batch, 16, 16, 16)).astype(np.float32)
    else:
        ops, d = vgg11_ops() if name == "vgg11" else resnet20_ops()
        wl["x"] = rng.standard_normal((nodes, batch, 32, 32, 3)).astype(np.float32)
        wl["labels"] = make_labels(nodes, batch, 10, rng, dirichlet_alpha)
    wl["ops"], wl["d"] = ops, d
    wl["params"] = init_params(ops, d, nodes, rng)
    wl["Wmix"] = ring_matrix(nodes)
    if name in ("resnet20_topk", "resnet20_topk_layerwise"):
        # public copies lag the models by a heavy-tailed residual, so that the
        # top 1% by magnitude is a non-trivial selection
        resid = rng.standard_normal((nodes, d)) * np.where(rng.random((nodes, d)) < 0.05, 1e-2, 1e-4)
        wl["x_hat"] = (wl["params"] - resid).astype(np.float32)
        wl["gamma"] = 0.1
        if name == "resnet20_topk_layerwise":
            wl["seg_offsets"] = layer_segments(ops, d)
        else:
            wl["seg_offsets"] = np.array([0, d], np.int64)
        wl["seg_k"] = np.maximum(1, np.diff(wl["seg_offsets"]) // 100).astype(np.int64)
    else:
        wl["x_hat"] = np.zeros((nodes, d), np.float32)
        wl["seg_offsets"] = np.array([0, d], np.int64)
        wl["seg_k"] = np.array([d], np.int64)
    return wl


def random_s8(rng, shape):
    """int8 iid uniform on {-127..127} (the contraction sweep's operands)."""
    return rng.integers(-127, 128, size=shape, dtype=np.int16).astype(np.int8)
