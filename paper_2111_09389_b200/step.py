"""One whole 8-bit training step of all simulated nodes, as a fixed sequence of
lpdt C-ABI calls on preallocated device buffers.

TrainStep walks a network op list (see `workloads`) forward and backward:
every conv/linear quantizes its input and weights per node, runs the int8
contraction and dequantizes; Range-EvoNorm follows in fp32; backward quantizes
each incoming layer gradient once and feeds both adjoint contractions, weight
gradients staying fp32; then the SGD half-step and the CHOCO gossip mix
(Section 3 and Algorithms 1 and 3 of the paper).  Python only orders the calls
and owns the buffers; all arithmetic runs in the CUDA library.
"""
import torch

from . import api


class TrainStep:
    def __init__(self, ops, d, nodes, batch, in_shape, ren_eps=1e-5, lr=0.1, gamma=1.0,
                 seg_offsets=None, seg_k=None, has_labels=True, grad_rounding=0, seed=0,
                 quantize_wgrad=False, input_grad=False, message_bits=32, recompute_norm_input=False,
                 node_groups=1, fuse_requantize=False, device="cuda"):
        if not torch.cuda.is_available():
            raise RuntimeError("TrainStep needs a CUDA device; there is no CPU path")
        self.ops, self.d, self.N, self.B = ops, d, nodes, batch
        self.eps, self.lr, self.gamma = float(ren_eps), float(lr), float(gamma)
        self.seg_offsets = [0, d] if seg_offsets is None else [int(v) for v in seg_offsets]
        self.seg_k = [d] if seg_k is None else [int(v) for v in seg_k]
        self.grad_rounding, self.seed = grad_rounding, seed
        self.quantize_wgrad, self.input_grad = quantize_wgrad, input_grad
        self.message_bits = message_bits          # 8: gossip messages as 8-bit codes with one range per (node, segment)
        # True: nothing but 8-bit tensors (and the small norm statistics) is kept from the forward to the
        # backward pass.  The fp32 input of every Range-EvoNorm layer, i.e. the output of the convolution
        # before it, is not stored per layer; the backward pass recomputes it from the saved 8-bit operands
        # into one shared buffer (same integer sums, same dequantization: bit-identical values).
        self.recompute_norm_input = recompute_norm_input
        self._shared_out = {}
        # True: a Range-EvoNorm layer whose result goes straight into a convolution's quantizer writes the 8-bit
        # codes itself where the shape allows (lpdt_range_evonorm_fwd_q8 / _bwd_q8: no fp32 round trip, no separate
        # quantizer launch; identical codes; a quarter fewer launches per ResNet-20 step).  Off by default: on the
        # benchmark workloads the step measured 2-8 % slower with it (the CTAs of a node have to meet before the
        # first code can be written).  Not with stochastic rounding of the layer gradients.
        self.fuse_requantize = bool(fuse_requantize)
        # node_groups > 1: the nodes are split into that many contiguous groups whose forward and backward passes
        # run side by side on streams of their own (the nodes are independent until the gossip mix).  Every call
        # then covers fewer nodes, and the launches of one group fill the gaps of the others; results do not
        # change.  Not with stochastic rounding, whose random numbers are keyed by the node's index inside a call.
        self.node_groups = max(1, min(int(node_groups), nodes)) if not grad_rounding else 1
        dev = torch.device(device)
        N, B = nodes, batch
        f32 = dict(dtype=torch.float32, device=dev)
        i8 = dict(dtype=torch.int8, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        self.params = torch.zeros(N, d, **f32)
        self.grads = torch.zeros(N, d, **f32)
        self.x_half = torch.zeros(N, d, **f32)
        self.x_hat = torch.zeros(N, d, **f32)
        self.x_out = torch.zeros(N, d, **f32)
        self.Wmix = torch.zeros(N, N, **f32)
        self.x = torch.zeros((N, B) + tuple(in_shape), **f32)
        self.labels = torch.zeros(N, B, **i32) if has_labels else None
        self.loss = torch.zeros(N, **f32)
        self.dev_status = torch.zeros(1, **i32)
        self.msg_scale = torch.zeros(N, len(self.seg_k), **f32)
        ws_bytes = max(api.lpdt_quantize_workspace_size(N),
                       api.lpdt_gossip_mix_workspace_size(N, d, len(self.seg_k)))
        self.buf = []
        shape = tuple(in_shape)
        # all layer weights are quantized by one batched call into one int8 buffer (256-byte aligned blocks)
        wlist = [op for op in ops if op["op"] in ("conv", "linear")]
        self.w_src, self.w_size, self.w_dst = [], [], []
        qbytes = 0
        for op in wlist:
            wn = op["cout"] * op["cin"] * (op["R"] * op["S"] if op["op"] == "conv" else 1)
            self.w_src.append(op["w_off"]); self.w_size.append(wn); self.w_dst.append(qbytes)
            qbytes += (N * wn + 255) // 256 * 256
        self.qW_all = torch.empty(max(qbytes, 256), **i8)
        # raw int32 weight-gradient sums of every layer, each a contiguous [nodes][size] block (256-byte aligned
        # starts): converted to fp32 by one batched launch at the end of the backward pass
        self.g_acc_off, n_acc = [], 0
        for wn in self.w_size:
            self.g_acc_off.append(n_acc)
            n_acc += (N * wn + 63) // 64 * 64
        self.g_acc = torch.empty(max(n_acc, 64), **i32)
        self.sW_all = torch.empty(max(len(wlist), 1), N, **f32)
        ws_bytes = max(ws_bytes, api.lpdt_quantize_batch_workspace_size(N, min(len(wlist), 64)))
        wi = 0
        for op in ops:
            k = op["op"]
            b = {}
            if k in ("conv", "linear"):
                if k == "linear":
                    H = W = 1; R = S = 1; stride = 1; pad = 0
                else:
                    H, W, R, S, stride, pad = op["H"], op["W"], op["R"], op["S"], op["stride"], op["pad"]
                desc = api.conv_desc(N, B, H, W, op["cin"], op["cout"], R, S, stride, pad)
                Ho = (H + 2 * pad - R) // stride + 1
                Wo = (W + 2 * pad - S) // stride + 1
                b.update(desc=desc, in_shape=(H, W, op["cin"]),
                         qA=torch.empty(N, B, H, W, op["cin"], **i8), sA=torch.empty(N, **f32),
                         qW=self.qW_all[self.w_dst[wi]:self.w_dst[wi] + N * self.w_size[wi]].view(N, op["cout"], R, S, op["cin"]),
                         sW=self.sW_all[wi],
                         out=self._conv_out((N, B, Ho, Wo, op["cout"]), f32),
                         E=torch.empty(N, B, Ho, Wo, op["cout"], **i8), sE=torch.empty(N, **f32),
                         dx=torch.empty(N, B, H, W, op["cin"], **f32),
                         wn=op["cout"] * R * S * op["cin"], wi=wi)
                b["gacc"] = self.g_acc[self.g_acc_off[wi]:self.g_acc_off[wi] + N * b["wn"]].view(N, b["wn"])
                if quantize_wgrad:
                    b.update(gq=torch.empty(N, b["wn"], **i8), gs=torch.empty(N, **f32),
                             gw=torch.empty(N, b["wn"], **f32))
                wi += 1
                for which in (0, 1, 2):
                    ws_bytes = max(ws_bytes, api.lpdt_qconv_workspace_size(desc, which))
                shape = (Ho, Wo, op["cout"])
            elif k == "ren":
                H, W, Cc, G = op["H"], op["W"], op["C"], op["groups"]
                b.update(out=torch.empty(N, B, H, W, Cc, **f32), dx=torch.empty(N, B, H, W, Cc, **f32),
                         gmin=torch.empty(N, B, G, **f32), gmax=torch.empty(N, B, G, **f32),
                         amin=torch.empty(N, B, G, **i32), amax=torch.empty(N, B, G, **i32))
                # per-sample partial sums of the parameter gradients: a buffer per layer, because their reduction
                # runs later, on the side stream
                b["ws_ren"] = torch.empty(api.lpdt_range_evonorm_bwd_workspace_size(N, B, Cc), dtype=torch.uint8,
                                          device=dev)
                b["q8_fwd"] = self.fuse_requantize and bool(api.lpdt_range_evonorm_fwd_q8_fits(B, H, W, Cc, G))
                b["q8_bwd"] = (self.fuse_requantize and not grad_rounding and
                               bool(api.lpdt_range_evonorm_bwd_q8_fits(B, H, W, Cc, G)))
                b["ctl"] = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(N), dtype=torch.uint8, device=dev)
            elif k == "add":
                Ho, Wo = (op["H"] + op["stride"] - 1) // op["stride"], (op["W"] + op["stride"] - 1) // op["stride"]
                b.update(out=torch.empty(N, B, Ho, Wo, op["C"], **f32))
            elif k == "save":
                b.update(dx=torch.empty(N, B, op["H"], op["W"], op["C"], **f32))
            elif k == "maxpool":
                H, W, Cc = op["H"], op["W"], op["C"]
                b.update(out=torch.empty(N, B, H // 2, W // 2, Cc, **f32),
                         idx=torch.empty(N, B, H // 2, W // 2, Cc, **i8),
                         dx=torch.empty(N, B, H, W, Cc, **f32))
                shape = (H // 2, W // 2, Cc)
            elif k == "avgpool":
                b.update(out=torch.empty(N, B, 1, 1, op["C"], **f32),
                         dx=torch.empty(N, B, op["H"], op["W"], op["C"], **f32))
                shape = (1, 1, op["C"])
            else:
                raise ValueError(k)
            self.buf.append(b)
        self.out_shape = shape
        # per-node ranges emitted by producers for the next quantizer: row li = forward output of op li,
        # row len(ops)+li = layer gradient leaving op li; zeroed once per step
        self.ranges = torch.zeros(2 * len(ops), N, **f32)
        self.dy = torch.zeros((N, B) + tuple(shape), **f32)      # upstream gradient / dlogits
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        # The weight-gradient contractions leave the critical path of the backward pass: each is issued on a
        # side stream (its own workspace) as soon as its quantized layer gradient exists, and joins before the
        # parameter update.  Captured into the step's CUDA graph the fork and join become graph edges.
        self.ws_side = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.side = torch.cuda.Stream(device=dev)
        self.groups = []
        if self.node_groups > 1:
            bounds = [N * g // self.node_groups for g in range(self.node_groups + 1)]
            self.groups = [self._node_view(bounds[g], bounds[g + 1], ws_bytes, dev) for g in range(self.node_groups)]

    def _node_view(self, n0, n1, ws_bytes, dev):
        """A TrainStep over nodes [n0, n1) that shares this one's storage: every per-node tensor is a slice,
        every convolution descriptor carries the group's node count; it has its own streams and workspaces."""
        N = self.N
        c = TrainStep.__new__(TrainStep)
        c.__dict__.update({k: v for k, v in self.__dict__.items() if not isinstance(v, (torch.Tensor, list, dict))})
        c.ops, c.w_src, c.w_size, c.w_dst, c.seg_offsets, c.seg_k = (self.ops, self.w_src, self.w_size, self.w_dst,
                                                                     self.seg_offsets, self.seg_k)
        c.N, c.node_groups, c.groups, c._shared_out = n1 - n0, 1, [], {}
        cut = lambda t: t[n0:n1] if isinstance(t, torch.Tensor) and t.dim() > 0 and t.shape[0] == N else t
        for name in ("params", "grads", "x", "labels", "loss", "dy"):
            setattr(c, name, cut(getattr(self, name)))
        c.dev_status = self.dev_status
        c.ranges = self.ranges[:, n0:n1]
        c.buf = []
        for op, b in zip(self.ops, self.buf):
            cb = {}
            for k, v in b.items():
                if k == "desc":
                    cb[k] = api.conv_desc(n1 - n0, v.B, v.H, v.W, v.Cin, v.Cout, v.R, v.S, v.stride, v.pad)
                elif k == "ws_ren":
                    per = v.numel() // N
                    cb[k] = v[n0 * per:n1 * per]
                elif k == "ctl":          # the meeting point of a group's own launches
                    cb[k] = torch.zeros(api.lpdt_range_evonorm_q8_ctl_size(n1 - n0), dtype=torch.uint8, device=dev)
                else:
                    cb[k] = cut(v)
            c.buf.append(cb)
        c.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        c.ws_side = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        c.stream = torch.cuda.Stream(device=dev)
        c.side = torch.cuda.Stream(device=dev)
        return c

    def _each_group(self, fn):
        """fn(step) for this step, or for every node group on its own stream between a fork and a join."""
        if not self.groups:
            fn(self)
            return
        main = torch.cuda.current_stream()
        for i, g in enumerate(self.groups):
            g.stream.wait_stream(main)
            api.GROUP = i + 1
            with torch.cuda.stream(g.stream):
                fn(g)
        api.GROUP = 0
        for g in self.groups:
            main.wait_stream(g.stream)

    def _conv_out(self, shape, f32):
        """fp32 output buffer of a convolution: one per layer, or (recompute_norm_input) one per distinct
        shape shared by all layers of that shape, since no layer's output has to outlive its consumers."""
        if not self.recompute_norm_input:
            return torch.empty(*shape, **f32)
        if shape not in self._shared_out:
            self._shared_out[shape] = torch.empty(*shape, **f32)
        return self._shared_out[shape]

    def saved_bytes_per_node(self):
        """Bytes one node keeps from its forward pass for its backward pass, by kind."""
        N = self.N
        rep = {"int8_activations": 0, "int8_weights": 0, "fp32_norm_inputs": 0, "norm_statistics": 0, "pool_indices": 0}
        for op, b in zip(self.ops, self.buf):
            k = op["op"]
            if k in ("conv", "linear"):
                rep["int8_activations"] += b["qA"].numel() // N
                rep["int8_weights"] += b["qW"].numel() // N
            elif k == "ren":
                if not self.recompute_norm_input:
                    rep["fp32_norm_inputs"] += 4 * self.B * op["H"] * op["W"] * op["C"]
                rep["norm_statistics"] += 4 * 4 * self.B * op["groups"]
            elif k == "maxpool":
                rep["pool_indices"] += b["idx"].numel() // N
        rep["total"] = sum(rep.values())
        return rep

    # ---- host -> device ------------------------------------------------------------
    def load(self, wl):
        self.params.copy_(torch.from_numpy(wl["params"]))
        self.x_hat.copy_(torch.from_numpy(wl["x_hat"]))
        self.Wmix.copy_(torch.from_numpy(wl["Wmix"]))
        self.x.copy_(torch.from_numpy(wl["x"]))
        if "labels" in wl and self.labels is not None:
            self.labels.copy_(torch.from_numpy(wl["labels"]))
        if "dy" in wl:
            self.dy.copy_(torch.from_numpy(wl["dy"]))

    # ---- host inputs, one batch ahead -------------------------------------------------
    def upload(self, x_host, labels_host=None):
        """Start copying a batch (pinned host tensors) into staging buffers on a copy stream; returns at once.
        The copy overlaps whatever step is running: the step's own input buffers are untouched until
        step_from_upload() takes the staged batch."""
        if not hasattr(self, "_copy"):
            self._copy = torch.cuda.Stream(device=self.x.device)
            self._x_stage = torch.empty_like(self.x)
            self._lab_stage = torch.empty_like(self.labels) if self.labels is not None else None
            self._staged = torch.cuda.Event()
            self._taken = torch.cuda.Event()
            self._taken.record()
        self._copy.wait_event(self._taken)                 # the previous batch has left the staging buffers
        with torch.cuda.stream(self._copy):
            self._x_stage.copy_(x_host, non_blocking=True)
            if labels_host is not None and self._lab_stage is not None:
                self._lab_stage.copy_(labels_host, non_blocking=True)
            self._staged.record()

    def step_from_upload(self, step=None):
        """Take the staged batch (device-to-device copy into the step's inputs, ordered after the upload) and
        run one step: `step` is run() by default, or replay() once the step has been captured."""
        cur = torch.cuda.current_stream()
        cur.wait_event(self._staged)
        self.x.copy_(self._x_stage, non_blocking=True)
        if self._lab_stage is not None:
            self.labels.copy_(self._lab_stage, non_blocking=True)
        self._taken.record()
        (step or self.run)()

    @classmethod
    def from_workload(cls, wl, **kw):
        st = cls(wl["ops"], wl["d"], wl["nodes"], wl["batch"], wl["x"].shape[2:], wl["ren_eps"], wl["lr"],
                 wl["gamma"], wl["seg_offsets"], wl["seg_k"], has_labels=("labels" in wl),
                 input_grad=("dy" in wl), **kw)
        st.load(wl)
        return st

    # ---- the step --------------------------------------------------------------------
    def _p(self, off):
        return self.params[:, off:]

    def _g(self, off):
        return self.grads[:, off:]

    def _prepare(self):
        """Once per step, all nodes: clear the range accumulators, quantize every layer's weights."""
        N, d = self.N, self.d
        api.lpdt_fill_zero(self.ranges)
        for lo in range(0, len(self.w_size), 64):        # every layer's weights, 64 tensors per call
            hi = min(lo + 64, len(self.w_size))
            api.lpdt_quantize_batch(self.params, N, d, self.w_src[lo:hi], self.w_size[lo:hi], self.w_dst[lo:hi],
                                    self.qW_all, self.sW_all[lo:hi], self.ws)

    def forward(self):
        self._prepare()
        self._each_group(lambda g: g._forward_layers())
        self.out = self.buf[-1]["out"]
        return self.out

    def _forward_layers(self):
        N, B, d = self.N, self.B, self.d
        cur = self.x
        cur_range = None          # per-node max|cur| when the producer of cur emitted it
        saved = []
        for li, (op, b) in enumerate(zip(self.ops, self.buf)):
            k = op["op"]
            if k in ("conv", "linear"):
                n_in = cur.numel() // N
                if b.pop("pre_quantized", False):
                    pass                            # the norm layer before it wrote qA and sA
                elif cur_range is not None:
                    api.lpdt_quantize_with_range(cur, N, n_in, n_in, cur_range, b["qA"], b["sA"])
                else:
                    api.lpdt_quantize(cur, N, n_in, n_in, b["qA"], b["sA"], self.ws)
                bias = self._p(op["b_off"]) if k == "linear" else None
                api.lpdt_qconv_fwd(b["desc"], b["qA"], b["sA"], b["qW"], b["sW"], Y=b["out"], bias=bias,
                                   bias_node_stride=d, ws=self.ws, dev_status=self.dev_status)
                cur, cur_range = b["out"], None
            elif k == "ren":
                Cc = op["C"]
                b["x"] = cur
                b["x_from"] = li - 1 if (li > 0 and self.ops[li - 1]["op"] in ("conv", "linear")) else None
                # an identity shortcut right after this layer is added inside the kernel
                nxt = self.ops[li + 1] if li + 1 < len(self.ops) else None
                fuse = nxt is not None and nxt["op"] == "add" and nxt["stride"] == 1 and nxt["Ca"] == nxt["C"]
                res = saved[-1] if fuse else None
                # the next operation that computes: a convolution right behind this layer (or behind the fused
                # shortcut and the block boundary) takes the 8-bit codes from this kernel
                lj = li + 1
                if fuse:
                    lj += 1
                while lj < len(self.ops) and self.ops[lj]["op"] == "save":
                    lj += 1
                to_conv = lj < len(self.ops) and self.ops[lj]["op"] in ("conv", "linear")
                if b["q8_fwd"] and to_conv:
                    cb = self.buf[lj]
                    # y itself is still needed when something else reads it: the shortcut of the next block
                    keep_y = lj != li + 1
                    api.lpdt_range_evonorm_fwd_q8(N, B, op["H"], op["W"], Cc, op["groups"], self.eps, cur,
                                                  self._p(op["p_off"]), self._p(op["p_off"] + Cc),
                                                  self._p(op["p_off"] + 2 * Cc), d, b["out"] if keep_y else None,
                                                  b["gmin"], b["gmax"], b["amin"], b["amax"], cb["qA"], cb["sA"],
                                                  b["ctl"], res=res, dev_status=self.dev_status)
                    cb["pre_quantized"] = True
                    cur, cur_range = b["out"], None
                else:
                    api.lpdt_range_evonorm_fwd(N, B, op["H"], op["W"], Cc, op["groups"], self.eps, cur,
                                               self._p(op["p_off"]), self._p(op["p_off"] + Cc),
                                               self._p(op["p_off"] + 2 * Cc), d, b["out"], b["gmin"], b["gmax"],
                                               b["amin"], b["amax"], amax_out=self.ranges[li], res=res)
                    cur, cur_range = b["out"], self.ranges[li]
                b["fused_add"] = fuse
            elif k == "save":
                saved.append(cur)
            elif k == "add":
                a = saved.pop()
                if self.buf[li - 1].get("fused_add"):
                    continue                        # already added by the Range-EvoNorm kernel before it
                api.lpdt_residual_add(N, B, op["H"], op["W"], op["Ca"], op["C"], op["stride"], op["ch_off"],
                                      cur, a, b["out"], amax_out=self.ranges[li])
                cur, cur_range = b["out"], self.ranges[li]
            elif k == "maxpool":
                api.lpdt_maxpool2x2(N, B, op["H"], op["W"], op["C"], cur, b["out"], b["idx"])
                cur = b["out"]        # max-pooling keeps max|x| only for non-negative maxima: range recomputed
                cur_range = None
            elif k == "avgpool":
                api.lpdt_avgpool(N, B, op["H"] * op["W"], op["C"], cur, b["out"])
                cur, cur_range = b["out"], None
        self.out = cur
        return cur

    def backward(self):
        self._each_group(lambda g: g._backward_layers())
        self._finish_gradients()
        if self.groups:
            self.input_grad_out = self.buf[0]["dx"] if self.input_grad else None
        return self.input_grad_out

    def _backward_layers(self):
        N, B, d = self.N, self.B, self.d
        if self.labels is not None:
            K = self.out.numel() // (N * B)
            api.lpdt_softmax_ce(N, B, K, self.out, self.labels, self.loss, self.dy, self.dev_status)
        g = self.dy
        g_range = None
        L = len(self.ops)
        sc = []
        fused_shortcut = False
        ctr = 0
        for li in range(len(self.ops) - 1, -1, -1):
            op, b = self.ops[li], self.buf[li]
            k = op["op"]
            if k in ("conv", "linear"):
                if k == "linear":
                    api.lpdt_colsum(N, B, op["cout"], g, self._g(op["b_off"]), d)
                n_out = b["E"].numel() // N
                if b.pop("E_ready", False):
                    pass                            # the norm layer behind it wrote E and sE
                elif g_range is not None:
                    api.lpdt_quantize_with_range(g, N, n_out, n_out, g_range, b["E"], b["sE"],
                                                 rounding=self.grad_rounding, seed=self.seed, ctr_offset=ctr)
                else:
                    api.lpdt_quantize(g, N, n_out, n_out, b["E"], b["sE"], self.ws, rounding=self.grad_rounding,
                                      seed=self.seed, ctr_offset=ctr)
                ctr += 1
                main = torch.cuda.current_stream()
                self.side.wait_stream(main)               # E (and, at the first use, everything before) is ready
                with torch.cuda.stream(self.side):
                    if self.quantize_wgrad:
                        api.lpdt_qconv_bwd_weight(b["desc"], b["E"], b["sE"], b["qA"], b["sA"], dW=b["gw"],
                                                  dw_node_stride=b["wn"], ws=self.ws_side, dev_status=self.dev_status)
                        api.lpdt_quantize(b["gw"], N, b["wn"], b["wn"], b["gq"], b["gs"], self.ws_side)
                        api.lpdt_dequantize(b["gq"], N, b["wn"], b["gs"], self._g(op["w_off"]), d)
                    else:
                        # raw sums now, one conversion launch for all layers after the last of them
                        api.lpdt_qconv_bwd_weight(b["desc"], b["E"], b["sE"], b["qA"], b["sA"], dWacc=b["gacc"],
                                                  ws=self.ws_side, dev_status=self.dev_status)
                if li > 0 or self.input_grad:
                    # first convolution of a residual block with an identity shortcut: the block-output gradient
                    # joins this gradient in the contraction's epilogue (no separate residual_add_bwd pass)
                    addend = None
                    if li > 0 and self.ops[li - 1]["op"] == "save" and sc:
                        aop = sc[-1][1]
                        if aop["stride"] == 1 and aop["Ca"] == aop["C"]:
                            addend = sc[-1][0]
                            fused_shortcut = True
                    b["addend"] = addend
                    api.lpdt_qconv_bwd_data(b["desc"], b["E"], b["sE"], b["qW"], b["sW"], dA=b["dx"],
                                            ws=self.ws, dev_status=self.dev_status, addend=addend)
                    g, g_range = b["dx"], None
                else:
                    g = None
            elif k == "ren":
                Cc = op["C"]
                if self.recompute_norm_input and b["x_from"] is not None:
                    # the layer's input again, from the convolution's saved 8-bit operands into the shared buffer
                    cb, cop = self.buf[b["x_from"]], self.ops[b["x_from"]]
                    api.lpdt_qconv_fwd(cb["desc"], cb["qA"], cb["sA"], cb["qW"], cb["sW"], Y=cb["out"],
                                       bias=self._p(cop["b_off"]) if cop["op"] == "linear" else None,
                                       bias_node_stride=d, ws=self.ws, dev_status=self.dev_status)
                # dx only; the parameter-gradient sums stay as partial sums and are reduced on the side stream
                if b["q8_bwd"] and li > 0 and self.ops[li - 1]["op"] == "conv":
                    # dx goes nowhere but into that convolution's quantizer: its codes are written here
                    cb = self.buf[li - 1]
                    api.lpdt_range_evonorm_bwd_q8(N, B, op["H"], op["W"], Cc, op["groups"], self.eps, g, b["x"],
                                                  self._p(op["p_off"]), self._p(op["p_off"] + Cc), d, b["gmin"],
                                                  b["gmax"], b["amin"], b["amax"], cb["E"], cb["sE"], None, None, None,
                                                  d, b["ws_ren"], b["ctl"], dev_status=self.dev_status)
                    cb["E_ready"] = True
                    g, g_range = None, None
                else:
                    api.lpdt_range_evonorm_bwd(N, B, op["H"], op["W"], Cc, op["groups"], self.eps, g, b["x"],
                                               self._p(op["p_off"]), self._p(op["p_off"] + Cc), d, b["gmin"],
                                               b["gmax"], b["amin"], b["amax"], b["dx"], None, None, None, d, b["ws_ren"],
                                               amax_out=self.ranges[L + li])
                    g, g_range = b["dx"], self.ranges[L + li]
            elif k == "add":
                sc.append((g, op))
            elif k == "save":
                dy_sc, aop = sc.pop()
                if fused_shortcut:                  # already added by the convolution above
                    fused_shortcut = False
                else:
                    api.lpdt_residual_add_bwd(N, B, aop["H"], aop["W"], aop["Ca"], aop["C"], aop["stride"],
                                              aop["ch_off"], dy_sc, g, b["dx"])
                    g, g_range = b["dx"], None
            elif k == "maxpool":
                api.lpdt_maxpool2x2_bwd(N, B, op["H"], op["W"], op["C"], g, b["idx"], b["dx"])
                g, g_range = b["dx"], None
            elif k == "avgpool":
                api.lpdt_avgpool_bwd(N, B, op["H"] * op["W"], op["C"], g, b["dx"])
                g, g_range = b["dx"], None
        torch.cuda.current_stream().wait_stream(self.side)      # this group's weight-gradient contractions are done
        self.input_grad_out = g
        return g

    def _finish_gradients(self):
        """After every group's backward pass, all nodes at once on the side stream: all norm layers'
        parameter-gradient sums in one launch, all layers' int32 weight-gradient sums to fp32 in another."""
        N, d = self.N, self.d
        pending_ren = [(op, b) for op, b in zip(self.ops, self.buf) if op["op"] == "ren"]
        self.side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(self.side):
            self._ren_param_sums(pending_ren)
            if not self.quantize_wgrad:
                convs = [(op, b) for op, b in zip(self.ops, self.buf) if op["op"] in ("conv", "linear")]
                for lo in range(0, len(convs), 64):
                    part = convs[lo:lo + 64]
                    api.lpdt_dequantize_acc_batch(self.g_acc, N, [self.g_acc_off[b["wi"]] for _, b in part],
                                                  [b["wn"] for _, b in part], [op["w_off"] for op, _ in part],
                                                  [b["sE"] for _, b in part], [b["sA"] for _, b in part],
                                                  self.grads, d)
        torch.cuda.current_stream().wait_stream(self.side)      # weight gradients complete before the update

    def _ren_param_sums(self, pending):
        """Reduce the Range-EvoNorm parameter-gradient partial sums of the layers in `pending` (current stream):
        one launch per 64 layers."""
        for lo in range(0, len(pending), 64):
            part = pending[lo:lo + 64]
            api.lpdt_range_evonorm_bwd_params_batch(self.N, self.B, [op["C"] for op, _ in part],
                                                    [b["ws_ren"] for _, b in part], [op["p_off"] for op, _ in part],
                                                    self.grads, self.d)
        pending.clear()

    def update(self):
        N, d = self.N, self.d
        dense = all(k >= hi - lo for k, lo, hi in zip(self.seg_k, self.seg_offsets[:-1], self.seg_offsets[1:]))
        if dense and self.message_bits != 8:
            # no compression: the half-step is computed inside the mix kernel (one pass over parameters and gradients)
            api.lpdt_sgd_gossip_mix(N, d, self.params, self.grads, self.lr, self.x_half, self.x_hat, self.x_out,
                                    self.Wmix, self.gamma)
            return
        api.lpdt_sgd_update(N * d, self.params, self.grads, self.lr, self.x_half)
        if self.message_bits == 8:
            api.lpdt_gossip_mix_q8(N, d, self.x_half, self.x_hat, self.x_out, self.Wmix, self.gamma,
                                   self.seg_offsets, self.seg_k, self.msg_scale, self.ws, self.dev_status)
        else:
            api.lpdt_gossip_mix(N, d, self.x_half, self.x_hat, self.x_out, self.Wmix, self.gamma,
                                self.seg_offsets, self.seg_k, self.ws, self.dev_status)

    def run(self):
        if self.groups:      # one fork for both passes: a group's backward pass follows its own forward pass
            self._prepare()
            self._each_group(lambda g: (g._forward_layers(), g._backward_layers()))
            self.out = self.buf[-1]["out"]
            self._finish_gradients()
            self.input_grad_out = self.buf[0]["dx"] if self.input_grad else None
        else:
            self.forward()
            self.backward()
        self.update()

    def record(self):
        """Run one step eagerly and return the log of its entry-point calls, in issue order:
        [(name, function, args, kwargs, contraction kernel or "", node group)].  The calls of a log can be issued
        again on the buffers the step left behind (every call reads and writes the same tensors)."""
        api.RECORD = log = []
        try:
            self.run()
        finally:
            api.RECORD = None
        return log

    def contractions(self, passes=("fwd", "bwd_data")):
        """Re-issue only the integer contractions of every layer, in step order, on the operands the
        last run() left in the buffers (results are overwritten with the same values).  For timing
        those kernels without the rest of the step; returns the number of calls made."""
        d, n = self.d, 0
        for li, (op, b) in enumerate(zip(self.ops, self.buf)):
            if op["op"] in ("conv", "linear") and "fwd" in passes:
                bias = self._p(op["b_off"]) if op["op"] == "linear" else None
                api.lpdt_qconv_fwd(b["desc"], b["qA"], b["sA"], b["qW"], b["sW"], Y=b["out"], bias=bias,
                                   bias_node_stride=d, ws=self.ws, dev_status=self.dev_status)
                n += 1
        for li in range(len(self.ops) - 1, -1, -1):
            op, b = self.ops[li], self.buf[li]
            if op["op"] not in ("conv", "linear"):
                continue
            if "bwd_weight" in passes and not self.quantize_wgrad:
                api.lpdt_qconv_bwd_weight(b["desc"], b["E"], b["sE"], b["qA"], b["sA"], dW=self._g(op["w_off"]),
                                          dw_node_stride=d, ws=self.ws, dev_status=self.dev_status)
                n += 1
            if "bwd_data" in passes and (li > 0 or self.input_grad):
                api.lpdt_qconv_bwd_data(b["desc"], b["E"], b["sE"], b["qW"], b["sW"], dA=b["dx"], ws=self.ws,
                                        dev_status=self.dev_status, addend=b.get("addend"))
                n += 1
        return n

    # ---- CUDA graph: the whole step as one replayable launch -------------------------------
    def capture(self):
        """Record run() into a CUDA graph (one warm-up run first so that every
        one-time kernel attribute is set before capture)."""
        self.run()
        torch.cuda.synchronize()
        before = api.lpdt_launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.run()
        self.graph_launches = api.lpdt_launch_count() - before
        self.graph = g
        return g

    def replay(self):
        self.graph.replay()
        api.add_replayed_launches(self.graph_launches)
