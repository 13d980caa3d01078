"""Layer chaining for the LeNet-5 / VGG-7 / ResNet-18 shaped workloads.

Nothing is computed here: every step is a call into the CUDA library through
`twn`.  This module only owns the device buffers (torch provides the memory) and the
order of the calls of a forward pass and of a training step (Algorithm 1: ternarize every
layer, forward through the ternary weights, backward for data through the same codes,
straight-through weight gradients for the fp32 master weights).

Activations and gradients are NHWC bf16; logits and weight gradients are fp32.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import datagen as dg
from . import twn


def _dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@dataclass
class Layer:
    name: str
    Cin: int
    Cout: int
    k: int = 1
    stride: int = 1
    pad: int = 0
    H: int = 1           # input extent (1 for fully connected layers)
    W: int = 1
    relu: bool = True
    affine: bool = False
    residual: str | None = None      # name of the activation added before the ReLU
    src: str = ""                    # name of the input activation
    out_f32: bool = False            # logits
    # filled by the net
    B: int = 0
    desc: object = None
    K: int = 0
    small_cin: bool = False
    fold: tuple | None = None      # (Hf, Wf, ldf) when the layer runs in folded form
    ldk: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def Ho(self):
        return (self.H + 2 * self.pad - self.k) // self.stride + 1

    @property
    def Wo(self):
        return (self.W + 2 * self.pad - self.k) // self.stride + 1

    @property
    def macs(self):
        return self.B * self.Ho * self.Wo * self.K * self.Cout


class TernaryNet:
    """A chain of ternary conv / FC layers with pooling glue, all buffers preallocated."""

    def __init__(self, name: str, batch: int, in_shape, ops, seed: int = 0, delta_factor: float = 0.7,
                 train: bool = False, optimizer: dict | None = None):
        """optimizer: None (the step ends with the weight gradients) or dict(lr, momentum, weight_decay):
        the step then ends with the SGD update of the master weights (Algorithm 1, UpdateParameters), which
        also leaves the next iteration's thresholds behind, so that later steps run only the coding sweep."""
        self.name, self.B, self.in_shape, self.ops = name, batch, in_shape, ops
        self.seed, self.delta_factor, self.train = seed, delta_factor, train
        self.optimizer = optimizer if train else None
        self._delta_ready = False
        self.layers: dict[str, Layer] = {op[1].name: op[1] for op in ops if op[0] == "layer"}
        self.act: dict[str, torch.Tensor] = {}
        self.aux: dict[str, torch.Tensor] = {}
        self.grad: dict[str, torch.Tensor] = {}
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        # the code re-layouts for the backward pass run on a side stream beside the forward pass
        self.side_streams = [torch.cuda.Stream()]
        self.dw_stream = torch.cuda.Stream()     # weight gradients run beside the backward-for-data chain
        self.timed = None          # when a list: (kind, name, flops, start event, end event)
        H, W, C = in_shape
        self.act["input"] = torch.zeros((batch, H, W, C), dtype=torch.bfloat16, device="cuda")
        self._build()

    # ------------------------------------------------------------------ construction
    def _build(self):
        B = self.B
        ws_dw = 0
        for op in self.ops:
            kind = op[0]
            if kind == "layer":
                L: Layer = op[1]
                L.B = B
                L.K = L.k * L.k * L.Cin
                L.desc = twn.conv_desc(B, L.H, L.W, L.Cin, L.Cout, L.k, L.stride, L.pad)
                L.small_cin = (L.Cin % 16 != 0) and not (L.k == 1 and L.Cin % 8 == 0)
                e = L.extra
                Wm = dg.he_normal(self.seed, f"{self.name}.{L.name}.weight", L.Cout, L.K)
                e["W"] = _dev(Wm)
                e["ld"] = twn.ld_for(L.K)
                e["packed"] = torch.zeros((L.Cout, e["ld"] // 16), dtype=torch.int32, device="cuda")
                e["stats"] = twn.new_stats()
                if L.affine:
                    e["scale"] = _dev(dg.draw(self.seed, f"{self.name}.{L.name}.scale", L.Cout, "normal", 1.0, float(np.sqrt(0.1))))
                    e["shift"] = _dev(dg.draw(self.seed, f"{self.name}.{L.name}.shift", L.Cout, "normal", 0.0, float(np.sqrt(0.1))))
                else:
                    e["scale"] = e["shift"] = None
                M = B * L.Ho * L.Wo
                # a stride-2 layer on very few channels runs in folded form, other small-Cin layers
                # through the patch matrix
                L.fold = twn.fold_dims(L.desc) if L.small_cin else None
                if L.fold:
                    Hf, Wf, ldf = L.fold
                    e["xf"] = torch.zeros((B, Hf, Wf, 16), dtype=torch.bfloat16, device="cuda")
                    e["packed_f"] = torch.zeros((L.Cout, ldf // 16), dtype=torch.int32, device="cuda")
                elif L.small_cin:
                    L.ldk = (L.K + 7) // 8 * 8
                    e["xcol"] = torch.zeros((M, L.ldk), dtype=torch.bfloat16, device="cuda")
                out_dtype = torch.float32 if L.out_f32 else torch.bfloat16
                self.act[L.name] = torch.zeros((B, L.Ho, L.Wo, L.Cout), dtype=out_dtype, device="cuda")
                res = self.act[L.residual] if L.residual else None
                e["epi"] = twn.epilogue(e["scale"], e["shift"], res, relu=L.relu,
                                        out_dtype=twn.F32 if L.out_f32 else twn.BF16)
                if self.optimizer:
                    if L.small_cin and not L.fold:
                        raise NotImplementedError("the update needs a weight gradient in the layout of the weights")
                    e["V"] = torch.zeros_like(e["W"])
                if self.train:
                    first = L.src == "input"
                    if not first:
                        e["ld_b"] = twn.ld_for(L.k * L.k * L.Cout)
                        e["packed_b"] = torch.zeros((L.Cin, e["ld_b"] // 16), dtype=torch.int32, device="cuda")
                    e["dz"] = torch.zeros((B, L.Ho, L.Wo, L.Cout), dtype=torch.bfloat16, device="cuda")
                    if L.fold:
                        e["dw_desc"] = L.desc
                        e["dW"] = torch.zeros((L.Cout, L.K), dtype=torch.float32, device="cuda")
                        ws_dw = max(ws_dw, twn.conv2d_bwd_weight_folded_workspace_bytes(L.desc))
                    elif L.small_cin:
                        e["dw_desc"] = twn.conv_desc(1, 1, M, L.ldk, L.Cout, 1, 1, 0)
                        e["dW"] = torch.zeros((L.Cout, L.ldk), dtype=torch.float32, device="cuda")
                        ws_dw = max(ws_dw, twn.conv2d_bwd_weight_workspace_bytes(e["dw_desc"]))
                    else:
                        e["dw_desc"] = L.desc
                        e["dW"] = torch.zeros((L.Cout, L.K), dtype=torch.float32, device="cuda")
                        ws_dw = max(ws_dw, twn.conv2d_bwd_weight_workspace_bytes(e["dw_desc"]))
            elif kind == "maxpool":
                _, name, src, k, s, p = op
                Bx, H, W, C = self.act[src].shape
                Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
                self.act[name] = torch.zeros((Bx, Ho, Wo, C), dtype=torch.bfloat16, device="cuda")
                if self.train:
                    self.aux[name] = torch.zeros((Bx, Ho, Wo, C), dtype=torch.uint8, device="cuda")
            elif kind == "avgpool":
                _, name, src = op
                Bx, H, W, C = self.act[src].shape
                self.act[name] = torch.zeros((Bx, 1, 1, C), dtype=torch.bfloat16, device="cuda")
            elif kind == "flatten":
                _, name, src = op
                a = self.act[src]
                self.act[name] = a.view(a.shape[0], 1, 1, -1)
        self.ws_tern = torch.empty(twn.ternarize_batch_workspace_bytes(min(len(self.layers), 32)),
                                   dtype=torch.uint8, device="cuda")
        if self.train:
            for name, a in self.act.items():
                if name != "input" and a.dtype == torch.bfloat16:
                    self.grad[name] = torch.zeros_like(a)
            self.ws_dw = torch.empty(max(ws_dw, 16), dtype=torch.uint8, device="cuda")

    def set_input(self, bits: np.ndarray):
        self.act["input"].copy_(_bf16(bits).view(self.act["input"].shape))

    # ------------------------------------------------------------------ timing hooks
    def _call(self, kind, name, flops, fn):
        if self.timed is None:
            fn()
            return
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        self.timed.append((kind, name, flops, e0, e1))

    # ------------------------------------------------------------------ Algorithm 1, first loop
    def ternarize_all(self, join: bool = True):
        """Algorithm 1, first loop: every layer's threshold, codes and scale, all layers in one
        batched call (two launches per 32 layers) on the current stream.  The re-layouts of the codes
        for the backward pass follow as one batched launch on a side stream, beside the forward pass;
        the backward pass waits for its event."""
        main = torch.cuda.current_stream()
        layers = list(self.layers.values())
        for i in range(0, len(layers), 32):
            group = layers[i:i + 32]
            items = [(L.extra["W"], L.Cout, L.K, L.extra["stats"], L.extra["packed"], L.extra["ld"], None)
                     for L in group]
            if self._delta_ready:
                # the thresholds were left behind by the previous step's update: coding sweep only
                self._call("ternarize", f"layers {i}..{i + len(group) - 1}", 0,
                           lambda: twn.ternarize_codes_batch(items, self.ws_tern))
            else:
                self._call("ternarize", f"layers {i}..{i + len(group) - 1}", 0,
                           lambda: twn.ternarize_batch(items, self.delta_factor, self.ws_tern))
        for L in layers:
            if L.fold:
                twn.fold_codes(L.desc, L.extra["packed"], L.extra["ld"], L.extra["packed_f"], L.fold[2])
        if self.train:
            # the re-layouts for the backward pass: one batched launch beside the forward pass
            st = self.side_streams[0]
            st.wait_stream(main)
            todo = [L for L in layers if "packed_b" in L.extra]
            with torch.cuda.stream(st):
                for i in range(0, len(todo), 32):
                    twn.transpose_codes_batch([(L.extra["packed"], L.extra["ld"], L.desc, L.extra["packed_b"],
                                                L.extra["ld_b"]) for L in todo[i:i + 32]])
                ev = torch.cuda.Event()
                ev.record(st)
            for L in todo:
                L.extra["ready_b"] = ev
            self._pending_join = True
        if join:
            self.join_side_streams()

    def _wait_codes(self, L, key="ready"):
        ev = L.extra.get(key)
        if ev is not None:
            torch.cuda.current_stream().wait_event(ev)

    def join_side_streams(self):
        """All side-stream work rejoins the current stream (required before a graph capture ends
        and before the master weights change)."""
        if getattr(self, "_pending_join", False):
            main = torch.cuda.current_stream()
            main.wait_stream(self.side_streams[0])      # the only side stream ternarize_all forks
            self._pending_join = False
            for L in self.layers.values():      # nothing left to wait for
                L.extra.pop("ready", None)
                L.extra.pop("ready_b", None)

    # ------------------------------------------------------------------ forward
    def forward(self):
        for op in self.ops:
            kind = op[0]
            if kind == "layer":
                L: Layer = op[1]
                e = L.extra
                x, y = self.act[L.src], self.act[L.name]
                fl = 2 * L.macs
                self._wait_codes(L)
                if L.fold:
                    twn.fold_input(L.desc, x, e["xf"])
                    self._call("tconv", L.name + ".fwd", fl, lambda: twn.conv2d_fwd_folded(
                        L.desc, e["xf"], e["packed_f"], L.fold[2], e["stats"], e["epi"], y, self.status))
                elif L.small_cin:
                    twn.im2col(L.desc, x, e["xcol"], L.ldk)
                    M = L.B * L.Ho * L.Wo
                    self._call("tconv", L.name + ".fwd", fl, lambda: twn.gemm(
                        e["xcol"], L.ldk, e["packed"], e["ld"], e["stats"], M, L.Cout, L.K, e["epi"], y,
                        L.Cout, self.status))
                else:
                    self._call("tconv", L.name + ".fwd", fl, lambda: twn.conv2d_fwd(
                        L.desc, x, e["packed"], e["ld"], e["stats"], e["epi"], y, self.status))
            elif kind == "maxpool":
                _, name, src, k, s, p = op
                x = self.act[src]
                Bx, H, W, C = x.shape
                twn.maxpool2d_fwd(x, Bx, H, W, C, k, s, p, self.act[name], self.aux.get(name))
            elif kind == "avgpool":
                _, name, src = op
                x = self.act[src]
                Bx, H, W, C = x.shape
                twn.avgpool_fwd(x, Bx, H * W, C, self.act[name])
        return self.act[self.ops[-1][1].name]

    # ------------------------------------------------------------------ backward
    def backward(self, dlogits: torch.Tensor):
        """dlogits: bf16 [B, classes], the gradient injected at the logits.  Fills extra['dW'] of
        every layer.  An activation with two consumers (the input of a residual block) gets its
        second contribution added through the residual input of the backward-for-data epilogue."""
        assert self.train
        last: Layer = self.ops[-1][1]
        acc: dict[str, torch.Tensor] = {last.name: dlogits.view(self.act[last.name].shape)}

        def emit_tensor(name, t):
            assert name not in acc, "a materialised gradient must be the first contribution"
            acc[name] = t

        def emit(name, fn):
            """fn(res, out): out = contribution (+ res).  The first contribution is written plainly."""
            if name == "input":
                return
            out = self.grad[name]
            fn(acc.get(name), out)
            acc[name] = out

        # A layer P = relu(z * scale + shift) whose output feeds exactly one convolution gets its
        # dZ straight from that convolution's backward-for-data pass (the ReLU gate and the scale
        # applied in its epilogue) instead of from an activation-backward sweep of its own.
        consumers: dict[str, list] = {}
        for op in self.ops:
            if op[0] == "layer":
                consumers.setdefault(op[1].src, []).append(op[1])
                if op[1].residual:
                    consumers.setdefault(op[1].residual, []).append(None)
            elif op[0] in ("maxpool", "avgpool", "flatten"):
                consumers.setdefault(op[2], []).append(op[1])
        FUSED = object()

        def fused_producer(L):
            P = self.layers.get(L.src)
            if P is None or not P.relu or P.residual or P.out_f32 or L.fold or L.small_cin:
                return None
            return P if consumers.get(P.name) == [L] else None

        # A projection shortcut (a layer read only as the residual input of another layer) shares its input with
        # the first convolution of its block.  Its backward pass is taken after that convolution's: the dense
        # gradient is written first, and the strided shortcut then adds into it in place, which lets
        # twn_conv2d_bwd_data skip the residue classes its single tap never reaches.
        def is_shortcut(L):
            if L.relu or L.residual or L.fold or L.small_cin or L.src == "input":
                return False
            users = consumers.get(L.name, [])
            return users == [None]
        order, deferred = [], {}
        for op in reversed(self.ops):
            if op[0] == "layer" and is_shortcut(op[1]):
                deferred[op[1].src] = op
                continue
            order.append(op)
            if op[0] == "layer" and op[1].src in deferred:
                order.append(deferred.pop(op[1].src))
        order.extend(deferred.values())

        main = torch.cuda.current_stream()
        self.dw_stream.wait_stream(main)
        for op in order:
            kind = op[0]
            if kind == "layer":
                L: Layer = op[1]
                e = L.extra
                dY = acc[L.name]
                if dY is not FUSED:
                    n = dY.numel()
                    y = self.act[L.name] if L.relu else None
                    dpre = None
                    if L.residual:
                        # the gradient before the ReLU also flows, unscaled, into the shortcut branch
                        dpre = e.get("dpre")
                        if dpre is None:
                            dpre = e["dpre"] = torch.zeros_like(e["dz"])
                    twn.act_bwd(dY, y, e["scale"], n, L.Cout, e["dz"], dpre)
                    if L.residual:
                        emit_tensor(L.residual, dpre)
                # dW needs only dz and the layer's input: it goes to its own stream (one after the
                # other there, they share the workspace) and overlaps the dX chain of the layers below
                dz_ready = torch.cuda.Event()
                dz_ready.record(main)
                with torch.cuda.stream(self.dw_stream):
                    self.dw_stream.wait_event(dz_ready)
                    if L.fold:
                        self._call("dw", L.name + ".dW", 2 * L.macs, lambda: twn.conv2d_bwd_weight_folded(
                            L.desc, e["xf"], e["dz"], e["dW"], self.ws_dw, self.status))
                    else:
                        x = e["xcol"] if L.small_cin else self.act[L.src]
                        self._call("dw", L.name + ".dW", 2 * L.macs, lambda: twn.conv2d_bwd_weight(
                            e["dw_desc"], x, e["dz"], e["dW"], self.ws_dw, self.status))
                P = fused_producer(L) if L.src != "input" else None
                if P is not None:
                    self._wait_codes(L, "ready_b")
                    epi = twn.epilogue(scale=P.extra["scale"], residual=self.act[P.name], out_dtype=twn.BF16,
                                       residual_op=twn.RESIDUAL_GATE)
                    self._call("tconv", L.name + ".dX", 2 * L.macs, lambda: twn.conv2d_bwd_data(
                        L.desc, e["dz"], e["packed_b"], e["ld_b"], e["stats"], epi, P.extra["dz"], self.status))
                    assert P.name not in acc
                    acc[P.name] = FUSED
                elif L.src != "input":
                    def bwd(res, out, L=L, e=e):
                        self._wait_codes(L, "ready_b")
                        epi = twn.epilogue(residual=res, out_dtype=twn.BF16)
                        self._call("tconv", L.name + ".dX", 2 * L.macs, lambda: twn.conv2d_bwd_data(
                            L.desc, e["dz"], e["packed_b"], e["ld_b"], e["stats"], epi, out, self.status))
                    emit(L.src, bwd)
            elif kind == "maxpool":
                _, name, src, k, s, p = op
                Bx, H, W, C = self.act[src].shape
                dY = acc[name]

                P = self.layers.get(src)
                if P is not None and P.relu and not P.residual and consumers.get(src) == [name]:
                    # the pool is the only reader of a ReLU layer: its backward pass writes that
                    # layer's dZ (gate by the pooled value, folded batch-norm scale) in one sweep
                    twn.maxpool2d_bwd_act(dY, self.aux[name], self.act[name], P.extra["scale"], Bx, H, W, C, k, s, p,
                                          P.extra["dz"])
                    acc[src] = FUSED
                    continue

                def mp(res, out, dY=dY, name=name, Bx=Bx, H=H, W=W, C=C, k=k, s=s, p=p):
                    assert res is None
                    twn.maxpool2d_bwd(dY, self.aux[name], Bx, H, W, C, k, s, p, out)
                emit(src, mp)
            elif kind == "avgpool":
                _, name, src = op
                Bx, H, W, C = self.act[src].shape
                dY = acc[name]

                def ap(res, out, dY=dY, Bx=Bx, H=H, W=W, C=C):
                    assert res is None
                    twn.avgpool_bwd(dY, Bx, H * W, C, out)
                emit(src, ap)
            elif kind == "flatten":
                _, name, src = op
                emit_tensor(src, acc[name].view(self.act[src].shape))
        main.wait_stream(self.dw_stream)
        self.last_grads = acc

    def sgd_step(self):
        """Algorithm 1, UpdateParameters: SGD with momentum and weight decay on every layer's master
        weights (one batched launch per 32 layers), which also writes the next thresholds."""
        o = self.optimizer
        layers = list(self.layers.values())
        for i in range(0, len(layers), 32):
            items = [(L.extra["W"], L.extra["dW"], L.extra["V"], L.extra["stats"]) for L in layers[i:i + 32]]
            twn.sgd_update_batch(items, o["lr"], o["momentum"], o["weight_decay"], self.delta_factor, self.ws_tern)
        self._delta_ready = True

    def train_step(self, dlogits):
        self.ternarize_all(join=False)
        self.forward()
        self.backward(dlogits)
        self.join_side_streams()
        if self.optimizer:
            self.sgd_step()

    def check_status(self):
        s = twn.read_status(self.status)
        if s != 0:
            raise twn.TwnError(s, "device status")

    def total_macs(self, train: bool | None = None):
        train = self.train if train is None else train
        f = sum(L.macs for L in self.layers.values())
        if train:
            f += sum(L.macs for L in self.layers.values())                       # dW
            f += sum(L.macs for L in self.layers.values() if L.src != "input")   # dX
        return f


# ---------------------------------------------------------------------- the three shapes
def lenet5_ops():
    return [
        ("layer", Layer("conv1", 1, 32, 5, 1, 0, 28, 28, src="input")),
        ("maxpool", "pool1", "conv1", 2, 2, 0),
        ("layer", Layer("conv2", 32, 64, 5, 1, 0, 12, 12, src="pool1")),
        ("maxpool", "pool2", "conv2", 2, 2, 0),
        ("flatten", "flat", "pool2"),
        ("layer", Layer("fc1", 1024, 512, src="flat")),
        ("layer", Layer("fc2", 512, 10, relu=False, src="fc1", out_f32=True)),
    ]


def lenet5(batch=100, train=False, seed=0):
    return TernaryNet("lenet5", batch, (28, 28, 1), lenet5_ops(), seed, train=train)


def vgg7_ops():
    ops, src, H = [], "input", 32
    cin = 3
    for i, c in enumerate([128, 128, 256, 256, 512, 512], 1):
        ops.append(("layer", Layer(f"conv{i}", cin, c, 3, 1, 1, H, H, affine=True, src=src)))
        src, cin = f"conv{i}", c
        if i % 2 == 0:
            ops.append(("maxpool", f"pool{i // 2}", src, 2, 2, 0))
            src, H = f"pool{i // 2}", H // 2
    ops.append(("flatten", "flat", src))
    ops.append(("layer", Layer("fc1", 8192, 1024, affine=True, src="flat")))
    ops.append(("layer", Layer("fc2", 1024, 10, relu=False, src="fc1", out_f32=True)))
    return ops


def vgg7(batch=128, train=False, seed=0):
    return TernaryNet("vgg7", batch, (32, 32, 3), vgg7_ops(), seed, train=train)


def resnet18_ops(image=224, classes=1000, widths=(64, 128, 256, 512)):
    """BasicBlock layout [2, 2, 2, 2] with a 7x7/2 first layer.  `widths` are the channels of the four
    stages; (96, 192, 384, 768) is the 1.5x wider "ResNet-18B" of the paper's ImageNet experiments."""
    w0 = widths[0]
    ops = [("layer", Layer("stem", 3, w0, 7, 2, 3, image, image, affine=True, src="input"))]
    H = (image + 6 - 7) // 2 + 1
    ops.append(("maxpool", "pool0", "stem", 3, 2, 1))
    H = (H + 2 - 3) // 2 + 1
    src, cin = "pool0", w0
    for li, c in enumerate(widths, 1):
        for b in range(2):
            stride = 2 if (li > 1 and b == 0) else 1
            p = f"l{li}.b{b}"
            Ho = (H + 2 - 3) // stride + 1
            ops.append(("layer", Layer(p + ".conv1", cin, c, 3, stride, 1, H, H, affine=True, src=src)))
            short = src
            if stride != 1 or cin != c:
                ops.append(("layer", Layer(p + ".down", cin, c, 1, stride, 0, H, H, relu=False, affine=True, src=src)))
                short = p + ".down"
            ops.append(("layer", Layer(p + ".conv2", c, c, 3, 1, 1, Ho, Ho, affine=True, residual=short,
                                       src=p + ".conv1")))
            src, cin, H = p + ".conv2", c, Ho
    ops.append(("avgpool", "gap", src))
    ops.append(("layer", Layer("fc", widths[-1], classes, relu=False, src="gap", out_f32=True)))
    return ops


def resnet18(batch=64, train=True, seed=0, image=224, classes=1000, widths=(64, 128, 256, 512), name="resnet18",
             optimizer=None):
    return TernaryNet(name, batch, (image, image, 3), resnet18_ops(image, classes, widths), seed, train=train,
                      optimizer=optimizer)


def resnet18b(batch=64, train=True, seed=0, image=224, classes=1000):
    return resnet18(batch, train, seed, image, classes, widths=(96, 192, 384, 768), name="resnet18b")
