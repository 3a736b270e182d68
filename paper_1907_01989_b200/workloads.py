"""Seeded synthetic workloads: network descriptions, weights and inputs.

This module only *describes* graphs (op kinds, shapes, attributes) and draws the
random numbers that fill them.  It performs none of the inference arithmetic and is
the one module that both the CUDA binding and the CPU oracle's tests consume, so the
two sides always see identical graphs, weights and inputs.

Recipe (stands in for the trained phone models of the paper's Section 6, which are
not available): inputs ~ U[-1, 1] rounded to fp16-representable values, weights
~ N(0, 1/fan_in) (fan_in = kh*kw*Cin for a full convolution, kh*kw for depthwise),
biases ~ U[-0.1, 0.1].  Array number k of workload number c is drawn from
numpy.random.Generator(PCG64([0, c, k])), so every array is independent of the batch
size and of every other array; image b of input i comes from PCG64([1, c, i, b]).  "same" padding follows the TensorFlow convention
(the paper's engine is TFLite's): Ho = ceil(H / s), total = max((Ho-1)*s +
(k-1)*d + 1 - H, 0), before = total // 2.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

CONV2D = "conv2d"
DEPTHWISE = "depthwise_conv2d"
ADD = "add"
ACTIVATION = "activation"
GLOBAL_AVG_POOL = "global_avg_pool"
RESIZE_BILINEAR = "resize_bilinear"
CONCAT = "concat"

ACT_NONE, ACT_RELU, ACT_RELU6 = "none", "relu", "relu6"


@dataclass
class OpSpec:
    kind: str
    inputs: List[int]
    output: int
    kh: int = 1
    kw: int = 1
    stride: Tuple[int, int] = (1, 1)
    dilation: Tuple[int, int] = (1, 1)
    pads: Tuple[int, int, int, int] = (0, 0, 0, 0)  # top, left, bottom, right
    cout: int = 0
    act: str = ACT_NONE  # ACTIVATION ops only
    out_hw: Tuple[int, int] = (0, 0)  # RESIZE_BILINEAR only
    align_corners: bool = True
    weights: Optional[np.ndarray] = None  # fp32, [Cout][kh][kw][Cin]; depthwise [1][kh][kw][C]
    bias: Optional[np.ndarray] = None  # fp32, [Cout]


@dataclass
class GraphSpec:
    name: str
    batch: int
    workload_id: int = 0
    shapes: Dict[int, Tuple[int, int, int]] = field(default_factory=dict)  # id -> (H, W, C)
    inputs: List[int] = field(default_factory=list)
    outputs: List[int] = field(default_factory=list)
    ops: List[OpSpec] = field(default_factory=list)


def same_pads(size: int, k: int, stride: int, dilation: int) -> Tuple[int, int, int]:
    """TensorFlow-SAME padding along one axis -> (out_size, before, after)."""
    out = -(-size // stride)
    total = max((out - 1) * stride + (k - 1) * dilation + 1 - size, 0)
    return out, total // 2, total - total // 2


class _Rng:
    """Array k of workload c comes from PCG64([0, c, k])."""

    def __init__(self, workload_id: int):
        self.c = workload_id
        self.k = 0

    def gen(self) -> np.random.Generator:
        g = np.random.Generator(np.random.PCG64([0, self.c, self.k]))
        self.k += 1
        return g


class GraphBuilder:
    def __init__(self, name: str, batch: int, workload_id: int):
        self.g = GraphSpec(name=name, batch=batch, workload_id=workload_id)
        self.rng = _Rng(workload_id)
        self._next = 0

    def _new(self, H: int, W: int, C: int) -> int:
        t = self._next
        self._next += 1
        self.g.shapes[t] = (H, W, C)
        return t

    def input(self, H: int, W: int, C: int) -> int:
        t = self._new(H, W, C)
        self.g.inputs.append(t)
        return t

    def output(self, t: int) -> None:
        self.g.outputs.append(t)

    def _conv(self, kind: str, x: int, cout: int, k: int, stride: int, dilation: int, bias: bool = True) -> int:
        H, W, C = self.g.shapes[x]
        Ho, pt, pb = same_pads(H, k, stride, dilation)
        Wo, pl, pr = same_pads(W, k, stride, dilation)
        if kind == DEPTHWISE:
            cout = C
            fan_in = k * k
            wshape = (1, k, k, C)
        else:
            fan_in = k * k * C
            wshape = (cout, k, k, C)
        w = (self.rng.gen().standard_normal(wshape) / np.sqrt(fan_in)).astype(np.float32)
        b = self.rng.gen().uniform(-0.1, 0.1, size=(cout,)).astype(np.float32) if bias else None
        if not bias:
            self.rng.gen()
        out = self._new(Ho, Wo, cout)
        self.g.ops.append(OpSpec(kind=kind, inputs=[x], output=out, kh=k, kw=k, stride=(stride, stride),
                                 dilation=(dilation, dilation), pads=(pt, pl, pb, pr), cout=cout,
                                 weights=w, bias=b))
        return out

    def conv2d(self, x: int, cout: int, k: int = 1, stride: int = 1, dilation: int = 1, bias: bool = True) -> int:
        return self._conv(CONV2D, x, cout, k, stride, dilation, bias)

    def depthwise(self, x: int, k: int = 3, stride: int = 1, dilation: int = 1, bias: bool = True) -> int:
        return self._conv(DEPTHWISE, x, 0, k, stride, dilation, bias)

    def activation(self, x: int, act: str) -> int:
        out = self._new(*self.g.shapes[x])
        self.g.ops.append(OpSpec(kind=ACTIVATION, inputs=[x], output=out, act=act))
        return out

    def add(self, a: int, b: int) -> int:
        out = self._new(*self.g.shapes[a])
        self.g.ops.append(OpSpec(kind=ADD, inputs=[a, b], output=out))
        return out

    def concat(self, a: int, b: Optional[int] = None) -> int:
        """Channels of `a`, then channels of `b`; with one input the identity."""
        H, W, Ca = self.g.shapes[a]
        Cb = 0 if b is None else self.g.shapes[b][2]
        out = self._new(H, W, Ca + Cb)
        self.g.ops.append(OpSpec(kind=CONCAT, inputs=[a] if b is None else [a, b], output=out))
        return out

    def identity_add(self, x: int) -> int:
        """An ADD with a single input: the identity (graph clean-up removes it)."""
        out = self._new(*self.g.shapes[x])
        self.g.ops.append(OpSpec(kind=ADD, inputs=[x], output=out))
        return out

    def global_avg_pool(self, x: int) -> int:
        _, _, C = self.g.shapes[x]
        out = self._new(1, 1, C)
        self.g.ops.append(OpSpec(kind=GLOBAL_AVG_POOL, inputs=[x], output=out))
        return out

    def resize_bilinear(self, x: int, oh: int, ow: int, align_corners: bool = True) -> int:
        _, _, C = self.g.shapes[x]
        out = self._new(oh, ow, C)
        self.g.ops.append(OpSpec(kind=RESIZE_BILINEAR, inputs=[x], output=out, out_hw=(oh, ow),
                                 align_corners=align_corners))
        return out

    def finish(self) -> GraphSpec:
        return self.g


def make_input(g: GraphSpec, images: Optional[List[int]] = None, index: int = 0) -> np.ndarray:
    """U[-1,1] NHWC input number `index` of a graph, rounded to fp16-representable fp32.

    Image b of the batch is drawn from its own stream PCG64([1, g.workload_id, index, b]),
    so a sub-batch (`images`) holds exactly the images the full batch holds.
    """
    H, W, C = g.shapes[g.inputs[index]]
    ids = list(range(g.batch)) if images is None else list(images)
    x = np.empty((len(ids), H, W, C), dtype=np.float32)
    for i, b in enumerate(ids):
        r = np.random.Generator(np.random.PCG64([1, g.workload_id, index, b]))
        x[i] = r.uniform(-1.0, 1.0, size=(H, W, C)).astype(np.float32)
    return x.astype(np.float16).astype(np.float32)


# ----------------------------------------------------------------------------------------
# Workload 1: one depthwise-separable block
# ----------------------------------------------------------------------------------------
def separable_block(batch: int = 1, H: int = 32, W: int = 32, C: int = 32, cout: int = 64) -> GraphSpec:
    b = GraphBuilder("separable_block", batch, 1)
    x = b.input(H, W, C)
    y = b.activation(b.depthwise(x, 3, 1), ACT_RELU6)
    y = b.activation(b.conv2d(y, cout, 1), ACT_RELU6)
    b.output(y)
    return b.finish()


# ----------------------------------------------------------------------------------------
# Workload 2: MobileNetV1 1.0
# ----------------------------------------------------------------------------------------
_V1_BLOCKS = [(64, 1), (128, 2), (128, 1), (256, 2), (256, 1), (512, 2), (512, 1), (512, 1), (512, 1),
              (512, 1), (512, 1), (1024, 2), (1024, 1)]


def mobilenet_v1(batch: int = 1, size: int = 224, classes: int = 1001) -> GraphSpec:
    b = GraphBuilder("mobilenet_v1", batch, 2)
    x = b.input(size, size, 3)
    y = b.activation(b.conv2d(x, 32, 3, 2), ACT_RELU6)
    for cout, s in _V1_BLOCKS:
        y = b.activation(b.depthwise(y, 3, s), ACT_RELU6)
        y = b.activation(b.conv2d(y, cout, 1), ACT_RELU6)
    y = b.global_avg_pool(y)
    y = b.conv2d(y, classes, 1)
    b.output(y)
    return b.finish()


# ----------------------------------------------------------------------------------------
# Workload 3: MobileNetV2 1.0; workload 4: the same backbone at output stride 16 + head
# ----------------------------------------------------------------------------------------
_V2_SETTINGS = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2),
                (6, 320, 1, 1)]


def _inverted_residual(b: GraphBuilder, x: int, t: int, cout: int, stride: int, dilation: int) -> int:
    cin = b.g.shapes[x][2]
    y = x
    if t != 1:
        y = b.activation(b.conv2d(y, cin * t, 1), ACT_RELU6)
    y = b.activation(b.depthwise(y, 3, stride, dilation), ACT_RELU6)
    y = b.conv2d(y, cout, 1)
    if stride == 1 and cin == cout:
        y = b.add(x, y)
    return y


def _v2_backbone(b: GraphBuilder, x: int, segmentation: bool) -> int:
    """17 inverted-residual blocks.  For segmentation at output stride 16 the stride of
    block 14 (first 160-channel block) is dropped, blocks 15-16 use dilation 2 and block 17
    dilation 4, so everything after block 7 runs at 1/16 resolution."""
    y = b.activation(b.conv2d(x, 32, 3, 2), ACT_RELU6)
    index = 0
    for t, c, n, s in _V2_SETTINGS:
        for i in range(n):
            index += 1
            stride, dilation = (s if i == 0 else 1), 1
            if segmentation and index >= 14:
                stride = 1
                dilation = {14: 1, 15: 2, 16: 2, 17: 4}[index]
            y = _inverted_residual(b, y, t, c, stride, dilation)
    return y


def mobilenet_v2(batch: int = 1, size: int = 224, classes: int = 1001) -> GraphSpec:
    b = GraphBuilder("mobilenet_v2", batch, 3)
    x = b.input(size, size, 3)
    y = _v2_backbone(b, x, False)
    y = b.activation(b.conv2d(y, 1280, 1), ACT_RELU6)
    y = b.global_avg_pool(y)
    y = b.conv2d(y, classes, 1)
    b.output(y)
    return b.finish()


def mobilenet_v2_segmentation(batch: int = 1, size: int = 513, classes: int = 21) -> GraphSpec:
    b = GraphBuilder("mobilenet_v2_seg_os16", batch, 4)
    x = b.input(size, size, 3)
    y = _v2_backbone(b, x, True)
    y = b.activation(b.conv2d(y, 256, 1), ACT_RELU)
    y = b.conv2d(y, classes, 1)
    y = b.resize_bilinear(y, size, size, True)
    b.output(y)
    return b.finish()


# ----------------------------------------------------------------------------------------
# Workload 5: single fused operators
# ----------------------------------------------------------------------------------------
def single_pointwise(batch: int, hw: int, cin: int, cout: int, residual: bool = False,
                     act: str = ACT_RELU6) -> GraphSpec:
    """1x1 conv + bias + activation (+ residual add read from a second graph input)."""
    b = GraphBuilder(f"pw_{batch}x{hw}x{cin}x{cout}", batch, 5)
    x = b.input(hw, hw, cin)
    r = b.input(hw, hw, cout) if residual else None
    y = b.conv2d(x, cout, 1)
    if act != ACT_NONE:
        y = b.activation(y, act)
    if residual:
        y = b.add(r, y)
    b.output(y)
    return b.finish()


def single_depthwise(batch: int, hw: int, c: int, stride: int = 1, dilation: int = 1,
                     residual: bool = False) -> GraphSpec:
    b = GraphBuilder(f"dw_{batch}x{hw}x{c}_s{stride}d{dilation}", batch, 6)
    x = b.input(hw, hw, c)
    ho = same_pads(hw, 3, stride, dilation)[0]
    r = b.input(ho, ho, c) if residual else None
    y = b.activation(b.depthwise(x, 3, stride, dilation), ACT_RELU6)
    if residual:
        y = b.add(r, y)
    b.output(y)
    return b.finish()


def depthwise_then_pointwise(batch: int, h: int, w: int, c: int, cout: int, stride: int = 1, residual: bool = False,
                             dw_act=ACT_RELU6, pw_act=None, post_act=None) -> GraphSpec:
    """Depthwise 3x3 (+ activation) feeding a 1x1 convolution (+ activation, + residual, + activation): the second
    half of an inverted-residual block, the pattern one kernel can run without storing the tensor in between."""
    b = GraphBuilder(f"dwpw_{batch}x{h}x{w}x{c}x{cout}_s{stride}", batch, 9)
    x = b.input(h, w, c)
    ho, wo = same_pads(h, 3, stride, 1)[0], same_pads(w, 3, stride, 1)[0]
    r = b.input(ho, wo, cout) if residual else None
    y = b.depthwise(x, 3, stride, 1)
    if dw_act is not None:
        y = b.activation(y, dw_act)
    y = b.conv2d(y, cout, 1)
    if pw_act is not None:
        y = b.activation(y, pw_act)
    if residual:
        y = b.add(r, y)
    if post_act is not None:
        y = b.activation(y, post_act)
    b.output(y)
    return b.finish()


def inverted_residual_block(batch: int, h: int, w: int, cin: int, hidden: int, cout: int, stride: int = 1,
                            act: str = ACT_RELU6, out_act: Optional[str] = None) -> GraphSpec:
    """One inverted-residual block of MobileNetV2 on its own: 1x1 expansion + activation, depthwise 3x3 + activation,
    linear 1x1 projection, and the residual sum where the block keeps shape (stride 1, cin == cout)."""
    b = GraphBuilder(f"block_{batch}x{h}x{w}_{cin}_{hidden}_{cout}_s{stride}", batch, 14)
    x = b.input(h, w, cin)
    y = b.conv2d(x, hidden, 1)
    if act != ACT_NONE:
        y = b.activation(y, act)
    y = b.depthwise(y, 3, stride, 1)
    if act != ACT_NONE:
        y = b.activation(y, act)
    y = b.conv2d(y, cout, 1)
    if stride == 1 and cin == cout:
        y = b.add(x, y)
    if out_act is not None:
        y = b.activation(y, out_act)
    b.output(y)
    return b.finish()


def pointwise_pair(batch: int, h: int, w: int, cin: int, cmid: int, cout: int, residual: bool = True,
                   mid_act: str = ACT_NONE, act: str = ACT_RELU6) -> GraphSpec:
    """The seam between two inverted-residual blocks on its own: the linear 1x1 projection of one block (plus the
    residual sum, the residual being a second graph input) followed by the 1x1 expansion + activation of the next.
    Both tensors are graph outputs: the narrow one is what the next block's residual sum would read."""
    b = GraphBuilder(f"pair_{batch}x{h}x{w}_{cin}_{cmid}_{cout}_{int(residual)}", batch, 15)
    x = b.input(h, w, cin)
    y = b.conv2d(x, cmid, 1)
    if mid_act != ACT_NONE:
        y = b.activation(y, mid_act)
    if residual:
        y = b.add(b.input(h, w, cmid), y)
    z = b.conv2d(y, cout, 1)
    if act != ACT_NONE:
        z = b.activation(z, act)
    b.output(y)
    b.output(z)
    return b.finish()


# ----------------------------------------------------------------------------------------
# Workload 10: a network of "fire" modules - squeeze 1x1, then a 1x1 and a 3x3 expansion whose outputs are
# concatenated - with a 2x2 stride-2 stem and a 3x3 stride-3 reduction: the operators and the kernel sizes /
# strides (1x1, 2x2, 3x3; 1 to 3) that the MobileNets do not use.  Channel counts are chosen so that one
# concatenation joins whole 4-channel slices and the others do not.
# ----------------------------------------------------------------------------------------
def _fire(b: GraphBuilder, x: int, squeeze: int, e1: int, e3: int) -> int:
    s = b.activation(b.conv2d(x, squeeze, 1), ACT_RELU)
    left = b.activation(b.conv2d(s, e1, 1), ACT_RELU)
    right = b.activation(b.conv2d(s, e3, 3), ACT_RELU)
    return b.concat(left, right)


def fire_network(batch: int = 1, size: int = 96, classes: int = 10) -> GraphSpec:
    b = GraphBuilder("fire_network", batch, 10)
    x = b.input(size, size, 3)
    y = b.activation(b.conv2d(x, 24, 2, 2), ACT_RELU)
    y = _fire(b, y, 8, 16, 16)
    y = _fire(b, y, 8, 18, 14)
    y = b.activation(b.conv2d(y, 48, 3, 3), ACT_RELU)
    y = _fire(b, y, 12, 23, 25)
    y = b.concat(y)
    skip = y
    y = _fire(b, y, 12, 24, 24)
    y = b.add(skip, y)
    y = b.identity_add(y)
    y = b.activation(b.conv2d(y, 64, 2, 1), ACT_RELU6)
    y = b.global_avg_pool(y)
    y = b.conv2d(y, classes, 1)
    b.output(y)
    return b.finish()


def single_concat(batch: int, h: int, w: int, ca: int, cb: int) -> GraphSpec:
    b = GraphBuilder(f"concat_{batch}x{h}x{w}x{ca}+{cb}", batch, 11)
    x = b.input(h, w, ca)
    y = b.input(h, w, cb)
    b.output(b.concat(x, y))
    return b.finish()


def single_conv(batch: int, h: int, w: int, cin: int, cout: int, k: int, stride: int, act: str = ACT_RELU) -> GraphSpec:
    b = GraphBuilder(f"conv{k}_{batch}x{h}x{w}x{cin}x{cout}_s{stride}", batch, 12)
    x = b.input(h, w, cin)
    y = b.conv2d(x, cout, k, stride)
    if act != ACT_NONE:
        y = b.activation(y, act)
    b.output(y)
    return b.finish()


def single_conv3x3(batch: int, hw: int, cin: int, cout: int, stride: int = 1) -> GraphSpec:
    b = GraphBuilder(f"conv3_{batch}x{hw}x{cin}x{cout}_s{stride}", batch, 7)
    x = b.input(hw, hw, cin)
    y = b.activation(b.conv2d(x, cout, 3, stride), ACT_RELU6)
    b.output(y)
    return b.finish()


SWEEP_CHANNELS_PW = [32, 64, 96, 144, 192, 384, 576, 960, 1280]
SWEEP_CHANNELS_DW = [32, 96, 144, 192, 384, 576, 960]
SWEEP_BATCH = [1, 8, 64, 256]
SWEEP_HW = [7, 14, 28, 56, 112]
