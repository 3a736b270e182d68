"""Oracle graph evaluation: runs a graph description op by op on the CPU.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Storage modes:
  "f32"  nothing is rounded; tensors are fp32.
  "f16"  emulates fp16 storage with fp32 arithmetic: weights are rounded to fp16 once,
         biases stay fp32, and every tensor that is *stored* (each executed op's output,
         and each graph input as it is packed) is rounded to fp16 after the op's whole
         epilogue; arithmetic between two stores is unrounded.

Evaluating the unfused graph stores after every op; evaluating the fused graph (the list
produced by compile.fuse) stores once per fused op.  A fused op is its leading op followed
by its folded element-wise ops in graph order, applied to the leading op's fp32 result.
"""
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import compile as oc
from . import ops


def _leading(op, x: Sequence[np.ndarray], f16: bool) -> np.ndarray:
    k = op.kind
    if k in oc.CONV_KINDS:
        w = ops.round_f16(op.weights) if f16 else op.weights
        fn = ops.conv2d if k == "conv2d" else ops.depthwise
        return fn(x[0], w, op.bias, op.stride, op.dilation, op.pads)
    if k == "activation":
        return ops.activation(x[0], op.act)
    if k in ("add", "concat") and len(x) == 1:
        return ops.activation(x[0], "none")  # a single-input ADD / CONCAT is the identity
    if k == "add":
        return ops.add(x[0], x[1])
    if k == "concat":
        return ops.concat(x[0], x[1])
    if k == "global_avg_pool":
        return ops.global_avg_pool(x[0])
    if k == "resize_bilinear":
        return ops.resize_bilinear(x[0], op.out_hw[0], op.out_hw[1], op.align_corners)
    raise ValueError(k)


def run(g, inputs: Sequence[np.ndarray], storage: str = "f16", fused: bool = True,
        fused_ops: Optional[List[oc.FusedOp]] = None, keep_all: bool = False) -> Dict[int, np.ndarray]:
    """Evaluate `g` on NHWC fp32 `inputs` (one per graph input, batch = inputs[0].shape[0]).

    Returns {tensor id: NHWC fp32 array} for the graph outputs, or for every stored tensor
    when keep_all is set.
    """
    f16 = storage == "f16"
    if storage not in ("f16", "f32"):
        raise ValueError(storage)
    store = (lambda a: ops.round_f16(a)) if f16 else (lambda a: np.ascontiguousarray(a, dtype=np.float32))
    val: Dict[int, np.ndarray] = {}
    for t, x in zip(g.inputs, inputs):
        assert tuple(x.shape[1:]) == tuple(g.shapes[t]), (x.shape, g.shapes[t])
        val[t] = store(x)
    if fused_ops is None:
        fused_ops = oc.fuse(g, enable=fused)
    last_use: Dict[int, int] = {}
    for i, f in enumerate(fused_ops):
        for t in f.reads():
            last_use[t] = i
    keep = set(g.outputs)
    for i, f in enumerate(fused_ops):
        op = g.ops[f.op_index]
        y = _leading(op, [val[t] for t in f.inputs], f16)
        for what, arg in f.epilogue:
            if what == "act":
                y = ops.activation(y, arg)
            else:
                y = ops.add(y, val[arg])
        assert tuple(y.shape[1:]) == tuple(g.shapes[f.output]), (f, y.shape, g.shapes[f.output])
        val[f.output] = store(y)
        if not keep_all:
            for t in set(f.reads()):
                if last_use[t] == i and t not in keep:
                    del val[t]
    if keep_all:
        return val
    return {t: val[t] for t in g.outputs}
