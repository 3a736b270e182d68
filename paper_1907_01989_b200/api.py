"""ctypes binding over libgi.so (declared in include/gi.h).

Argument marshalling only: every step of the inference path runs inside the library.
PyTorch is used for device memory and streams.  There is no fallback: if the library
has not been built, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

from . import workloads as wl

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgi.so")

GI_OK = 0
GI_E_INVALID, GI_E_UNSUPPORTED, GI_E_NOMEM, GI_E_CUDA, GI_E_STATE, GI_E_ARENA = -1, -2, -3, -4, -5, -6
GI_F16, GI_F32 = 1, 2
GI_NHWC, GI_PHWC4 = 0, 1
GI_OP_CONV2D, GI_OP_DEPTHWISE_CONV2D, GI_OP_ADD, GI_OP_ACTIVATION, GI_OP_GLOBAL_AVG_POOL, GI_OP_RESIZE_BILINEAR = 1, 2, 3, 4, 5, 6
GI_OP_CONCAT = 7
GI_EXEC_PACK, GI_EXEC_UNPACK = 100, 101
GI_ACT_NONE, GI_ACT_RELU, GI_ACT_RELU6 = 0, 1, 2
GI_PLAN_GREEDY_BY_SIZE, GI_PLAN_GREEDY_SHARED_OBJECTS, GI_PLAN_NAIVE, GI_PLAN_MIN_COST_FLOW = 0, 1, 2, 3
GI_PW_AUTO, GI_PW_SIMT, GI_PW_TC_PAIR, GI_PW_TC_LANE, GI_PW_TC_WIDE, GI_PW_RULE = 0, 1, 2, 3, 4, 5
GI_XOP_AUTO, GI_XOP_OFF, GI_XOP_ON, GI_XOP_CHAIN = 0, 1, 2, 3
GI_STATIC_ARENA_BYTES = 16 << 20
KERNEL_NAMES = {1: "pack", 2: "unpack", 3: "conv_simt", 4: "pointwise_tc", 5: "depthwise", 6: "eltwise", 7: "pool",
                8: "resize", 9: "conv3x3_tc", 10: "pointwise_ts", 11: "depthwise_pointwise", 12: "none", 13: "concat", 14: "conv_tc", 15: "inverted_residual", 16: "pointwise_mm", 17: "pointwise_chain"}

_KIND = {wl.CONV2D: GI_OP_CONV2D, wl.DEPTHWISE: GI_OP_DEPTHWISE_CONV2D, wl.ADD: GI_OP_ADD,
         wl.ACTIVATION: GI_OP_ACTIVATION, wl.GLOBAL_AVG_POOL: GI_OP_GLOBAL_AVG_POOL,
         wl.RESIZE_BILINEAR: GI_OP_RESIZE_BILINEAR, wl.CONCAT: GI_OP_CONCAT}
_ACT = {wl.ACT_NONE: GI_ACT_NONE, wl.ACT_RELU: GI_ACT_RELU, wl.ACT_RELU6: GI_ACT_RELU6}


class gi_op_desc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("inputs", C.c_int32 * 2), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride_h", C.c_int32), ("stride_w", C.c_int32), ("dilation_h", C.c_int32), ("dilation_w", C.c_int32),
                ("pad_t", C.c_int32), ("pad_l", C.c_int32), ("pad_b", C.c_int32), ("pad_r", C.c_int32),
                ("cout", C.c_int32), ("act", C.c_int32), ("out_h", C.c_int32), ("out_w", C.c_int32),
                ("align_corners", C.c_int32), ("weight_dtype", C.c_int32), ("weights", C.c_void_p),
                ("bias", C.c_void_p)]


class gi_compile_options(C.Structure):
    _fields_ = [("planner", C.c_int32), ("fuse", C.c_int32), ("align", C.c_int32), ("pointwise", C.c_int32),
                ("cross_op", C.c_int32)]


class gi_exec_info(C.Structure):
    _fields_ = [("n_ops", C.c_int32), ("n_fused_ops", C.c_int32), ("n_tensors", C.c_int32), ("batch", C.c_int32),
                ("storage", C.c_int32), ("arena_bytes", C.c_uint64), ("naive_bytes", C.c_uint64),
                ("lower_bound_bytes", C.c_uint64), ("weight_bytes", C.c_uint64)]


class gi_tensor_info(C.Structure):
    _fields_ = [("h", C.c_int32), ("w", C.c_int32), ("c", C.c_int32), ("alive", C.c_int32), ("intermediate", C.c_int32),
                ("first_op", C.c_int32), ("last_op", C.c_int32), ("bytes", C.c_uint64), ("offset", C.c_uint64)]


class gi_op_info(C.Structure):
    _fields_ = [("kind", C.c_int32), ("graph_op", C.c_int32), ("inputs", C.c_int32 * 2), ("residual", C.c_int32),
                ("output", C.c_int32), ("act_pre", C.c_int32), ("act_post", C.c_int32), ("kernel", C.c_int32),
                ("bytes", C.c_uint64), ("flops", C.c_uint64)]


EXPORTS = ["gi_graph_create", "gi_graph_input", "gi_add_op", "gi_graph_output", "gi_graph_destroy", "gi_compile",
           "gi_exec_query", "gi_exec_tensor", "gi_exec_op", "gi_exec_bind", "gi_run", "gi_run_static", "gi_run_timed", "gi_device_status", "gi_selftest_bounded_wait", "gi_exec_destroy",
           "gi_slice8_tensor_bytes", "gi_slice8_pointwise_blob_bytes", "gi_slice8_pointwise_pack", "gi_slice8_pointwise_run",
           "gi_status_str", "gi_last_error", "gi_tensor_bytes", "gi_f32_to_f16"]

_lib = None


class GiError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where}: status {status}: {detail}")
        self.status = status


def lib() -> C.CDLL:
    """Load libgi.so; raises if it has not been built (python -m paper_1907_01989_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python {os.path.join(_HERE, 'build.py')}`; "
                           "there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp = C.c_void_p
    L.gi_graph_create.argtypes = [C.POINTER(vp), C.c_int32, C.c_int32]
    L.gi_graph_input.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32)]
    L.gi_add_op.argtypes = [vp, C.POINTER(gi_op_desc), C.POINTER(C.c_int32)]
    L.gi_graph_output.argtypes = [vp, C.c_int32, C.c_int32]
    L.gi_graph_destroy.argtypes = [vp]
    L.gi_graph_destroy.restype = None
    L.gi_compile.argtypes = [vp, C.POINTER(gi_compile_options), C.POINTER(vp)]
    L.gi_exec_query.argtypes = [vp, C.POINTER(gi_exec_info)]
    L.gi_exec_tensor.argtypes = [vp, C.c_int32, C.POINTER(gi_tensor_info)]
    L.gi_exec_op.argtypes = [vp, C.c_int32, C.POINTER(gi_op_info)]
    L.gi_exec_bind.argtypes = [vp, vp, C.c_size_t, vp]
    L.gi_run.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, C.c_size_t, vp]
    L.gi_run_static.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp]
    L.gi_run_static.restype = C.c_int32
    L.gi_run_timed.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, C.c_size_t, vp, C.POINTER(C.c_float), C.c_int32]
    L.gi_device_status.argtypes = [C.POINTER(C.c_uint32)]
    L.gi_device_status.restype = C.c_int32
    L.gi_selftest_bounded_wait.argtypes = [C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(C.c_int32), vp]
    L.gi_selftest_bounded_wait.restype = C.c_int32
    L.gi_exec_destroy.argtypes = [vp]
    L.gi_exec_destroy.restype = None
    L.gi_slice8_tensor_bytes.argtypes = [C.c_int32] * 4
    L.gi_slice8_tensor_bytes.restype = C.c_uint64
    L.gi_slice8_pointwise_blob_bytes.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_uint64)]
    L.gi_slice8_pointwise_blob_bytes.restype = C.c_int32
    L.gi_slice8_pointwise_pack.argtypes = [vp, vp, C.c_int32, C.c_int32, vp, C.c_uint64]
    L.gi_slice8_pointwise_pack.restype = C.c_int32
    L.gi_slice8_pointwise_run.argtypes = [vp, vp, vp] + [C.c_int32] * 6 + [vp]
    L.gi_slice8_pointwise_run.restype = C.c_int32
    L.gi_status_str.argtypes = [C.c_int32]
    L.gi_status_str.restype = C.c_char_p
    L.gi_last_error.argtypes = []
    L.gi_last_error.restype = C.c_char_p
    L.gi_tensor_bytes.argtypes = [C.c_int32] * 6
    L.gi_tensor_bytes.restype = C.c_uint64
    L.gi_f32_to_f16.argtypes = [vp, vp, C.c_size_t]
    L.gi_f32_to_f16.restype = None
    for name in ("gi_graph_create", "gi_graph_input", "gi_add_op", "gi_graph_output", "gi_compile", "gi_exec_query",
                 "gi_exec_tensor", "gi_exec_op", "gi_exec_bind", "gi_run", "gi_run_timed"):
        getattr(L, name).restype = C.c_int32
    _lib = L
    return L


def _check(status: int, where: str) -> None:
    if status != GI_OK:
        L = lib()
        raise GiError(status, f"{where} [{L.gi_status_str(status).decode()}]", L.gi_last_error().decode())


def gi_tensor_bytes(batch, H, W, Cc, storage=GI_F16, align=256) -> int:
    return int(lib().gi_tensor_bytes(batch, H, W, Cc, storage, align))


def gi_f32_to_f16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().gi_f32_to_f16(x.ctypes.data, out.ctypes.data, x.size)
    return out


def gi_device_status() -> int:
    flags = C.c_uint32(0)
    _check(lib().gi_device_status(C.byref(flags)), "gi_device_status")
    return int(flags.value)


def gi_selftest_bounded_wait(limit_us: int, stream=None):
    """-> (microseconds the wait lasted on the device, True if it ended by running out)."""
    waited, gave_up = C.c_uint32(0), C.c_int32(0)
    _check(lib().gi_selftest_bounded_wait(limit_us, C.byref(waited), C.byref(gave_up), _stream_ptr(stream)), "gi_selftest_bounded_wait")
    return int(waited.value), bool(gave_up.value)


def gi_slice8_tensor_bytes(batch, H, W, Cc) -> int:
    return int(lib().gi_slice8_tensor_bytes(batch, H, W, Cc))


def gi_slice8_pointwise_pack(w: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """Packed weights + bias (uint8 array) of a 1x1 layer w[cout, cin] for gi_slice8_pointwise_run."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    cout, cin = w.shape
    n = C.c_uint64(0)
    _check(lib().gi_slice8_pointwise_blob_bytes(cin, cout, C.byref(n)), "gi_slice8_pointwise_blob_bytes")
    blob = np.zeros(int(n.value), dtype=np.uint8)
    _check(lib().gi_slice8_pointwise_pack(w.ctypes.data, bias.ctypes.data, cin, cout, blob.ctypes.data, blob.size), "gi_slice8_pointwise_pack")
    return blob


def gi_slice8_pointwise_run(dev_in: int, dev_out: int, dev_blob: int, batch, H, W, cin, cout, act, stream=None) -> None:
    """Argument marshalling only: the three pointers are device addresses (torch tensors' data_ptr())."""
    _check(lib().gi_slice8_pointwise_run(dev_in, dev_out, dev_blob, batch, H, W, cin, cout, act, _stream_ptr(stream)), "gi_slice8_pointwise_run")


class Graph:
    """gi_graph_create / gi_graph_input / gi_add_op / gi_graph_output."""

    def __init__(self, batch: int, storage: int = GI_F16):
        self._h = C.c_void_p()
        _check(lib().gi_graph_create(C.byref(self._h), batch, storage), "gi_graph_create")
        self.batch, self.storage = batch, storage

    def __del__(self):
        if getattr(self, "_h", None) is not None and self._h and _lib is not None:
            _lib.gi_graph_destroy(self._h)
            self._h = None

    def input(self, H: int, W: int, Cc: int, layout: int = GI_NHWC) -> int:
        t = C.c_int32(-1)
        _check(lib().gi_graph_input(self._h, H, W, Cc, layout, C.byref(t)), "gi_graph_input")
        return t.value

    def add_op(self, desc: gi_op_desc) -> int:
        t = C.c_int32(-1)
        _check(lib().gi_add_op(self._h, C.byref(desc), C.byref(t)), "gi_add_op")
        return t.value

    def output(self, t: int, layout: int = GI_NHWC) -> None:
        _check(lib().gi_graph_output(self._h, t, layout), "gi_graph_output")

    def compile(self, planner: int = GI_PLAN_GREEDY_BY_SIZE, fuse: bool = True, align: int = 256,
                pointwise: int = GI_PW_AUTO, cross_op: int = GI_XOP_AUTO) -> "Executable":
        opt = gi_compile_options(planner, 1 if fuse else 0, align, pointwise, cross_op)
        h = C.c_void_p()
        _check(lib().gi_compile(self._h, C.byref(opt), C.byref(h)), "gi_compile")
        return Executable(h, self)


def graph_from_spec(spec: wl.GraphSpec, storage: int = GI_F16, io_layout: int = GI_NHWC, out_layout: int = None):
    """Build a gi graph from a workload description.  Returns (Graph, {spec tensor id -> gi tensor id}).
    `io_layout` is the layout of the graph's inputs and, unless `out_layout` is given, of its outputs."""
    out_layout = io_layout if out_layout is None else out_layout
    g = Graph(spec.batch, storage)
    ids = {}
    for t in spec.inputs:
        H, W, Cc = spec.shapes[t]
        ids[t] = g.input(H, W, Cc, io_layout)
    for op in spec.ops:
        d = gi_op_desc()
        d.kind = _KIND[op.kind]
        d.inputs[0] = ids[op.inputs[0]]
        d.inputs[1] = ids[op.inputs[1]] if len(op.inputs) > 1 else -1
        keep = []
        if op.kind in (wl.CONV2D, wl.DEPTHWISE):
            d.kh, d.kw = op.kh, op.kw
            d.stride_h, d.stride_w = op.stride
            d.dilation_h, d.dilation_w = op.dilation
            d.pad_t, d.pad_l, d.pad_b, d.pad_r = op.pads
            d.cout = op.cout
            w = np.ascontiguousarray(op.weights, dtype=np.float32)
            keep.append(w)
            d.weight_dtype = GI_F32
            d.weights = w.ctypes.data
            if op.bias is not None:
                b = np.ascontiguousarray(op.bias, dtype=np.float32)
                keep.append(b)
                d.bias = b.ctypes.data
        elif op.kind == wl.ACTIVATION:
            d.act = _ACT[op.act]
        elif op.kind == wl.RESIZE_BILINEAR:
            d.out_h, d.out_w = op.out_hw
            d.align_corners = 1 if op.align_corners else 0
        ids[op.output] = g.add_op(d)
        del keep
    for t in spec.outputs:
        g.output(ids[t], out_layout)
    return g, ids


class Executable:
    """gi_exec_*: query, bind weights, run.  Device buffers are torch tensors owned here or by the caller."""

    def __init__(self, handle: C.c_void_p, graph: Graph):
        self._h = handle
        self.graph = graph
        self.info = gi_exec_info()
        _check(lib().gi_exec_query(self._h, C.byref(self.info)), "gi_exec_query")
        self._weights = None
        self._arena = None

    def __del__(self):
        if getattr(self, "_h", None) is not None and self._h and _lib is not None:
            _lib.gi_exec_destroy(self._h)
            self._h = None

    def tensor(self, t: int) -> gi_tensor_info:
        ti = gi_tensor_info()
        _check(lib().gi_exec_tensor(self._h, t, C.byref(ti)), "gi_exec_tensor")
        return ti

    def op(self, i: int) -> gi_op_info:
        oi = gi_op_info()
        _check(lib().gi_exec_op(self._h, i, C.byref(oi)), "gi_exec_op")
        return oi

    def ops(self) -> List[gi_op_info]:
        return [self.op(i) for i in range(self.info.n_ops)]

    # -- device side -------------------------------------------------------------------
    def bind(self, device="cuda:0", stream=None) -> None:
        """Allocate the weight blob and the arena as torch tensors and upload the packed weights."""
        import torch
        self._weights = torch.empty(max(int(self.info.weight_bytes), 256), dtype=torch.uint8, device=device)
        self._arena = torch.empty(max(int(self.info.arena_bytes), 256), dtype=torch.uint8, device=device)
        self.bind_raw(self._weights.data_ptr(), self._weights.numel(), stream)

    def bind_raw(self, dev_weights: int, nbytes: int, stream=None) -> None:
        _check(lib().gi_exec_bind(self._h, dev_weights, nbytes, _stream_ptr(stream)), "gi_exec_bind")

    @property
    def arena(self):
        return self._arena

    def run_raw(self, in_ptrs: Sequence[int], out_ptrs: Sequence[int], arena_ptr: int, arena_bytes: int,
                stream=None) -> None:
        ins = (C.c_void_p * max(len(in_ptrs), 1))(*in_ptrs)
        outs = (C.c_void_p * max(len(out_ptrs), 1))(*out_ptrs)
        _check(lib().gi_run(self._h, ins, outs, arena_ptr, arena_bytes, _stream_ptr(stream)), "gi_run")

    def run_static(self, inputs, outputs, stream=None) -> None:
        """gi_run_static: intermediates in the library's built-in arena; allocates nothing."""
        ins = (C.c_void_p * max(len(inputs), 1))(*[t.data_ptr() for t in inputs])
        outs = (C.c_void_p * max(len(outputs), 1))(*[t.data_ptr() for t in outputs])
        _check(lib().gi_run_static(self._h, ins, outs, _stream_ptr(stream)), "gi_run_static")

    def run_timed(self, inputs, outputs, stream=None) -> List[float]:
        """gi_run_timed: one run with an event around every executed op; returns per-op milliseconds."""
        n = int(self.info.n_ops)
        ms = (C.c_float * n)()
        ins = (C.c_void_p * max(len(inputs), 1))(*[t.data_ptr() for t in inputs])
        outs = (C.c_void_p * max(len(outputs), 1))(*[t.data_ptr() for t in outputs])
        _check(lib().gi_run_timed(self._h, ins, outs, self._arena.data_ptr(), self._arena.numel(), _stream_ptr(stream),
                                  ms, n), "gi_run_timed")
        return list(ms)

    def run(self, inputs, outputs, stream=None) -> None:
        """inputs / outputs: torch CUDA tensors in the declared layouts (contiguous, storage dtype)."""
        self.run_raw([t.data_ptr() for t in inputs], [t.data_ptr() for t in outputs], self._arena.data_ptr(),
                     self._arena.numel(), stream)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        if torch.cuda.is_available():
            return torch.cuda.current_stream().cuda_stream
        return None
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)
