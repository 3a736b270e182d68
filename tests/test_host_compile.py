"""Host-side tests of the C-ABI library (no GPU): exported symbols, error behaviour, and the
compile step compared bit-exactly with the oracle's independent implementation."""
import ctypes as C
import os
import random
import re

import numpy as np
import pytest

from oracle import compile as oc
from paper_1907_01989_b200 import api
from paper_1907_01989_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

KIND_NAME = {api.GI_OP_CONV2D: "conv2d", api.GI_OP_DEPTHWISE_CONV2D: "depthwise_conv2d", api.GI_OP_ADD: "add",
             api.GI_OP_ACTIVATION: "activation", api.GI_OP_GLOBAL_AVG_POOL: "global_avg_pool",
             api.GI_OP_RESIZE_BILINEAR: "resize_bilinear", api.GI_OP_CONCAT: "concat"}
ACT_NAME = {api.GI_ACT_NONE: None, api.GI_ACT_RELU: "relu", api.GI_ACT_RELU6: "relu6"}


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "gi.h")).read()
    declared = re.findall(r"^GI_API\s+[\w\s\*]+?\b(gi_\w+)\s*\(", header, flags=re.M)
    assert sorted(declared) == sorted(api.EXPORTS)
    L = api.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_f32_to_f16_matches_numpy():
    rng = np.random.default_rng(7)
    pos = np.arange(0, 0x7bff, dtype=np.uint16)
    lo = pos.view(np.float16).astype(np.float64)
    hi = (pos + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)
    edge = np.array([65504.0, 65519.99, 65520.0, 65536.0, 1e10, -65520.0, 2.0 ** -24, 2.0 ** -25, 2.0 ** -26, 6.1e-5,
                     2.0 ** -14, np.inf, -np.inf, 0.0, -0.0], dtype=np.float32)
    r = (rng.standard_normal(500_000) * np.exp(rng.uniform(-20, 12, 500_000))).astype(np.float32)
    allh = np.arange(65536, dtype=np.uint16).view(np.float16)
    allh = allh[~np.isnan(allh)].astype(np.float32)
    with np.errstate(over="ignore"):
        for x in (mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf)), -mid, edge, r, allh):
            assert np.array_equal(api.gi_f32_to_f16(x), x.astype(np.float16).view(np.uint16))


def test_tensor_bytes_matches_size_formula():
    for batch, shape in [(1, (8, 6, 12)), (1, (7, 7, 5)), (3, (7, 7, 4)), (256, (112, 112, 96)), (2, (1, 1, 1001)),
                         (16, (513, 513, 21))]:
        for storage, eb in ((api.GI_F16, 2), (api.GI_F32, 4)):
            for align in (256, 1024):
                assert api.gi_tensor_bytes(batch, *shape, storage, align) == oc.tensor_bytes(batch, shape, eb, align)


# ---------------------------------------------------------------------- compile step vs oracle
def exec_records(ex):
    """(ops, sizes, intermediates, lifetimes, offsets) as the library reports them."""
    ops = ex.ops()
    tensors = {t: ex.tensor(t) for t in range(ex.info.n_tensors)}
    return ops, tensors


def compare_with_oracle(spec, planner, fuse=True, storage=api.GI_F16, align=256):
    g, ids = api.graph_from_spec(spec, storage)
    assert all(ids[t] == t for t in ids)  # the builder and the library number tensors alike
    ex = g.compile(planner=planner, fuse=fuse, align=align)
    ops, tensors = exec_records(ex)
    fused = oc.fuse(spec, enable=fuse)
    n_in, n_out = len(spec.inputs), len(spec.outputs)
    assert ex.info.n_fused_ops == len(fused)
    assert ex.info.n_ops == len(fused) + n_in + n_out
    for k in range(n_in):
        assert ops[k].kind == api.GI_EXEC_PACK and ops[k].output == spec.inputs[k]
    for k in range(n_out):
        o = ops[n_in + len(fused) + k]
        assert o.kind == api.GI_EXEC_UNPACK and o.inputs[0] == spec.outputs[k]
    for f, o in zip(fused, ops[n_in:n_in + len(fused)]):
        assert KIND_NAME[o.kind] == f.kind and o.graph_op == f.op_index and o.output == f.output
        assert [t for t in (o.inputs[0], o.inputs[1]) if t >= 0] == f.inputs
        adds = [a for k, a in f.epilogue if k == "add"]
        assert (o.residual if o.residual >= 0 else None) == (adds[0] if adds else None)
        if f.kind in oc.CONV_KINDS:
            pre, post, seen_add = None, None, False
            for k, a in f.epilogue:
                if k == "add":
                    seen_add = True
                elif seen_add or pre is not None:
                    post = a
                else:
                    pre = a
            assert ACT_NAME[o.act_pre] == pre and ACT_NAME[o.act_post] == post
    eb = 2 if storage == api.GI_F16 else 4
    views = oc.concat_views(spec, fused) if fuse else {}
    p = oc.plan_problem(spec, fused, eb, align, convert_io=True, views=views)
    life = oc.lifetimes(p)
    for t, ti in tensors.items():
        assert bool(ti.alive) == (t in p.size or t in views)
        assert (ti.h, ti.w, ti.c) == tuple(spec.shapes[t])
        if t in views:
            assert ti.intermediate == 2 and t not in p.size
        if t in p.size:
            assert ti.intermediate == 1
            assert ti.bytes == p.size[t]
            assert (ti.first_op, ti.last_op) == life[t]
    if planner == api.GI_PLAN_NAIVE:
        off, total = oc.plan_naive(p)
    elif planner == api.GI_PLAN_GREEDY_SHARED_OBJECTS:
        off, total = oc.plan_greedy_shared_objects(p)[:2]
    elif planner == api.GI_PLAN_MIN_COST_FLOW:
        off, total = oc.plan_min_cost_flow(p)[:2]
    else:
        off, total = oc.plan_greedy_by_size(p)
    assert ex.info.arena_bytes == total
    assert ex.info.naive_bytes == oc.plan_naive(p)[1]
    assert ex.info.lower_bound_bytes == oc.lower_bound(p)
    for t in p.intermediate:
        assert tensors[t].offset == off[t], (t, tensors[t].offset, off[t])
        assert tensors[t].offset % align == 0
    oc.check_no_overlap(p, {t: tensors[t].offset for t in p.intermediate})
    for t, (root, first_slice) in views.items():
        H, W, _ = spec.shapes[t]
        assert tensors[t].offset == off[root] + first_slice * spec.batch * ((H * W + 1) // 2 * 2) * 4 * eb
    return ex


PLANNERS = [api.GI_PLAN_GREEDY_BY_SIZE, api.GI_PLAN_GREEDY_SHARED_OBJECTS, api.GI_PLAN_NAIVE, api.GI_PLAN_MIN_COST_FLOW]
NETS = [lambda: wl.separable_block(1), lambda: wl.mobilenet_v1(1), lambda: wl.mobilenet_v2(1),
        lambda: wl.mobilenet_v2_segmentation(1), lambda: wl.mobilenet_v2(256), lambda: wl.mobilenet_v2_segmentation(16),
        lambda: wl.single_pointwise(8, 14, 96, 576, residual=True), lambda: wl.single_depthwise(8, 7, 96, 2),
        lambda: wl.fire_network(4), lambda: wl.single_concat(3, 5, 5, 6, 7)]


@pytest.mark.parametrize("planner", PLANNERS)
@pytest.mark.parametrize("net", range(len(NETS)))
def test_plan_offsets_bit_exact_on_workloads(net, planner):
    spec = NETS[net]()
    compare_with_oracle(spec, planner)
    if net < 3:
        compare_with_oracle(spec, planner, fuse=False)
        compare_with_oracle(spec, planner, storage=api.GI_F32, align=1024)


def random_spec(rnd: random.Random, n_ops: int) -> wl.GraphSpec:
    b = wl.GraphBuilder("random", rnd.choice([1, 2, 3]), 99)
    live = [b.input(rnd.choice([5, 8, 9]), rnd.choice([4, 7, 8]), rnd.choice([3, 4, 6, 8]))]
    for _ in range(n_ops):
        x = rnd.choice(live[-4:])
        kind = rnd.choice(["conv1", "conv3", "dw", "act", "act", "add", "add", "pool", "conv2", "concat", "concat", "ident"])
        H, W, Cc = b.g.shapes[x]
        if kind == "conv1":
            y = b.conv2d(x, rnd.choice([4, 6, 8, Cc]), 1)
        elif kind == "conv3":
            y = b.conv2d(x, rnd.choice([4, 8, Cc]), 3, rnd.choice([1, 2]))
        elif kind == "dw":
            y = b.depthwise(x, 3, rnd.choice([1, 2]), rnd.choice([1, 2]))
        elif kind == "act":
            y = b.activation(x, rnd.choice([wl.ACT_RELU, wl.ACT_RELU6]))
        elif kind == "add":
            same = [t for t in live if b.g.shapes[t] == b.g.shapes[x]]
            y = b.add(rnd.choice(same), x)
        elif kind == "conv2":
            y = b.conv2d(x, rnd.choice([4, 5, 8]), rnd.choice([2, 3]), rnd.choice([1, 2, 3]))
        elif kind == "concat":
            same = [t for t in live if b.g.shapes[t][:2] == b.g.shapes[x][:2]]
            y = b.concat(rnd.choice(same), x)
        elif kind == "ident":
            y = b.identity_add(x) if rnd.random() < 0.5 else b.concat(x)
        else:
            if H * W == 1:
                continue
            y = b.global_avg_pool(x)
        live.append(y)
    used = {t for op in b.g.ops for t in op.inputs}
    outs = [t for t in live[1:] if t not in used] or [live[-1]]
    if live[-1] not in outs and live[-1] != live[0]:
        outs.append(live[-1])
    for t in outs:
        if t != live[0]:
            b.output(t)
    if not b.g.outputs:
        b.output(b.activation(live[0], wl.ACT_RELU))
    return b.finish()


@pytest.mark.parametrize("seed", range(40))
def test_plan_offsets_bit_exact_on_random_graphs(seed):
    rnd = random.Random(seed)
    spec = random_spec(rnd, rnd.randint(1, 30))
    for planner in PLANNERS:
        compare_with_oracle(spec, planner)
    compare_with_oracle(spec, api.GI_PLAN_GREEDY_BY_SIZE, fuse=False)


def test_expected_fused_counts_and_arena():
    for make, n_fused, mib in ((wl.mobilenet_v1, 29, 2.297), (wl.mobilenet_v2, 54, 2.871),
                               (wl.mobilenet_v2_segmentation, 54, 15.14)):
        g, _ = api.graph_from_spec(make(1))
        ex = g.compile()
        assert ex.info.n_fused_ops == n_fused and ex.info.n_ops == n_fused + 2
        assert abs(ex.info.arena_bytes / 2 ** 20 - mib) < 2e-3
        assert ex.info.arena_bytes == ex.info.lower_bound_bytes


def test_kernels_of_the_benchmark_step():
    """Which kernel runs which layer of MobileNetV2-224 at batch 256 (the bench configuration): the generated launch
    table and the cross-operator rule decide at compile time, so the mix is checked without a GPU.  The expansion
    layers from 24 input channels on and the 14x14 / 7x7 projections run on the lane-per-pixel kernel, the 112x112
    layers and the 56x56 / 28x28 projections on the pixel-pair kernel, the 7x7 layers with 576 or more input channels on
    the CTA-pair kernel, four 14x14 seams as one kernel each; no block runs as one kernel."""
    from collections import Counter
    ex = api.graph_from_spec(wl.mobilenet_v2(256), api.GI_F16)[0].compile()
    ops = ex.ops()
    mix = Counter(api.KERNEL_NAMES[o.kernel] for o in ops)
    assert mix["depthwise"] == 17 and mix["conv3x3_tc"] == 1 and mix["pool"] == 1 and mix["unpack"] == 1
    assert mix["pointwise_chain"] == 4 and mix["inverted_residual"] == 0 and mix["depthwise_pointwise"] == 0
    assert mix["pointwise_ts"] + mix["pointwise_tc"] + mix["pointwise_mm"] == 27
    assert mix["pointwise_mm"] >= 3 and mix["pointwise_ts"] >= 12
    assert sum(v for k, v in mix.items() if k != "none") == 51
    for o in ops:
        name = api.KERNEL_NAMES[o.kernel]
        if name in ("pointwise_ts", "pointwise_tc", "pointwise_mm"):
            tin, tout = ex.tensor(o.inputs[0]), ex.tensor(o.output)
            if tin.h == 7 and tin.c >= 576:
                assert name == "pointwise_mm", (tin.h, tin.c, tout.c)
            if tout.c >= 4 * tin.c and tin.c >= 24:
                assert name == "pointwise_ts", (tin.h, tin.c, tout.c)  # an expansion layer
            if tin.h == 112:
                assert name == "pointwise_tc", (tin.h, tin.c, tout.c)


# ---------------------------------------------------------------------- error behaviour
def _conv_desc(x, cout=8, k=1, **kw):
    d = api.gi_op_desc()
    d.kind = api.GI_OP_CONV2D
    d.inputs[0] = x
    d.inputs[1] = -1
    d.kh = d.kw = k
    d.stride_h = d.stride_w = d.dilation_h = d.dilation_w = 1
    d.cout = cout
    d.weight_dtype = api.GI_F32
    for key, v in kw.items():
        setattr(d, key, v)
    return d


def test_error_paths():
    L = api.lib()
    h = C.c_void_p()
    assert L.gi_graph_create(C.byref(h), 0, api.GI_F16) == api.GI_E_INVALID
    assert L.gi_graph_create(C.byref(h), 1, 7) == api.GI_E_INVALID
    assert L.gi_graph_create(None, 1, api.GI_F16) == api.GI_E_INVALID
    assert b"batch" in L.gi_last_error() or b"null" in L.gi_last_error()
    g = api.Graph(2)
    with pytest.raises(api.GiError):
        g.input(0, 4, 4)
    x = g.input(8, 8, 4)
    w = np.zeros((8, 5, 5, 4), dtype=np.float32)
    with pytest.raises(api.GiError) as ei:
        g.add_op(_conv_desc(x, k=5, weights=w.ctypes.data))
    assert ei.value.status == api.GI_E_UNSUPPORTED
    with pytest.raises(api.GiError) as ei:
        g.add_op(_conv_desc(x))  # no weights
    assert ei.value.status == api.GI_E_INVALID
    with pytest.raises(api.GiError):
        g.add_op(_conv_desc(17, weights=w.ctypes.data))  # unknown tensor
    with pytest.raises(api.GiError):
        g.add_op(_conv_desc(x, weights=w.ctypes.data, stride_h=0))
    with pytest.raises(api.GiError) as ei:
        g.add_op(_conv_desc(x, weights=w.ctypes.data, stride_h=4, stride_w=4))
    assert ei.value.status == api.GI_E_UNSUPPORTED
    d = _conv_desc(x, k=3, weights=w.ctypes.data, stride_h=3, stride_w=3)
    d.kind = api.GI_OP_DEPTHWISE_CONV2D
    with pytest.raises(api.GiError) as ei:
        g.add_op(d)  # depthwise: stride 3 has no kernel
    assert ei.value.status == api.GI_E_UNSUPPORTED
    d = api.gi_op_desc()
    d.kind = api.GI_OP_CONCAT
    d.inputs[0], d.inputs[1] = x, 17  # unknown second tensor
    with pytest.raises(api.GiError):
        g.add_op(d)
    y = g.add_op(_conv_desc(x, cout=8, weights=w.ctypes.data))
    d = api.gi_op_desc()
    d.kind = api.GI_OP_ADD
    d.inputs[0], d.inputs[1] = x, y  # 4 vs 8 channels
    with pytest.raises(api.GiError):
        g.add_op(d)
    d = api.gi_op_desc()
    d.kind = api.GI_OP_ACTIVATION
    d.inputs[0] = y
    with pytest.raises(api.GiError):
        g.add_op(d)  # act missing
    with pytest.raises(api.GiError):
        g.output(x)  # an input cannot be an output
    with pytest.raises(api.GiError):
        g.compile()  # no outputs yet
    g.output(y)
    with pytest.raises(api.GiError):
        g.output(y)
    with pytest.raises(api.GiError):
        g.compile(align=100)
    with pytest.raises(api.GiError):
        g.compile(planner=9)
    ex = g.compile()
    assert ex.info.n_ops == 3
    with pytest.raises(api.GiError):
        ex.tensor(99)
    with pytest.raises(api.GiError):
        ex.op(3)
    # gi_run before gi_exec_bind is refused before anything touches the device
    with pytest.raises(api.GiError) as ei:
        ex.run_raw([256], [256], 256, 1 << 30, stream=0)
    assert ei.value.status == api.GI_E_STATE


def test_graph_reusable_after_compile_and_weights_copied():
    spec = wl.separable_block(1)
    g, _ = api.graph_from_spec(spec)
    a = g.compile(planner=api.GI_PLAN_NAIVE)
    b = g.compile(planner=api.GI_PLAN_GREEDY_BY_SIZE)
    assert a.info.weight_bytes == b.info.weight_bytes > 0
    assert a.info.arena_bytes >= b.info.arena_bytes


def test_kernel_choice_options():
    """Kernel selection is a host decision: check it without a GPU."""
    def kernels(spec, **kw):
        return [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, api.GI_F16)[0].compile(**kw).ops()]

    even = wl.single_depthwise(2, 14, 32, 1)
    assert "depthwise" in kernels(even)
    g = api.graph_from_spec(even, api.GI_F16)[0]
    with pytest.raises(api.GiError):
        g.compile(pointwise=9)
    pw = wl.single_pointwise(128, 14, 16, 96)  # few input channels: the pixel-pair kernel by the rule
    assert "pointwise_tc" in kernels(pw) and "pointwise_ts" in kernels(pw, pointwise=api.GI_PW_TC_LANE)
    assert "pointwise_ts" in kernels(wl.single_pointwise(128, 14, 64, 384))  # an expansion with 24 or more input channels
    assert "conv_simt" in kernels(pw, pointwise=api.GI_PW_SIMT)
    # all pixels in one wave of 128-pixel tiles: the lane-per-pixel kernel whatever the channel counts
    small = wl.single_pointwise(2, 14, 64, 384)
    assert "pointwise_ts" in kernels(small) and "pointwise_tc" in kernels(small, pointwise=api.GI_PW_TC_PAIR)


def test_cross_op_option():
    """Depthwise + 1x1 convolution as one kernel: chosen at compile time, only where the pattern and the kernel allow."""
    def kernels(spec, storage=api.GI_F16, **kw):
        return [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, storage)[0].compile(**kw).ops()]

    pair = wl.depthwise_then_pointwise(4, 28, 28, 32, 24, 1, residual=True)
    assert "depthwise_pointwise" not in kernels(pair) and "depthwise_pointwise" not in kernels(pair, cross_op=api.GI_XOP_OFF)
    on = kernels(pair, cross_op=api.GI_XOP_ON, planner=api.GI_PLAN_NAIVE)
    assert on.count("depthwise_pointwise") == 1 and on.count("none") == 1 and "depthwise" not in on
    assert on.index("none") == on.index("depthwise_pointwise") + 1
    # fp32 storage, channels not a multiple of 16, planes wider than 128 columns: two kernels
    assert "depthwise_pointwise" not in kernels(pair, api.GI_F32, cross_op=api.GI_XOP_ON)
    assert "depthwise_pointwise" not in kernels(wl.depthwise_then_pointwise(2, 14, 14, 24, 16), cross_op=api.GI_XOP_ON)
    assert "depthwise_pointwise" not in kernels(wl.depthwise_then_pointwise(1, 8, 200, 16, 16), cross_op=api.GI_XOP_ON)
    # the tensor between the two ops must have no other reader: a graph output stays a stored tensor
    b = wl.GraphBuilder("dw_out_and_pw", 2, 11)
    x = b.input(14, 14, 16)
    y = b.activation(b.depthwise(x, 3, 1, 1), wl.ACT_RELU6)
    b.output(y)
    b.output(b.conv2d(y, 8, 1))
    assert "depthwise_pointwise" not in kernels(b.finish(), cross_op=api.GI_XOP_ON)
    # the plan is not affected: the tensor keeps its arena slot, the op count stays
    g = api.graph_from_spec(pair, api.GI_F16)[0]
    a, c = g.compile(cross_op=api.GI_XOP_OFF, planner=api.GI_PLAN_NAIVE), g.compile(cross_op=api.GI_XOP_ON, planner=api.GI_PLAN_NAIVE)
    assert a.info.arena_bytes == c.info.arena_bytes and a.info.n_ops == c.info.n_ops
    # whole network at batch 256: the ten blocks on 14x14 and 7x7 planes run as one kernel each (expansion, depthwise
    # and projection: two ops without a launch per block); of the seven blocks on larger planes the depthwise ->
    # projection pair runs as one kernel (one op without a launch each).  One kernel reads the pair's / block's input
    # while it writes its output, so where input and output share arena bytes (legal for separate ops: their
    # lifetimes do not meet) the ops stay separate kernels - never under the naive plan
    v2 = kernels(wl.mobilenet_v2(256), cross_op=api.GI_XOP_ON, planner=api.GI_PLAN_NAIVE)
    # (one more op without a launch: the layout conversion of the input, which the stem reads as NHWC itself)
    assert v2.count("inverted_residual") == 10 and v2.count("depthwise_pointwise") == 7 and v2.count("none") == 28
    assert v2[0] == "none" and v2[1] == "conv3x3_tc"
    # the library's own choice: no block as one kernel (measured: neither the 14x14 nor the 7x7 blocks are faster
    # that way than as three kernels), at any batch
    auto = kernels(wl.mobilenet_v2(256), planner=api.GI_PLAN_NAIVE)
    assert auto.count("inverted_residual") == 0 and auto.count("depthwise_pointwise") == 0
    assert "inverted_residual" not in kernels(wl.mobilenet_v2(1))
    gv2 = api.graph_from_spec(wl.mobilenet_v2(256), api.GI_F16)[0]
    for planner in (api.GI_PLAN_GREEDY_BY_SIZE, api.GI_PLAN_GREEDY_SHARED_OBJECTS, api.GI_PLAN_MIN_COST_FLOW):
        ex = gv2.compile(cross_op=api.GI_XOP_ON, planner=planner)
        ops = ex.ops()
        for i, o in enumerate(ops):
            name = api.KERNEL_NAMES[o.kernel]
            if name in ("depthwise_pointwise", "inverted_residual"):
                tin, tout = ex.tensor(o.inputs[0]), ex.tensor(ops[i + (1 if name == "depthwise_pointwise" else 2)].output)
                assert tin.offset + tin.bytes <= tout.offset or tout.offset + tout.bytes <= tin.offset
    names = [api.KERNEL_NAMES[o.kernel] for o in gv2.compile(cross_op=api.GI_XOP_ON).ops()]
    assert names.count("depthwise_pointwise") == 5 and names.count("inverted_residual") == 9
    with pytest.raises(api.GiError):
        g.compile(cross_op=7)


def test_pointwise_pair_option():
    """Two consecutive 1x1 convolutions as one kernel: chosen at compile time, only where pattern, kernel and memory plan allow."""
    def compiled(spec, storage=api.GI_F16, **kw):
        return api.graph_from_spec(spec, storage)[0].compile(**kw)

    def kernels(spec, storage=api.GI_F16, **kw):
        return [api.KERNEL_NAMES[o.kernel] for o in compiled(spec, storage, **kw).ops()]

    pair = wl.pointwise_pair(4, 14, 14, 384, 64, 384, True)
    on = kernels(pair, cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    assert on.count("pointwise_chain") == 1 and on.index("none") == on.index("pointwise_chain") + 1
    assert "pointwise_chain" not in kernels(pair, cross_op=api.GI_XOP_OFF) and "pointwise_chain" not in kernels(pair, cross_op=api.GI_XOP_ON)
    # fp32 storage, a second operator with a residual of its own, a strided second operator, too many channels in the middle
    assert "pointwise_chain" not in kernels(pair, api.GI_F32, cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    b = wl.GraphBuilder("pair_second_residual", 2, 15)
    x = b.input(8, 8, 32)
    y = b.conv2d(x, 32, 1)
    b.output(b.add(x, b.conv2d(y, 32, 1)))
    assert "pointwise_chain" not in kernels(b.finish(), cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    b = wl.GraphBuilder("pair_strided", 2, 15)
    b.output(b.conv2d(b.conv2d(b.input(8, 8, 32), 16, 1), 32, 1, 2))
    assert "pointwise_chain" not in kernels(b.finish(), cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    assert "pointwise_chain" not in kernels(wl.pointwise_pair(2, 7, 7, 960, 160, 960, True), cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    # the plan is not affected
    a, c = compiled(pair, cross_op=api.GI_XOP_OFF), compiled(pair, cross_op=api.GI_XOP_CHAIN)
    assert a.info.arena_bytes == c.info.arena_bytes and a.info.n_ops == c.info.n_ops
    # whole network: every projection -> expansion seam with at most 128 channels in the middle under the naive plan;
    # under the sharing plans the second output may lie on the bytes of the first operator's input or residual (their
    # lifetimes do not meet as separate ops): one kernel would read them while it writes it, so those stay two kernels
    gv2 = api.graph_from_spec(wl.mobilenet_v2(256), api.GI_F16)[0]
    assert [api.KERNEL_NAMES[o.kernel] for o in gv2.compile(cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE).ops()].count("pointwise_chain") == 13
    # (Algorithm 1 hands every hidden tensor the shared object its predecessor has just left: no seam qualifies there)
    for planner, expect in ((api.GI_PLAN_GREEDY_BY_SIZE, 11), (api.GI_PLAN_GREEDY_SHARED_OBJECTS, 0), (api.GI_PLAN_MIN_COST_FLOW, 12)):
        ex = gv2.compile(cross_op=api.GI_XOP_CHAIN, planner=planner)
        ops = ex.ops()
        n = 0
        for i, o in enumerate(ops):
            if api.KERNEL_NAMES[o.kernel] != "pointwise_chain":
                continue
            n += 1
            tout = ex.tensor(ops[i + 1].output)
            for t in (o.inputs[0], o.residual):
                if t >= 0:
                    tin = ex.tensor(t)
                    assert tin.offset + tin.bytes <= tout.offset or tout.offset + tout.bytes <= tin.offset
        assert n == expect
    # the library's own choice at batch 256: the four seams on 14x14 planes with 64 channels in the middle (measured);
    # none at batch 1 or 64, where the tiles would not fill the SMs twice
    auto = [api.KERNEL_NAMES[o.kernel] for o in gv2.compile().ops()]
    assert auto.count("pointwise_chain") == 4
    for batch in (1, 64):
        assert "pointwise_chain" not in kernels(wl.mobilenet_v2(batch))


def test_identity_resize_removed_like_the_oracle():
    """Graph clean-up (Section 3.1): the library drops the same identity ops as the oracle; plan and op list agree."""
    for extra in (False, True):
        b = wl.GraphBuilder("identity_ops", 2, 21)
        x = b.input(6, 5, 8)
        c = b.conv2d(x, 12, 1)
        a = b.activation(b.resize_bilinear(c, 6, 5, True), wl.ACT_RELU)
        r2 = b.resize_bilinear(a, 6, 5, False)
        if extra:
            b.output(r2)
        b.output(b.resize_bilinear(r2, 12, 10, True))
        spec = b.finish()
        for planner in PLANNERS:
            ex = compare_with_oracle(spec, planner)
        assert ex.info.n_fused_ops == (3 if extra else 2)
        compare_with_oracle(spec, api.GI_PLAN_GREEDY_BY_SIZE, fuse=False)


def _exact_bytes(spec, t, eb):
    H, W, Cc = spec.shapes[t]
    return ((Cc + 3) // 4) * spec.batch * ((H * W + 1) // 2 * 2) * 4 * eb


@pytest.mark.parametrize("planner", PLANNERS)
def test_concat_without_copy_memory_is_safe(planner):
    """Inputs of a CONCAT that were placed inside its output: they tile the output's slices exactly, the CONCAT
    launches nothing, and no two tensors that are in use at the same executed op share a byte - other than a
    tensor and the tensor that holds it.  Checked on the fire network and on random graphs, from the
    library's own answers (executed ops, offsets) with lifetimes recomputed here."""
    specs = [wl.fire_network(2)]
    for seed in range(60):
        rnd = random.Random(500 + seed)
        specs.append(random_spec(rnd, rnd.randint(4, 30)))
    seen_views = 0
    for spec in specs:
        g, _ = api.graph_from_spec(spec, api.GI_F16)
        ex = g.compile(planner=planner)
        ops, tensors = exec_records(ex)
        fused = oc.fuse(spec)
        views = oc.concat_views(spec, fused)
        seen_views += len(views)
        # every eligible CONCAT launches nothing; its parts tile it
        for f, o in zip(fused, ops[len(spec.inputs):]):
            if f.kind == "concat" and len(f.inputs) == 2 and views.get(f.inputs[0], (None,))[0] == f.output:
                a, b = f.inputs
                assert api.KERNEL_NAMES[o.kernel] == "none"
                assert tensors[a].offset == tensors[f.output].offset
                assert tensors[b].offset == tensors[a].offset + _exact_bytes(spec, a, 2)
                assert tensors[b].offset + _exact_bytes(spec, b, 2) == tensors[f.output].offset + _exact_bytes(spec, f.output, 2)
            elif f.kind == "concat" and len(f.inputs) == 2:
                assert api.KERNEL_NAMES[o.kernel] == "concat"
        # own lifetimes from the executed list
        life = {}
        for i, o in enumerate(ops):
            for t in (o.inputs[0], o.inputs[1], o.residual, o.output):
                if t >= 0 and tensors[t].alive and tensors[t].intermediate:
                    a, _ = life.get(t, (i, i))
                    life[t] = (a, i)
        ts = sorted(life)
        for x in ts:
            for y in ts:
                if x >= y or life[x][1] < life[y][0] or life[y][1] < life[x][0]:
                    continue
                if views.get(x, (None,))[0] == y or views.get(y, (None,))[0] == x:
                    continue
                x0, x1 = tensors[x].offset, tensors[x].offset + _exact_bytes(spec, x, 2)
                y0, y1 = tensors[y].offset, tensors[y].offset + _exact_bytes(spec, y, 2)
                assert x1 <= y0 or y1 <= x0, (spec.name, x, y, life[x], life[y])
        assert ex.info.arena_bytes >= max(tensors[t].offset + _exact_bytes(spec, t, 2) for t in ts)
    assert seen_views >= 6  # the cases above do exercise it


def test_concat_view_eligibility_rules():
    def fused_and_views(build):
        b = wl.GraphBuilder("views", 1, 60)
        build(b)
        spec = b.finish()
        return spec, oc.concat_views(spec, oc.fuse(spec))

    def ok(b):
        x = b.input(6, 6, 4)
        p, q = b.conv2d(x, 8, 1), b.conv2d(x, 6, 3)
        b.output(b.conv2d(b.concat(p, q), 4, 1))
    spec, v = fused_and_views(ok)
    assert v == {1: (3, 0), 2: (3, 2)}

    def ragged_first(b):
        x = b.input(6, 6, 4)
        p, q = b.conv2d(x, 6, 1), b.conv2d(x, 8, 3)
        b.output(b.conv2d(b.concat(p, q), 4, 1))
    assert fused_and_views(ragged_first)[1] == {}

    def reads_graph_input(b):
        x = b.input(6, 6, 4)
        b.output(b.conv2d(b.concat(x, b.conv2d(x, 8, 1)), 4, 1))
    assert fused_and_views(reads_graph_input)[1] == {}

    def is_graph_output(b):
        x = b.input(6, 6, 4)
        b.output(b.concat(b.conv2d(x, 8, 1), b.conv2d(x, 8, 3)))
    assert fused_and_views(is_graph_output)[1] == {}

    def nested(b):
        x = b.input(6, 6, 4)
        inner = b.concat(b.conv2d(x, 8, 1), b.conv2d(x, 8, 3))   # tensors 1, 2 -> 3
        outer = b.concat(inner, b.conv2d(x, 4, 1))                 # 3 holds tensors already: copied
        b.output(b.conv2d(outer, 4, 1))
    spec, v = fused_and_views(nested)
    assert v == {1: (3, 0), 2: (3, 2)}

    def same_twice_and_reused(b):
        x = b.input(6, 6, 4)
        p, q = b.conv2d(x, 8, 1), b.conv2d(x, 8, 3)
        c1 = b.concat(p, p)          # one tensor twice: copied
        c2 = b.concat(p, q)          # placed
        c3 = b.concat(q, p)          # both already placed: copied
        b.output(b.conv2d(b.add(b.add(c1, c2), c3), 4, 1))
    spec, v = fused_and_views(same_twice_and_reused)
    assert v == {1: (4, 0), 2: (4, 2)}


# ---------------------------------------------------------------------- launch table vs selection rule
def _launch_table():
    """Rows of csrc/launch_table.inc: (pixels, cin, cout, kernel id, ms pair, ms lane, ms wide)."""
    import re
    path = os.path.join(os.path.dirname(api.LIB_PATH), "csrc", "launch_table.inc")
    rows = []
    with open(path) as fh:
        for line in fh:
            m = re.match(r"\{(\d+)LL, (\d+), (\d+), (\d+), ([\d.]+)f, ([\d.]+)f, ([\d.]+)f\},", line.strip())
            if m:
                rows.append((int(m.group(1)), int(m.group(2)), int(m.group(3)), int(m.group(4)),
                             float(m.group(5)), float(m.group(6)), float(m.group(7))))
    return rows


def test_launch_table_and_rule_agree_where_both_apply():
    """The generated table of measured 1x1 kernel choices (the counterpart of the paper's work-group table,
    Section 4) is consulted before the selection rule.  Where a shape is in the table, either both name the same
    kernel, or the table's own measurements show the rule's kernel more than 3 % slower - and the executable
    follows the table.  Shapes outside the table take the rule."""
    rows = _launch_table()
    assert len(rows) >= 60
    col = {4: 4, 10: 5, 16: 6}  # kernel id -> column of its time
    overrides = 0
    for px, cin, cout, kern, *ms in rows:
        # a square plane with that many stored pixels at one of the tuned batches
        shape = None
        for b in (256, 64, 16):
            if px % b:
                continue
            for hw in (7, 14, 28, 56, 112, 33, 65, 129, 257):
                if (hw * hw + 1) // 2 * 2 == px // b:
                    shape = (b, hw)
        assert shape, (px, cin, cout)
        spec = wl.single_pointwise(shape[0], shape[1], cin, cout)
        pick = {}
        for mode in (api.GI_PW_AUTO, api.GI_PW_RULE):
            g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
            pick[mode] = g.compile(pointwise=mode).ops()[0].kernel
        assert pick[api.GI_PW_AUTO] == kern, (px, cin, cout)
        if pick[api.GI_PW_RULE] != kern:
            overrides += 1
            row = (px, cin, cout, kern) + tuple(ms)
            t_table, t_rule = row[col[kern]], row[col[pick[api.GI_PW_RULE]]]
            assert t_table > 0 and t_rule > 1.03 * t_table, (px, cin, cout, t_table, t_rule)
    assert overrides <= len(rows) // 10  # the rule was distilled from these measurements: it rarely loses
    # a shape that is not in the table takes the rule
    spec = wl.single_pointwise(3, 10, 40, 72)
    kernels = []
    for mode in (api.GI_PW_AUTO, api.GI_PW_RULE):
        g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
        kernels.append(g.compile(pointwise=mode).ops()[0].kernel)
    assert kernels[0] == kernels[1]


def test_depthwise_staging_table_is_sane_and_compiles():
    """The generated table of staging sizes for the depthwise stencil: an entry keeps the kernel's defaults (0, 0) unless
    its own measurements show another setting more than 3 % faster, every size is one the tuner tries, and every shape in
    it still compiles to the staged kernel (a setting the kernel cannot run falls back to the defaults)."""
    import re
    path = os.path.join(ROOT, "paper_1907_01989_b200", "csrc", "dw_table.inc")
    rows = [tuple(float(v.rstrip("f")) for v in m.group(1).split(",")) for m in re.finditer(r"^\{([^}]*)\},", open(path).read(), re.M)]
    assert len(rows) >= 30
    for b, h, w, c, stride, buf_kb, cta_kb, t0, t1 in rows:
        assert buf_kb in (0, 16, 24, 36, 48, 64) and cta_kb in (0, 56, 75, 110)
        assert (buf_kb, cta_kb) == (0, 0) or t1 * 1.03 < t0
        assert t1 <= t0
    for b, h, w, c, stride, *_ in rows[:12]:
        spec = wl.single_depthwise(int(b), int(h), int(c), int(stride), 1)
        g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
        assert [api.KERNEL_NAMES[o.kernel] for o in g.compile().ops()] == ["depthwise"]
    # the override used by the tuner: sizes from the environment at compile time, nonsense falls back to the defaults
    os.environ["GI_DW_BUF_KB"], os.environ["GI_DW_CTA_KB"] = "1", "1"
    try:
        g, _ = api.graph_from_spec(wl.single_depthwise(4, 56, 32, 1, 1), api.GI_F16, io_layout=api.GI_PHWC4)
        assert [api.KERNEL_NAMES[o.kernel] for o in g.compile().ops()] == ["depthwise"]
    finally:
        del os.environ["GI_DW_BUF_KB"], os.environ["GI_DW_CTA_KB"]



# ---------------------------------------------------------------------- layout experiment: host side
def test_slice8_host_side():
    """The host half of gi_slice8_pointwise_*: tensor sizes, argument checks, and where the packed weights of the
    CTA-pair kernel put each value (the first CTA of a pair gets the first half of a tile's output channels)."""
    import ctypes as C
    # [ceil(C/8)][batch][plane rounded up to even][8] halves
    assert api.gi_slice8_tensor_bytes(3, 7, 7, 20) == 3 * 3 * 50 * 16
    assert api.gi_slice8_tensor_bytes(1, 2, 2, 8) == 1 * 1 * 4 * 16
    assert api.gi_slice8_tensor_bytes(0, 2, 2, 8) == 0
    rng = np.random.default_rng(11)
    cin, cout = 72, 40  # two K chunks of 64 channels (the second one ragged), one output tile of 48 rows (two halves of 24)
    w = (rng.integers(-64, 64, size=(cout, cin)) / 64.0).astype(np.float32)  # exactly representable in fp16
    bias = rng.standard_normal(cout).astype(np.float32)
    blob = api.gi_slice8_pointwise_pack(w, bias)
    n_tile, half_rows, n_chunks = 48, 24, 2
    b_bytes = half_rows * 64 * 2
    assert blob.size == (n_chunks * 2 * b_bytes + 255) // 256 * 256 + n_tile * 4
    halves = blob[: n_chunks * 2 * b_bytes].view(np.float16).astype(np.float32).reshape(n_chunks, 2, 8, half_rows, 8)
    want = np.zeros((n_chunks, 2, 8, half_rows, 8), dtype=np.float32)
    for co in range(cout):
        for ci in range(cin):
            want[ci // 64, co // half_rows, (ci % 64) // 8, co % half_rows, ci % 8] = w[co, ci]
    assert np.array_equal(halves, want)
    off = (n_chunks * 2 * b_bytes + 255) // 256 * 256
    assert np.array_equal(blob[off: off + cout * 4].view(np.float32), bias)
    assert not blob[off + cout * 4:].any()
    # argument checks need no device
    L = api.lib()
    n = C.c_uint64(0)
    assert L.gi_slice8_pointwise_blob_bytes(0, 8, C.byref(n)) == api.GI_E_INVALID
    assert L.gi_slice8_pointwise_blob_bytes(8, 8, None) == api.GI_E_INVALID
    assert L.gi_slice8_pointwise_pack(None, None, 8, 8, None, 0) == api.GI_E_INVALID
    small = np.zeros(16, dtype=np.uint8)
    assert L.gi_slice8_pointwise_pack(w.ctypes.data, bias.ctypes.data, cin, cout, small.ctypes.data, small.size) == api.GI_E_INVALID
    assert L.gi_slice8_pointwise_run(None, None, None, 1, 2, 2, 8, 8, 0, None) == api.GI_E_INVALID
    assert L.gi_slice8_pointwise_run(16, 32, 256, 1, 2, 2, 8, 8, 7, None) == api.GI_E_INVALID   # unknown activation
    assert L.gi_slice8_pointwise_run(16, 40, 256, 1, 2, 2, 8, 8, 0, None) == api.GI_E_INVALID   # output not 16-byte aligned
    assert L.gi_slice8_pointwise_run(16, 32, 128, 1, 2, 2, 8, 8, 0, None) == api.GI_E_INVALID   # blob not 256-byte aligned
