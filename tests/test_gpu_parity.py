"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Tolerances: fp16 storage |gpu-oracle| <= 1e-2 + 1e-2*|oracle|; fp32 storage
<= 1e-4 + 1e-4*|oracle| (element-wise)."""
import numpy as np
import pytest

from oracle import graph as og
from oracle import ops as oops
from paper_1907_01989_b200 import api
from paper_1907_01989_b200 import workloads as wl

from gpu_util import DeviceRun, assert_close

pytestmark = pytest.mark.gpu

STORAGES = [api.GI_F16, api.GI_F32]
SNAME = {api.GI_F16: "f16", api.GI_F32: "f32"}


def check_all_tensors(spec, storage, pointwise=api.GI_PW_AUTO, fuse=True, cross_op=api.GI_XOP_AUTO):
    """Naive planner keeps every intermediate, so each stored tensor is compared, not only the output."""
    xs = [wl.make_input(spec, index=i) for i in range(len(spec.inputs))]
    ref = og.run(spec, xs, storage=SNAME[storage], fused=fuse, keep_all=True)
    run = DeviceRun(spec, storage, planner=api.GI_PLAN_NAIVE, pointwise=pointwise, fuse=fuse, guard_bytes=4096, cross_op=cross_op)
    outs = run.run(xs)
    assert run.guard_intact()
    worst = 0.0
    for t, r in ref.items():
        if t in run.on_chip:  # never stored: covered through the tensor computed from it
            continue
        got = outs[t] if t in outs else run.fetch(t)
        worst = max(worst, assert_close(got, r, storage, f"{spec.name} tensor {t}"))
    return worst


def check_outputs(spec, storage, images=None, **kw):
    xs = [wl.make_input(spec, index=i) for i in range(len(spec.inputs))]
    run = DeviceRun(spec, storage, guard_bytes=4096, **kw)
    outs = run.run(xs)
    assert run.guard_intact()
    sel = list(range(spec.batch)) if images is None else images
    ref = og.run(spec, [x[sel] for x in xs], storage=SNAME[storage], fused=True)
    for t in spec.outputs:
        assert_close(outs[t][sel], ref[t], storage, f"{spec.name} output {t}")
    return run, xs, outs


# ---------------------------------------------------------------------- config 1
@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("pointwise", [api.GI_PW_AUTO, api.GI_PW_SIMT])
def test_separable_block(storage, pointwise):
    check_all_tensors(wl.separable_block(1), storage, pointwise)
    check_all_tensors(wl.separable_block(3, 9, 7, 10, 22), storage, pointwise)  # ragged: odd plane, C % 4 != 0


@pytest.mark.parametrize("planner", [api.GI_PLAN_GREEDY_BY_SIZE, api.GI_PLAN_GREEDY_SHARED_OBJECTS, api.GI_PLAN_NAIVE,
                                     api.GI_PLAN_MIN_COST_FLOW])
def test_planners_give_same_result(planner):
    spec = wl.mobilenet_v2(2, size=64)
    run, xs, outs = check_outputs(spec, api.GI_F16, planner=planner)
    base = DeviceRun(spec, api.GI_F16, planner=api.GI_PLAN_NAIVE).run(xs)
    for t in spec.outputs:
        assert np.array_equal(outs[t], base[t])


# ---------------------------------------------------------------------- layout
@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("shape", [(1, 8, 6, 12), (2, 7, 7, 5), (3, 1, 1, 1001), (2, 5, 3, 3)])
def test_pack_layout_bit_exact(storage, shape):
    B, H, W, Cc = shape
    b = wl.GraphBuilder("layout", B, 50)
    x = b.input(H, W, Cc)
    b.output(b.activation(x, wl.ACT_RELU))
    spec = b.finish()
    xin = wl.make_input(spec)
    run = DeviceRun(spec, storage, planner=api.GI_PLAN_NAIVE)
    outs = run.run([xin])
    phys = oops.phwc4_pack(xin).reshape(-1)
    got = run.fetch_raw(spec.inputs[0]).astype(np.float32)
    assert np.array_equal(got[: phys.size], phys)  # includes zero pad lanes and the zero pad pixel
    assert np.array_equal(outs[spec.outputs[0]], np.maximum(xin, 0))


# ---------------------------------------------------------------------- single operators
PW_CASES = [  # batch, hw, cin, cout, residual, act
    (1, 7, 32, 64, False, wl.ACT_RELU6), (2, 7, 96, 24, True, wl.ACT_NONE), (3, 14, 144, 32, True, wl.ACT_NONE),
    (1, 28, 16, 96, False, wl.ACT_RELU6), (2, 9, 10, 22, False, wl.ACT_RELU), (1, 33, 320, 256, False, wl.ACT_RELU),
    (2, 5, 256, 21, False, wl.ACT_NONE), (4, 1, 1280, 1001, False, wl.ACT_NONE), (1, 56, 24, 144, False, wl.ACT_RELU6),
    (1, 14, 576, 160, False, wl.ACT_NONE), (5, 7, 960, 320, False, wl.ACT_NONE), (1, 20, 3, 5, True, wl.ACT_RELU6),
]


@pytest.mark.parametrize("case", PW_CASES)
def test_pointwise_fp32(case):
    batch, hw, cin, cout, residual, act = case
    spec = wl.single_pointwise(batch, hw, cin, cout, residual, act)
    check_all_tensors(spec, api.GI_F32)
    kernels = [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, api.GI_F32)[0].compile().ops()]
    assert "conv_simt" in kernels  # fp32 storage always takes the CUDA-core kernel


@pytest.mark.parametrize("mode,kernel", [(api.GI_PW_TC_PAIR, "pointwise_tc"), (api.GI_PW_TC_LANE, "pointwise_ts"),
                                         (api.GI_PW_TC_WIDE, "pointwise_mm")],
                         ids=["pair", "lane", "wide"])
@pytest.mark.parametrize("case", PW_CASES)
def test_pointwise_tensor_core(case, mode, kernel):
    """Both tensor-core variants on every case: operands by TMA (pixel pairs) and through tensor memory."""
    batch, hw, cin, cout, residual, act = case
    spec = wl.single_pointwise(batch, hw, cin, cout, residual, act)
    check_all_tensors(spec, api.GI_F16, pointwise=mode)
    kernels = [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, api.GI_F16)[0].compile(pointwise=mode).ops()]
    assert kernel in kernels
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("case", PW_CASES[:6])
def test_pointwise_simt_fp16(case):
    batch, hw, cin, cout, residual, act = case
    check_all_tensors(wl.single_pointwise(batch, hw, cin, cout, residual, act), api.GI_F16, pointwise=api.GI_PW_SIMT)


DW_CASES = [  # batch, hw, c, stride, dilation, residual
    (1, 7, 32, 1, 1, False), (2, 14, 96, 2, 1, False), (1, 33, 24, 1, 2, False), (1, 33, 8, 1, 4, True),
    (3, 9, 10, 2, 1, False), (1, 56, 144, 1, 1, True), (2, 112, 32, 2, 1, False), (1, 65, 12, 2, 1, False),
    (2, 3, 5, 1, 1, False), (1, 1, 7, 1, 1, False), (2, 2, 4, 2, 1, False),
    # dilated: even and odd planes, classes of unequal length, several planes per work item, a dilation larger than the plane
    (5, 20, 40, 1, 2, False), (3, 20, 12, 1, 4, True), (2, 10, 8, 1, 3, False), (2, 5, 4, 1, 4, False), (1, 3, 8, 1, 4, False),
    (16, 33, 96, 1, 2, False),
]


@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("case", DW_CASES)
def test_depthwise(storage, case):
    batch, hw, c, stride, dilation, residual = case
    check_all_tensors(wl.single_depthwise(batch, hw, c, stride, dilation, residual), storage)


def depthwise_spec(batch, h, w, c, stride, residual, act=wl.ACT_RELU6):
    b = wl.GraphBuilder(f"dwtc_{batch}x{h}x{w}x{c}_s{stride}", batch, 8)
    x = b.input(h, w, c)
    r = b.input(wl.same_pads(h, 3, stride, 1)[0], wl.same_pads(w, 3, stride, 1)[0], c) if residual else None
    y = b.depthwise(x, 3, stride, 1)
    if act is not None:
        y = b.activation(y, act)
    if residual:
        y = b.add(r, y)
    b.output(y)
    return b.finish()


EVEN_DW_CASES = [  # batch, H, W, C, stride, residual: even and non-square planes, many small planes per item
    (1, 14, 14, 32, 1, False), (3, 14, 14, 20, 1, False), (2, 28, 28, 192, 1, True), (1, 56, 56, 24, 1, False),
    (2, 112, 112, 8, 1, False), (5, 14, 14, 8, 1, False), (40, 4, 4, 8, 1, False), (1, 2, 2, 4, 1, False),
    (1, 20, 36, 12, 1, False), (1, 6, 252, 4, 1, True), (2, 14, 14, 96, 2, False), (2, 112, 112, 32, 2, False),
    (1, 56, 56, 144, 2, True), (2, 36, 20, 12, 2, False), (2, 2, 2, 4, 2, False), (37, 8, 8, 4, 2, False),
    (1, 64, 64, 8, 1, False), (2, 60, 128, 8, 2, False),
    # wide planes, stride 1: two output columns per thread
    (3, 40, 96, 8, 1, True), (1, 33, 130, 12, 1, False), (2, 100, 200, 4, 1, False), (5, 7, 128, 8, 1, True),
    (1, 1, 96, 4, 1, False), (2, 3, 254, 4, 1, True),
]


@pytest.mark.parametrize("case", EVEN_DW_CASES)
def test_depthwise_even_and_non_square_planes(case):
    batch, h, w, c, stride, residual = case
    check_all_tensors(depthwise_spec(batch, h, w, c, stride, residual), api.GI_F16)
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("act", [None, wl.ACT_RELU])
def test_depthwise_other_tails(act):
    check_all_tensors(depthwise_spec(2, 28, 28, 12, 1, False, act), api.GI_F16)
    check_all_tensors(depthwise_spec(2, 28, 28, 12, 2, True, act), api.GI_F16)
    check_all_tensors(depthwise_spec(2, 20, 112, 8, 1, False, act), api.GI_F16)
    check_all_tensors(depthwise_spec(1, 20, 112, 8, 1, True, act), api.GI_F16)
    assert api.gi_device_status() == 0


def depthwise_pointwise_spec(batch, h, w, c, cout, stride, residual, dw_act=wl.ACT_RELU6, pw_act=None, post_act=None):
    return wl.depthwise_then_pointwise(batch, h, w, c, cout, stride, residual, dw_act, pw_act, post_act)


DWPW_CASES = [  # batch, H, W, C, Cout, stride, residual
    (1, 32, 32, 32, 64, 1, False), (2, 112, 112, 32, 16, 1, False), (2, 56, 56, 144, 24, 1, True), (3, 28, 28, 192, 32, 1, True),
    (5, 14, 14, 384, 64, 1, True), (3, 14, 14, 576, 96, 1, False), (2, 112, 112, 96, 24, 2, False), (2, 56, 56, 144, 32, 2, False),
    (3, 28, 28, 192, 64, 2, False), (7, 7, 7, 64, 40, 1, True), (4, 14, 14, 48, 20, 2, False), (1, 20, 36, 16, 8, 1, False),
    (2, 60, 128, 16, 3, 2, False), (40, 4, 4, 16, 16, 1, False), (1, 2, 2, 16, 250, 1, False), (2, 9, 5, 32, 17, 2, True),
    (300, 14, 14, 32, 24, 1, False), (2, 64, 128, 16, 16, 1, False), (1200, 4, 4, 16, 16, 1, False), (1300, 6, 6, 16, 8, 2, True), (40, 56, 56, 16, 8, 1, True), (24, 112, 112, 16, 8, 1, False),
    (40, 56, 56, 16, 24, 2, False), (150, 28, 28, 32, 40, 1, True),
]


@pytest.mark.parametrize("case", DWPW_CASES)
def test_depthwise_pointwise_one_kernel(case):
    """A depthwise op and the 1x1 convolution that consumes it, run by one kernel: same results as the two
    operators one after the other (the tensor between them is rounded to fp16 on chip)."""
    batch, h, w, c, cout, stride, residual = case
    spec = depthwise_pointwise_spec(batch, h, w, c, cout, stride, residual)
    graph, _ = api.graph_from_spec(spec, api.GI_F16)
    names = [api.KERNEL_NAMES[o.kernel] for o in graph.compile(cross_op=api.GI_XOP_ON, planner=api.GI_PLAN_NAIVE).ops()]
    assert "depthwise_pointwise" in names and "none" in names, names
    check_all_tensors(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("dw_act,pw_act,post_act", [(None, wl.ACT_RELU, None), (wl.ACT_RELU, wl.ACT_RELU6, wl.ACT_RELU),
                                                    (wl.ACT_RELU6, None, wl.ACT_RELU6)])
def test_depthwise_pointwise_epilogues(dw_act, pw_act, post_act):
    for stride in (1, 2):
        spec = depthwise_pointwise_spec(3, 28, 28, 32, 24, stride, True, dw_act, pw_act, post_act)
        check_all_tensors(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("case", [(1, 32, 3, 32, 2), (2, 17, 3, 32, 2), (1, 12, 8, 12, 1), (2, 9, 5, 6, 2), (3, 21, 4, 21, 1),
                                  (1, 40, 2, 200, 2), (2, 224, 3, 32, 2), (3, 14, 4, 20, 2), (2, 6, 1, 8, 2), (1, 252, 3, 16, 2),
                                  (5, 2, 3, 128, 2), (2, 64, 3, 32, 2), (1, 128, 3, 32, 2), (2, 60, 3, 32, 2)])
def test_conv3x3(storage, case):
    spec = wl.single_conv3x3(*case)
    check_all_tensors(spec, storage)
    kernels = [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, storage)[0].compile().ops()]
    # one input slice and fp16 storage: the tensor-core kernel; anything else: the CUDA-core kernel
    assert ("conv3x3_tc" in kernels) == (storage == api.GI_F16 and case[2] <= 4)
    if storage == api.GI_F16:
        check_all_tensors(spec, storage, pointwise=api.GI_PW_SIMT)
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("storage", STORAGES)
def test_standalone_elementwise_pool_resize(storage):
    b = wl.GraphBuilder("misc", 2, 51)
    x = b.input(9, 7, 10)
    a = b.activation(x, wl.ACT_RELU6)          # producer is not a convolution: standalone activation
    c = b.conv2d(a, 10, 1)
    d = b.add(c, c)                              # x + x: standalone add
    e = b.add(b.activation(b.conv2d(d, 10, 3), wl.ACT_RELU), a)  # act, add fold
    f = b.activation(e, wl.ACT_RELU6)           # second act folds too
    p = b.global_avg_pool(f)
    r = b.resize_bilinear(f, 33, 25, True)
    r2 = b.resize_bilinear(f, 5, 4, False)
    for t in (p, r, r2):
        b.output(t)
    spec = b.finish()
    check_all_tensors(spec, storage)
    check_all_tensors(spec, storage, fuse=False)


# ---------------------------------------------------------------------- whole networks, batch 1: every tensor
@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("make", [wl.mobilenet_v1, wl.mobilenet_v2], ids=["v1", "v2"])
def test_network_batch1_every_tensor(make, storage):
    check_all_tensors(make(1), storage)


@pytest.mark.parametrize("mode", [api.GI_PW_TC_PAIR, api.GI_PW_TC_LANE], ids=["pair", "lane"])
def test_network_with_one_pointwise_variant(mode):
    check_all_tensors(wl.mobilenet_v2(3, size=160), api.GI_F16, pointwise=mode)


def test_segmentation_batch1_every_tensor():
    check_all_tensors(wl.mobilenet_v2_segmentation(1), api.GI_F16)


def test_segmentation_small_fp32():
    check_all_tensors(wl.mobilenet_v2_segmentation(2, size=97), api.GI_F32)


# ---------------------------------------------------------------------- full sizes, in the benchmark's launch configuration
def test_mobilenet_v2_batch256_sampled_images():
    spec = wl.mobilenet_v2(256)
    run, xs, outs = check_outputs(spec, api.GI_F16, images=[0, 101, 255])
    # determinism: a second run gives bit-identical logits
    again = run.run(xs)
    for t in spec.outputs:
        assert np.array_equal(outs[t], again[t])
    # images are independent: the same image in another slot gives the same answer up to kernel tiling
    assert np.isfinite(outs[spec.outputs[0]]).all()


def test_mobilenet_v2_batch64_one_kernel_pairs_sampled_images():
    """With cross-operator kernels on, the blocks on 14x14 and 7x7 planes run as one kernel each and, of the remaining
    depthwise -> projection pairs, those that qualify run as one kernel per pair."""
    spec = wl.mobilenet_v2(64)
    run, xs, outs = check_outputs(spec, api.GI_F16, images=[0, 33, 63], cross_op=api.GI_XOP_ON)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert names.count("depthwise_pointwise") >= 4 and names.count("inverted_residual") >= 8, names
    again = run.run(xs)
    for t in spec.outputs:
        assert np.array_equal(outs[t], again[t])
    assert api.gi_device_status() == 0


def test_mobilenet_v1_batch256_sampled_images():
    check_outputs(wl.mobilenet_v1(256), api.GI_F16, images=[0, 77, 255])


def test_segmentation_batch16_sampled_images():
    check_outputs(wl.mobilenet_v2_segmentation(16), api.GI_F16, images=[0, 15])


# ---------------------------------------------------------------------- run-time argument checks
def test_run_argument_checks():
    import torch
    spec = wl.separable_block(1)
    run = DeviceRun(spec, api.GI_F16)
    x = torch.zeros((1, 32, 32, 32), dtype=torch.float16, device="cuda:0")
    out = run.outs[0]
    nb = int(run.ex.info.arena_bytes)
    with pytest.raises(api.GiError) as ei:
        run.ex.run_raw([x.data_ptr()], [out.data_ptr()], run.arena.data_ptr(), nb - 1)
    assert ei.value.status == api.GI_E_ARENA
    with pytest.raises(api.GiError) as ei:
        run.ex.run_raw([x.data_ptr()], [out.data_ptr()], run.arena.data_ptr() + 8, nb)
    assert ei.value.status == api.GI_E_ARENA
    with pytest.raises(api.GiError) as ei:
        run.ex.run_raw([0], [out.data_ptr()], run.arena.data_ptr(), nb)
    assert ei.value.status == api.GI_E_INVALID
    g2, _ = api.graph_from_spec(spec)
    ex2 = g2.compile()
    with pytest.raises(api.GiError) as ei:
        ex2.run_raw([x.data_ptr()], [out.data_ptr()], run.arena.data_ptr(), nb)
    assert ei.value.status == api.GI_E_STATE
    # the context is still healthy
    run.ex.run_raw([x.data_ptr()], [out.data_ptr()], run.arena.data_ptr(), nb)
    torch.cuda.synchronize()


def test_phwc4_io_layout_skips_conversions():
    import torch
    spec = wl.separable_block(2, 9, 7, 12, 20)
    xin = wl.make_input(spec)
    g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
    ex = g.compile()
    assert ex.info.n_ops == ex.info.n_fused_ops == 2
    ex.bind()
    x = torch.from_numpy(oops.phwc4_pack(xin)).to("cuda:0").half().contiguous()
    H, W, Cc = spec.shapes[spec.outputs[0]]
    out = torch.zeros(api.gi_tensor_bytes(2, H, W, Cc) // 2, dtype=torch.float16, device="cuda:0")
    ex.run([x], [out])
    torch.cuda.synchronize()
    ref = og.run(spec, [xin], storage="f16")[spec.outputs[0]]
    got = oops.phwc4_unpack(out.float().cpu().numpy(), 2, H, W, Cc)
    assert_close(got, ref, api.GI_F16, "phwc4 io")


@pytest.mark.gpu
@pytest.mark.parametrize("graphs", [False, True], ids=["launches", "cuda_graphs"])
def test_host_pipeline_matches_plain_runs(graphs):
    """Batches submitted through the two-slot host pipeline come back in order and equal to plain runs."""
    import torch
    from paper_1907_01989_b200.pipeline import HostPipeline
    spec = wl.mobilenet_v2(2, 96)
    g, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = g.compile()
    ex.bind("cuda:0")
    shape_in = (spec.batch,) + tuple(spec.shapes[spec.inputs[0]])
    shape_out = (spec.batch,) + tuple(spec.shapes[spec.outputs[0]])
    xs = [torch.from_numpy(wl.make_input(spec) * (0.5 + 0.25 * i)).half().pin_memory() for i in range(5)]
    want = []
    for x in xs:
        out = torch.empty(shape_out, dtype=torch.float16, device="cuda:0")
        ex.run([x.to("cuda:0")], [out])
        torch.cuda.synchronize()
        want.append(out.cpu())
    pipe = HostPipeline(ex, [shape_in], [shape_out], torch.float16, "cuda:0", graphs=graphs)
    assert len(pipe.graphs) == (2 if graphs else 0)
    got = [torch.empty(shape_out, dtype=torch.float16).pin_memory() for _ in xs]
    for x, o in zip(xs, got):
        pipe.submit([x], [o])
    pipe.synchronize()
    for w, o in zip(want, got):
        assert torch.equal(w, o)
    assert len({float(w.float().abs().sum()) for w in want}) == len(want)  # the batches really differ


@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("case", [(3, 3, 200, 150, True), (3, 3, 200, 150, False), (9, 7, 1, 1, True), (9, 7, 9, 7, True),
                                  (17, 5, 4, 40, False), (2, 33, 65, 513, True)])
def test_resize_shapes(storage, case):
    """Row intervals longer than one chunk of weights, a single output row, identity, mixed up / down scaling."""
    h, w, oh, ow, align = case
    b = wl.GraphBuilder(f"resize_{h}x{w}_{oh}x{ow}_{int(align)}", 2, 52)
    x = b.input(h, w, 6)
    b.output(b.resize_bilinear(b.conv2d(x, 6, 1), oh, ow, align))
    check_all_tensors(b.finish(), storage)


# ---------------------------------------------------------------------- random graphs
def _random_spec(rnd, n_ops):
    """Random DAG of all operator kinds on small, ragged shapes (odd planes, C % 4 != 0)."""
    b = wl.GraphBuilder("random_gpu", rnd.choice([1, 2, 5]), 98)
    live = [b.input(rnd.choice([5, 8, 9, 16]), rnd.choice([4, 7, 8, 18]), rnd.choice([3, 4, 6, 8, 20]))]
    for _ in range(n_ops):
        x = rnd.choice(live[-4:])
        kind = rnd.choice(["conv1", "conv1", "conv3", "dw", "dw", "act", "add", "pool", "resize", "conv2", "concat", "concat", "ident"])
        H, W, Cc = b.g.shapes[x]
        if kind == "conv1":
            y = b.conv2d(x, rnd.choice([4, 6, 8, 24, Cc]), 1)
        elif kind == "conv3":
            y = b.conv2d(x, rnd.choice([4, 8, Cc]), 3, rnd.choice([1, 2]))
        elif kind == "dw":
            y = b.depthwise(x, 3, rnd.choice([1, 2]), rnd.choice([1, 1, 2]))
        elif kind == "act":
            y = b.activation(x, rnd.choice([wl.ACT_RELU, wl.ACT_RELU6]))
        elif kind == "add":
            same = [t for t in live if b.g.shapes[t] == b.g.shapes[x]]
            y = b.add(rnd.choice(same), x)
        elif kind == "conv2":
            y = b.conv2d(x, rnd.choice([4, 5, 8, 24]), rnd.choice([2, 3]), rnd.choice([1, 2, 3]))
        elif kind == "concat":
            same = [t for t in live if b.g.shapes[t][:2] == b.g.shapes[x][:2]]
            y = b.concat(rnd.choice(same), x)
        elif kind == "ident":
            y = b.identity_add(x) if rnd.random() < 0.5 else b.concat(x)
        elif kind == "pool":
            if H * W == 1:
                continue
            y = b.global_avg_pool(x)
        else:
            y = b.resize_bilinear(x, rnd.choice([1, 3, H, 2 * H + 1]), rnd.choice([2, W, 3 * W]), rnd.choice([True, False]))
        live.append(y)
    used = {t for op in b.g.ops for t in op.inputs}
    outs = [t for t in live[1:] if t not in used] or [live[-1]]
    for t in outs:
        if t != live[0]:
            b.output(t)
    if not b.g.outputs:
        b.output(b.activation(live[0], wl.ACT_RELU))
    return b.finish()


@pytest.mark.parametrize("seed", range(24))
def test_random_graphs(seed):
    """Every stored tensor of a random graph against the oracle, fp16 (tensor-core kernels) and fp32, fused."""
    import random
    rnd = random.Random(1000 + seed)
    spec = _random_spec(rnd, rnd.randint(3, 14))
    check_all_tensors(spec, api.GI_F16)  # small launches: every 1x1 takes the lane-per-pixel kernel
    check_all_tensors(spec, api.GI_F16, pointwise=api.GI_PW_TC_PAIR)
    check_all_tensors(spec, api.GI_F32)
    check_outputs(spec, api.GI_F16)  # greedy-by-size arena: tensors share memory
    # depthwise -> 1x1 pairs as one kernel wherever the pattern occurs (the tensor in between is not stored)
    check_all_tensors(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    assert api.gi_device_status() == 0


def test_identity_resize_removed():
    """A resize to the input's own size is dropped at compile time (Section 3.1); results are those of the oracle,
    whose own clean-up is pinned to change nothing."""
    b = wl.GraphBuilder("identity_ops", 3, 21)
    x = b.input(10, 6, 8)
    c = b.conv2d(x, 12, 1)
    a = b.activation(b.resize_bilinear(c, 10, 6, True), wl.ACT_RELU6)
    r2 = b.resize_bilinear(a, 10, 6, False)
    b.output(r2)
    b.output(b.resize_bilinear(b.depthwise(r2, 3, 1, 1), 20, 12, True))
    spec = b.finish()
    for storage in STORAGES:
        check_all_tensors(spec, storage)
        check_outputs(spec, storage)


# ---------------------------------------------------------------------- second workload: CONCAT, 2x2 kernels, stride 3
CONCAT_CASES = [  # batch, H, W, Ca, Cb: whole slices, ragged first input, ragged second input, odd planes, one channel each
    (2, 8, 8, 8, 8), (3, 7, 5, 4, 6), (2, 9, 9, 6, 8), (1, 5, 3, 3, 3), (4, 1, 1, 1, 1), (2, 14, 14, 96, 32), (1, 33, 31, 5, 11),
    (2, 6, 6, 7, 1), (300, 3, 3, 2, 9),
]


@pytest.mark.gpu
@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("case", CONCAT_CASES)
def test_concat_bit_exact(storage, case):
    """CONCAT moves values without arithmetic: the result is the oracle's, bit for bit, and lanes beyond the last
    channel and the padding pixel of an odd plane are zero in memory."""
    spec = wl.single_concat(*case)
    xs = [wl.make_input(spec, index=i) for i in range(2)]
    ref = og.run(spec, xs, storage=SNAME[storage])[spec.outputs[0]]
    run = DeviceRun(spec, storage, guard_bytes=4096)
    got = run.run(xs)[spec.outputs[0]]
    assert run.guard_intact()
    assert np.array_equal(got, ref)
    assert "concat" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    # the stored PHWC4 tensor (the unpack kernel reads it from the arena): padding is zero
    t = spec.outputs[0]
    B, H, W, Cc = (case[0], case[1], case[2], case[3] + case[4])
    S, P = (Cc + 3) // 4, (H * W + 1) // 2 * 2
    raw = run.fetch_raw(t)[: S * B * P * 4].reshape(S, B, P, 4).astype(np.float32)
    assert not raw[:, :, H * W:, :].any()
    if Cc % 4:
        assert not raw[S - 1, :, :, Cc % 4:].any()
    assert api.gi_device_status() == 0


CONV_K_S_CASES = [  # batch, H, W, Cin, Cout, k, stride
    (2, 8, 8, 3, 8, 2, 1), (2, 9, 7, 5, 6, 2, 2), (1, 16, 16, 8, 24, 2, 3), (3, 10, 11, 4, 5, 3, 3), (2, 7, 7, 6, 4, 1, 3),
    (1, 96, 96, 3, 24, 2, 2), (2, 24, 24, 32, 48, 3, 3), (2, 5, 5, 12, 40, 2, 1), (1, 1, 1, 4, 4, 2, 3),
]


@pytest.mark.gpu
@pytest.mark.parametrize("storage", STORAGES)
@pytest.mark.parametrize("case", CONV_K_S_CASES)
def test_conv_2x2_and_stride_3(storage, case):
    """Kernel sizes and strides of the paper's search space that the MobileNets do not use (Section 4)."""
    spec = wl.single_conv(*case)
    check_all_tensors(spec, storage)
    check_all_tensors(spec, storage, fuse=False)
    assert api.gi_device_status() == 0


@pytest.mark.gpu
@pytest.mark.parametrize("storage", STORAGES)
def test_fire_network_every_tensor(storage):
    for spec in (wl.fire_network(2), wl.fire_network(3, size=77)):
        check_all_tensors(spec, storage)
        for planner in (api.GI_PLAN_GREEDY_BY_SIZE, api.GI_PLAN_GREEDY_SHARED_OBJECTS, api.GI_PLAN_MIN_COST_FLOW):
            check_outputs(spec, storage, planner=planner)
    check_all_tensors(wl.fire_network(2), storage, fuse=False)
    assert api.gi_device_status() == 0


@pytest.mark.gpu
def test_fire_network_batch64_sampled_images():
    spec = wl.fire_network(64, size=192)
    check_outputs(spec, api.GI_F16, images=[0, 31, 63])
    assert api.gi_device_status() == 0


@pytest.mark.gpu
def test_single_input_add_and_concat():
    """Removed at compile time unless they are graph outputs, where they run as copies (Section 3.1)."""
    b = wl.GraphBuilder("ident_gpu", 3, 22)
    x = b.input(7, 5, 6)
    y = b.activation(b.conv2d(x, 10, 1), wl.ACT_RELU)
    z = b.concat(b.identity_add(y))
    out1 = b.activation(b.conv2d(z, 6, 3), wl.ACT_RELU6)
    b.output(b.concat(out1))
    b.output(b.identity_add(out1))
    spec = b.finish()
    for storage in STORAGES:
        run, xs, outs = check_outputs(spec, storage)
        names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
        assert names.count("eltwise") == 2 and "concat" not in names
        check_all_tensors(spec, storage)


CONV_TC_CASES = [  # batch, H, W, Cin, Cout, k, stride, dilation, residual, act, post_act
    (2, 12, 12, 8, 16, 3, 1, 1, False, wl.ACT_RELU, None),        # 5 chunks of 16 pixel-slices, the last one ragged
    (3, 9, 7, 5, 6, 3, 2, 1, False, wl.ACT_RELU6, None),          # ragged channels both sides, odd planes
    (2, 24, 24, 48, 64, 3, 1, 1, True, wl.ACT_NONE, wl.ACT_RELU),  # 7 chunks, residual then activation
    (1, 20, 20, 64, 64, 3, 1, 2, False, wl.ACT_RELU, None),       # dilation 2, 9 chunks
    (2, 16, 16, 16, 256, 3, 2, 1, False, wl.ACT_RELU6, None),     # all 512 accumulator columns
    (2, 17, 15, 32, 48, 3, 3, 1, False, wl.ACT_RELU, None),       # stride 3
    (2, 16, 16, 24, 40, 2, 2, 1, True, wl.ACT_RELU, wl.ACT_RELU6),  # 2x2
    (4, 14, 14, 96, 24, 1, 2, 1, False, wl.ACT_NONE, None),       # strided 1x1
    (70, 9, 9, 12, 20, 3, 1, 1, False, wl.ACT_RELU, None),        # many tiles: every CTA walks several
    (1, 3, 3, 6, 4, 3, 1, 1, False, wl.ACT_NONE, None),           # a single, mostly empty tile
]


@pytest.mark.parametrize("case", CONV_TC_CASES)
def test_conv_kxk_tensor_core(case):
    B, H, W, cin, cout, k, stride, dil, residual, act, post = case
    b = wl.GraphBuilder(f"convtc_{B}x{H}x{W}x{cin}x{cout}_k{k}s{stride}d{dil}", B, 13)
    x = b.input(H, W, cin)
    r = b.input(wl.same_pads(H, k, stride, dil)[0], wl.same_pads(W, k, stride, dil)[0], cout) if residual else None
    y = b.conv2d(x, cout, k, stride, dil)
    if act != wl.ACT_NONE:
        y = b.activation(y, act)
    if residual:
        y = b.add(r, y)
    if post is not None:
        y = b.activation(y, post)
    b.output(y)
    spec = b.finish()
    run = DeviceRun(spec, api.GI_F16)
    assert [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()].count("conv_tc") == 1
    check_all_tensors(spec, api.GI_F16)
    check_outputs(spec, api.GI_F16)
    check_all_tensors(spec, api.GI_F16, pointwise=api.GI_PW_SIMT)  # same graph on the CUDA-core kernel
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("case", [(2, 14, 14, 96, 96, 3, 2), (1, 9, 9, 128, 144, 3, 1), (1, 6, 6, 256, 256, 3, 1), (3, 5, 5, 8, 300, 2, 1)])
def test_conv_kxk_output_channels_split_over_cta_groups(case):
    """Weights beyond the shared-memory budget (or more than 256 output channels): each CTA group computes a range
    of output channels."""
    spec = wl.single_conv(*case)
    run = DeviceRun(spec, api.GI_F16)
    assert "conv_tc" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    check_all_tensors(spec, api.GI_F16)
    assert api.gi_device_status() == 0


def test_conv_kxk_weights_far_too_large_take_the_cuda_core_kernel():
    spec = wl.single_conv(1, 4, 4, 512, 512, 3, 1)
    run = DeviceRun(spec, api.GI_F16)
    assert "conv_simt" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    check_all_tensors(spec, api.GI_F16)


def _names(spec, **kw):
    return [api.KERNEL_NAMES[o.kernel] for o in api.graph_from_spec(spec, api.GI_F16)[0].compile(**kw).ops()]


@pytest.mark.parametrize("case", [(2, 32, 48, 16), (1, 224, 224, 32), (3, 6, 2, 24), (2, 2, 2, 8), (5, 62, 30, 40), (1, 130, 258, 16)])
def test_stem_reads_nhwc_input_itself(case):
    """3-channel NHWC fp16 input, 3x3 stride-2 convolution, even H and W: the layout conversion launches nothing and
    the convolution gathers from the caller's tensor; results are those of the oracle (which knows no layouts)."""
    B, H, W, cout = case
    b = wl.GraphBuilder(f"stem_nhwc_{B}x{H}x{W}x{cout}", B, 14)
    x = b.input(H, W, 3)
    y = b.activation(b.conv2d(x, cout, 3, 2), wl.ACT_RELU6)
    b.output(b.activation(b.depthwise(y, 3, 1), wl.ACT_RELU))
    spec = b.finish()
    assert _names(spec)[:2] == ["none", "conv3x3_tc"]
    assert _names(spec, fuse=False)[0] == "pack"
    check_all_tensors(spec, api.GI_F16)
    check_outputs(spec, api.GI_F16)
    assert api.gi_device_status() == 0


def test_stem_keeps_the_layout_conversion_where_it_must():
    def first_two(build, B=2):
        b = wl.GraphBuilder("stem_pack", B, 15)
        build(b)
        spec = b.finish()
        check_all_tensors(spec, api.GI_F16)
        return _names(spec)[:2]

    def odd(b):
        b.output(b.activation(b.conv2d(b.input(33, 32, 3), 16, 3, 2), wl.ACT_RELU6))
    assert first_two(odd) == ["pack", "conv3x3_tc"]

    def stride1(b):
        b.output(b.activation(b.conv2d(b.input(32, 32, 3), 16, 3, 1), wl.ACT_RELU6))
    assert first_two(stride1) == ["pack", "conv3x3_tc"]

    def four_channels(b):
        b.output(b.activation(b.conv2d(b.input(32, 32, 4), 16, 3, 2), wl.ACT_RELU6))
    assert first_two(four_channels) == ["pack", "conv3x3_tc"]

    def second_reader(b):
        x = b.input(32, 32, 3)
        b.output(b.activation(b.conv2d(x, 16, 3, 2), wl.ACT_RELU6))
        b.output(b.activation(b.depthwise(x, 3, 2), wl.ACT_RELU6))
    assert first_two(second_reader) == ["pack", "conv3x3_tc"]
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("cross_op", [api.GI_XOP_OFF, api.GI_XOP_ON])
def test_fire_network_with_caller_owned_phwc4_buffers(cross_op):
    """PHWC4 input and output (no layout conversions): the first convolution reads the caller's buffer, the
    copy-free concatenations still apply (they are interior), the result is the oracle's."""
    import torch
    spec = wl.fire_network(3, size=64)
    xin = wl.make_input(spec)
    g, _ = api.graph_from_spec(spec, api.GI_F16, io_layout=api.GI_PHWC4)
    ex = g.compile(cross_op=cross_op)
    names = [api.KERNEL_NAMES[o.kernel] for o in ex.ops()]
    assert names.count("none") == 2 and "pack" not in names and "unpack" not in names
    ex.bind()
    x = torch.from_numpy(oops.phwc4_pack(xin)).to("cuda:0").half().contiguous()
    H, W, Cc = spec.shapes[spec.outputs[0]]
    out = torch.zeros(api.gi_tensor_bytes(3, H, W, Cc) // 2, dtype=torch.float16, device="cuda:0")
    for _ in range(2):  # a second run over the same arena gives the same answer
        ex.run([x], [out])
        torch.cuda.synchronize()
        got = oops.phwc4_unpack(out.float().cpu().numpy(), 3, H, W, Cc)
        assert_close(got, og.run(spec, [xin], storage="f16")[spec.outputs[0]], api.GI_F16, "fire network, phwc4 io")
    assert api.gi_device_status() == 0


# ---------------------------------------------------------------------- the single-operator sweep at the sizes it is timed at
# Corners of the single-operator grid that `bench.py --sweep` times: the tensor-bound 1x1 shapes (streamed weights, tens of
# K chunks, many output tiles per pixel tile), the deep and narrow 7x7 layers, the widest plane with a residual, and the
# depthwise shapes at batch 64 / 256.  Every image of the batch is drawn; three sampled images (first, middle, last: the
# last one lies in the ragged tail tile) are compared element by element with the oracle.
SWEEP_PW_CASES = [(256, 14, 576, 576, False), (256, 14, 960, 960, False), (256, 14, 1280, 1280, False), (256, 7, 960, 160, False),
                  (256, 7, 320, 1280, False), (256, 112, 16, 96, True), (64, 56, 192, 192, True), (8, 28, 384, 384, False)]
SWEEP_DW_CASES = [(256, 112, 96, 1), (256, 112, 96, 2), (256, 14, 576, 2), (64, 7, 960, 1), (256, 28, 192, 1), (64, 56, 144, 2)]


@pytest.mark.parametrize("case", SWEEP_PW_CASES, ids=lambda c: "b%d_%dx%d_%dto%d%s" % (c[0], c[1], c[1], c[2], c[3], "_res" if c[4] else ""))
def test_sweep_pointwise_points_at_full_size(case):
    b, hw, cin, cout, res = case
    spec = wl.single_pointwise(b, hw, cin, cout, residual=res)
    run, _, _ = check_outputs(spec, api.GI_F16, images=[0, b // 2 + 1, b - 1])
    assert any(api.KERNEL_NAMES[o.kernel] in ("pointwise_tc", "pointwise_ts", "pointwise_mm") for o in run.ex.ops())
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("mode", [api.GI_PW_TC_PAIR, api.GI_PW_TC_LANE, api.GI_PW_TC_WIDE], ids=["pair", "lane", "wide"])
@pytest.mark.parametrize("case", [(256, 14, 576, 576), (64, 14, 1280, 1280)], ids=["576", "1280"])
def test_sweep_tensor_bound_points_both_variants(case, mode):
    b, hw, cin, cout = case
    check_outputs(wl.single_pointwise(b, hw, cin, cout), api.GI_F16, images=[0, b - 1], pointwise=mode)


@pytest.mark.parametrize("case", SWEEP_DW_CASES, ids=lambda c: "b%d_%dx%dx%d_s%d" % (c[0], c[1], c[1], c[2], c[3]))
def test_sweep_depthwise_points_at_full_size(case):
    b, hw, c, stride = case
    spec = wl.single_depthwise(b, hw, c, stride, 1)
    run, _, _ = check_outputs(spec, api.GI_F16, images=[0, b // 2 + 1, b - 1])
    assert "depthwise" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert api.gi_device_status() == 0


# ---------------------------------------------------------------------- one executable, several host threads / several arenas
def test_two_threads_run_one_executable_with_their_own_arenas():
    """gi_run may be called on one executable from several host threads as long as the runs use different arenas
    and outputs; and a single thread that alternates between arenas gets the same answers every time."""
    import threading
    import torch
    spec = wl.mobilenet_v2(2, size=96)
    x_np = wl.make_input(spec)
    ref = og.run(spec, [x_np], storage="f16")[spec.outputs[0]]
    g, _ = api.graph_from_spec(spec, api.GI_F16)
    ex = g.compile()
    ex.bind("cuda:0")
    nb = max(int(ex.info.arena_bytes), 256)
    x = torch.from_numpy(x_np).to("cuda:0").half().contiguous()
    out_shape = (spec.batch,) + tuple(spec.shapes[spec.outputs[0]])
    n_threads, rounds = 3, 8
    arenas = [torch.full((nb,), 0xFF, dtype=torch.uint8, device="cuda:0") for _ in range(n_threads)]
    outs = [torch.zeros(out_shape, dtype=torch.float16, device="cuda:0") for _ in range(n_threads)]
    streams = [torch.cuda.Stream() for _ in range(n_threads)]
    torch.cuda.synchronize()
    errors = []

    def work(i):
        try:
            for _ in range(rounds):
                ex.run_raw([x.data_ptr()], [outs[i].data_ptr()], arenas[i].data_ptr(), nb, streams[i])
            streams[i].synchronize()
        except Exception as exc:  # reported by the main thread
            errors.append(exc)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(n_threads)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    first = outs[0].float().cpu().numpy()
    assert_close(first, ref, api.GI_F16, "threaded run")
    for o in outs[1:]:
        assert np.array_equal(o.float().cpu().numpy(), first)
    # one thread, alternating arenas
    for k in range(6):
        outs[k % 2].zero_()
        ex.run_raw([x.data_ptr()], [outs[k % 2].data_ptr()], arenas[k % 3].data_ptr(), nb)
        torch.cuda.synchronize()
        assert np.array_equal(outs[k % 2].float().cpu().numpy(), first)
    assert api.gi_device_status() == 0


# ---------------------------------------------------------------------- a whole inverted-residual block as one kernel
# (batch, H, W, Cin, hidden, Cout, stride): the block shapes of MobileNetV2 on 14x14 and 7x7 planes, small and odd
# planes, hidden widths that are not a multiple of the 64-channel chunk, a batch that leaves the last unit half empty
IR_CASES = [(3, 14, 14, 64, 384, 64, 1), (2, 14, 14, 64, 384, 96, 1), (2, 14, 14, 96, 576, 96, 1), (3, 14, 14, 96, 576, 160, 2),
            (5, 7, 7, 160, 960, 160, 1), (4, 7, 7, 160, 960, 320, 1), (1, 7, 7, 16, 64, 16, 1), (3, 9, 5, 32, 100, 24, 1),
            (2, 10, 12, 16, 72, 20, 2), (7, 3, 3, 48, 128, 48, 1), (2, 16, 16, 32, 192, 32, 1), (3, 11, 13, 16, 40, 16, 1)]


@pytest.mark.parametrize("case", IR_CASES, ids=lambda c: "b%d_%dx%d_%d_%d_%d_s%d" % c)
def test_inverted_residual_block_one_kernel(case):
    b, h, w, cin, hidden, cout, stride = case
    spec = wl.inverted_residual_block(b, h, w, cin, hidden, cout, stride)
    run, xs, outs = check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert names.count("inverted_residual") == 1 and names.count("none") == 2, names
    again = run.run(xs)
    for t in spec.outputs:
        assert np.array_equal(outs[t], again[t])
    assert api.gi_device_status() == 0


@pytest.mark.parametrize("act,out_act", [(wl.ACT_RELU, None), (wl.ACT_NONE, wl.ACT_RELU6), (wl.ACT_RELU6, wl.ACT_RELU)])
def test_inverted_residual_block_epilogues(act, out_act):
    spec = wl.inverted_residual_block(3, 7, 7, 32, 96, 32, 1, act=act, out_act=out_act)
    run, _, _ = check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_ON)
    assert "inverted_residual" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]


def test_mobilenet_v2_batch32_blocks_as_one_kernel_every_tensor():
    """Every stored tensor of the network with the ten 14x14 / 7x7 blocks as one kernel each (the hidden tensors of
    those blocks are never stored: they are covered through the block outputs computed from them)."""
    spec = wl.mobilenet_v2(4, size=224)
    xs = [wl.make_input(spec)]
    ref = og.run(spec, xs, storage="f16", fused=True, keep_all=True)
    run = DeviceRun(spec, api.GI_F16, planner=api.GI_PLAN_NAIVE, guard_bytes=4096, cross_op=api.GI_XOP_ON)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert names.count("inverted_residual") == 10, names
    outs = run.run(xs)
    assert run.guard_intact()
    for t, r in ref.items():
        if t in run.on_chip:
            continue
        assert_close(outs[t] if t in outs else run.fetch(t), r, api.GI_F16, f"tensor {t}")
    assert api.gi_device_status() == 0


# ---------------------------------------------------------------------- 1x1 -> 1x1 as one kernel
# (batch, H, W, Cin, Cmid, Cout, residual): the projection -> expansion seams of MobileNetV2 (every plane size), a
# middle width that is not a multiple of 16 (24, 20), one that is not a multiple of 4 (10), input widths that leave the
# last 32-channel chunk ragged, odd planes, a single pixel, more tiles than one wave of SMs
PC_CASES = [(3, 14, 14, 384, 64, 384, True), (2, 14, 14, 384, 96, 576, False), (2, 14, 14, 576, 96, 576, True),
            (3, 7, 7, 576, 112, 672, False), (5, 7, 7, 960, 80, 480, True), (2, 28, 28, 192, 32, 192, True),
            (2, 28, 28, 144, 32, 192, False), (1, 56, 56, 144, 24, 144, True), (1, 56, 56, 96, 24, 144, False),
            (1, 112, 112, 32, 16, 96, False), (3, 9, 5, 40, 20, 70, True), (2, 3, 3, 17, 10, 33, True), (4, 1, 1, 64, 16, 64, False),
            (40, 28, 28, 48, 16, 48, True), (2, 6, 6, 100, 112, 130, False)]


@pytest.mark.parametrize("case", PC_CASES, ids=lambda c: "b%d_%dx%d_%d_%d_%d_r%d" % c)
def test_pointwise_pair_one_kernel(case):
    b, h, w, cin, cmid, cout, residual = case
    spec = wl.pointwise_pair(b, h, w, cin, cmid, cout, residual)
    # every tensor its own memory: under a sharing plan the second output may lie on the first input's bytes, and the
    # pair then stays two kernels (covered by the host tests)
    run, xs, outs = check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert names.count("pointwise_chain") == 1 and names.count("none") == 1, names
    again = run.run(xs)
    for t in spec.outputs:
        assert np.array_equal(outs[t], again[t])
    # the same two tensors from two kernels: identical bits (same products, same fp32 sums per output, same rounding)
    two = DeviceRun(spec, api.GI_F16, cross_op=api.GI_XOP_OFF, planner=api.GI_PLAN_NAIVE).run(xs)
    for t in spec.outputs:
        assert_close(outs[t], two[t], api.GI_F16, f"{spec.name} output {t} against the two-kernel path")
    assert api.gi_device_status() == 0


def test_pointwise_pair_too_wide_for_one_kernel_stays_two():
    """160 channels in the middle: the two weight rings, the operand tile and the residual strips no longer fit shared
    memory together; the pair must fall back to two kernels and still be right."""
    spec = wl.pointwise_pair(3, 7, 7, 960, 160, 960, True)
    run, _, _ = check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert "pointwise_chain" not in names and "none" not in names, names


@pytest.mark.parametrize("mid_act,act", [(wl.ACT_RELU, wl.ACT_NONE), (wl.ACT_RELU6, wl.ACT_RELU), (wl.ACT_NONE, wl.ACT_RELU6)])
def test_pointwise_pair_epilogues(mid_act, act):
    spec = wl.pointwise_pair(3, 10, 10, 48, 32, 80, True, mid_act=mid_act, act=act)
    run, _, _ = check_outputs(spec, api.GI_F16, cross_op=api.GI_XOP_CHAIN, planner=api.GI_PLAN_NAIVE)
    assert "pointwise_chain" in [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]


def test_mobilenet_v2_seams_as_one_kernel_every_tensor():
    """Every stored tensor of the network with each projection -> expansion seam as one kernel."""
    spec = wl.mobilenet_v2(4, size=224)
    xs = [wl.make_input(spec)]
    ref = og.run(spec, xs, storage="f16", fused=True, keep_all=True)
    run = DeviceRun(spec, api.GI_F16, planner=api.GI_PLAN_NAIVE, guard_bytes=4096, cross_op=api.GI_XOP_CHAIN)
    names = [api.KERNEL_NAMES[o.kernel] for o in run.ex.ops()]
    assert names.count("pointwise_chain") == 13, names  # all seams but the three with 160 channels in the middle
    outs = run.run(xs)
    assert run.guard_intact()
    for t, r in ref.items():
        if t in run.on_chip:
            continue
        assert_close(outs[t] if t in outs else run.fetch(t), r, api.GI_F16, f"tensor {t}")
    assert api.gi_device_status() == 0


# ---------------------------------------------------------------------- layout experiment: slices of eight channels
S8_CASES = [  # batch, hw, cin, cout, act: ragged channels and planes, one CTA pair half empty, many output tiles, long K
    (2, 9, 10, 22, wl.ACT_RELU), (3, 14, 144, 32, wl.ACT_NONE), (1, 33, 320, 256, wl.ACT_RELU6),
    (4, 1, 1280, 1001, wl.ACT_NONE), (16, 14, 512, 512, wl.ACT_RELU6), (5, 7, 960, 320, wl.ACT_NONE),
]


@pytest.mark.parametrize("case", S8_CASES)
def test_slice8_pointwise_matches_the_oracle(case):
    """The wide-tile 1x1 kernel on tensors stored in slices of 8 channels (gi_slice8_pointwise_*): the tiled copy lands
    operand rows directly.  Same seeded layer and input as the PHWC4 path, every output element against the oracle; the
    output buffer starts as NaN bytes, so padding lanes and the padding pixel must be written (as zeros)."""
    import torch
    from tests.gpu_util import pack_slice8, unpack_slice8, POISON
    batch, hw, cin, cout, act = case
    spec = wl.single_pointwise(batch, hw, cin, cout, False, act)
    x = wl.make_input(spec)
    ref = og.run(spec, [x], storage="f16", fused=True)[spec.outputs[0]]
    conv = [o for o in spec.ops if o.kind == wl.CONV2D][0]
    blob = torch.from_numpy(api.gi_slice8_pointwise_pack(conv.weights.reshape(cout, cin), conv.bias)).to("cuda:0")
    x_dev = torch.from_numpy(pack_slice8(x.astype(np.float16))).to("cuda:0")
    assert x_dev.numel() * 2 == api.gi_slice8_tensor_bytes(batch, hw, hw, cin)
    out_bytes = api.gi_slice8_tensor_bytes(batch, hw, hw, cout)
    out_dev = torch.full((out_bytes,), POISON, dtype=torch.uint8, device="cuda:0")
    api.gi_slice8_pointwise_run(x_dev.data_ptr(), out_dev.data_ptr(), blob.data_ptr(), batch, hw, hw, cin, cout, api._ACT[act])
    torch.cuda.synchronize()
    assert api.gi_device_status() == 0
    raw = out_dev.cpu().numpy().view(np.float16).astype(np.float32)
    assert_close(unpack_slice8(raw, batch, hw, hw, cout), ref, api.GI_F16, f"slice8 {case}")
    # every stored value is finite (a later 1x1 layer multiplies padding lanes and the padding pixel by zero weights,
    # and 0 x NaN = NaN), and the lanes beyond the last channel hold zeros
    S, P = (cout + 7) // 8, (hw * hw + 1) // 2 * 2
    phys = raw[: S * batch * P * 8].reshape(S, batch, P, 8)
    assert np.isfinite(phys).all()
    if cout % 8:
        assert np.all(phys[S - 1, :, : hw * hw, cout % 8:] == 0)


# ---------------------------------------------------------------------- the give-up path of the device-side waits
def test_bounded_wait_runs_out_and_the_context_survives():
    """Every wait in the kernels is bounded; here one is made to run out on purpose and safely: a warp waits on a
    barrier that nothing completes, with a limit of a few milliseconds.  The wait must end by its limit (not hang,
    not trap), report it, and leave the context healthy: a real inference afterwards still matches the oracle and the
    kernels' own status word stays clean."""
    waited_us, gave_up = api.gi_selftest_bounded_wait(3000)
    assert gave_up
    assert 2500 <= waited_us <= 50000, waited_us
    waited_us, gave_up = api.gi_selftest_bounded_wait(200)
    assert gave_up and 100 <= waited_us <= 20000, waited_us
    with pytest.raises(api.GiError):
        api.gi_selftest_bounded_wait(0)
    assert api.gi_device_status() == 0
    check_outputs(wl.separable_block(2), api.GI_F16)
    assert api.gi_device_status() == 0
