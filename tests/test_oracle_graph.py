"""Pins for the oracle's graph evaluation: an independent float64 numpy evaluation of the same
graph descriptions (sliding windows + einsum, no shared code), and fused == unfused."""
import numpy as np
import pytest
from numpy.lib.stride_tricks import sliding_window_view

from oracle import compile as oc
from oracle import graph as og
from paper_1907_01989_b200 import workloads as wl


def np_eval(g, x):
    """Evaluate the *unfused* graph in float64 with numpy only."""
    val = {g.inputs[0]: x.astype(np.float64)}
    for k, t in enumerate(g.inputs[1:], 1):
        raise AssertionError("single-input graphs only")
    for op in g.ops:
        a = val[op.inputs[0]]
        if op.kind in ("conv2d", "depthwise_conv2d"):
            pt, pl, pb, pr = op.pads
            ap = np.pad(a, ((0, 0), (pt, pb), (pl, pr), (0, 0)))
            kh, kw = op.kh, op.kw
            eh, ew = (kh - 1) * op.dilation[0] + 1, (kw - 1) * op.dilation[1] + 1
            win = sliding_window_view(ap, (eh, ew), axis=(1, 2))          # B, H', W', C, eh, ew
            win = win[:, ::op.stride[0], ::op.stride[1], :, ::op.dilation[0], ::op.dilation[1]]
            w = op.weights.astype(np.float64)
            if op.kind == "conv2d":
                y = np.einsum("bhwcyx,oyxc->bhwo", win, w, optimize=True)
            else:
                y = np.einsum("bhwcyx,yxc->bhwc", win, w[0], optimize=True)
            if op.bias is not None:
                y = y + op.bias.astype(np.float64)
        elif op.kind == "activation":
            y = np.maximum(a, 0.0)
            if op.act == "relu6":
                y = np.minimum(y, 6.0)
        elif op.kind in ("add", "concat") and len(op.inputs) == 1:
            y = a
        elif op.kind == "add":
            y = a + val[op.inputs[1]]
        elif op.kind == "concat":
            y = np.concatenate([a, val[op.inputs[1]]], axis=3)
        elif op.kind == "global_avg_pool":
            y = a.mean(axis=(1, 2), keepdims=True)
        elif op.kind == "resize_bilinear":
            oh, ow = op.out_hw
            H, W = a.shape[1:3]
            if op.align_corners:  # the corner samples of input and output coincide
                fy = np.linspace(0.0, H - 1.0, oh) if oh > 1 else np.zeros(1)
                fx = np.linspace(0.0, W - 1.0, ow) if ow > 1 else np.zeros(1)
            else:                 # output sample o sits at o / out of the way along the input's extent
                fy = np.arange(oh) / oh * H
                fx = np.arange(ow) / ow * W
            y0 = np.minimum(np.floor(fy).astype(int), H - 1)
            x0 = np.minimum(np.floor(fx).astype(int), W - 1)
            y1, x1 = np.minimum(y0 + 1, H - 1), np.minimum(x0 + 1, W - 1)
            wy, wx = (fy - y0)[None, :, None, None], (fx - x0)[None, None, :, None]
            rows0 = a[:, y0][:, :, x0] * (1 - wx) + a[:, y0][:, :, x1] * wx
            rows1 = a[:, y1][:, :, x0] * (1 - wx) + a[:, y1][:, :, x1] * wx
            y = rows0 * (1 - wy) + rows1 * wy
        else:
            raise ValueError(op.kind)
        val[op.output] = y
    return val


def resize_chain():
    """Bilinear resizes in both corner conventions, up and down, with H != W and odd factors."""
    b = wl.GraphBuilder("resize_chain", 2, 61)
    x = b.input(9, 7, 5)
    y = b.conv2d(x, 6, 1)
    y = b.resize_bilinear(y, 23, 10, False)
    y = b.activation(b.depthwise(y, 3, 1), wl.ACT_RELU6)
    y = b.resize_bilinear(y, 7, 25, False)
    y = b.resize_bilinear(y, 15, 9, True)
    y = b.resize_bilinear(y, 30, 4, False)
    b.output(y)
    return b.finish()


NETS = [
    ("separable_block", lambda: wl.separable_block(2)),
    ("mobilenet_v1", lambda: wl.mobilenet_v1(1, size=96)),
    ("mobilenet_v2", lambda: wl.mobilenet_v2(1, size=96)),
    ("segmentation", lambda: wl.mobilenet_v2_segmentation(1, size=65)),
    ("fire_network", lambda: wl.fire_network(2)),
    ("fire_network_odd", lambda: wl.fire_network(1, size=77)),
    ("resize_both_corner_conventions", lambda: resize_chain()),
]


@pytest.mark.parametrize("name,make", NETS)
def test_oracle_matches_float64_numpy_on_every_tensor(name, make):
    g = make()
    x = wl.make_input(g)
    ref = np_eval(g, x)
    got = og.run(g, [x], storage="f32", fused=False, keep_all=True)
    # the only tensors the oracle does not compute are the outputs of the identity operators its clean-up removes
    removed = {op.output for op in g.ops if op.kind in ("add", "concat") and len(op.inputs) == 1 and op.output not in g.outputs}
    assert set(ref) - set(got) == removed and set(got) <= set(ref)
    for t in got:
        scale = max(1.0, float(np.abs(ref[t]).max()))
        np.testing.assert_allclose(got[t], ref[t], rtol=0, atol=2e-5 * scale, err_msg=f"{name} tensor {t}")
    # fused evaluation agrees with the same reference on the tensors that survive fusion
    fused = og.run(g, [x], storage="f32", fused=True, keep_all=True)
    for t in fused:
        scale = max(1.0, float(np.abs(ref[t]).max()))
        np.testing.assert_allclose(fused[t], ref[t], rtol=0, atol=2e-5 * scale)


def test_full_size_mobilenet_v2_against_numpy():
    g = wl.mobilenet_v2(1)
    x = wl.make_input(g)
    ref = np_eval(g, x)
    got = og.run(g, [x], storage="f32", fused=True)
    out = g.outputs[0]
    assert got[out].shape == (1, 1, 1, 1001)
    np.testing.assert_allclose(got[out], ref[out], rtol=0, atol=2e-5 * max(1.0, np.abs(ref[out]).max()))


@pytest.mark.parametrize("name,make", NETS)
def test_fused_equals_unfused(name, make):
    g = make()
    x = wl.make_input(g)
    a = og.run(g, [x], storage="f32", fused=True)
    b = og.run(g, [x], storage="f32", fused=False)
    for t in g.outputs:
        assert np.array_equal(a[t], b[t])  # same fp32 values through the same epilogue order: bit-exact
    a = og.run(g, [x], storage="f16", fused=True, keep_all=True)
    b = og.run(g, [x], storage="f16", fused=False, keep_all=True)
    for t in a:
        # fp16 storage: the unfused graph rounds between conv, activation and add; fusing removes
        # roundings, so the two differ by a few fp16 ulps that then propagate
        assert np.all(np.abs(a[t] - b[t]) <= 1e-2 + 1e-2 * np.abs(b[t])), (name, t)


def test_f16_storage_values_are_representable():
    g = wl.separable_block(1)
    x = wl.make_input(g)
    r = og.run(g, [x], storage="f16", keep_all=True)
    for t, v in r.items():
        assert np.array_equal(v, v.astype(np.float16).astype(np.float32))


def test_input_generator_is_batch_independent():
    g4, g2 = wl.mobilenet_v2(4, size=32), wl.mobilenet_v2(2, size=32)
    x4 = wl.make_input(g4)
    assert np.array_equal(wl.make_input(g2, images=[1, 3]), x4[[1, 3]])
    assert np.array_equal(x4, x4.astype(np.float16).astype(np.float32))
    assert x4.min() >= -1 and x4.max() <= 1
    for a, b in zip(g4.ops, g2.ops):
        if a.weights is not None:
            assert np.array_equal(a.weights, b.weights) and np.array_equal(a.bias, b.bias)


def test_resize_to_the_same_size_is_the_identity_and_removing_it_changes_nothing():
    """The premise of the identity-removal pass: bilinear resize to the input's own size returns the input
    bit for bit (both corner conventions), so the cleaned graph computes exactly what the original does."""
    from oracle import ops
    rnd = np.random.default_rng(3)
    x = rnd.standard_normal((2, 6, 5, 7)).astype(np.float32)
    for ac in (True, False):
        assert np.array_equal(ops.resize_bilinear(x, 6, 5, ac), x)
    # the same network with and without the identity ops
    def build(with_identities):
        b = wl.GraphBuilder("identity_ops", 2, 21)
        t = b.input(6, 5, 8)
        y = b.conv2d(t, 12, 1)
        if with_identities:
            y = b.resize_bilinear(y, 6, 5, True)
        y = b.activation(y, wl.ACT_RELU)
        if with_identities:
            y = b.resize_bilinear(y, 6, 5, False)
        y = b.resize_bilinear(y, 12, 10, True)
        b.output(y)
        return b.finish()
    ga, gb = build(True), build(False)
    xs = [wl.make_input(ga, index=0)]
    for storage in ("f16", "f32"):
        ya = og.run(ga, xs, storage=storage)[ga.outputs[0]]
        yb = og.run(gb, xs, storage=storage)[gb.outputs[0]]
        assert np.array_equal(ya, yb)


def test_concat_then_1x1_convolution_is_the_sum_of_the_convolutions_of_the_parts():
    """Pins the channel order of CONCAT: a 1x1 convolution of concat(a, b) with weights [Wa | Wb] equals the
    convolution of a with Wa plus that of b with Wb (bias counted once)."""
    r = np.random.default_rng(5)
    from oracle import ops
    a = r.standard_normal((2, 5, 3, 6)).astype(np.float32)
    b = r.standard_normal((2, 5, 3, 5)).astype(np.float32)
    w = r.standard_normal((7, 1, 1, 11)).astype(np.float32)
    bias = r.standard_normal(7).astype(np.float32)
    whole = ops.conv2d(ops.concat(a, b), w, bias)
    parts = (ops.conv2d(a, np.ascontiguousarray(w[..., :6]), bias).astype(np.float64)
             + ops.conv2d(b, np.ascontiguousarray(w[..., 6:]), None).astype(np.float64))
    np.testing.assert_allclose(whole, parts, rtol=0, atol=1e-5)
    # and the values themselves: channel c of the result is channel c of a, then channel c - 6 of b
    y = ops.concat(a, b)
    assert y.shape == (2, 5, 3, 11)
    assert np.array_equal(y[1, 4, 2], np.array(list(a[1, 4, 2]) + list(b[1, 4, 2]), dtype=np.float32))
    swapped = ops.concat(b, a)
    assert not np.array_equal(swapped, y) and np.array_equal(swapped[..., 5:], a)


def test_single_input_add_and_concat_are_identities_and_removing_them_changes_nothing():
    b = wl.GraphBuilder("ident", 2, 77)
    x = b.input(6, 5, 7)
    y = b.activation(b.conv2d(x, 10, 1), wl.ACT_RELU)
    z = b.concat(b.identity_add(y))
    out1 = b.activation(b.conv2d(z, 6, 3), wl.ACT_RELU6)
    kept = b.concat(out1)  # a graph output: stays, as a copy
    b.output(kept)
    g = b.finish()
    fused = oc.fuse(g)
    assert [f.kind for f in fused] == ["conv2d", "conv2d", "concat"]
    assert fused[1].inputs == [fused[0].output] and fused[2].inputs == [out1]
    xin = wl.make_input(g)
    a = og.run(g, [xin], storage="f32", fused=True)[kept]
    ref = np_eval(g, xin)[kept]
    np.testing.assert_allclose(a, ref, rtol=0, atol=2e-5)
