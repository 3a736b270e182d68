"""Pins for the oracle's operators: each check compares oracle/ops.c with something that is
not itself - brute force in another loop order and precision, a library routine for a special
case, a closed form, or an invariant."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import ops

RNG = np.random.default_rng(1234)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------- convolution
def brute_conv(x, w, bias, stride, dilation, pads):
    """Seven nested loops, channel loop outermost, exact summation with math.fsum."""
    B, H, W, Cin = x.shape
    Cout, kh, kw, _ = w.shape
    pt, pl, pb, pr = pads
    Ho = (H + pt + pb - ((kh - 1) * dilation[0] + 1)) // stride[0] + 1
    Wo = (W + pl + pr - ((kw - 1) * dilation[1] + 1)) // stride[1] + 1
    out = np.zeros((B, Ho, Wo, Cout), dtype=np.float64)
    for co in range(Cout):
        for b in range(B):
            for ox in range(Wo):
                for oy in range(Ho):
                    terms = [float(bias[co])] if bias is not None else []
                    for ci in range(Cin):
                        for kx in range(kw):
                            for ky in range(kh):
                                iy = oy * stride[0] - pt + ky * dilation[0]
                                ix = ox * stride[1] - pl + kx * dilation[1]
                                if 0 <= iy < H and 0 <= ix < W:
                                    terms.append(float(x[b, iy, ix, ci]) * float(w[co, ky, kx, ci]))
                    out[b, oy, ox, co] = math.fsum(terms)
    return out


CONV_CASES = [
    # H, W, Cin, Cout, k, stride, dilation, pads
    (5, 6, 3, 4, 3, (1, 1), (1, 1), (1, 1, 1, 1)),
    (7, 5, 2, 3, 3, (2, 2), (1, 1), (0, 0, 1, 1)),
    (9, 8, 2, 2, 3, (1, 1), (2, 2), (2, 2, 2, 2)),
    (6, 7, 5, 3, 1, (1, 1), (1, 1), (0, 0, 0, 0)),
    (8, 8, 1, 2, 3, (2, 1), (1, 2), (1, 2, 0, 2)),
    (4, 4, 3, 2, 2, (1, 1), (1, 1), (0, 0, 1, 1)),
    (9, 7, 3, 2, 2, (2, 2), (1, 1), (0, 0, 1, 1)),
    (10, 11, 2, 3, 3, (3, 3), (1, 1), (1, 0, 0, 1)),
    (8, 8, 2, 2, 2, (3, 3), (1, 1), (0, 0, 0, 0)),
    (7, 9, 4, 5, 1, (3, 2), (1, 1), (0, 0, 0, 0)),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv2d_brute_force(case):
    H, W, Cin, Cout, k, stride, dilation, pads = case
    x = RNG.standard_normal((2, H, W, Cin)).astype(np.float32)
    w = RNG.standard_normal((Cout, k, k, Cin)).astype(np.float32)
    b = RNG.standard_normal(Cout).astype(np.float32)
    got = ops.conv2d(x, w, b, stride, dilation, pads)
    ref = brute_conv(x, w, b, stride, dilation, pads)
    assert got.shape == ref.shape
    # double accumulation rounded once to fp32: at most half an ulp from the exact sum (+ double rounding slack)
    np.testing.assert_allclose(got, ref, rtol=1e-6, atol=1e-6)
    assert np.array_equal(got, ref.astype(np.float32)) or np.max(np.abs(got - ref.astype(np.float32))) <= 1e-6


def test_conv1x1_is_matmul():
    x = RNG.standard_normal((2, 6, 5, 40)).astype(np.float32)
    w = RNG.standard_normal((24, 1, 1, 40)).astype(np.float32)
    b = RNG.standard_normal(24).astype(np.float32)
    got = ops.conv2d(x, w, b)
    ref = x.reshape(-1, 40).astype(np.float64) @ w.reshape(24, 40).astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_allclose(got.reshape(-1, 24), ref, rtol=2e-7, atol=1e-6)


def test_conv_delta_input_reads_out_flipped_weights():
    # a single 1 at (3,3) of channel ci: out[oy,ox,co] = w[co, 3-oy+1, 3-ox+1, ci] where that tap exists
    w = RNG.standard_normal((3, 3, 3, 2)).astype(np.float32)
    for ci in range(2):
        x = np.zeros((1, 7, 7, 2), dtype=np.float32)
        x[0, 3, 3, ci] = 1.0
        y = ops.conv2d(x, w, None, pads=(1, 1, 1, 1))
        for oy, ox in itertools.product(range(7), range(7)):
            ky, kx = 3 - oy + 1, 3 - ox + 1
            for co in range(3):
                want = w[co, ky, kx, ci] if 0 <= ky < 3 and 0 <= kx < 3 else 0.0
                assert y[0, oy, ox, co] == want


@pytest.mark.parametrize("stride,dilation", [(1, 1), (2, 1), (1, 2), (1, 4)])
def test_conv_all_ones_counts_valid_taps(stride, dilation):
    H = W = 9
    pad = dilation
    x = np.ones((1, H, W, 1), dtype=np.float32)
    w = np.ones((1, 3, 3, 1), dtype=np.float32)
    y = ops.conv2d(x, w, None, (stride, stride), (dilation, dilation), (pad, pad, pad, pad))
    for oy in range(y.shape[1]):
        for ox in range(y.shape[2]):
            ny = sum(0 <= oy * stride - pad + k * dilation < H for k in range(3))
            nx = sum(0 <= ox * stride - pad + k * dilation < W for k in range(3))
            assert y[0, oy, ox, 0] == ny * nx
    if stride == 1 and dilation == 1:
        assert y[0, 0, 0, 0] == 4 and y[0, 0, 4, 0] == 6 and y[0, 4, 4, 0] == 9


def test_conv3x3_centre_tap_is_1x1():
    x = RNG.standard_normal((1, 6, 6, 5)).astype(np.float32)
    w1 = RNG.standard_normal((4, 1, 1, 5)).astype(np.float32)
    w3 = np.zeros((4, 3, 3, 5), dtype=np.float32)
    w3[:, 1, 1, :] = w1[:, 0, 0, :]
    assert np.array_equal(ops.conv2d(x, w3, None, pads=(1, 1, 1, 1)), ops.conv2d(x, w1, None))


def test_out_size_formula_examples():
    # 224 -> 112 at stride 2 with TF-SAME pads (0 before, 1 after); 513 -> 257 with (1, 1)
    assert ops.out_size(224, 3, 2, 1, 0, 1) == 112
    assert ops.out_size(513, 3, 2, 1, 1, 1) == 257
    assert ops.out_size(33, 3, 1, 4, 4, 4) == 33
    assert ops.out_size(7, 1, 1, 1, 0, 0) == 7


# ---------------------------------------------------------------------- depthwise
def test_depthwise_identity_kernel_returns_input():
    x = RNG.standard_normal((2, 7, 9, 6)).astype(np.float32)
    w = np.zeros((3, 3, 6), dtype=np.float32)
    w[1, 1, :] = 1.0
    assert np.array_equal(ops.depthwise(x, w, None, pads=(1, 1, 1, 1)), x)


@pytest.mark.parametrize("stride,dilation,pads", [((1, 1), (1, 1), (1, 1, 1, 1)), ((2, 2), (1, 1), (0, 0, 1, 1)),
                                                  ((1, 1), (2, 2), (2, 2, 2, 2)), ((2, 1), (1, 1), (1, 0, 1, 2))])
def test_depthwise_equals_block_diagonal_conv(stride, dilation, pads):
    C = 5
    x = RNG.standard_normal((2, 8, 7, C)).astype(np.float32)
    w = RNG.standard_normal((3, 3, C)).astype(np.float32)
    b = RNG.standard_normal(C).astype(np.float32)
    full = np.zeros((C, 3, 3, C), dtype=np.float32)
    for c in range(C):
        full[c, :, :, c] = w[:, :, c]
    a = ops.depthwise(x, w, b, stride, dilation, pads)
    ref = brute_conv(x, full, b, stride, dilation, pads)
    np.testing.assert_allclose(a, ref, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("d", [2, 4])
def test_depthwise_dilation_equals_phase_subsampling(d):
    # dilation d with pad d on an image == dilation 1 with pad 1 on each of the d*d phase images
    C, H, W = 3, 4 * d, 3 * d
    x = RNG.standard_normal((1, H, W, C)).astype(np.float32)
    w = RNG.standard_normal((3, 3, C)).astype(np.float32)
    y = ops.depthwise(x, w, None, (1, 1), (d, d), (d, d, d, d))
    for py in range(d):
        for px in range(d):
            sub = np.ascontiguousarray(x[:, py::d, px::d, :])
            ys = ops.depthwise(sub, w, None, (1, 1), (1, 1), (1, 1, 1, 1))
            assert np.array_equal(y[:, py::d, px::d, :], ys)


def test_depthwise_stride2_equals_stride1_subsampled():
    C = 4
    x = RNG.standard_normal((1, 10, 12, C)).astype(np.float32)
    w = RNG.standard_normal((3, 3, C)).astype(np.float32)
    b = RNG.standard_normal(C).astype(np.float32)
    s1 = ops.depthwise(x, w, b, (1, 1), (1, 1), (0, 0, 1, 1))
    s2 = ops.depthwise(x, w, b, (2, 2), (1, 1), (0, 0, 1, 1))
    assert np.array_equal(s2, s1[:, ::2, ::2, :])


# ---------------------------------------------------------------------- element-wise, pool
def test_activation_exact_values():
    v = np.array([-1.0, -0.0, 0.0, 3.0, 6.0, 7.0, np.float32(5.9999995)], dtype=np.float32)
    assert list(ops.activation(v, "relu")) == [0.0, 0.0, 0.0, 3.0, 6.0, 7.0, np.float32(5.9999995)]
    assert list(ops.activation(v, "relu6")) == [0.0, 0.0, 0.0, 3.0, 6.0, 6.0, np.float32(5.9999995)]
    assert np.array_equal(ops.activation(v, "none"), v)


def test_add_is_fp32_add():
    a = RNG.standard_normal(1000).astype(np.float32)
    b = RNG.standard_normal(1000).astype(np.float32) * 1e-3
    assert np.array_equal(ops.add(a, b), a + b)


def test_pool_constant_and_depthwise_equivalence():
    x = np.full((2, 7, 7, 5), 0.37, dtype=np.float32)
    np.testing.assert_allclose(ops.global_avg_pool(x), np.float32(0.37), rtol=1e-7)
    x = RNG.standard_normal((2, 7, 7, 5)).astype(np.float32)
    got = ops.global_avg_pool(x)
    ref = x.astype(np.float64).mean(axis=(1, 2), keepdims=True)
    np.testing.assert_allclose(got, ref, rtol=1e-6, atol=1e-7)
    # mean == 1/(HW) * depthwise conv with a full-size all-ones kernel, no padding
    w = np.ones((7, 7, 5), dtype=np.float32)
    dw = ops.depthwise(x, w, None) / np.float32(49.0)
    np.testing.assert_allclose(got, dw, rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------------- bilinear
def test_bilinear_constant_ramp_and_samples():
    c = np.full((1, 5, 4, 2), 1.25, dtype=np.float32)
    assert np.array_equal(ops.resize_bilinear(c, 65, 49, True), np.full((1, 65, 49, 2), 1.25, dtype=np.float32))
    # align_corners, 33 -> 513: scale exactly 1/16; a linear ramp stays the same linear ramp
    yy, xx = np.meshgrid(np.arange(33, dtype=np.float32), np.arange(33, dtype=np.float32), indexing="ij")
    ramp = (2.0 * yy - 3.0 * xx + 1.0)[None, :, :, None].astype(np.float32)
    up = ops.resize_bilinear(ramp, 513, 513, True)
    oy, ox = np.meshgrid(np.arange(513, dtype=np.float64), np.arange(513, dtype=np.float64), indexing="ij")
    want = 2.0 * oy / 16.0 - 3.0 * ox / 16.0 + 1.0
    np.testing.assert_allclose(up[0, :, :, 0], want, rtol=0, atol=1e-5)
    # outputs at multiples of 16 are the input samples
    r = RNG.standard_normal((1, 33, 33, 3)).astype(np.float32)
    up = ops.resize_bilinear(r, 513, 513, True)
    assert np.array_equal(up[:, ::16, ::16, :], r)
    # midpoint between two samples along x
    np.testing.assert_allclose(up[0, 0, 8, :], (r[0, 0, 0, :].astype(np.float64) + r[0, 0, 1, :]) / 2, rtol=1e-6)
    np.testing.assert_allclose(up[0, 24, 0, :], (r[0, 1, 0, :].astype(np.float64) + r[0, 2, 0, :]) / 2, rtol=1e-6,
                               atol=1e-7)


def test_bilinear_without_align_corners_closed_forms():
    """Corner convention 0 (src = o * in / out, no half-pixel shift) against closed forms that do not
    repeat that expression.  Each fails for the two plausible misreadings, a scale of (in-1)/(out-1)
    and half-pixel centres."""
    x = RNG.standard_normal(7).astype(np.float32)
    # exact 2x up-sampling along W: even outputs are the samples, odd ones the mean of two neighbours,
    # the last one repeats the last sample (its right neighbour is clamped)
    col = x[None, None, :, None]
    up = ops.resize_bilinear(col, 1, 14, False)[0, 0, :, 0]
    assert np.array_equal(up[0::2], x)
    np.testing.assert_allclose(up[1:-1:2], (x[:-1].astype(np.float64) + x[1:]) / 2, rtol=1e-6, atol=1e-7)
    assert up[-1] == x[-1]
    # the same along H (a transposed scale or axis would show here: H and W differ)
    row = x[None, :, None, None]
    up = ops.resize_bilinear(np.repeat(row, 3, axis=2), 14, 3, False)[0, :, :, 0]
    for w in range(3):
        assert np.array_equal(up[0::2, w], x)
        np.testing.assert_allclose(up[1:-1:2, w], (x[:-1].astype(np.float64) + x[1:]) / 2, rtol=1e-6, atol=1e-7)
        assert up[-1, w] == x[-1]
    # exact 2x down-sampling picks every second sample
    y = RNG.standard_normal((2, 8, 6, 3)).astype(np.float32)
    assert np.array_equal(ops.resize_bilinear(y, 4, 3, False), y[:, ::2, ::2, :])
    # a linear ramp of 5 samples resized to 13: the ramp evaluated at min(o * 5/13, 4)
    ramp = (0.75 * np.arange(5, dtype=np.float64) - 1.5)
    got = ops.resize_bilinear(ramp.astype(np.float32)[None, None, :, None], 1, 13, False)[0, 0, :, 0]
    want = 0.75 * np.minimum(np.arange(13) * 5.0 / 13.0, 4.0) - 1.5
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)
    got = ops.resize_bilinear(ramp.astype(np.float32)[None, :, None, None], 13, 1, False)[0, :, 0, 0]
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)
    # and both axes at once, different sizes: 5x3 -> 13x4
    yy, xx = np.meshgrid(np.arange(5, dtype=np.float64), np.arange(3, dtype=np.float64), indexing="ij")
    plane = (0.5 * yy - 2.0 * xx + 0.25)
    got = ops.resize_bilinear(plane.astype(np.float32)[None, :, :, None], 13, 4, False)[0, :, :, 0]
    sy = np.minimum(np.arange(13) * 5.0 / 13.0, 4.0)[:, None]
    sx = np.minimum(np.arange(4) * 3.0 / 4.0, 2.0)[None, :]
    np.testing.assert_allclose(got, 0.5 * sy - 2.0 * sx + 0.25, rtol=0, atol=1e-6)


# ---------------------------------------------------------------------- fp16 rounding
def test_f16_rounding_matches_numpy_everywhere_it_matters():
    # all 65536 half patterns round-trip
    allh = np.arange(65536, dtype=np.uint16)
    f = ops.f16_bits_to_f32(allh)
    ref = allh.view(np.float16).astype(np.float32)
    assert np.array_equal(f.view(np.uint32), ref.view(np.uint32))
    back = ops.f32_to_f16_bits(f)
    nan = np.isnan(ref)
    assert np.array_equal(back[~nan], allh[~nan])
    assert np.all((back[nan] & 0x7c00) == 0x7c00) and np.all((back[nan] & 0x3ff) != 0)
    # exact midpoints between adjacent non-negative finite halves (ties to even), and their fp32 neighbours
    pos = np.arange(0, 0x7bff, dtype=np.uint16)
    lo = pos.view(np.float16).astype(np.float64)
    hi = (pos + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)  # exactly representable in fp32
    for cand in (mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf)), -mid):
        assert np.array_equal(ops.f32_to_f16_bits(cand), cand.astype(np.float16).view(np.uint16))
    # overflow and subnormal boundaries
    edge = np.array([65504.0, 65519.99, 65520.0, 65536.0, 1e10, -65520.0, 2.0 ** -24, 2.0 ** -25,
                     np.nextafter(np.float32(2.0 ** -25), np.float32(1)), 2.0 ** -26, 6.1e-5, 6.0975552e-05,
                     2.0 ** -14, np.inf, -np.inf, 0.0, -0.0], dtype=np.float32)
    with np.errstate(over="ignore"):
        assert np.array_equal(ops.f32_to_f16_bits(edge), edge.astype(np.float16).view(np.uint16))
    # a million random floats over many magnitudes
    r = (RNG.standard_normal(1_000_000) * np.exp(RNG.uniform(-20, 12, 1_000_000))).astype(np.float32)
    with np.errstate(over="ignore"):
        assert np.array_equal(ops.f32_to_f16_bits(r), r.astype(np.float16).view(np.uint16))
        assert np.array_equal(ops.round_f16(r).view(np.uint32), r.astype(np.float16).astype(np.float32).view(np.uint32))


# ---------------------------------------------------------------------- PHWC4
def _read_kv(path):
    kv = {}
    with open(path) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                kv[k] = int(v)
    return kv


def test_phwc4_fig1_example():
    kv = _read_kv(os.path.join(GOLDEN, "fig1_phwc4.txt"))
    H, W, C = kv["H"], kv["W"], kv["C"]
    x = np.arange(H * W * C, dtype=np.float32).reshape(1, H, W, C)
    p = ops.phwc4_pack(x)
    # stored sequentially as a 2-D array of (H*C/4, 4*W)
    arr = p.reshape(-1)
    assert arr.size == kv["rows"] * kv["cols"]
    arr2d = arr.reshape(kv["rows"], kv["cols"])
    for h, w, c in itertools.product(range(H), range(W), range(C)):
        s = c // 4
        assert arr2d[s * H + h, 4 * w + c % 4] == x[0, h, w, c]
        assert ops.phwc4_index(1, H, W, 0, h, w, c) == (s * H + h) * 4 * W + 4 * w + c % 4


@pytest.mark.parametrize("shape", [(1, 3, 3, 3), (2, 7, 7, 5), (3, 1, 1, 1001), (2, 4, 5, 8), (1, 10, 10, 6)])
def test_phwc4_round_trip_and_zero_padding(shape):
    B, H, W, C = shape
    x = RNG.standard_normal(shape).astype(np.float32) + 10.0  # no zeros in the data
    p = ops.phwc4_pack(x)
    S = (C + 3) // 4
    assert p.shape == (S, B, (H * W + 1) // 2 * 2, 4)  # C = 5 costs as much as C = 8
    assert np.array_equal(ops.phwc4_unpack(p, B, H, W, C), x)
    assert np.count_nonzero(p) == x.size  # everything that is not data is zero
    if C % 4:
        assert np.all(p[S - 1, :, :, C % 4:] == 0)
    if (H * W) % 2:
        assert np.all(p[:, :, H * W:, :] == 0)
