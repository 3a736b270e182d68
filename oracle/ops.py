"""numpy-facing wrappers over oracle/ops.c (test infrastructure; see oracle/__init__.py)."""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())
_f = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_u16 = np.ctypeslib.ndpointer(dtype=np.uint16, flags="C_CONTIGUOUS")
_fopt = C.c_void_p
_i = C.c_int

_lib.orc_out_size.restype = _i
_lib.orc_out_size.argtypes = [_i] * 6
_lib.orc_conv2d.argtypes = [_f, _i, _i, _i, _i, _f, _fopt, _i] + [_i] * 10 + [_f]
_lib.orc_depthwise.argtypes = [_f, _i, _i, _i, _i, _f, _fopt] + [_i] * 10 + [_f]
_lib.orc_relu.argtypes = [_f, C.c_size_t]
_lib.orc_relu6.argtypes = [_f, C.c_size_t]
_lib.orc_add.argtypes = [_f, _f, _f, C.c_size_t]
_lib.orc_global_avg_pool.argtypes = [_f, _i, _i, _i, _i, _f]
_lib.orc_resize_bilinear.argtypes = [_f, _i, _i, _i, _i, _f, _i, _i, _i]
_lib.orc_f32_to_f16_bits.argtypes = [_f, _u16, C.c_size_t]
_lib.orc_f16_bits_to_f32.argtypes = [_u16, _f, C.c_size_t]
_lib.orc_round_f16.argtypes = [_f, C.c_size_t]
_lib.orc_phwc4_index.restype = C.c_size_t
_lib.orc_phwc4_index.argtypes = [_i] * 8
_lib.orc_phwc4_pack.argtypes = [_f, _i, _i, _i, _i, _i, _f]
_lib.orc_phwc4_unpack.argtypes = [_f, _i, _i, _i, _i, _i, _f]
_lib.orc_num_threads.restype = _i
_lib.orc_set_threads.argtypes = [_i]


def _c(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(_lib.orc_num_threads())


def set_threads(n: int) -> None:
    _lib.orc_set_threads(int(n))


def out_size(n, k, stride, dilation, pad_before, pad_after) -> int:
    return int(_lib.orc_out_size(n, k, stride, dilation, pad_before, pad_after))


def conv2d(x, w, bias, stride=(1, 1), dilation=(1, 1), pads=(0, 0, 0, 0)):
    x, w = _c(x), _c(w)
    bias = None if bias is None else _c(bias)
    B, H, W, Cin = x.shape
    Cout, kh, kw, wc = w.shape
    assert wc == Cin
    pt, pl, pb, pr = pads
    Ho = out_size(H, kh, stride[0], dilation[0], pt, pb)
    Wo = out_size(W, kw, stride[1], dilation[1], pl, pr)
    out = np.empty((B, Ho, Wo, Cout), dtype=np.float32)
    _lib.orc_conv2d(x, B, H, W, Cin, w, _ptr(bias), Cout, kh, kw, stride[0], stride[1], dilation[0], dilation[1],
                    pt, pl, pb, pr, out)
    return out


def depthwise(x, w, bias, stride=(1, 1), dilation=(1, 1), pads=(0, 0, 0, 0)):
    x, w = _c(x), _c(w)
    bias = None if bias is None else _c(bias)
    B, H, W, Cc = x.shape
    if w.ndim == 4:
        assert w.shape[0] == 1
        w = w[0]
    kh, kw, wc = w.shape
    assert wc == Cc
    w = np.ascontiguousarray(w)
    pt, pl, pb, pr = pads
    Ho = out_size(H, kh, stride[0], dilation[0], pt, pb)
    Wo = out_size(W, kw, stride[1], dilation[1], pl, pr)
    out = np.empty((B, Ho, Wo, Cc), dtype=np.float32)
    _lib.orc_depthwise(x, B, H, W, Cc, w, _ptr(bias), kh, kw, stride[0], stride[1], dilation[0], dilation[1],
                       pt, pl, pb, pr, out)
    return out


def activation(x, kind: str):
    y = _c(x).copy()
    if kind == "relu":
        _lib.orc_relu(y.reshape(-1), y.size)
    elif kind == "relu6":
        _lib.orc_relu6(y.reshape(-1), y.size)
    elif kind != "none":
        raise ValueError(kind)
    return y


def add(a, b):
    a, b = _c(a), _c(b)
    assert a.shape == b.shape
    out = np.empty_like(a)
    _lib.orc_add(a.reshape(-1), b.reshape(-1), out.reshape(-1), a.size)
    return out


def concat(a, b):
    """Channel concatenation (Section 3.1 lists CONCAT among the operators): out[..., :Ca] = a, out[..., Ca:] = b."""
    a, b = _c(a), _c(b)
    assert a.shape[:3] == b.shape[:3]
    out = np.empty(a.shape[:3] + (a.shape[3] + b.shape[3],), dtype=np.float32)
    for c in range(a.shape[3]):
        out[..., c] = a[..., c]
    for c in range(b.shape[3]):
        out[..., a.shape[3] + c] = b[..., c]
    return out


def global_avg_pool(x):
    x = _c(x)
    B, H, W, Cc = x.shape
    out = np.empty((B, 1, 1, Cc), dtype=np.float32)
    _lib.orc_global_avg_pool(x, B, H, W, Cc, out.reshape(-1))
    return out


def resize_bilinear(x, oh, ow, align_corners=True):
    x = _c(x)
    B, H, W, Cc = x.shape
    out = np.empty((B, oh, ow, Cc), dtype=np.float32)
    _lib.orc_resize_bilinear(x, B, H, W, Cc, out, oh, ow, 1 if align_corners else 0)
    return out


def f32_to_f16_bits(x):
    x = _c(x)
    out = np.empty(x.shape, dtype=np.uint16)
    _lib.orc_f32_to_f16_bits(x.reshape(-1), out.reshape(-1), x.size)
    return out


def f16_bits_to_f32(h):
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, dtype=np.float32)
    _lib.orc_f16_bits_to_f32(h.reshape(-1), out.reshape(-1), h.size)
    return out


def round_f16(x):
    y = _c(x).copy()
    _lib.orc_round_f16(y.reshape(-1), y.size)
    return y


def plane_pixels(H: int, W: int) -> int:
    """Pixels per stored plane: H*W rounded up to even (a whole number of 16-byte fp16 units)."""
    return (H * W + 1) // 2 * 2


def phwc4_index(B, H, W, b, h, w, c) -> int:
    return int(_lib.orc_phwc4_index(B, H, W, plane_pixels(H, W), b, h, w, c))


def phwc4_pack(x):
    x = _c(x)
    B, H, W, Cc = x.shape
    S = (Cc + 3) // 4
    out = np.empty((S, B, plane_pixels(H, W), 4), dtype=np.float32)
    _lib.orc_phwc4_pack(x, B, H, W, Cc, plane_pixels(H, W), out.reshape(-1))
    return out


def phwc4_unpack(p, B, H, W, Cc):
    p = _c(p)
    out = np.empty((B, H, W, Cc), dtype=np.float32)
    _lib.orc_phwc4_unpack(p.reshape(-1), B, H, W, Cc, plane_pixels(H, W), out)
    return out
