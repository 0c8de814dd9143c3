"""numpy-facing wrapper around ``dybit_oracle.c`` (test infrastructure only).

Argument marshalling and nothing else: every number comes out of the C file.
The shared object is compiled on first use with
``gcc -O2 -ffp-contract=off -fopenmp`` (no fast-math, no FMA contraction, so
each fp32 operation rounds once, as the text of the oracle says).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dybit_oracle.c")
_LIB = os.path.join(_HERE, "libdybit_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object next to it."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                 "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        i64, i32, f32, u32 = C.c_int64, C.c_int, C.c_float, C.c_uint
        vp = C.c_void_p
        lib.orc_threads.restype = i32
        lib.orc_decode_mag.restype = C.c_double
        lib.orc_decode_mag.argtypes = [i32, u32]
        lib.orc_decode.restype = C.c_double
        lib.orc_decode.argtypes = [i32, i32, u32]
        lib.orc_decode_table.argtypes = [i32, i32, vp]
        lib.orc_decode_fields.argtypes = [i32, u32, C.POINTER(i32), C.POINTER(u32)]
        lib.orc_absmax_scale.argtypes = [vp, i64, i32, i32, C.POINTER(f32), C.POINTER(f32)]
        lib.orc_encode_one.restype = u32
        lib.orc_encode_one.argtypes = [f32, f32, i32, i32]
        lib.orc_quantize.argtypes = [vp, i64, i32, i32, f32, vp]
        lib.orc_pack.argtypes = [vp, i64, i32, vp, i64]
        lib.orc_unpack.argtypes = [vp, i64, i32, vp]
        lib.orc_pack_rows.argtypes = [vp, i64, i64, i32, vp, i64]
        lib.orc_unpack_rows.argtypes = [vp, i64, i64, i32, i64, vp]
        lib.orc_dequantize.argtypes = [vp, i64, i32, i32, f32, vp]
        lib.orc_alpha.restype = f32
        lib.orc_alpha.argtypes = [f32, i32, i32, f32, i32, i32]
        lib.orc_gemm.argtypes = [i64, i64, i64, vp, i32, i32, f32, vp, i32, i32, f32, vp, vp]
        lib.orc_gemm_sampled.argtypes = [i64, i64, vp, i32, i32, f32, vp, i32, i32, f32,
                                         vp, vp, i64, vp, vp]
        lib.orc_conv2d.argtypes = [i32] * 10 + [vp, i32, i32, f32, vp, i32, i32, f32, vp, vp]
        lib.orc_rmse.argtypes = [vp, i64, i32, i32, f32, f32, vp]
        lib.orc_depthwise_conv2d.argtypes = [i32] * 9 + [vp, i32, i32, f32, vp, i32, i32, f32, vp, vp]
        lib.orc_conv2d_sampled.argtypes = [i32] * 10 + [vp, i32, i32, f32, f32, vp, i32, i32, f32, vp, i64, vp, vp]
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def threads() -> int:
    return int(_load().orc_threads())


def decode_mag(m: int, c: int) -> float:
    return float(_load().orc_decode_mag(m, c))


def decode(bits: int, is_signed: bool, code: int) -> float:
    return float(_load().orc_decode(bits, int(is_signed), code))


def decode_table(bits: int, is_signed: bool) -> np.ndarray:
    out = np.zeros(1 << bits, dtype=np.float64)
    _load().orc_decode_table(bits, int(is_signed), _p(out))
    return out


def decode_fields(m: int, c: int):
    e, man = C.c_int(0), C.c_uint(0)
    _load().orc_decode_fields(m, c, C.byref(e), C.byref(man))
    return int(e.value), int(man.value)


def absmax_scale(x, bits: int, is_signed: bool):
    x = _f32(x).ravel()
    s, inv = C.c_float(0), C.c_float(0)
    _load().orc_absmax_scale(_p(x), x.size, bits, int(is_signed), C.byref(s), C.byref(inv))
    return np.float32(s.value), np.float32(inv.value)


def encode_one(x, inv, bits: int, is_signed: bool) -> int:
    return int(_load().orc_encode_one(float(np.float32(x)), float(np.float32(inv)),
                                      bits, int(is_signed)))


def quantize(x, bits: int, is_signed: bool, inv) -> np.ndarray:
    """fp32 tensor -> one code per byte (unpacked), same shape."""
    x = _f32(x)
    codes = np.zeros(x.shape, dtype=np.uint8)
    _load().orc_quantize(_p(x), x.size, bits, int(is_signed), float(np.float32(inv)), _p(codes))
    return codes


def packed_bytes(n: int, bits: int) -> int:
    """ceil(n*bits/8) rounded up to 16 bytes (zero-filled tail)."""
    return ((n * bits + 7) // 8 + 15) // 16 * 16


def row_stride_bytes(k: int, bits: int) -> int:
    """Row stride of a matrix operand: columns padded to a multiple of 128 codes."""
    return (k + 127) // 128 * 128 * bits // 8


def pack(codes, bits: int) -> np.ndarray:
    codes = _u8(codes).ravel()
    out = np.zeros(packed_bytes(codes.size, bits), dtype=np.uint8)
    _load().orc_pack(_p(codes), codes.size, bits, _p(out), out.size)
    return out


def unpack(packed, n: int, bits: int) -> np.ndarray:
    packed = _u8(packed).ravel()
    codes = np.zeros(n, dtype=np.uint8)
    _load().orc_unpack(_p(packed), n, bits, _p(codes))
    return codes


def pack_rows(codes, bits: int, row_stride: int | None = None) -> np.ndarray:
    codes = _u8(codes)
    rows, cols = codes.shape
    rs = row_stride_bytes(cols, bits) if row_stride is None else row_stride
    out = np.zeros((rows, rs), dtype=np.uint8)
    _load().orc_pack_rows(_p(codes), rows, cols, bits, _p(out), rs)
    return out


def unpack_rows(packed, rows: int, cols: int, bits: int) -> np.ndarray:
    packed = _u8(packed)
    rs = packed.shape[-1] if packed.ndim == 2 else packed.size // rows
    codes = np.zeros((rows, cols), dtype=np.uint8)
    _load().orc_unpack_rows(_p(packed), rows, cols, bits, rs, _p(codes))
    return codes


def dequantize(codes, bits: int, is_signed: bool, scale) -> np.ndarray:
    codes = _u8(codes)
    out = np.zeros(codes.shape, dtype=np.float32)
    _load().orc_dequantize(_p(codes), codes.size, bits, int(is_signed),
                           float(np.float32(scale)), _p(out))
    return out


def alpha(scale_a, fmt_a, scale_b, fmt_b) -> np.float32:
    return np.float32(_load().orc_alpha(float(np.float32(scale_a)), fmt_a[0], int(fmt_a[1]),
                                        float(np.float32(scale_b)), fmt_b[0], int(fmt_b[1])))


def gemm(codes_a, fmt_a, scale_a, codes_b, fmt_b, scale_b):
    """codes_a: [M][K], codes_b: [N][K] -> (S int64 [M][N], C fp32 [M][N])."""
    a, b = _u8(codes_a), _u8(codes_b)
    m, k = a.shape
    n, k2 = b.shape
    assert k == k2
    s = np.zeros((m, n), dtype=np.int64)
    c = np.zeros((m, n), dtype=np.float32)
    _load().orc_gemm(m, n, k, _p(a), fmt_a[0], int(fmt_a[1]), float(np.float32(scale_a)),
                     _p(b), fmt_b[0], int(fmt_b[1]), float(np.float32(scale_b)), _p(s), _p(c))
    return s, c


def gemm_sampled(codes_a, fmt_a, scale_a, codes_b, fmt_b, scale_b, rows_idx, cols_idx):
    a, b = _u8(codes_a), _u8(codes_b)
    m, k = a.shape
    n, _ = b.shape
    ri = np.ascontiguousarray(rows_idx, dtype=np.int64)
    ci = np.ascontiguousarray(cols_idx, dtype=np.int64)
    assert ri.shape == ci.shape and ri.max(initial=0) < m and ci.max(initial=0) < n
    s = np.zeros(ri.size, dtype=np.int64)
    c = np.zeros(ri.size, dtype=np.float32)
    _load().orc_gemm_sampled(n, k, _p(a), fmt_a[0], int(fmt_a[1]), float(np.float32(scale_a)),
                             _p(b), fmt_b[0], int(fmt_b[1]), float(np.float32(scale_b)),
                             _p(ri), _p(ci), ri.size, _p(s), _p(c))
    return s, c


def conv_out_hw(h, w, r, s, stride, pad, dilation=1):
    return ((h + 2 * pad - dilation * (r - 1) - 1) // stride + 1,
            (w + 2 * pad - dilation * (s - 1) - 1) // stride + 1)


def conv2d(codes_x, fmt_x, scale_x, codes_w, fmt_w, scale_w, stride=1, pad=0, dilation=1):
    """codes_x: [n][h][w][c]; codes_w: [k][r][s][c] -> (S int64, Y fp32) [n][oh][ow][k]."""
    x, wt = _u8(codes_x), _u8(codes_w)
    n, h, w, c = x.shape
    k, r, s, c2 = wt.shape
    assert c == c2
    oh, ow = conv_out_hw(h, w, r, s, stride, pad, dilation)
    acc = np.zeros((n, oh, ow, k), dtype=np.int64)
    y = np.zeros((n, oh, ow, k), dtype=np.float32)
    _load().orc_conv2d(n, h, w, c, k, r, s, stride, pad, dilation,
                       _p(x), fmt_x[0], int(fmt_x[1]), float(np.float32(scale_x)),
                       _p(wt), fmt_w[0], int(fmt_w[1]), float(np.float32(scale_w)),
                       _p(acc), _p(y))
    return acc, y


def depthwise_conv2d(codes_x, fmt_x, scale_x, codes_w, fmt_w, scale_w, stride=1, pad=0, dilation=1):
    """codes_x: [n][h][w][c]; codes_w: [c][r][s] (one filter per channel) -> (S int64, Y fp32) [n][oh][ow][c]."""
    x, wt = _u8(codes_x), _u8(codes_w)
    n, h, w, c = x.shape
    c2, r, s = wt.shape
    assert c2 == c
    oh, ow = conv_out_hw(h, w, r, s, stride, pad, dilation)
    acc = np.zeros((n, oh, ow, c), dtype=np.int64)
    y = np.zeros((n, oh, ow, c), dtype=np.float32)
    _load().orc_depthwise_conv2d(n, h, w, c, r, s, stride, pad, dilation,
                                 _p(x), fmt_x[0], int(fmt_x[1]), float(np.float32(scale_x)),
                                 _p(wt), fmt_w[0], int(fmt_w[1]), float(np.float32(scale_w)),
                                 _p(acc), _p(y))
    return acc, y


def conv2d_sampled(x_fp32, fmt_x, scale_pair_x, codes_w, fmt_w, scale_w, flat_idx, stride=1, pad=0, dilation=1):
    """Chosen outputs of the convolution, quantising the needed fp32 activations on the spot.

    x_fp32: [n][h][w][c] float32; scale_pair_x: (scale, inv); flat_idx: indices into Y[n][oh][ow][k].
    Returns (S int64, Y fp32), one entry per index."""
    x, wt = _f32(x_fp32), _u8(codes_w)
    n, h, w, c = x.shape
    k, r, s, c2 = wt.shape
    assert c == c2
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    oh, ow = conv_out_hw(h, w, r, s, stride, pad, dilation)
    assert idx.size == 0 or (idx.min() >= 0 and idx.max() < n * oh * ow * k)
    acc = np.zeros(idx.size, dtype=np.int64)
    y = np.zeros(idx.size, dtype=np.float32)
    _load().orc_conv2d_sampled(n, h, w, c, k, r, s, stride, pad, dilation, _p(x), fmt_x[0], int(fmt_x[1]),
                               float(np.float32(scale_pair_x[0])), float(np.float32(scale_pair_x[1])),
                               _p(wt), fmt_w[0], int(fmt_w[1]), float(np.float32(scale_w)),
                               _p(idx), idx.size, _p(acc), _p(y))
    return acc, y


def rmse(x, bits: int, is_signed: bool, scale_pair):
    """Eq. 2: (RMSE, sigma, mse) of quantizing x to the format with {scale, inv}."""
    x = _f32(x).ravel()
    out = np.zeros(3, dtype=np.float64)
    _load().orc_rmse(_p(x), x.size, bits, int(is_signed), float(np.float32(scale_pair[0])),
                     float(np.float32(scale_pair[1])), _p(out))
    return float(out[0]), float(out[1]), float(out[2])


def fake_quant(x, bits: int, is_signed: bool, scale_pair) -> np.ndarray:
    """QAT forward: the fp32 image of x under the format, decode(encode(x)) with {scale, inv}."""
    x = _f32(x)
    codes = quantize(x, bits, is_signed, scale_pair[1])
    return dequantize(codes, bits, is_signed, scale_pair[0]).reshape(x.shape)


def fake_quant_backward(x, grad_out, bits: int, is_signed: bool, scale_pair) -> np.ndarray:
    """Straight-through estimator with clipping: the gradient passes where x lies inside the closed range the
    format covers under this scale, [-hi, hi] (signed) or [0, hi] (unsigned), hi = fl32(scale * 2^(m-1)) by Eq. 1."""
    x, g = _f32(x), _f32(grad_out)
    m = bits - (1 if is_signed else 0)
    hi = np.float32(scale_pair[0]) * np.float32(2.0 ** (m - 1))
    lo = -hi if is_signed else np.float32(0.0)
    out = np.zeros(x.shape, dtype=np.float32)
    for i in np.ndindex(x.shape):
        if lo <= x[i] <= hi:          # NaN compares false: no gradient
            out[i] = g[i]
    return out
