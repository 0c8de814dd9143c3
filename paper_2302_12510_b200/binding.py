"""ctypes binding of libdybit.so: argument marshalling only.

Function names follow include/dybit.h.  torch supplies device memory and the
current stream; every computation happens inside the library's kernels.
There is no fallback: if libdybit.so is absent the import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import NamedTuple, Optional, Tuple

import torch

from . import _build

__all__ = [
    "Fmt", "ConvDesc", "DybitError", "lib", "CONTAINER_NAMES",
    "dybit_status_string", "dybit_packed_bytes", "dybit_row_stride_bytes", "dybit_decode_table",
    "dybit_choose_container", "dybit_gemm_workspace_bytes", "dybit_conv2d_workspace_bytes",
    "dybit_conv2d_out_hw", "dybit_absmax_scale", "dybit_quantize_pack", "dybit_quantize_pack_2d",
    "dybit_decode", "dybit_gemm", "dybit_conv2d", "dybit_last_device_status",
    "dybit_launch_count", "dybit_set_conv_lowering", "dybit_set_gemm_decode", "dybit_selftest_wait_timeout", "dybit_profile_next_gemm", "dybit_profile_next_gemm_clock", "dybit_gemm_static_ws", "STATIC_WS_BYTES",
    "dybit_gemm_requant", "dybit_conv2d_requant", "dybit_depthwise_conv2d", "dybit_gemm_batched",
    "dybit_quantize_conv2d", "dybit_quantize_conv2d_requant",
    "ConvLayers", "dybit_quantize_expand_layers", "dybit_conv2d_prepared", "dybit_conv2d_prepared_layers",
    "dybit_gemm_batched_workspace_bytes", "dybit_rmse", "dybit_rmse_sweep", "dybit_fake_quant", "dybit_fake_quant_backward",
    "dybit_search_bitwidths",
]


class Fmt(NamedTuple):
    bits: int
    is_signed: bool


class _CFmt(C.Structure):
    _fields_ = [("bits", C.c_int), ("is_signed", C.c_int)]


class _CConvDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n", "h", "w", "c", "k", "r", "s", "stride", "pad", "dilation")]


class _CConvLayer(C.Structure):
    _fields_ = [("desc", _CConvDesc), ("X", C.c_void_p), ("fx", _CFmt), ("scale_x", C.c_void_p),
                ("scale_x_out", C.c_void_p), ("X_packed", C.c_void_p), ("W", C.c_void_p), ("fw", _CFmt),
                ("scale_w", C.c_void_p), ("ldw_bytes", C.c_int64), ("Y", C.c_void_p), ("Y_raw", C.c_void_p),
                ("ws", C.c_void_p), ("ws_bytes", C.c_size_t), ("Q", C.c_void_p), ("fq", _CFmt),
                ("scale_q", C.c_void_p), ("bias", C.c_void_p), ("relu", C.c_int)]


class ConvDesc(NamedTuple):
    n: int
    h: int
    w: int
    c: int
    k: int
    r: int
    s: int
    stride: int = 1
    pad: int = 0
    dilation: int = 1


class DybitError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dybit_status_string(status)} (status {status})")


CONTAINER_NAMES = {0: "int8", 1: "e4m3", 2: "bf16"}


def _load() -> C.CDLL:
    # DYBIT_LIBRARY=debug selects the range-checked build (libdybit_debug.so); anything else is the product library
    path = _build.DEBUG_LIB_PATH if os.environ.get("DYBIT_LIBRARY", "") == "debug" else _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2302_12510_b200._build` "
            "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(path)
    i64, i32, sz, vp = C.c_int64, C.c_int, C.c_size_t, C.c_void_p
    lib.dybit_status_string.restype = C.c_char_p
    lib.dybit_status_string.argtypes = [i32]
    lib.dybit_packed_bytes.restype = sz
    lib.dybit_packed_bytes.argtypes = [i64, i32]
    lib.dybit_row_stride_bytes.restype = sz
    lib.dybit_row_stride_bytes.argtypes = [i64, i32]
    lib.dybit_decode_table.argtypes = [_CFmt, C.POINTER(C.c_float)]
    lib.dybit_choose_container.argtypes = [_CFmt, _CFmt, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.dybit_gemm_workspace_bytes.restype = sz
    lib.dybit_gemm_workspace_bytes.argtypes = [i64, i64, i64, _CFmt, _CFmt]
    lib.dybit_conv2d_workspace_bytes.restype = sz
    lib.dybit_conv2d_workspace_bytes.argtypes = [C.POINTER(_CConvDesc), _CFmt, _CFmt]
    lib.dybit_conv2d_out_hw.argtypes = [C.POINTER(_CConvDesc), C.POINTER(i32), C.POINTER(i32)]
    lib.dybit_absmax_scale.argtypes = [vp, i64, _CFmt, vp, vp]
    lib.dybit_quantize_pack.argtypes = [vp, i64, _CFmt, vp, vp, vp, vp]
    lib.dybit_quantize_pack_2d.argtypes = [vp, i64, i64, i64, _CFmt, vp, vp, i64, vp, vp]
    lib.dybit_decode.argtypes = [vp, i64, _CFmt, vp, vp, vp]
    lib.dybit_gemm.argtypes = [i64, i64, i64, vp, _CFmt, vp, i64, vp, _CFmt, vp, i64,
                               vp, i64, vp, vp, sz, vp]
    lib.dybit_conv2d.argtypes = [C.POINTER(_CConvDesc), vp, _CFmt, vp, vp, _CFmt, vp, i64,
                                 vp, vp, vp, sz, vp]
    lib.dybit_last_device_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.dybit_launch_count.restype = C.c_uint64
    lib.dybit_launch_count.argtypes = []
    lib.dybit_set_conv_lowering.argtypes = [i32]
    lib.dybit_set_gemm_decode.argtypes = [i32]
    lib.dybit_selftest_wait_timeout.argtypes = [C.c_uint64, vp, vp]
    lib.dybit_profile_next_gemm.argtypes = [vp, vp]
    lib.dybit_profile_next_gemm_clock.argtypes = [vp]
    lib.dybit_gemm_requant.argtypes = [i64, i64, i64, vp, _CFmt, vp, i64, vp, _CFmt, vp, i64,
                                       _CFmt, vp, vp, i32, vp, i64, vp, sz, vp]
    lib.dybit_conv2d_requant.argtypes = [C.POINTER(_CConvDesc), vp, _CFmt, vp, vp, _CFmt, vp, i64,
                                         _CFmt, vp, vp, i32, vp, vp, sz, vp]
    lib.dybit_quantize_conv2d_requant.argtypes = [C.POINTER(_CConvDesc), vp, _CFmt, vp, vp, vp, vp, _CFmt, vp, i64,
                                                  _CFmt, vp, vp, i32, vp, vp, sz, vp]
    lib.dybit_rmse.argtypes = [vp, i64, _CFmt, vp, vp, vp]
    lib.dybit_quantize_conv2d.argtypes = [C.POINTER(_CConvDesc), vp, _CFmt, vp, vp, vp, vp, _CFmt, vp, i64,
                                          vp, vp, vp, sz, vp]
    lib.dybit_quantize_expand_layers.argtypes = [C.POINTER(_CConvLayer), i32, vp]
    lib.dybit_conv2d_prepared.argtypes = [C.POINTER(_CConvLayer), vp]
    lib.dybit_conv2d_prepared_layers.argtypes = [C.POINTER(_CConvLayer), i32, vp]
    lib.dybit_gemm_batched_workspace_bytes.restype = sz
    lib.dybit_gemm_batched_workspace_bytes.argtypes = [i64, i64, i64, i64, _CFmt, _CFmt]
    lib.dybit_gemm_batched.argtypes = [i64, i64, i64, i64, vp, _CFmt, vp, i64, i64, vp, _CFmt, vp, i64, i64,
                                       vp, i64, i64, vp, vp, sz, vp]
    lib.dybit_depthwise_conv2d.argtypes = [C.POINTER(_CConvDesc), vp, _CFmt, vp, vp, _CFmt, vp, i64, vp, vp]
    lib.dybit_rmse_sweep.argtypes = [vp, i64, i32, C.POINTER(_CFmt), vp, vp, vp, vp]
    lib.dybit_fake_quant.argtypes = [vp, i64, _CFmt, vp, vp, vp]
    lib.dybit_fake_quant_backward.argtypes = [vp, vp, i64, _CFmt, vp, vp, vp]
    lib.dybit_search_bitwidths.argtypes = [i32, C.POINTER(C.c_double), C.POINTER(C.c_double), i32, C.c_double, i32,
                                           C.POINTER(i32), C.POINTER(i32)]
    lib.dybit_gemm_static_ws.argtypes = [i64, i64, i64, vp, _CFmt, vp, i64, vp, _CFmt, vp, i64, vp, i64, vp, vp]
    return lib


lib = _load()


def _fmt(f) -> _CFmt:
    bits, sg = f
    return _CFmt(int(bits), int(bool(sg)))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status: int, where: str):
    if status != 0:
        raise DybitError(status, where)


def _dev_f32(x: torch.Tensor, name: str) -> torch.Tensor:
    if not (x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous float32 CUDA tensor")
    return x


# ---------------------------------------------------------------- host helpers

def dybit_status_string(status: int) -> str:
    return lib.dybit_status_string(int(status)).decode()


def dybit_packed_bytes(n: int, bits: int) -> int:
    return int(lib.dybit_packed_bytes(int(n), int(bits)))


def dybit_row_stride_bytes(k: int, bits: int) -> int:
    return int(lib.dybit_row_stride_bytes(int(k), int(bits)))


def dybit_decode_table(fmt) -> list:
    buf = (C.c_float * 256)()
    _check(lib.dybit_decode_table(_fmt(fmt), buf), "dybit_decode_table")
    return list(buf)


def dybit_choose_container(fa, fb) -> Tuple[int, int, int]:
    c, ea, eb = C.c_int(-1), C.c_int(0), C.c_int(0)
    _check(lib.dybit_choose_container(_fmt(fa), _fmt(fb), C.byref(c), C.byref(ea), C.byref(eb)),
           "dybit_choose_container")
    return c.value, ea.value, eb.value


def dybit_gemm_workspace_bytes(M: int, N: int, K: int, fa, fb) -> int:
    return int(lib.dybit_gemm_workspace_bytes(int(M), int(N), int(K), _fmt(fa), _fmt(fb)))


def _cdesc(d: ConvDesc) -> _CConvDesc:
    return _CConvDesc(*[int(v) for v in d])


def dybit_conv2d_workspace_bytes(desc: ConvDesc, fx, fw) -> int:
    cd = _cdesc(desc)
    return int(lib.dybit_conv2d_workspace_bytes(C.byref(cd), _fmt(fx), _fmt(fw)))


def dybit_conv2d_out_hw(desc: ConvDesc) -> Tuple[int, int]:
    cd = _cdesc(desc)
    oh, ow = C.c_int(0), C.c_int(0)
    _check(lib.dybit_conv2d_out_hw(C.byref(cd), C.byref(oh), C.byref(ow)), "dybit_conv2d_out_hw")
    return oh.value, ow.value


# ---------------------------------------------------------------- device entry points

def dybit_absmax_scale(x: torch.Tensor, fmt, scale_out: Optional[torch.Tensor] = None, stream=None):
    _dev_f32(x, "x")
    if scale_out is None:
        scale_out = torch.empty(2, dtype=torch.float32, device=x.device)
    _check(lib.dybit_absmax_scale(_ptr(x), x.numel(), _fmt(fmt), _ptr(scale_out), _stream(stream)),
           "dybit_absmax_scale")
    return scale_out


def dybit_quantize_pack(x: torch.Tensor, fmt, scale: Optional[torch.Tensor] = None,
                        packed: Optional[torch.Tensor] = None,
                        scale_out: Optional[torch.Tensor] = None, stream=None):
    """Returns (packed uint8 tensor, scale tensor {scale, 1/scale})."""
    _dev_f32(x, "x")
    n = x.numel()
    if packed is None:
        packed = torch.empty(dybit_packed_bytes(n, fmt[0]), dtype=torch.uint8, device=x.device)
    if scale is None and scale_out is None:
        scale_out = torch.empty(2, dtype=torch.float32, device=x.device)
    _check(lib.dybit_quantize_pack(_ptr(x), n, _fmt(fmt), _ptr(scale), _ptr(packed), _ptr(scale_out),
                                   _stream(stream)), "dybit_quantize_pack")
    return packed, (scale if scale is not None else scale_out)


def dybit_quantize_pack_2d(x: torch.Tensor, fmt, scale: Optional[torch.Tensor] = None,
                           packed: Optional[torch.Tensor] = None, row_stride_bytes: Optional[int] = None,
                           scale_out: Optional[torch.Tensor] = None, ld: Optional[int] = None,
                           cols: Optional[int] = None, stream=None):
    """x: [rows][ld] float32 (cols <= ld used).  Returns (packed [rows][row_stride] uint8, scale)."""
    if not (x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1):
        raise ValueError("x must be a 2-D float32 CUDA tensor with unit inner stride")
    rows = x.shape[0]
    cols = x.shape[1] if cols is None else cols
    ld = x.stride(0) if ld is None else ld
    if row_stride_bytes is None:
        row_stride_bytes = dybit_row_stride_bytes(cols, fmt[0])
    if packed is None:
        packed = torch.empty((rows, row_stride_bytes), dtype=torch.uint8, device=x.device)
    if scale is None and scale_out is None:
        scale_out = torch.empty(2, dtype=torch.float32, device=x.device)
    _check(lib.dybit_quantize_pack_2d(_ptr(x), rows, cols, ld, _fmt(fmt), _ptr(scale), _ptr(packed),
                                      row_stride_bytes, _ptr(scale_out), _stream(stream)),
           "dybit_quantize_pack_2d")
    return packed, (scale if scale is not None else scale_out)


def dybit_decode(packed: torch.Tensor, n: int, fmt, scale: Optional[torch.Tensor] = None,
                 out: Optional[torch.Tensor] = None, stream=None):
    if out is None:
        out = torch.empty(n, dtype=torch.float32, device=packed.device)
    _check(lib.dybit_decode(_ptr(packed), int(n), _fmt(fmt), _ptr(scale), _ptr(out), _stream(stream)),
           "dybit_decode")
    return out


def dybit_gemm(M: int, N: int, K: int, A: torch.Tensor, fa, scale_a: torch.Tensor,
               B: torch.Tensor, fb, scale_b: torch.Tensor, C_out: Optional[torch.Tensor] = None,
               want_raw: bool = False, C_raw: Optional[torch.Tensor] = None,
               ws: Optional[torch.Tensor] = None, lda_bytes: Optional[int] = None,
               ldb_bytes: Optional[int] = None, stream=None):
    """C = sA*sB * value(A) @ value(B)^T.  Returns (C fp32 [M][N], C_raw int32 or None)."""
    lda = A.stride(0) if lda_bytes is None else lda_bytes
    ldb = B.stride(0) if ldb_bytes is None else ldb_bytes
    if C_out is None:
        C_out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    if want_raw and C_raw is None:
        C_raw = torch.empty((M, N), dtype=torch.int32, device=A.device)
    if ws is None:
        ws = torch.empty(dybit_gemm_workspace_bytes(M, N, K, fa, fb) + 1024, dtype=torch.uint8, device=A.device)
    off = (-ws.data_ptr()) % 1024
    ws_ptr = C.c_void_p(ws.data_ptr() + off)
    _check(lib.dybit_gemm(M, N, K, _ptr(A), _fmt(fa), _ptr(scale_a), lda, _ptr(B), _fmt(fb), _ptr(scale_b), ldb,
                          _ptr(C_out), C_out.stride(0), _ptr(C_raw), ws_ptr, ws.numel() - off, _stream(stream)),
           "dybit_gemm")
    return C_out, C_raw


def dybit_conv2d(desc: ConvDesc, X: torch.Tensor, fx, scale_x: torch.Tensor,
                 W: torch.Tensor, fw, scale_w: torch.Tensor, Y: Optional[torch.Tensor] = None,
                 want_raw: bool = False, Y_raw: Optional[torch.Tensor] = None,
                 ws: Optional[torch.Tensor] = None, ldw_bytes: Optional[int] = None, stream=None):
    """Returns (Y fp32 [n][oh][ow][k], Y_raw int32 or None)."""
    oh, ow = dybit_conv2d_out_hw(desc)
    ldw = W.stride(0) if ldw_bytes is None else ldw_bytes
    if Y is None:
        Y = torch.empty((desc.n, oh, ow, desc.k), dtype=torch.float32, device=X.device)
    if want_raw and Y_raw is None:
        Y_raw = torch.empty((desc.n, oh, ow, desc.k), dtype=torch.int32, device=X.device)
    if ws is None:
        ws = torch.empty(dybit_conv2d_workspace_bytes(desc, fx, fw) + 1024, dtype=torch.uint8, device=X.device)
    off = (-ws.data_ptr()) % 1024
    ws_ptr = C.c_void_p(ws.data_ptr() + off)
    cd = _cdesc(desc)
    _check(lib.dybit_conv2d(C.byref(cd), _ptr(X), _fmt(fx), _ptr(scale_x), _ptr(W), _fmt(fw), _ptr(scale_w), ldw,
                            _ptr(Y), _ptr(Y_raw), ws_ptr, ws.numel() - off, _stream(stream)), "dybit_conv2d")
    return Y, Y_raw


def dybit_last_device_status(stream=None) -> Tuple[int, int]:
    detail = C.c_uint32(0)
    st = lib.dybit_last_device_status(_stream(stream), C.byref(detail))
    return int(st), int(detail.value)


def dybit_launch_count() -> int:
    return int(lib.dybit_launch_count())


def dybit_selftest_wait_timeout(limit_ns: int, device=None) -> torch.Tensor:
    """Runs the library's bounded wait on a barrier nobody signals; returns the two result words (device tensor)."""
    result = torch.zeros(2, dtype=torch.int32, device=device or torch.device("cuda", torch.cuda.current_device()))
    _check(lib.dybit_selftest_wait_timeout(int(limit_ns), result.data_ptr(), _stream(None)), "dybit_selftest_wait_timeout")
    return result


def dybit_set_gemm_decode(mode: int) -> None:
    """0: expand pass for both operands; 1: decode B in the GEMM's main loop wherever possible; 2: by shape (default)."""
    _check(lib.dybit_set_gemm_decode(int(mode)), "dybit_set_gemm_decode")


def dybit_set_conv_lowering(mode: int) -> None:
    """0: by shape (default); 1: halo tiles wherever they apply; 2: never halo tiles."""
    _check(lib.dybit_set_conv_lowering(int(mode)), "dybit_set_conv_lowering")


def dybit_profile_next_gemm(ev_start: Optional[torch.cuda.Event], ev_stop: Optional[torch.cuda.Event]):
    """Arms event recording around the next GEMM/conv tensor-core kernel (events need enable_timing=True)."""
    if ev_start is None:
        _check(lib.dybit_profile_next_gemm(None, None), "dybit_profile_next_gemm")
        return
    for ev in (ev_start, ev_stop):
        if not ev.cuda_event:           # torch creates the handle lazily on first record
            ev.record()
    _check(lib.dybit_profile_next_gemm(C.c_void_p(ev_start.cuda_event), C.c_void_p(ev_stop.cuda_event)),
           "dybit_profile_next_gemm")


def dybit_profile_next_gemm_clock(t2: Optional[torch.Tensor]):
    """Arms device-clock recording for the next GEMM/conv tensor-core kernel: t2 is an int64 device tensor of two
    elements, initialised to {-1 (all ones), 0}, that receives {first start, last end} in nanoseconds."""
    if t2 is not None and (t2.dtype != torch.int64 or t2.numel() < 2 or not t2.is_cuda):
        raise ValueError("t2 must be an int64 CUDA tensor of two elements")
    _check(lib.dybit_profile_next_gemm_clock(_ptr(t2)), "dybit_profile_next_gemm_clock")


STATIC_WS_BYTES = 16 * 1024 * 1024   # DYBIT_STATIC_WS_BYTES in include/dybit.h


def dybit_gemm_static_ws(M: int, N: int, K: int, A: torch.Tensor, fa, scale_a: torch.Tensor,
                         B: torch.Tensor, fb, scale_b: torch.Tensor, C_out: torch.Tensor,
                         C_raw: Optional[torch.Tensor] = None, lda_bytes: Optional[int] = None,
                         ldb_bytes: Optional[int] = None, stream=None):
    """dybit_gemm without a workspace argument, for callers that cannot allocate device memory.

    The caller passes every input and output buffer (C_out too: this wrapper creates no tensor);
    the library's built-in scratch array holds the expanded operands.  Problems that need more
    than STATIC_WS_BYTES raise DybitError (status 4).  Calls share the scratch: keep them on one
    stream per device.
    """
    lda = A.stride(0) if lda_bytes is None else lda_bytes
    ldb = B.stride(0) if ldb_bytes is None else ldb_bytes
    _check(lib.dybit_gemm_static_ws(M, N, K, _ptr(A), _fmt(fa), _ptr(scale_a), lda, _ptr(B), _fmt(fb),
                                    _ptr(scale_b), ldb, _ptr(C_out), C_out.stride(0), _ptr(C_raw),
                                    _stream(stream)), "dybit_gemm_static_ws")
    return C_out, C_raw


def _ws_ptr(ws: torch.Tensor):
    off = (-ws.data_ptr()) % 1024
    return C.c_void_p(ws.data_ptr() + off), ws.numel() - off


def _bias_ptr(bias, n):
    if bias is None:
        return None
    if not (bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous() and bias.numel() == n):
        raise ValueError("bias must be a contiguous float32 device tensor with one value per output column")
    return _ptr(bias)


def dybit_gemm_requant(M: int, N: int, K: int, A: torch.Tensor, fa, scale_a: torch.Tensor,
                       B: torch.Tensor, fb, scale_b: torch.Tensor, fq, scale_q: torch.Tensor, relu: bool = False,
                       bias: Optional[torch.Tensor] = None, Q: Optional[torch.Tensor] = None, ldq_bytes: Optional[int] = None,
                       ws: Optional[torch.Tensor] = None, stream=None):
    """GEMM whose result is written as packed DyBit codes of format fq (scale given).  Returns Q [M][ldq] uint8."""
    if ldq_bytes is None:
        ldq_bytes = N * fq[0] // 8
    if Q is None:
        Q = torch.zeros((M, ldq_bytes), dtype=torch.uint8, device=A.device)
    if ws is None:
        ws = torch.empty(dybit_gemm_workspace_bytes(M, N, K, fa, fb) + 1024, dtype=torch.uint8, device=A.device)
    wp, wn = _ws_ptr(ws)
    _check(lib.dybit_gemm_requant(M, N, K, _ptr(A), _fmt(fa), _ptr(scale_a), A.stride(0), _ptr(B), _fmt(fb),
                                  _ptr(scale_b), B.stride(0), _fmt(fq), _ptr(scale_q), _bias_ptr(bias, N), int(bool(relu)),
                                  _ptr(Q), ldq_bytes, wp, wn, _stream(stream)), "dybit_gemm_requant")
    return Q


def dybit_conv2d_requant(desc: ConvDesc, X: torch.Tensor, fx, scale_x: torch.Tensor, W: torch.Tensor, fw,
                         scale_w: torch.Tensor, fq, scale_q: torch.Tensor, relu: bool = False,
                         bias: Optional[torch.Tensor] = None, Q: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """Convolution whose result is the dense NHWK stream of packed codes (the next layer's X).  Returns Q (1-D uint8)."""
    oh, ow = dybit_conv2d_out_hw(desc)
    if Q is None:
        Q = torch.zeros(dybit_packed_bytes(desc.n * oh * ow * desc.k, fq[0]), dtype=torch.uint8, device=X.device)
    if ws is None:
        ws = torch.empty(dybit_conv2d_workspace_bytes(desc, fx, fw) + 1024, dtype=torch.uint8, device=X.device)
    wp, wn = _ws_ptr(ws)
    cd = _cdesc(desc)
    _check(lib.dybit_conv2d_requant(C.byref(cd), _ptr(X), _fmt(fx), _ptr(scale_x), _ptr(W), _fmt(fw), _ptr(scale_w),
                                    W.stride(0), _fmt(fq), _ptr(scale_q), _bias_ptr(bias, desc.k), int(bool(relu)),
                                    _ptr(Q), wp, wn,
                                    _stream(stream)), "dybit_conv2d_requant")
    return Q


def dybit_quantize_conv2d_requant(desc: ConvDesc, X: torch.Tensor, fx, W: torch.Tensor, fw, scale_w: torch.Tensor,
                                  fq, scale_q: torch.Tensor, relu: bool = False, bias: Optional[torch.Tensor] = None,
                                  scale_x: Optional[torch.Tensor] = None, scale_out: Optional[torch.Tensor] = None,
                                  packed: Optional[torch.Tensor] = None, Q: Optional[torch.Tensor] = None,
                                  ws: Optional[torch.Tensor] = None, stream=None):
    """Quantize + pack the fp32 NHWC activation X, convolve its codes with W and write the result as packed codes.
    Returns (Q uint8 dense NHWK stream, packed codes of X uint8, scale of X float32[2])."""
    _dev_f32(X, "X")
    if X.numel() != desc.n * desc.h * desc.w * desc.c:
        raise ValueError("X does not match the descriptor")
    oh, ow = dybit_conv2d_out_hw(desc)
    if Q is None:
        Q = torch.zeros(dybit_packed_bytes(desc.n * oh * ow * desc.k, fq[0]), dtype=torch.uint8, device=X.device)
    if packed is None:
        packed = torch.empty(dybit_packed_bytes(X.numel(), fx[0]), dtype=torch.uint8, device=X.device)
    if scale_out is None:
        scale_out = torch.empty(2, dtype=torch.float32, device=X.device)
    if ws is None:
        ws = torch.empty(dybit_conv2d_workspace_bytes(desc, fx, fw) + 1024, dtype=torch.uint8, device=X.device)
    wp, wn = _ws_ptr(ws)
    cd = _cdesc(desc)
    _check(lib.dybit_quantize_conv2d_requant(C.byref(cd), _ptr(X), _fmt(fx), _ptr(scale_x), _ptr(scale_out), _ptr(packed),
                                             _ptr(W), _fmt(fw), _ptr(scale_w), W.stride(0), _fmt(fq), _ptr(scale_q),
                                             _bias_ptr(bias, desc.k), int(bool(relu)), _ptr(Q), wp, wn, _stream(stream)),
           "dybit_quantize_conv2d_requant")
    return Q, packed, scale_out


def dybit_gemm_batched_workspace_bytes(batch: int, M: int, N: int, K: int, fa, fb) -> int:
    return int(lib.dybit_gemm_batched_workspace_bytes(int(batch), int(M), int(N), int(K), _fmt(fa), _fmt(fb)))


def dybit_gemm_batched(M: int, N: int, K: int, A: torch.Tensor, fa, scale_a: torch.Tensor, B: torch.Tensor, fb,
                       scale_b: torch.Tensor, want_raw: bool = False, C: Optional[torch.Tensor] = None,
                       ws: Optional[torch.Tensor] = None, stream=None):
    """C[b] = A[b] * B[b]^T for packed A [batch][M][row bytes], B [batch][N][row bytes] (uint8, one scale per operand).
    Returns (C float32 [batch][M][N], C_raw int32 or None)."""
    if A.dim() != 3 or B.dim() != 3 or A.shape[0] != B.shape[0] or A.shape[1] != M or B.shape[1] != N:
        raise ValueError("A must be [batch][M][row bytes] and B [batch][N][row bytes]")
    if A.stride(2) != 1 or B.stride(2) != 1:
        raise ValueError("rows of A and B must be contiguous")
    batch = A.shape[0]
    if C is None:
        C = torch.empty((batch, M, N), dtype=torch.float32, device=A.device)
    raw = torch.empty(C.shape, dtype=torch.int32, device=A.device) if want_raw else None
    if raw is not None and not C.is_contiguous():
        raise ValueError("want_raw needs a contiguous C")
    if ws is None:
        ws = torch.empty(dybit_gemm_batched_workspace_bytes(batch, M, N, K, fa, fb) + 1024, dtype=torch.uint8,
                         device=A.device)
    wp, wn = _ws_ptr(ws)
    _check(lib.dybit_gemm_batched(batch, M, N, K, _ptr(A), _fmt(fa), _ptr(scale_a), A.stride(1), A.stride(0),
                                  _ptr(B), _fmt(fb), _ptr(scale_b), B.stride(1), B.stride(0),
                                  _ptr(C), C.stride(1), C.stride(0), _ptr(raw), wp, wn, _stream(stream)),
           "dybit_gemm_batched")
    return C, raw


def dybit_quantize_conv2d(desc: ConvDesc, X: torch.Tensor, fx, W: torch.Tensor, fw, scale_w: torch.Tensor,
                          scale_x: Optional[torch.Tensor] = None, scale_out: Optional[torch.Tensor] = None,
                          packed: Optional[torch.Tensor] = None, want_raw: bool = False,
                          Y: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """Quantize + pack the fp32 NHWC activation X and convolve its codes with the packed weights W in one call.
    Returns (Y float32 [n][oh][ow][k], Y_raw int32 or None, packed codes uint8, scale float32[2])."""
    _dev_f32(X, "X")
    if X.numel() != desc.n * desc.h * desc.w * desc.c:
        raise ValueError("X does not match the descriptor")
    oh, ow = dybit_conv2d_out_hw(desc)
    if Y is None:
        Y = torch.empty((desc.n, oh, ow, desc.k), dtype=torch.float32, device=X.device)
    raw = torch.empty(Y.shape, dtype=torch.int32, device=X.device) if want_raw else None
    if packed is None:
        packed = torch.empty(dybit_packed_bytes(X.numel(), fx[0]), dtype=torch.uint8, device=X.device)
    if scale_out is None:
        scale_out = torch.empty(2, dtype=torch.float32, device=X.device)
    if ws is None:
        ws = torch.empty(dybit_conv2d_workspace_bytes(desc, fx, fw) + 1024, dtype=torch.uint8, device=X.device)
    wp, wn = _ws_ptr(ws)
    cd = _cdesc(desc)
    _check(lib.dybit_quantize_conv2d(C.byref(cd), _ptr(X), _fmt(fx), _ptr(scale_x), _ptr(scale_out), _ptr(packed),
                                     _ptr(W), _fmt(fw), _ptr(scale_w), W.stride(0), _ptr(Y), _ptr(raw), wp, wn,
                                     _stream(stream)), "dybit_quantize_conv2d")
    return Y, raw, packed, scale_out


class ConvLayers:
    """Arguments of dybit_quantize_conv2d for several independent layers, marshalled once into the C array that
    dybit_quantize_expand_layers / dybit_conv2d_prepared take.  Each entry of `layers` is a dict with the keyword
    arguments of dybit_quantize_conv2d (desc, X, fx, W, fw, scale_w and optionally scale_x, scale_out, packed, Y,
    want_raw, ws) or, with fq and scale_q given, of dybit_quantize_conv2d_requant (relu, bias, Q): that layer then
    leaves as packed codes in self.Q[i] instead of fp32 in self.Y[i].  Missing outputs and workspaces are allocated
    here, one workspace per layer."""

    def __init__(self, layers):
        self.n = len(layers)
        self.array = (_CConvLayer * self.n)()
        self.Y, self.raw, self.packed, self.scale, self.Q, self._keep = [], [], [], [], [], []
        for i, a in enumerate(layers):
            desc, X, fx, W, fw = a["desc"], _dev_f32(a["X"], "X"), a["fx"], a["W"], a["fw"]
            if X.numel() != desc.n * desc.h * desc.w * desc.c:
                raise ValueError("X does not match the descriptor")
            oh, ow = dybit_conv2d_out_hw(desc)
            requant = a.get("fq") is not None
            Y, Q, raw = a.get("Y"), a.get("Q"), None
            if requant:
                if Q is None:
                    Q = torch.zeros(dybit_packed_bytes(desc.n * oh * ow * desc.k, a["fq"][0]), dtype=torch.uint8, device=X.device)
                Y = None
            else:
                if Y is None:
                    Y = torch.empty((desc.n, oh, ow, desc.k), dtype=torch.float32, device=X.device)
                if a.get("want_raw"):
                    raw = torch.empty(Y.shape, dtype=torch.int32, device=X.device)
            packed = a.get("packed")
            if packed is None:
                packed = torch.empty(dybit_packed_bytes(X.numel(), fx[0]), dtype=torch.uint8, device=X.device)
            scale_out = a.get("scale_out")
            if scale_out is None:
                scale_out = torch.empty(2, dtype=torch.float32, device=X.device)
            ws = a.get("ws")
            if ws is None:
                ws = torch.empty(dybit_conv2d_workspace_bytes(desc, fx, fw) + 1024, dtype=torch.uint8, device=X.device)
            wp, wn = _ws_ptr(ws)
            c = self.array[i]
            c.desc = _cdesc(desc)
            addr = lambda t: None if t is None else t.data_ptr()
            c.X, c.fx, c.scale_x = addr(X), _fmt(fx), addr(a.get("scale_x"))
            c.scale_x_out, c.X_packed = addr(scale_out), addr(packed)
            c.W, c.fw, c.scale_w, c.ldw_bytes = addr(W), _fmt(fw), addr(a["scale_w"]), W.stride(0)
            c.Y, c.Y_raw, c.ws, c.ws_bytes = addr(Y), addr(raw), wp.value, wn
            if requant:
                bias = a.get("bias")
                c.Q, c.fq, c.scale_q, c.relu = addr(Q), _fmt(a["fq"]), addr(a["scale_q"]), int(bool(a.get("relu")))
                c.bias = None if bias is None else _bias_ptr(bias, desc.k).value
                self._keep.append((a["scale_q"], bias))
            self.Q.append(Q)
            self.Y.append(Y)
            self.raw.append(raw)
            self.packed.append(packed)
            self.scale.append(scale_out)
            self._keep.append((X, W, a["scale_w"], a.get("scale_x"), ws))


def dybit_quantize_expand_layers(layers: ConvLayers, stream=None):
    """Max-abs scales, codes and expanded operands of all the layers, in few launches on one stream."""
    _check(lib.dybit_quantize_expand_layers(layers.array, layers.n, _stream(stream)), "dybit_quantize_expand_layers")


def dybit_conv2d_prepared(layers: ConvLayers, i: int, stream=None):
    """The tensor-core part of layer i, after dybit_quantize_expand_layers.  Returns (Y, Y_raw or None), or (Q, None)
    for a layer with the re-quantizing epilogue."""
    _check(lib.dybit_conv2d_prepared(C.byref(layers.array[i]), _stream(stream)), "dybit_conv2d_prepared")
    return (layers.Y[i] if layers.Q[i] is None else layers.Q[i]), layers.raw[i]


def dybit_conv2d_prepared_layers(layers: ConvLayers, stream=None):
    """The tensor-core part of all layers on one stream, layers of one kernel configuration sharing launches."""
    _check(lib.dybit_conv2d_prepared_layers(layers.array, layers.n, _stream(stream)), "dybit_conv2d_prepared_layers")


def dybit_depthwise_conv2d(desc: ConvDesc, X: torch.Tensor, fx, scale_x: torch.Tensor, W: torch.Tensor, fw,
                           scale_w: torch.Tensor, Y: Optional[torch.Tensor] = None, stream=None):
    """Depth-wise convolution (desc.k == desc.c).  X: dense NHWC code stream; W: [c][row bytes] rows of r*s codes
    (dybit_quantize_pack_2d of the [c][r*s] filter matrix).  Returns Y [n][oh][ow][c] float32."""
    oh, ow = dybit_conv2d_out_hw(desc)
    if Y is None:
        Y = torch.empty((desc.n, oh, ow, desc.c), dtype=torch.float32, device=X.device)
    cd = _cdesc(desc)
    _check(lib.dybit_depthwise_conv2d(C.byref(cd), _ptr(X), _fmt(fx), _ptr(scale_x), _ptr(W), _fmt(fw), _ptr(scale_w),
                                      W.stride(0), _ptr(Y), _stream(stream)), "dybit_depthwise_conv2d")
    return Y


def dybit_rmse(x: torch.Tensor, fmt, scale: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None):
    """Eq. 2.  Returns a float64 device tensor {RMSE, sigma, mse, n}."""
    _dev_f32(x, "x")
    if out is None:
        out = torch.empty(4, dtype=torch.float64, device=x.device)
    _check(lib.dybit_rmse(_ptr(x), x.numel(), _fmt(fmt), _ptr(scale), _ptr(out), _stream(stream)), "dybit_rmse")
    return out


def dybit_rmse_sweep(x: torch.Tensor, fmts, scales: torch.Tensor, stream=None):
    """Eq. 2 for several candidate (format, scale) pairs in one pass over x.  scales: float32 device tensor
    [len(fmts)][2] of {scale, 1/scale}.  Returns (float64 device tensor [len(fmts)][4] of {RMSE, sigma, mse, n},
    int32 device tensor holding the index of the smallest RMSE)."""
    _dev_f32(x, "x")
    nc = len(fmts)
    if not (scales.is_cuda and scales.dtype == torch.float32 and scales.is_contiguous() and scales.numel() == 2 * nc):
        raise ValueError("scales must be a contiguous float32 device tensor with two values per candidate")
    arr = (_CFmt * max(nc, 1))(*[_fmt(f) for f in fmts])
    out = torch.empty((nc, 4), dtype=torch.float64, device=x.device)
    best = torch.empty(1, dtype=torch.int32, device=x.device)
    _check(lib.dybit_rmse_sweep(_ptr(x), x.numel(), nc, arr, _ptr(scales), _ptr(out), _ptr(best), _stream(stream)),
           "dybit_rmse_sweep")
    return out, best


def dybit_fake_quant(x: torch.Tensor, fmt, scale: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None):
    """Quantize-dequantize image of x (QAT forward) in one pass; returns a float32 tensor shaped like x."""
    _dev_f32(x, "x")
    if out is None:
        out = torch.empty_like(x)
    _dev_f32(out, "out")
    _check(lib.dybit_fake_quant(_ptr(x), x.numel(), _fmt(fmt), _ptr(scale), _ptr(out), _stream(stream)),
           "dybit_fake_quant")
    return out


def dybit_fake_quant_backward(x: torch.Tensor, grad_out: torch.Tensor, fmt, scale: torch.Tensor,
                              out: Optional[torch.Tensor] = None, stream=None):
    """Clipped straight-through gradient of dybit_fake_quant with respect to x."""
    _dev_f32(x, "x")
    _dev_f32(grad_out, "grad_out")
    if grad_out.numel() != x.numel():
        raise ValueError("grad_out must have as many elements as x")
    if out is None:
        out = torch.empty_like(x)
    _dev_f32(out, "out")
    _check(lib.dybit_fake_quant_backward(_ptr(x), _ptr(grad_out), x.numel(), _fmt(fmt), _ptr(scale), _ptr(out),
                                         _stream(stream)), "dybit_fake_quant_backward")
    return out


def dybit_search_bitwidths(lat, rmse, num_layers: int, strategy: str, constraint: float, top_k: int):
    """Algorithm 1.  lat / rmse: flat sequences of num_layers*9 numbers, index (layer*3 + a_idx)*3 + w_idx with
    idx 0, 1, 2 <-> 8, 4, 2 bits.  strategy "speedup" (constraint = alpha) or "rmse" (constraint = beta).
    Returns (weight bits, activation bits) as two lists."""
    if len(lat) != num_layers * 9 or len(rmse) != num_layers * 9:
        raise ValueError("lat and rmse need num_layers * 9 entries")
    if strategy not in ("speedup", "rmse"):
        raise ValueError("strategy must be 'speedup' or 'rmse'")
    la = (C.c_double * len(lat))(*[float(v) for v in lat])
    ra = (C.c_double * len(rmse))(*[float(v) for v in rmse])
    w = (C.c_int * num_layers)()
    a = (C.c_int * num_layers)()
    _check(lib.dybit_search_bitwidths(num_layers, la, ra, 0 if strategy == "speedup" else 1, float(constraint),
                                      int(top_k), w, a), "dybit_search_bitwidths")
    return list(w), list(a)
