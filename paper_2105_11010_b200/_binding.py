"""ctypes binding with the same names as the C ABI in ``include/sparq.h``.

Argument marshalling only.  Tensors must already live on the CUDA device (the
raw ``data_ptr`` is handed to the library) and work is enqueued on torch's
current stream unless a stream is given.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

MODE_NONE, MODE_BSPARQ, MODE_VSPARQ = 0, 1, 2
ROUND_TRUNCATE, ROUND_NEAREST = 0, 1
SET_5OPT, SET_3OPT, SET_2OPT, SET_6OPT, SET_7OPT = 0x1F, 0x15, 0x11, 0x3F, 0x7F

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libsparq_b200.so")


class SparqError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"sparq error {code}: {text}")
        self.code = code


class _CParams(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("window_bits", ctypes.c_int32),
                ("placement_mask", ctypes.c_uint32), ("rounding", ctypes.c_int32)]


class _CEpilogue(ctypes.Structure):
    _fields_ = [("scale", ctypes.c_void_p), ("bias", ctypes.c_void_p),
                ("relu", ctypes.c_int32), ("inv_out_scale", ctypes.c_float),
                ("acc_out", ctypes.c_void_p), ("f32_out", ctypes.c_void_p),
                ("u8_out", ctypes.c_void_p), ("next_transform", ctypes.POINTER(_CParams)),
                ("residual", ctypes.c_void_p), ("residual_scale", ctypes.c_float)]


@dataclass(frozen=True)
class SparqParams:
    """Mirror of ``sparq_params``."""
    mode: int = MODE_VSPARQ
    window_bits: int = 4
    placement_mask: int = SET_5OPT
    rounding: int = ROUND_NEAREST

    def _c(self) -> _CParams:
        return _CParams(self.mode, self.window_bits, self.placement_mask, self.rounding)


_lib: Optional[ctypes.CDLL] = None


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads the built C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2105_11010_b200.build` "
                "(needs nvcc); this package has no CPU fallback")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
        L.sparq_quantize.argtypes = [vp, vp, sz, sz, ctypes.POINTER(_CParams), vp]
        L.sparq_quantize.restype = i32
        L.sparq_gemm_s8.argtypes = [vp, i64, vp, i64, i64, i64, i64,
                                    ctypes.POINTER(_CParams), ctypes.POINTER(_CEpilogue), vp]
        L.sparq_gemm_s8.restype = i32
        L.sparq_conv2d_nhwc_s8.argtypes = [vp, i32, i32, i32, i32, vp, i32, i32, i32,
                                           i32, i32, i32, i32,
                                           ctypes.POINTER(_CParams), ctypes.POINTER(_CEpilogue), vp]
        L.sparq_conv2d_nhwc_s8.restype = i32
        L.sparq_packed_ctrl_bits.argtypes = [ctypes.POINTER(_CParams)]
        L.sparq_packed_ctrl_bits.restype = i32
        L.sparq_pack.argtypes = [vp, sz, sz, ctypes.POINTER(_CParams), vp, vp, vp]
        L.sparq_pack.restype = i32
        L.sparq_unpack.argtypes = [vp, vp, sz, sz, ctypes.POINTER(_CParams), vp, vp]
        L.sparq_unpack.restype = i32
        L.sparq_absmax.argtypes = [vp, i32, sz, vp, vp]
        L.sparq_absmax.restype = i32
        L.sparq_quantize_act_u8.argtypes = [vp, i32, sz, vp, vp, vp]
        L.sparq_quantize_act_u8.restype = i32
        L.sparq_quantize_weight_s8.argtypes = [vp, i64, i64, vp, vp, vp]
        L.sparq_quantize_weight_s8.restype = i32
        L.sparq_sparse24_expanded_k.argtypes = [i64, ctypes.POINTER(_CParams)]
        L.sparq_sparse24_expanded_k.restype = i64
        L.sparq_sparse24_expand_weights.argtypes = [vp, vp, i64, i64, ctypes.POINTER(_CParams), vp, vp]
        L.sparq_sparse24_expand_weights.restype = i32
        L.sparq_sparse24_expand_activations.argtypes = [vp, sz, sz, ctypes.POINTER(_CParams), vp, vp]
        L.sparq_sparse24_expand_activations.restype = i32
        L.sparq_gemm_s8_sparse24.argtypes = [vp, vp, i64, i64, i64, ctypes.POINTER(_CParams),
                                             ctypes.POINTER(_CEpilogue), vp, vp]
        L.sparq_gemm_s8_sparse24.restype = i32
        L.sparq_quantize_host.argtypes = L.sparq_quantize.argtypes
        L.sparq_quantize_host.restype = i32
        L.sparq_gemm_s8_host.argtypes = L.sparq_gemm_s8.argtypes
        L.sparq_gemm_s8_host.restype = i32
        L.sparq_conv2d_nhwc_s8_host.argtypes = L.sparq_conv2d_nhwc_s8.argtypes
        L.sparq_conv2d_nhwc_s8_host.restype = i32
        L.sparq_gemm_s8_static.argtypes = L.sparq_gemm_s8.argtypes
        L.sparq_gemm_s8_static.restype = i32
        L.sparq_selftest_wait_timeout.argtypes = [i64, i32, vp, vp]
        L.sparq_selftest_wait_timeout.restype = i32
        L.sparq_selftest_mma_rate.argtypes = [i32, i32, vp, vp]
        L.sparq_selftest_mma_rate.restype = i32
        L.sparq_check.argtypes = [vp]
        L.sparq_check.restype = i32
        L.sparq_last_error.argtypes = []
        L.sparq_last_error.restype = ctypes.c_char_p
        L.sparq_shutdown.argtypes = []
        L.sparq_shutdown.restype = i32
        _lib = L
    return _lib


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _dev(t: Optional[torch.Tensor], dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr() or None


def _raise(code: int) -> None:
    if code != 0:
        raise SparqError(code, sparq_last_error())


def sparq_last_error() -> str:
    return load_library().sparq_last_error().decode()


def sparq_check(stream=None) -> None:
    _raise(load_library().sparq_check(_stream_ptr(stream)))


def sparq_selftest_wait_timeout(limit_cycles: int, report: torch.Tensor, use_static_word: bool = False,
                                stream=None) -> None:
    """Diagnostic launch whose bounded wait runs out; ``report`` is 4 int32/uint32 words on the device."""
    if report.numel() < 4 or report.element_size() != 4 or not report.is_cuda:
        raise ValueError("report must hold four 32-bit words on the device")
    _raise(load_library().sparq_selftest_wait_timeout(int(limit_cycles), int(bool(use_static_word)),
                                                      report.data_ptr(), _stream_ptr(stream)))


def sparq_selftest_mma_rate(bn: int, iters: int, cycles_out: torch.Tensor, stream=None) -> int:
    """MMA-only loop on every SM; ``cycles_out`` (int64, one per SM, device) receives each CTA's cycles.
    Returns the number of CTAs launched."""
    if cycles_out.dtype != torch.int64 or not cycles_out.is_cuda or cycles_out.numel() < 256:
        raise ValueError("cycles_out must be an int64 device tensor of at least 256 elements")
    rc = load_library().sparq_selftest_mma_rate(int(bn), int(iters), cycles_out.data_ptr(), _stream_ptr(stream))
    if rc < 0:
        _raise(rc)
    return rc


def sparq_shutdown() -> None:
    _raise(load_library().sparq_shutdown())


def sparq_quantize(inp: torch.Tensor, out: torch.Tensor, rows: int, row_len: int,
                   params: SparqParams, stream=None) -> None:
    """``out = T(inp)`` for ``rows`` rows of ``row_len`` uint8 activations."""
    if inp.numel() < rows * row_len or out.numel() < rows * row_len:
        raise ValueError("tensor smaller than rows * row_len")
    p = params._c()
    _raise(load_library().sparq_quantize(_dev(inp, torch.uint8, "inp"), _dev(out, torch.uint8, "out"),
                                         rows, row_len, ctypes.byref(p), _stream_ptr(stream)))


def _next(next_transform):
    """(pointer for the struct, object that keeps the pointee alive)"""
    if next_transform is None:
        return None, None
    c = next_transform._c()
    return ctypes.pointer(c), c


def _epilogue(n_cols: int, scale, bias, relu, inv_out_scale, acc_out, f32_out, u8_out, next_transform=None,
              residual=None, residual_scale=0.0) -> _CEpilogue:
    for name, t in (("scale", scale), ("bias", bias)):
        if t is not None and t.numel() < n_cols:
            raise ValueError(f"{name} has fewer than N elements")
    return _CEpilogue(_dev(scale, torch.float32, "scale"), _dev(bias, torch.float32, "bias"),
                      int(bool(relu)), float(inv_out_scale),
                      _dev(acc_out, torch.int32, "acc_out"), _dev(f32_out, torch.float32, "f32_out"),
                      _dev(u8_out, torch.uint8, "u8_out"), _next(next_transform)[0],
                      _dev(residual, torch.uint8, "residual"), float(residual_scale))


def sparq_gemm_s8(A: torch.Tensor, B: torch.Tensor, params: SparqParams, *,
                  scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                  relu: bool = False, inv_out_scale: float = 1.0,
                  acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                  u8_out: Optional[torch.Tensor] = None,
                  next_transform: Optional[SparqParams] = None,
                  residual: Optional[torch.Tensor] = None, residual_scale: float = 0.0, stream=None) -> None:
    """``acc = T(A) @ B^T`` with A (M, K) uint8 and B (N, K) int8, then the epilogue."""
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    for name, t in (("acc_out", acc_out), ("f32_out", f32_out), ("u8_out", u8_out), ("residual", residual)):
        if t is not None and t.numel() < M * N:
            raise ValueError(f"{name} has fewer than M*N elements")
    p = params._c()
    e = _epilogue(N, scale, bias, relu, inv_out_scale, acc_out, f32_out, u8_out, next_transform,
                  residual, residual_scale)
    _raise(load_library().sparq_gemm_s8(_dev(A, torch.uint8, "A"), K, _dev(B, torch.int8, "B"), K,
                                        M, N, K, ctypes.byref(p), ctypes.byref(e), _stream_ptr(stream)))


def sparq_conv2d_nhwc_s8(x: torch.Tensor, w: torch.Tensor, stride, pad, params: SparqParams, *,
                         scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                         relu: bool = False, inv_out_scale: float = 1.0,
                         acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                         u8_out: Optional[torch.Tensor] = None,
                  next_transform: Optional[SparqParams] = None,
                  residual: Optional[torch.Tensor] = None, residual_scale: float = 0.0, stream=None) -> None:
    """Fused convolution of NHWC uint8 ``x`` with [cout][r][s][c] int8 ``w``."""
    nb, h, wd, c = x.shape
    cout, r, s, c2 = w.shape
    if c != c2:
        raise ValueError("x and w disagree on the channel count")
    ho = (h + 2 * pad[0] - r) // stride[0] + 1
    wo = (wd + 2 * pad[1] - s) // stride[1] + 1
    m = nb * ho * wo
    for name, t in (("acc_out", acc_out), ("f32_out", f32_out), ("u8_out", u8_out), ("residual", residual)):
        if t is not None and t.numel() < m * cout:
            raise ValueError(f"{name} has fewer than N*Ho*Wo*Cout elements")
    p = params._c()
    e = _epilogue(cout, scale, bias, relu, inv_out_scale, acc_out, f32_out, u8_out, next_transform,
                  residual, residual_scale)
    _raise(load_library().sparq_conv2d_nhwc_s8(_dev(x, torch.uint8, "x"), nb, h, wd, c,
                                               _dev(w, torch.int8, "w"), cout, r, s,
                                               stride[0], stride[1], pad[0], pad[1],
                                               ctypes.byref(p), ctypes.byref(e), _stream_ptr(stream)))


# ---- packed stream ------------------------------------------------------------------------

def sparq_packed_ctrl_bits(params: SparqParams) -> int:
    """Control bits per pair of the packed stream for these parameters."""
    p = params._c()
    rc = load_library().sparq_packed_ctrl_bits(ctypes.byref(p))
    if rc < 0:
        _raise(rc)
    return rc


def _rows(t: torch.Tensor):
    row_len = t.shape[-1] if t.dim() else 1
    return (t.numel() // row_len if row_len else 0), row_len


def sparq_pack(inp: torch.Tensor, params: SparqParams, data: torch.Tensor, ctrl: torch.Tensor, stream=None) -> None:
    """Packed stream of ``inp`` (rows along the last axis) into the caller's ``data``
    (numel / 16 * 2 * window_bits bytes) and ``ctrl`` (numel / 16 * ctrl_bits bytes) planes."""
    rows, row_len = _rows(inp)
    cb = sparq_packed_ctrl_bits(params)
    if data.numel() < inp.numel() // 16 * 2 * params.window_bits or ctrl.numel() < inp.numel() // 16 * cb:
        raise ValueError("data / ctrl plane too small")
    p = params._c()
    _raise(load_library().sparq_pack(_dev(inp, torch.uint8, "inp"), rows, row_len, ctypes.byref(p),
                                     _dev(data, torch.uint8, "data"), _dev(ctrl, torch.uint8, "ctrl"),
                                     _stream_ptr(stream)))


def sparq_unpack(data: torch.Tensor, ctrl: torch.Tensor, params: SparqParams, out: torch.Tensor, stream=None) -> None:
    """``out`` (rows along the last axis) = T(x) of the packed stream."""
    rows, row_len = _rows(out)
    cb = sparq_packed_ctrl_bits(params)
    if data.numel() < out.numel() // 16 * 2 * params.window_bits or ctrl.numel() < out.numel() // 16 * cb:
        raise ValueError("data / ctrl plane too small")
    p = params._c()
    _raise(load_library().sparq_unpack(_dev(data, torch.uint8, "data"), _dev(ctrl, torch.uint8, "ctrl"),
                                       rows, row_len, ctypes.byref(p), _dev(out, torch.uint8, "out"),
                                       _stream_ptr(stream)))


# ---- uniform min-max quantization front end -----------------------------------------------

DTYPE_F32, DTYPE_BF16 = 0, 1


def _float_ptr(x: torch.Tensor, name: str):
    if x is None or not x.is_cuda or not x.is_contiguous() or x.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"{name} must be a contiguous CUDA tensor of float32 or bfloat16")
    return x.data_ptr(), (DTYPE_BF16 if x.dtype == torch.bfloat16 else DTYPE_F32)


def sparq_absmax(x: torch.Tensor, max_inout: torch.Tensor, stream=None) -> None:
    """``max_inout[0] = max(max_inout[0], max |x|)`` on the device (float32, 1 element)."""
    ptr, dt = _float_ptr(x, "x")
    _raise(load_library().sparq_absmax(ptr, dt, x.numel(), _dev(max_inout, torch.float32, "max_inout"),
                                       _stream_ptr(stream)))


def sparq_quantize_act_u8(x: torch.Tensor, max_dev: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """Unsigned symmetric per-layer quantization of ``x`` onto [0, max] in 255 steps."""
    ptr, dt = _float_ptr(x, "x")
    if out.numel() < x.numel():
        raise ValueError("out is smaller than x")
    _raise(load_library().sparq_quantize_act_u8(ptr, dt, x.numel(), _dev(max_dev, torch.float32, "max_dev"),
                                                _dev(out, torch.uint8, "out"), _stream_ptr(stream)))


def sparq_quantize_weight_s8(w: torch.Tensor, out: torch.Tensor, scale_out: torch.Tensor, stream=None) -> None:
    """Signed symmetric per-kernel quantization of float32 ``w`` (kernels along axis 0)."""
    cout = w.shape[0]
    k = w.numel() // cout if cout else 0
    if out.numel() < w.numel() or scale_out.numel() < cout:
        raise ValueError("out / scale_out too small")
    _raise(load_library().sparq_quantize_weight_s8(_dev(w, torch.float32, "w"), cout, k, _dev(out, torch.int8, "out"),
                                                   _dev(scale_out, torch.float32, "scale_out"), _stream_ptr(stream)))


# ---- 2:4 sparse weights ---------------------------------------------------------------------

def sparq_sparse24_expanded_k(K: int, params: SparqParams) -> int:
    p = params._c()
    rc = load_library().sparq_sparse24_expanded_k(K, ctypes.byref(p))
    if rc < 0:
        _raise(int(rc))
    return int(rc)


def sparq_sparse24_expand_weights(vals: torch.Tensor, pos: torch.Tensor, params: SparqParams, w_exp: torch.Tensor,
                                  stream=None) -> None:
    """Compressed 2:4 weights (vals, pos: (N, K/2)) -> ``w_exp`` (N, K')."""
    N = vals.shape[0]
    K = 2 * (vals.numel() // N) if N else 0
    if pos.numel() != vals.numel() or w_exp.numel() < N * sparq_sparse24_expanded_k(K, params):
        raise ValueError("pos / w_exp size does not match vals")
    p = params._c()
    _raise(load_library().sparq_sparse24_expand_weights(_dev(vals, torch.int8, "vals"), _dev(pos, torch.uint8, "pos"),
                                                        N, K, ctypes.byref(p), _dev(w_exp, torch.int8, "w_exp"),
                                                        _stream_ptr(stream)))


def sparq_sparse24_expand_activations(A: torch.Tensor, params: SparqParams, a_exp: torch.Tensor, stream=None) -> None:
    """Activations (rows along the last axis, K) -> ``a_exp`` with K' per row."""
    rows, K = _rows(A)
    if a_exp.numel() < rows * sparq_sparse24_expanded_k(K, params):
        raise ValueError("a_exp too small")
    p = params._c()
    _raise(load_library().sparq_sparse24_expand_activations(_dev(A, torch.uint8, "A"), rows, K, ctypes.byref(p),
                                                            _dev(a_exp, torch.uint8, "a_exp"), _stream_ptr(stream)))


def sparq_gemm_s8_sparse24(A: torch.Tensor, w_exp: torch.Tensor, params: SparqParams, *,
                           workspace: Optional[torch.Tensor] = None,
                           scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                           relu: bool = False, inv_out_scale: float = 1.0,
                           acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                           u8_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """``acc[m][j] = sum_g T2(selected pair) . (v0, v1)`` for 2:4 weights expanded by
    :func:`sparq_sparse24_expand_weights`, then the epilogue."""
    M, K = A.shape
    N = w_exp.shape[0]
    kx = sparq_sparse24_expanded_k(K, params)
    if w_exp.numel() != N * kx:
        raise ValueError("w_exp does not have N * K' elements")
    if workspace is not None and workspace.numel() < M * kx:
        raise ValueError("workspace smaller than M * K'")
    p = params._c()
    e = _epilogue(N, scale, bias, relu, inv_out_scale, acc_out, f32_out, u8_out)
    _raise(load_library().sparq_gemm_s8_sparse24(_dev(A, torch.uint8, "A"), _dev(w_exp, torch.int8, "w_exp"), M, N, K,
                                                 ctypes.byref(p), ctypes.byref(e),
                                                 _dev(workspace, torch.uint8, "workspace"), _stream_ptr(stream)))


# ---- host-buffer forms ------------------------------------------------------------------

def _host(t: Optional[torch.Tensor], dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda:
        raise ValueError(f"{name} must be a CPU tensor (pinned for asynchronous copies)")
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous {dtype} tensor")
    return t.data_ptr() or None


def sparq_quantize_host(inp: torch.Tensor, out: torch.Tensor, rows: int, row_len: int,
                        params: SparqParams, stream=None) -> None:
    """Host-buffer form of :func:`sparq_quantize`; returns after the result is in ``out``."""
    if inp.numel() < rows * row_len or out.numel() < rows * row_len:
        raise ValueError("tensor smaller than rows * row_len")
    p = params._c()
    _raise(load_library().sparq_quantize_host(_host(inp, torch.uint8, "inp"), _host(out, torch.uint8, "out"),
                                              rows, row_len, ctypes.byref(p), _stream_ptr(stream)))


def sparq_gemm_s8_host(A: torch.Tensor, B: torch.Tensor, params: SparqParams, *,
                       scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                       relu: bool = False, inv_out_scale: float = 1.0,
                       acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                       u8_out: Optional[torch.Tensor] = None,
                  residual: Optional[torch.Tensor] = None, residual_scale: float = 0.0, stream=None) -> None:
    """Host-buffer form of :func:`sparq_gemm_s8`: ``A`` and the outputs are CPU tensors."""
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    for name, t in (("acc_out", acc_out), ("f32_out", f32_out), ("u8_out", u8_out), ("residual", residual)):
        if t is not None and t.numel() < M * N:
            raise ValueError(f"{name} has fewer than M*N elements")
    p = params._c()
    e = _CEpilogue(_dev(scale, torch.float32, "scale"), _dev(bias, torch.float32, "bias"),
                   int(bool(relu)), float(inv_out_scale),
                   _host(acc_out, torch.int32, "acc_out"), _host(f32_out, torch.float32, "f32_out"),
                   _host(u8_out, torch.uint8, "u8_out"), None,
                   _host(residual, torch.uint8, "residual"), float(residual_scale))
    _raise(load_library().sparq_gemm_s8_host(_host(A, torch.uint8, "A"), K, _dev(B, torch.int8, "B"), K,
                                             M, N, K, ctypes.byref(p), ctypes.byref(e), _stream_ptr(stream)))


def sparq_conv2d_nhwc_s8_host(x: torch.Tensor, w: torch.Tensor, stride, pad, params: SparqParams, *,
                              scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                              relu: bool = False, inv_out_scale: float = 1.0,
                              acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                              u8_out: Optional[torch.Tensor] = None,
                  residual: Optional[torch.Tensor] = None, residual_scale: float = 0.0, stream=None) -> None:
    """Host-buffer form of :func:`sparq_conv2d_nhwc_s8`: ``x`` and the outputs are CPU tensors."""
    nb, h, wd, c = x.shape
    cout, r, s, c2 = w.shape
    if c != c2:
        raise ValueError("x and w disagree on the channel count")
    ho = (h + 2 * pad[0] - r) // stride[0] + 1
    wo = (wd + 2 * pad[1] - s) // stride[1] + 1
    m = nb * ho * wo
    for name, t in (("acc_out", acc_out), ("f32_out", f32_out), ("u8_out", u8_out), ("residual", residual)):
        if t is not None and t.numel() < m * cout:
            raise ValueError(f"{name} has fewer than N*Ho*Wo*Cout elements")
    p = params._c()
    e = _CEpilogue(_dev(scale, torch.float32, "scale"), _dev(bias, torch.float32, "bias"),
                   int(bool(relu)), float(inv_out_scale),
                   _host(acc_out, torch.int32, "acc_out"), _host(f32_out, torch.float32, "f32_out"),
                   _host(u8_out, torch.uint8, "u8_out"), None,
                   _host(residual, torch.uint8, "residual"), float(residual_scale))
    _raise(load_library().sparq_conv2d_nhwc_s8_host(_host(x, torch.uint8, "x"), nb, h, wd, c,
                                                    _dev(w, torch.int8, "w"), cout, r, s,
                                                    stride[0], stride[1], pad[0], pad[1],
                                                    ctypes.byref(p), ctypes.byref(e), _stream_ptr(stream)))


STATIC_SCRATCH_BYTES = 8 << 20


def sparq_gemm_s8_static(A: torch.Tensor, B: torch.Tensor, params: SparqParams, *,
                         scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                         relu: bool = False, inv_out_scale: float = 1.0,
                         acc_out: Optional[torch.Tensor] = None, f32_out: Optional[torch.Tensor] = None,
                         u8_out: Optional[torch.Tensor] = None,
                  next_transform: Optional[SparqParams] = None,
                  residual: Optional[torch.Tensor] = None, residual_scale: float = 0.0, stream=None) -> None:
    """``sparq_gemm_s8`` for hosts that must not allocate device memory once running
    (all free memory already belongs to a framework's pool, or an allocation's
    device-wide synchronization is not acceptable).  Same result, computed as transform
    kernel + plain GEMM with the transformed activations in a fixed scratch array inside
    the library (``M * K <= STATIC_SCRATCH_BYTES``).  Synchronous; one call at a time per
    device.  The first call on a device performs the address look-up: make it before any
    stream capture."""
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    for name, t in (("acc_out", acc_out), ("f32_out", f32_out), ("u8_out", u8_out), ("residual", residual)):
        if t is not None and t.numel() < M * N:
            raise ValueError(f"{name} has fewer than M*N elements")
    p = params._c()
    e = _epilogue(N, scale, bias, relu, inv_out_scale, acc_out, f32_out, u8_out, next_transform,
                  residual, residual_scale)
    _raise(load_library().sparq_gemm_s8_static(_dev(A, torch.uint8, "A"), K, _dev(B, torch.int8, "B"), K,
                                               M, N, K, ctypes.byref(p), ctypes.byref(e), _stream_ptr(stream)))
