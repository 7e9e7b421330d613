"""ctypes access to the CPU oracle (``sparq_oracle.c``) -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  The CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparq_oracle.c")
_LIB = os.path.join(_HERE, "libsparq_oracle.so")

MODE_NONE, MODE_BSPARQ, MODE_VSPARQ = 0, 1, 2
ROUND_TRUNCATE, ROUND_NEAREST = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no intrinsics, no fp contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-std=c11",
             "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u, i, p = ctypes.c_uint, ctypes.c_int, ctypes.c_void_p
        i64, sz, f32 = ctypes.c_int64, ctypes.c_size_t, ctypes.c_float
        L.oracle_window_shift.argtypes = [u, i, u]
        L.oracle_window_shift.restype = i
        L.oracle_bsparq.argtypes = [u, i, u, i]
        L.oracle_bsparq.restype = u
        L.oracle_bsparq_window.argtypes = [u, i, u, i, ctypes.POINTER(i)]
        L.oracle_bsparq_window.restype = u
        L.oracle_vsparq_pair.argtypes = [u, u, i, u, i, ctypes.POINTER(u), ctypes.POINTER(u)]
        L.oracle_vsparq_pair.restype = None
        L.oracle_transform.argtypes = [p, p, sz, sz, i, i, u, i]
        L.oracle_transform.restype = None
        L.oracle_pair_fields.argtypes = [u, u, i, u, i, ctypes.POINTER(u), ctypes.POINTER(i),
                                         ctypes.POINTER(u), ctypes.POINTER(i), ctypes.POINTER(i)]
        L.oracle_pair_fields.restype = None
        L.oracle_pack_states.argtypes = [i, u]
        L.oracle_pack_states.restype = i
        L.oracle_pack_ctrl_bits.argtypes = [i, u]
        L.oracle_pack_ctrl_bits.restype = i
        L.oracle_pack.argtypes = [p, sz, sz, i, u, i, p, p]
        L.oracle_pack.restype = i
        L.oracle_unpack.argtypes = [p, p, sz, sz, i, u, p]
        L.oracle_unpack.restype = i
        L.oracle_pair_fields_n.argtypes = [u, u, i, i, u, i, ctypes.POINTER(u), ctypes.POINTER(i),
                                           ctypes.POINTER(u), ctypes.POINTER(i), ctypes.POINTER(i)]
        L.oracle_pair_fields_n.restype = None
        L.oracle_pack_states_n.argtypes = [i, i, u]
        L.oracle_pack_states_n.restype = i
        L.oracle_pack_ctrl_bits_n.argtypes = [i, i, u]
        L.oracle_pack_ctrl_bits_n.restype = i
        L.oracle_pack_n.argtypes = [p, sz, sz, i, i, u, i, p, p]
        L.oracle_pack_n.restype = i
        L.oracle_unpack_n.argtypes = [p, p, sz, sz, i, i, u, p]
        L.oracle_unpack_n.restype = i
        L.oracle_gemm.argtypes = [p, p, p, i64, i64, i64, i, i, u, i]
        L.oracle_gemm.restype = None
        L.oracle_gemm_sparse24.argtypes = [p, p, p, p, i64, i64, i64, i, i, u, i]
        L.oracle_gemm_sparse24.restype = i
        L.oracle_gemm_i64.argtypes = [p, p, p, i64, i64, i64, i, i, u, i]
        L.oracle_gemm_i64.restype = None
        L.oracle_conv2d_nhwc.argtypes = [p, i, i, i, i, p, i, i, i, i, i, i, i, i, i, u, i, p, i64, p]
        L.oracle_conv2d_nhwc.restype = None
        L.oracle_epilogue.argtypes = [p, i64, i64, p, p, i, f32, p, p]
        L.oracle_epilogue.restype = None
        L.oracle_epilogue_residual.argtypes = [p, i64, i64, p, p, p, f32, i, f32, p, p]
        L.oracle_epilogue_residual.restype = None
        L.oracle_absmax.argtypes = [p, i, sz]
        L.oracle_absmax.restype = f32
        L.oracle_quantize_act.argtypes = [p, i, sz, f32, p]
        L.oracle_quantize_act.restype = None
        L.oracle_quantize_weight.argtypes = [p, i64, i64, p, p]
        L.oracle_quantize_weight.restype = None
        L.oracle_num_threads.restype = i
        L.oracle_set_num_threads.argtypes = [i]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


# ---- scalar definitions ---------------------------------------------------

def window_shift(x: int, n: int, mask: int) -> int:
    return lib().oracle_window_shift(x, n, mask)


def bsparq(x: int, n: int, mask: int, rnd: int) -> int:
    return lib().oracle_bsparq(x, n, mask, rnd)


def bsparq_window(x: int, n: int, mask: int, rnd: int) -> Tuple[int, int]:
    """(window bits, shift) of the quantized value."""
    s = ctypes.c_int(0)
    w = lib().oracle_bsparq_window(x, n, mask, rnd, ctypes.byref(s))
    return int(w), int(s.value)


def vsparq_pair(a: int, b: int, n: int, mask: int, rnd: int) -> Tuple[int, int]:
    qa, qb = ctypes.c_uint(0), ctypes.c_uint(0)
    lib().oracle_vsparq_pair(a, b, n, mask, rnd, ctypes.byref(qa), ctypes.byref(qb))
    return int(qa.value), int(qb.value)


# ---- tensor definitions ---------------------------------------------------

def transform(x: np.ndarray, mode: int, n: int, mask: int, rnd: int) -> np.ndarray:
    """T over the last axis (pairs are adjacent along it and never cross rows)."""
    x = _c(x, np.uint8)
    out = np.empty_like(x)
    row_len = x.shape[-1] if x.ndim else 1
    rows = x.size // row_len if row_len else 0
    if x.size:
        lib().oracle_transform(_ptr(x), _ptr(out), rows, row_len, mode, n, mask, rnd)
    return out


# ---- encoded form (Eq. 4, n = 4) -----------------------------------------------

def pair_fields(a: int, b: int, mode: int, mask: int, rnd: int) -> Tuple[int, int, int, int, int]:
    """(in1, opt1, in2, opt2, mux) that the multiplier of Eq. 4 receives for the pair."""
    in1, in2 = ctypes.c_uint(0), ctypes.c_uint(0)
    o1, o2, mux = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    lib().oracle_pair_fields(a, b, mode, mask, rnd, ctypes.byref(in1), ctypes.byref(o1),
                             ctypes.byref(in2), ctypes.byref(o2), ctypes.byref(mux))
    return int(in1.value), int(o1.value), int(in2.value), int(o2.value), int(mux.value)


def pack_states(mode: int, mask: int) -> int:
    return lib().oracle_pack_states(mode, mask)


def pack_ctrl_bits(mode: int, mask: int) -> int:
    return lib().oracle_pack_ctrl_bits(mode, mask)


def pack(x: np.ndarray, mode: int, mask: int, rnd: int) -> Tuple[np.ndarray, np.ndarray]:
    """(data plane, control plane) of the packed stream; rows are the last axis."""
    x = _c(x, np.uint8)
    row_len = x.shape[-1]
    rows = x.size // row_len if row_len else 0
    cb = pack_ctrl_bits(mode, mask)
    data = np.empty(x.size // 2, dtype=np.uint8)
    ctrl = np.empty(x.size // 16 * cb, dtype=np.uint8)
    if lib().oracle_pack(_ptr(x), rows, row_len, mode, mask, rnd, _ptr(data), _ptr(ctrl)) != 0:
        raise ValueError("row length must be a multiple of 16")
    return data, ctrl


def unpack(data: np.ndarray, ctrl: np.ndarray, shape, mode: int, mask: int) -> np.ndarray:
    data, ctrl = _c(data, np.uint8), _c(ctrl, np.uint8)
    out = np.empty(shape, dtype=np.uint8)
    row_len = out.shape[-1]
    rows = out.size // row_len if row_len else 0
    if lib().oracle_unpack(_ptr(data), _ptr(ctrl), rows, row_len, mode, mask, _ptr(out)) != 0:
        raise ValueError("row length must be a multiple of 16")
    return out


# ---- encoded form for any window width (Section 5.1) -------------------------------

def pair_fields_n(a: int, b: int, mode: int, n: int, mask: int, rnd: int) -> Tuple[int, int, int, int, int]:
    """(in1, opt1, in2, opt2, mux) for n-bit windows; a lone value is split into two n-bit halves."""
    in1, in2 = ctypes.c_uint(0), ctypes.c_uint(0)
    o1, o2, mux = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    lib().oracle_pair_fields_n(a, b, mode, n, mask, rnd, ctypes.byref(in1), ctypes.byref(o1),
                               ctypes.byref(in2), ctypes.byref(o2), ctypes.byref(mux))
    return int(in1.value), int(o1.value), int(in2.value), int(o2.value), int(mux.value)


def pack_states_n(mode: int, n: int, mask: int) -> int:
    return lib().oracle_pack_states_n(mode, n, mask)


def pack_ctrl_bits_n(mode: int, n: int, mask: int) -> int:
    return lib().oracle_pack_ctrl_bits_n(mode, n, mask)


def pack_n(x: np.ndarray, mode: int, n: int, mask: int, rnd: int) -> Tuple[np.ndarray, np.ndarray]:
    """(data plane, control plane) for n-bit windows: 2n data bytes and cb control bytes per 16 activations."""
    x = _c(x, np.uint8)
    row_len = x.shape[-1]
    rows = x.size // row_len if row_len else 0
    cb = pack_ctrl_bits_n(mode, n, mask)
    data = np.empty(x.size // 16 * 2 * n, dtype=np.uint8)
    ctrl = np.empty(x.size // 16 * cb, dtype=np.uint8)
    if lib().oracle_pack_n(_ptr(x), rows, row_len, mode, n, mask, rnd, _ptr(data), _ptr(ctrl)) != 0:
        raise ValueError("row length must be a multiple of 16")
    return data, ctrl


def unpack_n(data: np.ndarray, ctrl: np.ndarray, shape, mode: int, n: int, mask: int) -> np.ndarray:
    data, ctrl = _c(data, np.uint8), _c(ctrl, np.uint8)
    out = np.empty(shape, dtype=np.uint8)
    row_len = out.shape[-1]
    rows = out.size // row_len if row_len else 0
    if lib().oracle_unpack_n(_ptr(data), _ptr(ctrl), rows, row_len, mode, n, mask, _ptr(out)) != 0:
        raise ValueError("row length must be a multiple of 16")
    return out


def gemm(A: np.ndarray, B: np.ndarray, mode: int, n: int, mask: int, rnd: int) -> np.ndarray:
    """int32 ``T(A) @ B`` with A (M, K) uint8 and B the logical (K, N) int8 matrix."""
    A, B = _c(A, np.uint8), _c(B, np.int8)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    acc = np.zeros((M, N), dtype=np.int32)
    if acc.size:
        lib().oracle_gemm(_ptr(A), _ptr(B), _ptr(acc), M, N, K, mode, n, mask, rnd)
    return acc


def gemm_sparse24(A: np.ndarray, vals: np.ndarray, pos: np.ndarray, mode: int, n: int, mask: int, rnd: int) -> np.ndarray:
    """int32 product of A (M, K) uint8 with 2:4-compressed weights: vals (N, K/2) int8 and
    their coordinates pos (N, K/2) uint8 inside each group of four; the SPARQ pair is the
    pair of activations the coordinates select."""
    A, vals, pos = _c(A, np.uint8), _c(vals, np.int8), _c(pos, np.uint8)
    M, K = A.shape
    N = vals.shape[0]
    assert vals.shape == (N, K // 2) and pos.shape == (N, K // 2)
    acc = np.zeros((M, N), dtype=np.int32)
    if acc.size and lib().oracle_gemm_sparse24(_ptr(A), _ptr(vals), _ptr(pos), _ptr(acc), M, N, K, mode, n, mask, rnd) != 0:
        raise ValueError("K must be a multiple of 4 and coordinates strictly increasing in 0..3")
    return acc


def gemm_i64(A: np.ndarray, B: np.ndarray, mode: int, n: int, mask: int, rnd: int) -> np.ndarray:
    A, B = _c(A, np.uint8), _c(B, np.int8)
    M, K = A.shape
    _, N = B.shape
    acc = np.zeros((M, N), dtype=np.int64)
    if acc.size:
        lib().oracle_gemm_i64(_ptr(A), _ptr(B), _ptr(acc), M, N, K, mode, n, mask, rnd)
    return acc


def conv2d_nhwc(x: np.ndarray, w: np.ndarray, stride: Tuple[int, int], pad: Tuple[int, int],
                mode: int, n: int, mask: int, rnd: int,
                pixels: Optional[Sequence[int]] = None) -> np.ndarray:
    """int32 direct convolution of NHWC uint8 ``x`` with [cout][r][s][c] int8 ``w``.

    Returns (N, Ho, Wo, Cout), or (len(pixels), Cout) for the listed linear output
    pixel indices only."""
    x, w = _c(x, np.uint8), _c(w, np.int8)
    nb, h, wd, c = x.shape
    cout, r, s, c2 = w.shape
    assert c == c2
    ho = (h + 2 * pad[0] - r) // stride[0] + 1
    wo = (wd + 2 * pad[1] - s) // stride[1] + 1
    if pixels is None:
        acc = np.zeros((nb, ho, wo, cout), dtype=np.int32)
        pix, npix = None, 0
    else:
        pix = _c(pixels, np.int64)
        npix = pix.size
        acc = np.zeros((npix, cout), dtype=np.int32)
    if acc.size:
        lib().oracle_conv2d_nhwc(_ptr(x), nb, h, wd, c, _ptr(w), cout, r, s,
                                 stride[0], stride[1], pad[0], pad[1],
                                 mode, n, mask, rnd, _ptr(pix), npix, _ptr(acc))
    return acc


def epilogue(acc: np.ndarray, scale: np.ndarray, bias: Optional[np.ndarray], relu: bool,
             inv_out_scale: float, residual: Optional[np.ndarray] = None,
             residual_scale: float = 0.0) -> Tuple[np.ndarray, np.ndarray]:
    """(fp32 output, requantized uint8 output) of the int32 accumulators; the
    channel axis is the last one.  `residual` (uint8, same shape) times
    `residual_scale` is added before the ReLU."""
    acc = _c(acc, np.int32)
    N = acc.shape[-1]
    M = acc.size // N if N else 0
    scale = _c(scale, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    f = np.empty(acc.shape, dtype=np.float32)
    q = np.empty(acc.shape, dtype=np.uint8)
    r = None if residual is None else _c(residual, np.uint8)
    if r is not None and r.shape != acc.shape:
        raise ValueError("residual must have the accumulators' shape")
    if acc.size:
        lib().oracle_epilogue_residual(_ptr(acc), M, N, _ptr(scale), _ptr(b), _ptr(r),
                                       ctypes.c_float(residual_scale), int(bool(relu)),
                                       ctypes.c_float(inv_out_scale), _ptr(f), _ptr(q))
    return f, q


# ---- uniform min-max quantization (Section 5) ---------------------------------

def _fp(x: np.ndarray):
    """(contiguous array, is_bf16): float32 arrays as they are, uint16 arrays as bf16 patterns."""
    if x.dtype == np.uint16:
        return np.ascontiguousarray(x), 1
    return _c(x, np.float32), 0


def absmax(x: np.ndarray) -> float:
    x, bf = _fp(x)
    return float(lib().oracle_absmax(_ptr(x), bf, x.size)) if x.size else 0.0


def quantize_act(x: np.ndarray, max_value: float) -> np.ndarray:
    x, bf = _fp(x)
    out = np.empty(x.shape, dtype=np.uint8)
    if x.size:
        lib().oracle_quantize_act(_ptr(x), bf, x.size, ctypes.c_float(max_value), _ptr(out))
    return out


def quantize_weight(w: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(int8 weights, per-kernel scale) of a float32 tensor whose first axis is the kernel."""
    w = _c(w, np.float32)
    cout = w.shape[0]
    k = w.size // cout if cout else 0
    q = np.empty(w.shape, dtype=np.int8)
    sc = np.empty(cout, dtype=np.float32)
    if w.size:
        lib().oracle_quantize_weight(_ptr(w), cout, k, _ptr(q), _ptr(sc))
    return q, sc


def num_threads() -> int:
    return lib().oracle_num_threads()


def set_num_threads(t: int) -> None:
    lib().oracle_set_num_threads(int(t))
