"""ctypes wrapper of the CPU oracle (``qfmt_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the benchmark's CPU-baseline
leg.  The product package never imports this module, and this module never imports the
product package.  Marshalling only: every piece of arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qfmt_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

STATS_WORDS = 264
ST_TOTAL, ST_ZERO_IN, ST_DENORMAL, ST_UNDERFLOW, ST_OVERFLOW, ST_NAN, ST_INF_IN = range(256, 263)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent outputs only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib: Optional[ctypes.CDLL] = None


def _L() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u32, i32, i64, sz, vp = (ctypes.c_uint32, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t,
                                 ctypes.c_void_p)
        for name in ("oracle_bias", "oracle_emax", "oracle_emin", "oracle_min_normal_log2"):
            getattr(lib, name).argtypes = [i32]
            getattr(lib, name).restype = i32
        lib.oracle_min_denormal_log2.argtypes = [i32, i32]
        lib.oracle_min_denormal_log2.restype = i32
        lib.oracle_max_normal.argtypes = [i32, i32]
        lib.oracle_max_normal.restype = ctypes.c_double
        lib.oracle_scale_bits.argtypes = [u32, u32]
        lib.oracle_scale_bits.restype = u32
        lib.oracle_quantize_bits.argtypes = [u32, i32, i32, i32, ctypes.POINTER(ctypes.c_int)]
        lib.oracle_quantize_bits.restype = u32
        lib.oracle_decode_code.argtypes = [u32, i32, i32]
        lib.oracle_decode_code.restype = u32
        lib.oracle_encode_code.argtypes = [u32, i32, i32]
        lib.oracle_encode_code.restype = u32
        lib.oracle_quantize_stats.argtypes = [vp, vp, sz, i32, i32, i32, u32, vp]
        lib.oracle_quantize_stats.restype = None
        lib.oracle_quantize_stats_threads.argtypes = [vp, vp, sz, i32, i32, i32, u32, vp, i32]
        lib.oracle_quantize_stats_threads.restype = None
        lib.oracle_gemm.argtypes = [vp, i64, i32, vp, i64, i32, i64, i64, i64, vp, vp]
        lib.oracle_gemm.restype = None
        lib.oracle_gemm_sampled.argtypes = [vp, i64, i32, vp, i64, i32, i64, vp, vp, i64, vp, vp]
        lib.oracle_gemm_sampled.restype = None
        lib.oracle_conv.argtypes = [i32, vp, vp, vp, vp, i64, vp, vp]
        lib.oracle_conv.restype = None
        lib.oracle_add_round_bits.argtypes = [u32, u32, i32, i32, i32]
        lib.oracle_add_round_bits.restype = u32
        lib.oracle_fmac_bits.argtypes = [u32, u32, u32, i32, i32, i32]
        lib.oracle_fmac_bits.restype = u32
        lib.oracle_bias_quantize_stats.argtypes = [vp, i64, i64, i64, vp, vp, i64, i32, i32, i32, u32, vp]
        lib.oracle_bias_quantize_stats.restype = None
        lib.oracle_fmac8_gemm.argtypes = [vp, i64, i32, vp, i64, i32, i64, i64, i64, i32, i32, i32, i32, vp, vp]
        lib.oracle_fmac8_gemm.restype = None
        lib.oracle_fmac8_gemm_sampled.argtypes = [vp, i64, i32, vp, i64, i32, i64, i32, i32, i32, i32, vp, vp,
                                                  i64, vp]
        lib.oracle_fmac8_gemm_sampled.restype = None
        lib.oracle_quantize_stats_pack16.argtypes = [vp, vp, sz, i32, i32, i32, u32, vp]
        lib.oracle_quantize_stats_pack16.restype = None
        lib.oracle_unpack16.argtypes = [vp, vp, sz, i32, i32]
        lib.oracle_unpack16.restype = None
        lib.oracle_dls_update.argtypes = [vp, vp, i64]
        lib.oracle_dls_update.restype = None
        lib.oracle_conv_fmac8.argtypes = [i32, vp, vp, vp, i32, i32, i32, i32, vp, i64, vp, vp]
        lib.oracle_conv_fmac8.restype = None
        _lib = lib
    return _lib


def _f32_bits(x: float) -> int:
    return int(np.array([x], dtype=np.float32).view(np.uint32)[0])


# ---- format constants -------------------------------------------------------------------------
def bias(e: int) -> int:
    return _L().oracle_bias(e)


def emin(e: int) -> int:
    return _L().oracle_emin(e)


def emax(e: int) -> int:
    return _L().oracle_emax(e)


def min_denormal_log2(e: int, m: int) -> int:
    return _L().oracle_min_denormal_log2(e, m)


def max_normal(e: int, m: int) -> float:
    return _L().oracle_max_normal(e, m)


# ---- scalar entry points ----------------------------------------------------------------------
def scale_bits(xbits: int, sbits: int) -> int:
    return _L().oracle_scale_bits(xbits, sbits)


def quantize_bits(ybits: int, e: int, m: int, denormals: int = 1) -> Tuple[int, int]:
    flag = ctypes.c_int(0)
    q = _L().oracle_quantize_bits(ybits, e, m, denormals, ctypes.byref(flag))
    return q, flag.value


def decode_code(code: int, e: int, m: int) -> int:
    return _L().oracle_decode_code(code, e, m)


def encode_code(qbits: int, e: int, m: int) -> int:
    return _L().oracle_encode_code(qbits, e, m)


def add_round_bits(abits: int, bbits: int, e: int, m: int, denormals: int = 1) -> int:
    """round(a + b) to (e, m): the exact sum of two fp32 words, rounded once."""
    return _L().oracle_add_round_bits(abits, bbits, e, m, denormals)


def fmac_bits(abits: int, xbits: int, ybits: int, e: int, m: int, denormals: int = 1) -> int:
    """FMAC: round(a + x*y) to (e, m), one rounding of the exact value."""
    return _L().oracle_fmac_bits(abits, xbits, ybits, e, m, denormals)


# ---- tensors ----------------------------------------------------------------------------------
def quantize_stats(x: np.ndarray, e: int, m: int, denormals: int = 1, loss_scale: float = 1.0,
                   want_q: bool = True, want_stats: bool = True, threads: int = 1):
    """Returns (q as float32 array shaped like x or None, stats as uint64[264] or None).
    threads > 1 cuts the tensor into that many pieces handled in parallel (records summed)."""
    xf = np.ascontiguousarray(x, dtype=np.float32)
    xb = xf.view(np.uint32).reshape(-1)
    q = np.empty_like(xb) if want_q else None
    st = np.zeros(STATS_WORDS, dtype=np.uint64) if want_stats else None
    args = (xb.ctypes.data, q.ctypes.data if want_q else None, xb.size, e, m, int(denormals), _f32_bits(loss_scale),
            st.ctypes.data if want_stats else None)
    if threads > 1:
        _L().oracle_quantize_stats_threads(*args, int(threads))
    else:
        _L().oracle_quantize_stats(*args)
    return (q.view(np.float32).reshape(xf.shape) if want_q else None), st


def quantize_stats_pack16(x: np.ndarray, e: int, m: int, denormals: int = 1, loss_scale: float = 1.0):
    """Rounded tensor as packed 16-bit codes (uint16, shaped like x) and its statistics."""
    xf = np.ascontiguousarray(x, dtype=np.float32)
    xb = xf.view(np.uint32).reshape(-1)
    codes = np.empty(xb.size, dtype=np.uint16)
    st = np.zeros(STATS_WORDS, dtype=np.uint64)
    _L().oracle_quantize_stats_pack16(xb.ctypes.data, codes.ctypes.data, xb.size, e, m, int(denormals),
                                      _f32_bits(loss_scale), st.ctypes.data)
    return codes.reshape(xf.shape), st


def unpack16(codes: np.ndarray, e: int, m: int) -> np.ndarray:
    """fp32 containers of packed 16-bit codes."""
    c = np.ascontiguousarray(codes, dtype=np.uint16)
    q = np.empty(c.size, dtype=np.uint32)
    _L().oracle_unpack16(c.ctypes.data, q.ctypes.data, c.size, e, m)
    return q.view(np.float32).reshape(c.shape)


def _mat(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.ndim == 2
    return a


def gemm(A: np.ndarray, B: np.ndarray, transA: bool = False, transB: bool = False):
    """C = op(A) op(B) in fp64 and T = |op(A)||op(B)|; A, B are the STORED row-major matrices."""
    A, B = _mat(A), _mat(B)
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    K2, N = (B.shape[1], B.shape[0]) if transB else B.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.float64)
    T = np.empty((M, N), dtype=np.float64)
    _L().oracle_gemm(A.ctypes.data, A.shape[1], int(transA), B.ctypes.data, B.shape[1], int(transB),
                     M, N, K, C.ctypes.data, T.ctypes.data)
    return C, T


def gemm_sampled(A: np.ndarray, B: np.ndarray, ii: np.ndarray, jj: np.ndarray,
                 transA: bool = False, transB: bool = False):
    A, B = _mat(A), _mat(B)
    K = A.shape[0] if transA else A.shape[1]
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    c = np.empty(ii.size, dtype=np.float64)
    t = np.empty(ii.size, dtype=np.float64)
    _L().oracle_gemm_sampled(A.ctypes.data, A.shape[1], int(transA), B.ctypes.data, B.shape[1],
                             int(transB), K, ii.ctypes.data, jj.ctypes.data, ii.size, c.ctypes.data,
                             t.ctypes.data)
    return c, t


def bias_quantize_stats(acc: np.ndarray, bias: Optional[np.ndarray], e: int, m: int, denormals: int = 1,
                        loss_scale: float = 1.0):
    """Y = R(R(S acc) + R(S bias)) with statistics of Y; acc is rows x cols, bias has cols entries."""
    a = _mat(acc)
    rows, cols = a.shape
    out = np.empty((rows, cols), dtype=np.uint32)
    st = np.zeros(STATS_WORDS, dtype=np.uint64)
    b = None
    if bias is not None:
        b = np.ascontiguousarray(bias, dtype=np.float32).reshape(-1)
        assert b.size == cols
    _L().oracle_bias_quantize_stats(a.ctypes.data, rows, cols, cols, b.ctypes.data if b is not None else None,
                                    out.ctypes.data, cols, e, m, int(denormals), _f32_bits(loss_scale),
                                    st.ctypes.data)
    return out.view(np.float32), st


def _check_narrow(a: np.ndarray) -> None:
    # the FMAC routines take operands with at most 12 significant bits (formats with m <= 11)
    if np.any(a.view(np.uint32) & np.uint32(0xFFF)):
        raise ValueError("FMAC operands must hold values of a format with m <= 11")


def fmac8_gemm(A: np.ndarray, B: np.ndarray, e: int, m: int, denormals: int = 1, transA: bool = False,
               transB: bool = False, group: int = 8, want_master: bool = False):
    """Algorithm 1 for every output of op(A) op(B); returns the rounded results as float32
    (and, if asked, the fp32 master accumulators before the final rounding)."""
    A, B = _mat(A), _mat(B)
    _check_narrow(A)
    _check_narrow(B)
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    K2, N = (B.shape[1], B.shape[0]) if transB else B.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.uint32)
    master = np.empty((M, N), dtype=np.uint32) if want_master else None
    _L().oracle_fmac8_gemm(A.ctypes.data, A.shape[1], int(transA), B.ctypes.data, B.shape[1], int(transB),
                           M, N, K, e, m, int(denormals), group, C.ctypes.data,
                           master.ctypes.data if want_master else None)
    return (C.view(np.float32), master.view(np.float32)) if want_master else C.view(np.float32)


def fmac8_gemm_sampled(A: np.ndarray, B: np.ndarray, ii: np.ndarray, jj: np.ndarray, e: int, m: int,
                       denormals: int = 1, transA: bool = False, transB: bool = False,
                       group: int = 8) -> np.ndarray:
    A, B = _mat(A), _mat(B)
    _check_narrow(A)
    _check_narrow(B)
    K = A.shape[0] if transA else A.shape[1]
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    c = np.empty(ii.size, dtype=np.uint32)
    _L().oracle_fmac8_gemm_sampled(A.ctypes.data, A.shape[1], int(transA), B.ctypes.data, B.shape[1],
                                   int(transB), K, e, m, int(denormals), group, ii.ctypes.data,
                                   jj.ctypes.data, ii.size, c.ctypes.data)
    return c.view(np.float32)


class DlsState(ctypes.Structure):
    """Dynamic-loss-scale controller state (same field order as the C struct in qfmt_oracle.c)."""
    _fields_ = [("scale", ctypes.c_float), ("growth", ctypes.c_float), ("backoff", ctypes.c_float),
                ("min_scale", ctypes.c_float), ("max_scale", ctypes.c_float),
                ("growth_interval", ctypes.c_int32), ("clean_steps", ctypes.c_int32), ("skip", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("n_steps", ctypes.c_uint64), ("n_skipped", ctypes.c_uint64)]


def dls_update(state: DlsState, stats: np.ndarray) -> None:
    """One controller step on the statistics records (uint64[n][264]) of a step's gradient tensors."""
    st = np.ascontiguousarray(stats, dtype=np.uint64).reshape(-1, STATS_WORDS)
    _L().oracle_dls_update(ctypes.byref(state), st.ctypes.data, st.shape[0])


CONV_FWD, CONV_DGRAD, CONV_WGRAD = 0, 1, 2


def conv(which: int, P: np.ndarray, Q: np.ndarray, geom, idx: Optional[np.ndarray] = None):
    """Direct convolution definitions on NCHW tensors.

    geom = (n, ci, h, w, co, r, s, pad_h, pad_w).  Operands (P, Q): forward (X, W); data
    gradient (dY, W); filter gradient (dY, X).  Returns (c, t) as flat fp64 arrays over the
    output tensor ([n][co][oh][ow], [n][ci][h][w] or [co][ci][r][s]) or over ``idx``.
    """
    n, ci, h, w, co, r, s, ph, pw = [int(v) for v in geom]
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    total = {CONV_FWD: n * co * oh * ow, CONV_DGRAD: n * ci * h * w, CONV_WGRAD: co * ci * r * s}[which]
    P = np.ascontiguousarray(P, dtype=np.float32)
    Q = np.ascontiguousarray(Q, dtype=np.float32)
    g = np.array([n, ci, h, w, co, r, s, ph, pw], dtype=np.int64)
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
        count = idx.size
    else:
        count = total
    c = np.empty(count, dtype=np.float64)
    t = np.empty(count, dtype=np.float64)
    _L().oracle_conv(which, g.ctypes.data, P.ctypes.data, Q.ctypes.data,
                     idx.ctypes.data if idx is not None else None, count, c.ctypes.data, t.ctypes.data)
    return c, t


def conv_fmac8(which: int, P: np.ndarray, Q: np.ndarray, geom, e: int, m: int, denormals: int = 1, group: int = 8,
               idx: Optional[np.ndarray] = None, want_master: bool = False):
    """Algorithm 1 applied to a convolution's sums (NCHW tensors, operands and index spaces as for
    ``conv``): runs of ``group`` FMACs along the reduction in the order stated in qfmt_oracle.c, padding
    positions as zero factors.  Returns the rounded results as float32, flat (and, if asked, the fp32
    totals before the final rounding)."""
    n, ci, h, w, co, r, s, ph, pw = [int(v) for v in geom]
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    total = {CONV_FWD: n * co * oh * ow, CONV_DGRAD: n * ci * h * w, CONV_WGRAD: co * ci * r * s}[which]
    P = np.ascontiguousarray(P, dtype=np.float32)
    Q = np.ascontiguousarray(Q, dtype=np.float32)
    _check_narrow(P.reshape(-1))
    _check_narrow(Q.reshape(-1))
    g = np.array([n, ci, h, w, co, r, s, ph, pw], dtype=np.int64)
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
        count = idx.size
    else:
        count = total
    out = np.empty(count, dtype=np.uint32)
    master = np.empty(count, dtype=np.uint32) if want_master else None
    _L().oracle_conv_fmac8(which, g.ctypes.data, P.ctypes.data, Q.ctypes.data, e, m, int(denormals), int(group),
                           idx.ctypes.data if idx is not None else None, count, out.ctypes.data,
                           master.ctypes.data if want_master else None)
    return (out.view(np.float32), master.view(np.float32)) if want_master else out.view(np.float32)
