"""Python binding of the qfmt C-ABI library (``include/qfmt.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of ``libqfmt.so``.
PyTorch is used by callers for device memory and streams; this module accepts torch tensors
or raw integer addresses.  There is no CPU fallback: if the shared library cannot be loaded,
the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqfmt.so")

QFMT_OK = 0
QFMT_ERR_BAD_FORMAT = -1
QFMT_ERR_BAD_ARG = -2
QFMT_ERR_UNSUPPORTED_ARCH = -3
QFMT_ERR_CUDA = -4
QFMT_ERR_TIMEOUT = -5
QFMT_ERR_SCRATCH_LIMIT = -6

STATS_WORDS = 264  # 256 histogram bins + 8 counters, all uint64
(ST_TOTAL, ST_ZERO_IN, ST_DENORMAL, ST_UNDERFLOW, ST_OVERFLOW, ST_NAN, ST_INF_IN) = range(256, 263)


class QfmtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().qfmt_status_string(status).decode()
        if status == QFMT_ERR_CUDA:
            msg += f" (cudaError {lib().qfmt_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


class qfmt_format_t(ctypes.Structure):
    _fields_ = [("e", ctypes.c_int32), ("m", ctypes.c_int32), ("denormals", ctypes.c_int32),
                ("rounding", ctypes.c_int32), ("loss_scale", ctypes.c_float)]


class qfmt_matrix_t(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("ld", ctypes.c_int64), ("trans", ctypes.c_int32)]


class qfmt_conv_t(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("n", "c_in", "h", "w", "c_out", "r", "s", "pad_h", "pad_w")]


QFMT_CONV_FWD, QFMT_CONV_DGRAD, QFMT_CONV_WGRAD = 0, 1, 2


class qfmt_stats_t(ctypes.Structure):
    _fields_ = [("hist", ctypes.c_uint64 * 256), ("n_total", ctypes.c_uint64),
                ("n_zero_in", ctypes.c_uint64), ("n_denormal", ctypes.c_uint64),
                ("n_underflow", ctypes.c_uint64), ("n_overflow", ctypes.c_uint64),
                ("n_nan", ctypes.c_uint64), ("n_inf_in", ctypes.c_uint64), ("reserved", ctypes.c_uint64)]


class qfmt_dls_t(ctypes.Structure):
    _fields_ = [("scale", ctypes.c_float), ("growth", ctypes.c_float), ("backoff", ctypes.c_float),
                ("min_scale", ctypes.c_float), ("max_scale", ctypes.c_float),
                ("growth_interval", ctypes.c_int32), ("clean_steps", ctypes.c_int32), ("skip", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("n_steps", ctypes.c_uint64), ("n_skipped", ctypes.c_uint64)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2103_15940_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        fmtp = ctypes.POINTER(qfmt_format_t)
        L.qfmt_quantize_stats.argtypes = [vp, vp, sz, fmtp, vp, ci, vp]
        L.qfmt_quantize_stats.restype = ci
        L.qfmt_quantize_stats_transpose.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, fmtp, vp, ci, vp]
        L.qfmt_quantize_stats_transpose.restype = ci
        L.qfmt_bias_quantize_stats.argtypes = [vp, ctypes.c_int64, vp, vp, ctypes.c_int64, ctypes.c_int64,
                                               ctypes.c_int64, fmtp, vp, ci, vp]
        L.qfmt_bias_quantize_stats.restype = ci
        L.qfmt_bias_quantize_stats_pack16.argtypes = L.qfmt_bias_quantize_stats.argtypes
        L.qfmt_bias_quantize_stats_pack16.restype = ci
        L.qfmt_quantize_stats_pack16.argtypes = [vp, vp, sz, fmtp, vp, ci, vp]
        L.qfmt_quantize_stats_pack16.restype = ci
        L.qfmt_unpack16.argtypes = [vp, vp, sz, fmtp, vp]
        L.qfmt_unpack16.restype = ci
        L.qfmt_quantize_stats_host.argtypes = [vp, vp, sz, fmtp, vp, vp, sz, vp]
        L.qfmt_quantize_stats_host.restype = ci
        L.qfmt_quantize_stats_host_work_bytes.argtypes = [sz]
        L.qfmt_quantize_stats_host_work_bytes.restype = sz
        L.qfmt_last_cuda_error.argtypes = []
        L.qfmt_last_cuda_error.restype = ci
        L.qfmt_status_string.argtypes = [ci]
        L.qfmt_status_string.restype = ctypes.c_char_p
        L.qfmt_version.argtypes = []
        L.qfmt_version.restype = ci
        _bind_optional(L)
        _lib = L
    return _lib


def _bind_optional(L: ctypes.CDLL) -> None:
    """Signatures of the contraction entry points; see include/qfmt.h."""
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    matp = ctypes.POINTER(qfmt_matrix_t)
    L.qfmt_gemm.argtypes = [matp, matp, vp, ctypes.c_int64, ctypes.POINTER(qfmt_format_t), vp, sz, vp]
    L.qfmt_gemm.restype = ci
    L.qfmt_gemm_workspace_bytes.argtypes = [matp, matp]
    L.qfmt_gemm_workspace_bytes.restype = sz
    i64 = ctypes.c_int64
    L.qfmt_gemm_packed16.argtypes = [matp, matp, vp, i64, ctypes.POINTER(qfmt_format_t), vp, sz, vp]
    L.qfmt_gemm_packed16.restype = ci
    L.qfmt_gemm_packed16_workspace_bytes.argtypes = [matp, matp]
    L.qfmt_gemm_packed16_workspace_bytes.restype = sz
    L.qfmt_gemm_fmac8.argtypes = [matp, matp, vp, ctypes.c_int64, ctypes.POINTER(qfmt_format_t), vp, ci, ci, vp]
    L.qfmt_gemm_fmac8.restype = ci
    L.qfmt_dls_update.argtypes = [vp, vp, ctypes.c_int64, vp]
    L.qfmt_dls_update.restype = ci
    L.qfmt_quantize_stats_dls.argtypes = [vp, vp, sz, ctypes.POINTER(qfmt_format_t), vp, vp, ci, vp]
    L.qfmt_quantize_stats_dls.restype = ci
    L.qfmt_linear_forward.argtypes = [matp, matp, vp, vp, ctypes.c_int64, ctypes.POINTER(qfmt_format_t), vp, ci, vp, sz, vp]
    L.qfmt_linear_forward.restype = ci
    L.qfmt_linear_fusion_policy.argtypes = [ci]
    L.qfmt_linear_fusion_policy.restype = ci
    L.qfmt_linear_forward_workspace_bytes.argtypes = [matp, matp]
    L.qfmt_linear_forward_workspace_bytes.restype = sz
    L.qfmt_gemm_tile_policy.argtypes = [ci]
    L.qfmt_gemm_tile_policy.restype = ci
    L.qfmt_conv_tile_policy.argtypes = [ci]
    L.qfmt_conv_tile_policy.restype = ci
    L.qfmt_device_status.argtypes = [vp, vp]
    L.qfmt_device_status.restype = ci
    convp = ctypes.POINTER(qfmt_conv_t)
    L.qfmt_conv.argtypes = [ctypes.c_int32, convp, vp, vp, vp, ctypes.POINTER(qfmt_format_t), vp, sz, vp]
    L.qfmt_conv.restype = ci
    L.qfmt_conv_workspace_bytes.argtypes = [ctypes.c_int32, convp]
    L.qfmt_conv_workspace_bytes.restype = sz
    L.qfmt_conv_fmac8.argtypes = [ctypes.c_int32, convp, vp, vp, vp, ctypes.POINTER(qfmt_format_t), vp, ci, ci, vp]
    L.qfmt_conv_fmac8.restype = ci
    L.qfmt_gemm_builtin_scratch.argtypes = [matp, matp, vp, ctypes.c_int64, ctypes.POINTER(qfmt_format_t), vp, vp]
    L.qfmt_gemm_builtin_scratch.restype = ci
    L.qfmt_selftest_bounded_wait.argtypes = [vp, ctypes.c_uint32, vp, vp]
    L.qfmt_selftest_bounded_wait.restype = ci
    L.qfmt_selftest_pair_schedule.argtypes = [i64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp]
    L.qfmt_selftest_pair_schedule.restype = ci


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_format(e: int, m: int, denormals: int = 1, loss_scale: float = 1.0, rounding: int = 0) -> qfmt_format_t:
    return qfmt_format_t(int(e), int(m), int(denormals), int(rounding), float(loss_scale))


def _check(status: int, where: str) -> None:
    if status != QFMT_OK:
        raise QfmtError(status, where)


def qfmt_quantize_stats(d_in, d_out, n: int, fmt: qfmt_format_t, d_stats=None, accumulate: int = 0,
                        stream=None) -> None:
    """Device buffers in, device buffers out; see qfmt_quantize_stats in include/qfmt.h."""
    _check(lib().qfmt_quantize_stats(_ptr(d_in), _ptr(d_out), int(n), ctypes.byref(fmt), _ptr(d_stats),
                                     int(accumulate), _stream_handle(stream)), "qfmt_quantize_stats")


def qfmt_quantize_stats_transpose(d_in, d_out, batch: int, rows: int, cols: int, fmt: qfmt_format_t, d_stats=None,
                                  accumulate: int = 0, stream=None) -> None:
    """[batch][rows][cols] -> rounded [batch][cols][rows]; see include/qfmt.h."""
    _check(lib().qfmt_quantize_stats_transpose(_ptr(d_in), _ptr(d_out), int(batch), int(rows), int(cols),
                                               ctypes.byref(fmt), _ptr(d_stats), int(accumulate),
                                               _stream_handle(stream)), "qfmt_quantize_stats_transpose")


def qfmt_bias_quantize_stats(d_acc, ld_acc: int, d_bias, d_out, ld_out: int, rows: int, cols: int,
                             fmt: qfmt_format_t, d_stats=None, accumulate: int = 0, stream=None) -> None:
    """Y = R(R(acc) + R(bias)) with the statistics of Y; see qfmt_bias_quantize_stats in include/qfmt.h."""
    _check(lib().qfmt_bias_quantize_stats(_ptr(d_acc), int(ld_acc), _ptr(d_bias), _ptr(d_out), int(ld_out),
                                          int(rows), int(cols), ctypes.byref(fmt), _ptr(d_stats), int(accumulate),
                                          _stream_handle(stream)), "qfmt_bias_quantize_stats")


def qfmt_bias_quantize_stats_pack16(d_acc, ld_acc: int, d_bias, d_codes, ld_codes: int, rows: int, cols: int,
                                    fmt: qfmt_format_t, d_stats=None, accumulate: int = 0, stream=None) -> None:
    """Y = R(R(acc) + R(bias)) as packed 16-bit codes, with the statistics of Y; see include/qfmt.h."""
    _check(lib().qfmt_bias_quantize_stats_pack16(_ptr(d_acc), int(ld_acc), _ptr(d_bias), _ptr(d_codes), int(ld_codes),
                                                 int(rows), int(cols), ctypes.byref(fmt), _ptr(d_stats),
                                                 int(accumulate), _stream_handle(stream)),
           "qfmt_bias_quantize_stats_pack16")


def qfmt_quantize_stats_pack16(d_in, d_codes, n: int, fmt: qfmt_format_t, d_stats=None, accumulate: int = 0,
                               stream=None) -> None:
    """Rounding pass that stores packed 16-bit codes; see qfmt_quantize_stats_pack16 in include/qfmt.h."""
    _check(lib().qfmt_quantize_stats_pack16(_ptr(d_in), _ptr(d_codes), int(n), ctypes.byref(fmt), _ptr(d_stats),
                                            int(accumulate), _stream_handle(stream)), "qfmt_quantize_stats_pack16")


def qfmt_unpack16(d_codes, d_out, n: int, fmt: qfmt_format_t, stream=None) -> None:
    """Packed 16-bit codes to fp32 containers; see qfmt_unpack16 in include/qfmt.h."""
    _check(lib().qfmt_unpack16(_ptr(d_codes), _ptr(d_out), int(n), ctypes.byref(fmt), _stream_handle(stream)),
           "qfmt_unpack16")


def qfmt_quantize_stats_host_work_bytes(n: int) -> int:
    return int(lib().qfmt_quantize_stats_host_work_bytes(int(n)))


def qfmt_quantize_stats_host(h_in, h_out, n: int, fmt: qfmt_format_t, h_stats, d_work, work_bytes: int,
                             stream=None) -> None:
    """Host buffers in and out (copies inside the call); see include/qfmt.h."""
    _check(lib().qfmt_quantize_stats_host(_ptr(h_in), _ptr(h_out), int(n), ctypes.byref(fmt), _ptr(h_stats),
                                          _ptr(d_work), int(work_bytes), _stream_handle(stream)),
           "qfmt_quantize_stats_host")


def qfmt_version() -> int:
    return int(lib().qfmt_version())


def qfmt_status_string(status: int) -> str:
    return lib().qfmt_status_string(int(status)).decode()


def make_matrix(t, trans: bool = False, rows: Optional[int] = None, cols: Optional[int] = None,
                ld: Optional[int] = None) -> qfmt_matrix_t:
    """Operand descriptor of a 2-D row-major torch tensor (or of a raw address with rows/cols/ld)."""
    if hasattr(t, "shape") and rows is None:
        assert t.dim() == 2 and t.stride(1) == 1
        rows, cols, ld = t.shape[0], t.shape[1], t.stride(0)
    return qfmt_matrix_t(_ptr(t), int(rows), int(cols), int(ld if ld is not None else cols), 1 if trans else 0)


def qfmt_gemm_workspace_bytes(A: qfmt_matrix_t, B: qfmt_matrix_t) -> int:
    return int(lib().qfmt_gemm_workspace_bytes(ctypes.byref(A), ctypes.byref(B)))


def qfmt_gemm(A: qfmt_matrix_t, B: qfmt_matrix_t, d_C, ldc: int, fmt: qfmt_format_t, d_workspace,
              workspace_bytes: int, stream=None) -> None:
    """C = op(A) op(B), exact products, fp32 accumulation; see qfmt_gemm in include/qfmt.h."""
    _check(lib().qfmt_gemm(ctypes.byref(A), ctypes.byref(B), _ptr(d_C), int(ldc), ctypes.byref(fmt),
                           _ptr(d_workspace), int(workspace_bytes), _stream_handle(stream)), "qfmt_gemm")


qfmt_matrix16_t = qfmt_matrix_t  # the same record with a pointer to 16-bit codes; make_matrix builds both


def qfmt_gemm_packed16_workspace_bytes(A: qfmt_matrix_t, B: qfmt_matrix_t) -> int:
    return int(lib().qfmt_gemm_packed16_workspace_bytes(ctypes.byref(A), ctypes.byref(B)))


def qfmt_gemm_packed16(A: qfmt_matrix_t, B: qfmt_matrix_t, d_C, ldc: int, fmt: qfmt_format_t, d_workspace,
                       workspace_bytes: int, stream=None) -> None:
    """C = op(A) op(B) on packed binary16 / bfloat16 codes; see qfmt_gemm_packed16 in include/qfmt.h."""
    _check(lib().qfmt_gemm_packed16(ctypes.byref(A), ctypes.byref(B), _ptr(d_C), int(ldc), ctypes.byref(fmt),
                                    _ptr(d_workspace), int(workspace_bytes), _stream_handle(stream)),
           "qfmt_gemm_packed16")


def qfmt_gemm_fmac8(A: qfmt_matrix_t, B: qfmt_matrix_t, d_C, ldc: int, fmt: qfmt_format_t, d_stats=None,
                    accumulate: int = 0, path: int = 0, stream=None) -> None:
    """C = op(A) op(B) with FMAC-8 accumulation (Algorithm 1); see qfmt_gemm_fmac8 in include/qfmt.h."""
    _check(lib().qfmt_gemm_fmac8(ctypes.byref(A), ctypes.byref(B), _ptr(d_C), int(ldc), ctypes.byref(fmt),
                                 _ptr(d_stats), int(accumulate), int(path), _stream_handle(stream)), "qfmt_gemm_fmac8")


def qfmt_dls_update(d_state, d_stats, n_records: int, stream=None) -> None:
    """One dynamic-loss-scale controller step on device records; see qfmt_dls_update in include/qfmt.h."""
    _check(lib().qfmt_dls_update(_ptr(d_state), _ptr(d_stats), int(n_records), _stream_handle(stream)), "qfmt_dls_update")


def qfmt_quantize_stats_dls(d_in, d_out, n: int, fmt: qfmt_format_t, d_state, d_stats=None, accumulate: int = 0,
                            stream=None) -> None:
    """qfmt_quantize_stats with the loss scale read from a device-resident qfmt_dls_t; see include/qfmt.h."""
    _check(lib().qfmt_quantize_stats_dls(_ptr(d_in), _ptr(d_out), int(n), ctypes.byref(fmt), _ptr(d_state),
                                         _ptr(d_stats), int(accumulate), _stream_handle(stream)),
           "qfmt_quantize_stats_dls")


def qfmt_linear_fusion_policy(policy: int) -> None:
    """0 automatic, 1 epilogue inside the GEMM kernel when it applies, 2 two kernels; see include/qfmt.h."""
    _check(lib().qfmt_linear_fusion_policy(int(policy)), "qfmt_linear_fusion_policy")


def qfmt_linear_forward_workspace_bytes(A: qfmt_matrix_t, B: qfmt_matrix_t) -> int:
    return int(lib().qfmt_linear_forward_workspace_bytes(ctypes.byref(A), ctypes.byref(B)))


def qfmt_linear_forward(A: qfmt_matrix_t, B: qfmt_matrix_t, d_bias, d_Y, ldy: int, fmt: qfmt_format_t, d_stats,
                        accumulate: int, d_workspace, workspace_bytes: int, stream=None) -> None:
    """Y = R(R(op(A) op(B)) + R(bias)) with the statistics of Y; see qfmt_linear_forward in include/qfmt.h."""
    _check(lib().qfmt_linear_forward(ctypes.byref(A), ctypes.byref(B), _ptr(d_bias), _ptr(d_Y), int(ldy),
                                     ctypes.byref(fmt), _ptr(d_stats), int(accumulate), _ptr(d_workspace),
                                     int(workspace_bytes), _stream_handle(stream)), "qfmt_linear_forward")


def qfmt_device_status(d_workspace, stream=None) -> int:
    return int(lib().qfmt_device_status(_ptr(d_workspace), _stream_handle(stream)))


def qfmt_gemm_builtin_scratch(A: qfmt_matrix_t, B: qfmt_matrix_t, d_C, ldc: int, fmt: qfmt_format_t,
                              d_status_out=None, stream=None) -> None:
    """qfmt_gemm for callers that cannot allocate: the workspace is a fixed 16 MiB array inside the
    library (shared by all calls on a GPU; keep them on one stream).  See include/qfmt.h."""
    _check(lib().qfmt_gemm_builtin_scratch(ctypes.byref(A), ctypes.byref(B), _ptr(d_C), int(ldc), ctypes.byref(fmt),
                                           _ptr(d_status_out), _stream_handle(stream)), "qfmt_gemm_builtin_scratch")


def qfmt_selftest_bounded_wait(d_status, limit_cycles: int, d_trace, stream=None) -> None:
    """Runs the library's bounded-wait self-test kernel; see qfmt_selftest_bounded_wait in include/qfmt.h."""
    _check(lib().qfmt_selftest_bounded_wait(_ptr(d_status), int(limit_cycles), _ptr(d_trace), _stream_handle(stream)),
           "qfmt_selftest_bounded_wait")


def qfmt_selftest_pair_schedule(tiles: int, chunks_per_tile: int, pair: int, j: int):
    """Piece j of a pair under the balanced schedule as (tile, first chunk, chunks, partial, head, pieces per
    pair); host only.  See qfmt_selftest_pair_schedule in include/qfmt.h."""
    out = (ctypes.c_int32 * 6)()
    _check(lib().qfmt_selftest_pair_schedule(int(tiles), int(chunks_per_tile), int(pair), int(j),
                                             ctypes.cast(out, ctypes.c_void_p)), "qfmt_selftest_pair_schedule")
    return tuple(int(v) for v in out)


def qfmt_conv_workspace_bytes(op: int, geom: qfmt_conv_t) -> int:
    return int(lib().qfmt_conv_workspace_bytes(int(op), ctypes.byref(geom)))


def qfmt_conv(op: int, geom: qfmt_conv_t, d_p, d_q, d_out, fmt: qfmt_format_t, d_workspace, workspace_bytes: int,
              stream=None) -> None:
    """Forward / data-gradient / filter-gradient product of a convolution on channels-last tensors;
    see qfmt_conv in include/qfmt.h."""
    _check(lib().qfmt_conv(int(op), ctypes.byref(geom), _ptr(d_p), _ptr(d_q), _ptr(d_out), ctypes.byref(fmt),
                           _ptr(d_workspace), int(workspace_bytes), _stream_handle(stream)), "qfmt_conv")


def qfmt_conv_fmac8(op: int, geom: qfmt_conv_t, d_p, d_q, d_out, fmt: qfmt_format_t, d_stats=None, accumulate: int = 0,
                    path: int = 0, stream=None) -> None:
    """A convolution's forward / data-gradient / filter-gradient product with FMAC-8 accumulation; see
    qfmt_conv_fmac8 in include/qfmt.h."""
    _check(lib().qfmt_conv_fmac8(int(op), ctypes.byref(geom), _ptr(d_p), _ptr(d_q), _ptr(d_out), ctypes.byref(fmt),
                                 _ptr(d_stats), int(accumulate), int(path), _stream_handle(stream)), "qfmt_conv_fmac8")


def qfmt_conv_tile_policy(policy: int) -> None:
    """0 automatic, 1 single-CTA kernel, 2 CTA pairs on whole tiles, 3 CTA pairs under the balanced schedule,
    for conv forward / data gradient; see include/qfmt.h."""
    _check(lib().qfmt_conv_tile_policy(int(policy)), "qfmt_conv_tile_policy")


def qfmt_gemm_tile_policy(policy: int) -> None:
    """0 automatic, 1 single-CTA tiles, 2 CTA-pair tiles, 3 CTA-pair tiles under the balanced schedule; see
    include/qfmt.h."""
    _check(lib().qfmt_gemm_tile_policy(int(policy)), "qfmt_gemm_tile_policy")
