"""The C-ABI library loads without a GPU, exports every symbol the header declares, and its
host-side argument checks answer before any device work (no compute calls here)."""
import ctypes
import os
import re

import pytest

import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import build as qbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    qbuild.build()
    return qf.lib()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(qfmt_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert "qfmt_quantize_stats" in names
    for name in names:
        assert hasattr(lib, name), name


def test_python_binding_has_the_same_names(lib):
    for name in declared_symbols():
        assert hasattr(qf, name) or hasattr(lib, name)
    assert callable(qf.qfmt_quantize_stats)


def test_version_and_status_strings(lib):
    assert qf.qfmt_version() >= 100
    for code in (0, -1, -2, -3, -4, -5, -99):
        assert len(qf.qfmt_status_string(code)) > 0


def test_struct_layouts(lib):
    assert ctypes.sizeof(qf.qfmt_stats_t) == 264 * 8
    assert ctypes.sizeof(qf.qfmt_format_t) == 20


@pytest.mark.parametrize("kw,code", [
    (dict(e=1, m=9), qf.QFMT_ERR_BAD_FORMAT), (dict(e=9, m=9), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=0), qf.QFMT_ERR_BAD_FORMAT), (dict(e=6, m=24), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=9, rounding=1), qf.QFMT_ERR_BAD_FORMAT), (dict(e=6, m=9, denormals=2), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=9, loss_scale=0.0), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=9, loss_scale=-2.0), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=9, loss_scale=float("inf")), qf.QFMT_ERR_BAD_FORMAT),
    (dict(e=6, m=9, loss_scale=float("nan")), qf.QFMT_ERR_BAD_FORMAT),
])
def test_bad_formats_are_rejected_on_the_host(lib, kw, code):
    fmt = qf.make_format(**kw)
    rc = lib.qfmt_quantize_stats(None, None, 0, ctypes.byref(fmt), None, 0, None)
    assert rc == code


def test_null_format_and_bad_flags(lib):
    assert lib.qfmt_quantize_stats(None, None, 0, None, None, 0, None) == qf.QFMT_ERR_BAD_ARG
    fmt = qf.make_format(6, 9)
    assert lib.qfmt_quantize_stats(None, None, 0, ctypes.byref(fmt), None, 7, None) == qf.QFMT_ERR_BAD_ARG
    assert lib.qfmt_quantize_stats(None, None, 16, ctypes.byref(fmt), None, 0, None) == qf.QFMT_ERR_BAD_ARG
    assert lib.qfmt_quantize_stats(ctypes.c_void_p(0x1002), None, 16, ctypes.byref(fmt), None, 0, None) \
        == qf.QFMT_ERR_BAD_ARG
    assert lib.qfmt_quantize_stats_host(None, None, 16, ctypes.byref(fmt), None, None, 0, None) == qf.QFMT_ERR_BAD_ARG
    assert qf.qfmt_quantize_stats_host_work_bytes(100) >= 400 + 264 * 8


def test_builtin_scratch_refuses_on_the_host_what_does_not_fit(lib):
    """qfmt_gemm_builtin_scratch answers QFMT_ERR_SCRATCH_LIMIT from host arithmetic alone (no device
    call has happened yet, so this runs without a GPU) whenever the product's whole workspace --
    256-byte header included -- exceeds the built-in 16 MiB.  The BERT-large stack has such a product:
    the out-projection's weight gradient, 1024 x 1024 outputs over K = 8192 tokens, planned in four
    K splits of 4 MiB each."""
    limit = 16 << 20
    fmt = qf.make_format(6, 9)
    refused = 0
    # (M, N, K) as op(A) [M x K] = stored [K x M] transposed, B stored [K x N]
    for M, N, K in ((1024, 1024, 8192), (1024, 2048, 32768), (2048, 2048, 65536), (512, 512, 1 << 20)):
        a = qf.qfmt_matrix_t(0x10000, K, M, M, 1)
        b = qf.qfmt_matrix_t(0x20000, K, N, N, 0)
        need = qf.qfmt_gemm_workspace_bytes(a, b)
        if need > limit:
            rc = lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(0x30000), N,
                                               ctypes.byref(fmt), None, None)
            assert rc == qf.QFMT_ERR_SCRATCH_LIMIT, (M, N, K, need)
            refused += 1
    assert refused >= 1, "no candidate product needs more than the built-in scratch: pick larger ones"
    # argument errors are reported before the size check and before any device call
    a = qf.qfmt_matrix_t(0x10000, 8192, 1024, 1024, 1)
    b = qf.qfmt_matrix_t(0x20000, 8192, 1024, 1024, 0)
    bad = qf.make_format(6, 11)
    assert lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(0x30000), 1024,
                                         ctypes.byref(bad), None, None) == qf.QFMT_ERR_BAD_FORMAT
    assert lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(0x30000), 512,
                                         ctypes.byref(fmt), None, None) == qf.QFMT_ERR_BAD_ARG  # ldc < N
    assert lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(0x30002), 1024,
                                         ctypes.byref(fmt), None, None) == qf.QFMT_ERR_BAD_ARG  # misaligned C


def test_conv_workspace_planning_without_a_gpu(lib):
    """qfmt_conv_workspace_bytes is host arithmetic: 0 for geometries the kernels refuse, the status
    header otherwise, plus the split-K partial sums of a filter gradient."""
    fwd, dgrad, wgrad = qf.QFMT_CONV_FWD, qf.QFMT_CONV_DGRAD, qf.QFMT_CONV_WGRAD
    ws = qf.qfmt_conv_workspace_bytes
    assert ws(fwd, qf.qfmt_conv_t(1, 30, 8, 8, 32, 3, 3, 1, 1)) == 0      # channels not a multiple of 32
    assert ws(fwd, qf.qfmt_conv_t(1, 32, 8, 200, 32, 3, 3, 1, 1)) == 0    # forward rows longer than a tile
    assert ws(dgrad, qf.qfmt_conv_t(1, 32, 8, 200, 32, 3, 3, 1, 1)) == 0
    assert ws(fwd, qf.qfmt_conv_t(1, 32, 2, 2, 32, 5, 5, 0, 0)) == 0      # empty output
    assert ws(7, qf.qfmt_conv_t(1, 32, 8, 8, 32, 3, 3, 1, 1)) == 0        # no such product
    # filter gradients take rows of any length (32-pixel stages); long pixel dimensions are split
    small = ws(wgrad, qf.qfmt_conv_t(1, 32, 2, 40, 32, 3, 3, 1, 1))
    assert 256 <= small < 256 + 2 * 32 * 9 * 32 * 4                        # four stages: one split, no partial sums
    g = qf.qfmt_conv_t(8, 64, 56, 56, 64, 3, 3, 1, 1)
    big = ws(wgrad, g)
    out_bytes = 64 * 9 * 64 * 4
    assert big >= 256 + 2 * out_bytes and (big - 256) % out_bytes == 0     # whole partial results behind the header
    assert (big - 256) // out_bytes <= 32                                  # at most 32 splits
    assert ws(wgrad, qf.qfmt_conv_t(1, 32, 8, 200, 32, 3, 3, 1, 1)) > 0
    # forward / data gradient: header, and the hand-over words when CTA pairs may run the balanced schedule
    assert 256 <= ws(fwd, g) <= 256 + 8192
    assert 256 <= ws(dgrad, g) <= 256 + 8192
