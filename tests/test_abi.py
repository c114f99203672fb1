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
