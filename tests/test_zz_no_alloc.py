"""qfmt_gemm_builtin_scratch: the GEMM for callers that cannot allocate device memory.

Such callers (code living inside another framework's memory plan, loops that must not allocate
once they run, processes whose device memory is owned by someone else's pool) cannot provide the
workspace qfmt_gemm asks for, so this entry point uses a fixed 16 MiB array inside the library.
The test calls it through the C ABI twice in a row on different problems -- the second call
finds the array as the first one left it -- and requires the same bits as qfmt_gemm, whose own
results are checked against the oracle elsewhere.  The file name sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def operands(seed, M, N, K, transA, transB):
    rng = workloads.rng_for(900 + seed)
    A = workloads.lognormal_tensor(rng, (K, M) if transA else (M, K), -4.0, 3.0, p_zero=0.01)
    B = workloads.lognormal_tensor(rng, (N, K) if transB else (K, N), -4.0, 3.0, p_zero=0.01)
    dA, dB = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
    fmt = qf.make_format(6, 9)
    qf.qfmt_quantize_stats(dA, dA, dA.numel(), fmt)
    qf.qfmt_quantize_stats(dB, dB, dB.numel(), fmt)
    return dA, dB


def test_two_calls_in_a_row_match_qfmt_gemm():
    lib = qf.lib()
    fmt = qf.make_format(6, 9)
    problems = [(0, 300, 520, 1500, False, False), (1, 260, 384, 2100, True, False)]
    status = torch.full((4,), 77, dtype=torch.int32, device=DEV)
    for seed, M, N, K, ta, tb in problems:
        dA, dB = operands(seed, M, N, K, ta, tb)
        a, b = qf.make_matrix(dA, ta), qf.make_matrix(dB, tb)
        # existing entry point, caller-allocated workspace
        ws = torch.zeros(max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=DEV)
        C_ref = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
        qf.qfmt_gemm(a, b, C_ref, N, fmt, ws, ws.numel())
        assert qf.qfmt_device_status(ws) == qf.QFMT_OK
        # new entry point, straight through the C ABI: inputs, outputs, nothing else
        C_new = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
        stream = torch.cuda.current_stream().cuda_stream
        rc = lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), C_new.data_ptr(), N, ctypes.byref(fmt),
                                           status.data_ptr(), stream)
        assert rc == qf.QFMT_OK
        assert int(status.cpu()[0]) == qf.QFMT_OK and int(status.cpu()[1]) == 77   # one int32 is written, no more
        got, ref = C_new.cpu().numpy(), C_ref.cpu().numpy()
        assert np.all(np.isfinite(ref))
        # same kernel, same fixed summation order: identical bits (stricter than the 2^-20 bound)
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_argument_errors_enqueue_nothing():
    lib = qf.lib()
    d = torch.ones(64, 64, dtype=torch.float32, device=DEV)
    a, b = qf.make_matrix(d), qf.make_matrix(d)
    bad = qf.make_format(6, 11)
    assert lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), d.data_ptr(), 64, ctypes.byref(bad),
                                         None, None) == qf.QFMT_ERR_BAD_FORMAT
    assert lib.qfmt_gemm_builtin_scratch(None, ctypes.byref(b), d.data_ptr(), 64, ctypes.byref(bad),
                                         None, None) == qf.QFMT_ERR_BAD_ARG
    assert "16 MiB" in qf.qfmt_status_string(qf.QFMT_ERR_SCRATCH_LIMIT)
    torch.cuda.synchronize()
    assert torch.all(d == 1.0)


def test_a_product_beyond_the_limit_is_refused_and_nothing_runs():
    """The BERT-large out-projection's weight gradient (1024 x 1024 outputs over 8192 tokens) is planned
    with K splits whose partial sums, plus the 256-byte header, exceed the 16 MiB array: the call must
    say QFMT_ERR_SCRATCH_LIMIT, leave the output and the status word alone, and qfmt_gemm with a
    caller's workspace must still do the product."""
    lib = qf.lib()
    fmt = qf.make_format(6, 9)
    M = N = 1024
    K = 8192
    X = torch.ones(K, M, dtype=torch.float32, device=DEV)
    G = torch.ones(K, N, dtype=torch.float32, device=DEV)
    a, b = qf.make_matrix(X, True), qf.make_matrix(G, False)
    need = qf.qfmt_gemm_workspace_bytes(a, b)
    if need <= (16 << 20):
        pytest.skip("this product fits the built-in scratch under the current plan")
    C = torch.full((M, N), -5.0, dtype=torch.float32, device=DEV)
    status = torch.full((4,), 77, dtype=torch.int32, device=DEV)
    rc = lib.qfmt_gemm_builtin_scratch(ctypes.byref(a), ctypes.byref(b), C.data_ptr(), N, ctypes.byref(fmt),
                                       status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == qf.QFMT_ERR_SCRATCH_LIMIT
    torch.cuda.synchronize()
    assert torch.all(C == -5.0) and torch.all(status == 77)
    ws = torch.zeros(need, dtype=torch.uint8, device=DEV)
    qf.qfmt_gemm(a, b, C, N, fmt, ws, need)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    assert torch.all(C == float(K))
