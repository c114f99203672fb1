"""The error path of a device-side wait that does not end.

Every wait inside the contraction kernels is bounded: when it runs out the waiting role records
QFMT_ERR_TIMEOUT in the status word, raises a block-wide flag, the other roles leave at their next
check and the kernel returns.  The library's self-test kernel takes exactly that path on a barrier
nothing arrives on (the wait gives up by itself, so the GPU is never left spinning); here its status
and trace are checked, and that the next ordinary product on the same GPU is still right."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("limit", [1 << 12, 1 << 16, 1 << 20])
def test_wait_runs_out_and_the_status_says_so(limit):
    status = torch.full((4,), 123, dtype=torch.int32, device=DEV)
    trace = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    qf.qfmt_selftest_bounded_wait(status, limit, trace)
    assert qf.qfmt_device_status(status) == qf.QFMT_ERR_TIMEOUT
    t = trace.cpu().numpy()
    assert t[0] == 1, "the waiting warp did not see its wait expire"
    assert t[1] == 1, "the other warp did not see the abort flag"
    assert t[2] >= limit, "the wait gave up before its limit"
    assert t[2] < 64 * limit + (1 << 22), "the wait overran its limit by far"
    assert "wait" in qf.qfmt_status_string(qf.QFMT_ERR_TIMEOUT)


def test_context_is_usable_afterwards():
    """After a timeout has been reported the same GPU runs an ordinary product bit-correctly, and a
    fresh workspace reports QFMT_OK."""
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    trace = torch.zeros(4, dtype=torch.int32, device=DEV)
    qf.qfmt_selftest_bounded_wait(status, 1 << 14, trace)
    assert qf.qfmt_device_status(status) == qf.QFMT_ERR_TIMEOUT
    rng = np.random.default_rng(3)
    A = rng.integers(-6, 7, size=(300, 200)).astype(np.float32)
    B = rng.integers(-6, 7, size=(200, 260)).astype(np.float32)
    dA, dB = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
    a, b = qf.make_matrix(dA), qf.make_matrix(dB)
    ws = torch.zeros(max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=DEV)
    C = torch.empty(300, 260, dtype=torch.float32, device=DEV)
    qf.qfmt_gemm(a, b, C, 260, qf.make_format(6, 9), ws, ws.numel())
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    ref, _ = oracle.gemm(A, B)
    assert np.array_equal(C.cpu().numpy().astype(np.float64), ref)


def test_argument_checks():
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    for limit in (0, (1 << 24) + 1):
        with pytest.raises(qf.QfmtError):
            qf.qfmt_selftest_bounded_wait(status, limit, status)
    with pytest.raises(qf.QfmtError):
        qf.qfmt_selftest_bounded_wait(None, 1 << 12, status)
