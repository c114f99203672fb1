"""GPU tests of qfmt_linear_forward, Y = R(R(op(A) op(B)) + R(bias)) with the statistics of Y
(Section IV-A's worked example).  The call must give the bits of its two parts, qfmt_gemm followed
by qfmt_bias_quantize_stats (with the same K-summation plan), whether the epilogue runs inside
the GEMM kernel (K <= 1024, e <= 6) or after it; the parts are checked against the oracle in their own tests, and once more here."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(autouse=True, params=[1, 0], ids=["in-kernel", "default"])
def fusion(request):
    """Every test runs with the epilogue inside the GEMM kernel (where it applies) and with the
    default plan."""
    qf.qfmt_linear_fusion_policy(request.param)
    yield request.param
    qf.qfmt_linear_fusion_policy(0)
    qf.qfmt_gemm_tile_policy(0)


def in_kernel(K, e):
    """True when qfmt_linear_forward runs the epilogue inside the GEMM kernel under policy 1."""
    return K <= 1024 and e <= 6


def two_step(a, b, d_bias, M, N, fmt, fused=True):
    """qfmt_gemm then qfmt_bias_quantize_stats.  The fused kernel never splits K, so its reference
    gets a workspace too small for split-K partial sums (same summation order, same bits); the
    unfused path inside qfmt_linear_forward plans like qfmt_gemm with the recommended workspace."""
    acc = torch.empty(M, N, dtype=torch.float32, device=DEV)
    ws = torch.zeros(256 if fused else max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=DEV)
    qf.qfmt_gemm(a, b, acc, N, fmt, ws, ws.numel())
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    y = torch.empty_like(acc)
    st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    qf.qfmt_bias_quantize_stats(acc, N, d_bias, y, N, M, N, fmt, st)
    torch.cuda.synchronize()
    return acc, y, st


def run_case(fusion, A, B, bias, e, m, den, transA=False, transB=False, ldy=None, check_oracle=False):
    """A, B: STORED matrices (numpy), already holding format values."""
    fmt = qf.make_format(e, m, den)
    dA, dB = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
    d_bias = torch.from_numpy(bias).to(DEV)
    a, b = qf.make_matrix(dA, transA), qf.make_matrix(dB, transB)
    M = A.shape[1] if transA else A.shape[0]
    N = B.shape[0] if transB else B.shape[1]
    K = A.shape[0] if transA else A.shape[1]
    acc, y_ref, st_ref = two_step(a, b, d_bias, M, N, fmt, fused=(fusion == 1 and in_kernel(K, e)))
    ldy = ldy or N
    buf = torch.full((M * ldy + 8,), 7.0, dtype=torch.float32, device=DEV)
    y = buf[:M * ldy].view(M, ldy)
    st = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV)
    wb = qf.qfmt_linear_forward_workspace_bytes(a, b)
    ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
    qf.qfmt_linear_forward(a, b, d_bias, y, ldy, fmt, st, 0, ws, wb)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    torch.cuda.synchronize()
    got = y[:, :N].cpu().numpy()
    want = y_ref.cpu().numpy()
    bad = np.nonzero(got.view(np.uint32) != want.view(np.uint32))
    assert bad[0].size == 0, (bad[0][:4], bad[1][:4], got[bad][:4], want[bad][:4])
    assert torch.all(y[:, N:] == 7.0) and torch.all(buf[M * ldy:] == 7.0)
    g, w = st.cpu().numpy().view(np.uint64), st_ref.cpu().numpy().view(np.uint64)
    assert np.array_equal(g, w), (g[np.nonzero(g != w)], w[np.nonzero(g != w)])
    if check_oracle:
        y_o, st_o = oracle.bias_quantize_stats(acc.cpu().numpy(), bias, e, m, den, 1.0)
        assert np.array_equal(got.view(np.uint32), y_o.view(np.uint32)) and np.array_equal(g, st_o)
    return g


def operands(seed, shape_a, shape_b, e, m, den, mu=-3.0, sigma=2.0):
    rng = workloads.rng_for(seed)
    A = oracle.quantize_stats(workloads.lognormal_tensor(rng, shape_a, mu, sigma, p_zero=0.02), e, m, den, 1.0,
                              want_stats=False)[0]
    B = oracle.quantize_stats(workloads.normal_tensor(rng, shape_b, 0.05), e, m, den, 1.0, want_stats=False)[0]
    return A, B


@pytest.mark.parametrize("policy", [1, 2])
@pytest.mark.parametrize("M,N,K", [(256, 256, 64), (300, 260, 200), (129, 516, 1024), (512, 1024, 96), (77, 30, 17)])
def test_fused_matches_two_step(fusion, policy, M, N, K):
    """K <= 1024: the epilogue runs inside the GEMM kernel (both tile shapes, ragged tiles, and an N
    that is not a multiple of 4, which takes the scalar store path).  Operands sit in buffers whose
    leading dimensions are padded to a multiple of 4, as the TMA loads need."""
    qf.qfmt_gemm_tile_policy(policy)
    e, m = 6, 9
    fmt = qf.make_format(e, m, 1)
    K4, N4 = (K + 3) // 4 * 4, (N + 3) // 4 * 4
    A, B = operands(600 + M + K, (M, K4), (K4, N4), e, m, 1)
    dA, dB = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
    a = qf.make_matrix(dA.data_ptr(), False, M, K, K4)
    b = qf.make_matrix(dB.data_ptr(), False, K, N, N4)
    bias = workloads.normal_tensor(workloads.rng_for(601, N), (N,), 0.05)
    d_bias = torch.from_numpy(bias).to(DEV)
    acc, y_ref, st_ref = two_step(a, b, d_bias, M, N, fmt, fused=(fusion == 1))
    y = torch.empty(M, N, dtype=torch.float32, device=DEV)
    st = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV)
    wb = qf.qfmt_linear_forward_workspace_bytes(a, b)
    ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
    qf.qfmt_linear_forward(a, b, d_bias, y, N, fmt, st, 0, ws, wb)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32))
    assert torch.equal(st, st_ref), (st[st != st_ref], st_ref[st != st_ref])
    if policy == 1 and M == 300:
        y_o, st_o = oracle.bias_quantize_stats(acc.cpu().numpy(), bias, e, m, 1, 1.0)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), y_o.view(np.uint32))
        assert np.array_equal(st.cpu().numpy().view(np.uint64), st_o)


@pytest.mark.parametrize("e,m,den", [(5, 10, 1), (5, 10, 0), (6, 9, 0), (7, 8, 1)])
def test_formats_and_flushing(fusion, e, m, den):
    A, B = operands(610 + e, (260, 128), (128, 264), e, m, den, mu=-8.0, sigma=3.0)   # small sums: denormals
    bias = workloads.lognormal_tensor(workloads.rng_for(611), (264,), -12.0, 3.0)
    st = run_case(fusion, A, B, bias, e, m, den, check_oracle=True)
    assert int(st[oracle.ST_DENORMAL]) > 0 or (e, m) != (5, 10)


def test_transposed_operands_and_leading_dimension(fusion):
    A, B = operands(620, (96, 260), (264, 96), 6, 9, 1)        # stored K x M and N x K
    bias = workloads.normal_tensor(workloads.rng_for(621), (264,), 0.05)
    run_case(fusion, A, B, bias, 6, 9, 1, transA=True, transB=True, ldy=272)


def test_long_contraction_and_bfloat16_family_run_the_two_kernels(fusion):
    """K > 1024 (sums leave the registers between groups) and e = 8 take the unfused path."""
    A, B = operands(630, (200, 1100), (1100, 256), 6, 9, 1)
    bias = workloads.normal_tensor(workloads.rng_for(631), (256,), 0.05)
    run_case(fusion, A, B, bias, 6, 9, 1)
    A, B = operands(632, (130, 64), (64, 256), 8, 7, 1)
    run_case(fusion, A, B, bias, 8, 7, 1, check_oracle=True)


def test_special_values_pass_through_the_epilogue(fusion):
    A, B = operands(640, (128, 64), (64, 256), 6, 9, 1)
    A[0, 0], A[1, 1], A[2, 2] = np.inf, -np.inf, np.nan
    B[:, 7] = 0.0
    bias = workloads.normal_tensor(workloads.rng_for(641), (256,), 0.05)
    bias[7], bias[8], bias[9] = -0.0, np.inf, np.nan
    run_case(fusion, A, B, bias, 6, 9, 1, check_oracle=True)


@pytest.mark.parametrize("layer", [0, 1, 2])
def test_config5_forward_layers_full_size(fusion, layer):
    """BERT-large forward products with K = 1024 at full size, in the benchmark's launch
    configuration: fused output and statistics equal the two-step result bit for bit."""
    c = workloads.config5_layer(layer, 0)
    e, m = 6, 9
    fmt = qf.make_format(e, m, 1)
    dX, dW = torch.from_numpy(c["X"]).to(DEV), torch.from_numpy(c["W"]).to(DEV)
    qf.qfmt_quantize_stats(dX, dX, dX.numel(), fmt)
    qf.qfmt_quantize_stats(dW, dW, dW.numel(), fmt)
    M, N = dX.shape[0], dW.shape[1]
    bias = workloads.normal_tensor(workloads.rng_for(650, layer), (N,), 0.02)
    d_bias = torch.from_numpy(bias).to(DEV)
    a, b = qf.make_matrix(dX), qf.make_matrix(dW)
    acc, y_ref, st_ref = two_step(a, b, d_bias, M, N, fmt, fused=(fusion == 1))
    y = torch.empty(M, N, dtype=torch.float32, device=DEV)
    st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    wb = qf.qfmt_linear_forward_workspace_bytes(a, b)
    ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
    qf.qfmt_linear_forward(a, b, d_bias, y, N, fmt, st, 0, ws, wb)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32)) and torch.equal(st, st_ref)
    # sampled rows against the oracle's formula on the GPU's own accumulator values
    rows = np.array([0, 1, M // 2, M - 1])
    y_o, _ = oracle.bias_quantize_stats(acc[rows].cpu().numpy(), bias, e, m, 1, 1.0)
    assert np.array_equal(y[rows].cpu().numpy().view(np.uint32), y_o.view(np.uint32))


def test_errors():
    d = torch.ones(256 * 256, dtype=torch.float32, device=DEV)
    a = qf.make_matrix(d.data_ptr(), False, 256, 256, 256)
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_linear_forward(a, a, d, d, 256, qf.make_format(6, 9, 1, 2.0), None, 0, ws, ws.numel())
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT      # a loss scale has no place in the forward formula
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_linear_forward(a, a, None, d, 256, qf.make_format(6, 9), None, 0, ws, ws.numel())
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_linear_forward(a, a, d, d, 256, qf.make_format(6, 9), None, 0, ws, 256)
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG         # no room for the rounded bias
