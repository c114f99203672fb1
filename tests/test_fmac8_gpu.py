"""GPU parity of qfmt_gemm_fmac8 (Algorithm 1, FMAC-8) against the CPU oracle.  The algorithm
fixes every rounding, so outputs and statistics must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def quantized(x, e, m, den):
    return oracle.quantize_stats(x, e, m, den, 1.0, want_stats=False)[0]


def run_gpu(A, B, e, m, den, transA=False, transB=False, path=0, want_stats=True, ldc=None, off=0):
    """A, B are the STORED matrices (numpy float32)."""
    M = A.shape[1] if transA else A.shape[0]
    N = B.shape[0] if transB else B.shape[1]
    ldc = ldc or N
    dA = torch.zeros(A.size + 8, dtype=torch.float32, device=DEV)[off:off + A.size].view(A.shape)
    dB = torch.zeros(B.size + 8, dtype=torch.float32, device=DEV)[off:off + B.size].view(B.shape)
    dA.copy_(torch.from_numpy(A))
    dB.copy_(torch.from_numpy(B))
    buf = torch.full((M * ldc + 16,), 7.0, dtype=torch.float32, device=DEV)
    dC = buf[off:off + M * ldc]
    st = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV) if want_stats else None
    a = qf.make_matrix(dA.data_ptr(), transA, A.shape[0], A.shape[1], A.shape[1])
    b = qf.make_matrix(dB.data_ptr(), transB, B.shape[0], B.shape[1], B.shape[1])
    qf.qfmt_gemm_fmac8(a, b, dC, ldc, qf.make_format(e, m, den), st, 0, path)
    torch.cuda.synchronize()
    full = dC.view(M, ldc).cpu().numpy() if M else np.zeros((0, ldc), np.float32)
    assert np.all(full[:, N:] == 7.0)
    assert torch.all(buf[:off] == 7.0) and torch.all(buf[off + M * ldc:] == 7.0)
    return np.ascontiguousarray(full[:, :N]), (st.cpu().numpy().view(np.uint64) if want_stats else None)


def check(A, B, e, m, den, transA=False, transB=False, paths=(0,), **kw):
    c_ref, master = oracle.fmac8_gemm(A, B, e, m, den, transA, transB, want_master=True)
    _, st_ref = oracle.quantize_stats(master, e, m, den, 1.0)
    for path in paths:
        c, st = run_gpu(A, B, e, m, den, transA, transB, path, **kw)
        bad = np.nonzero(c.view(np.uint32) != c_ref.view(np.uint32))
        assert bad[0].size == 0, (path, bad[0][:5], bad[1][:5], c[bad][:5], c_ref[bad][:5])
        if st is not None:
            assert np.array_equal(st, st_ref), (path, st[np.nonzero(st != st_ref)], st_ref[np.nonzero(st != st_ref)])
    return c_ref, st_ref


def paths_for(e, m):
    return (0, 1, 2) if (e, m) in ((5, 10), (8, 7)) else (0, 1)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (7, 8), (4, 3), (8, 7)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("mu", [-2.0, -9.0])
def test_random_operands_all_transposes(e, m, den, mu):
    """Signed log-normal operands: with mu = -9 the products of 1/5/10 live in the denormal range
    of the small accumulator, with mu = -2 they are normal and cancel."""
    rng = workloads.rng_for(400 + e, int(-mu))
    M, N, K = 150, 77, 109          # two tiles in M and N for the general kernel, ragged everywhere
    for tA in (False, True):
        for tB in (False, True):
            A = quantized(workloads.lognormal_tensor(rng, (K, M) if tA else (M, K), mu, 2.0, p_zero=0.02), e, m, den)
            B = quantized(workloads.lognormal_tensor(rng, (N, K) if tB else (K, N), mu, 2.0, p_zero=0.02), e, m, den)
            check(A, B, e, m, den, tA, tB, paths_for(e, m))


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9)])
def test_small_integers_force_ties(e, m):
    """Integer operands around 2^(m+1): partial sums sit exactly on halfway points again and again,
    so any rounding other than one nearest-even rounding per FMAC shows."""
    rng = np.random.default_rng(410 + e)
    M, N, K = 64, 48, 40
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float32)
    A[:, ::5] = rng.choice([1 << m, 1 << (m + 1), -(1 << (m + 1)), 3 << m], size=(M, (K + 4) // 5)).astype(np.float32)
    B = rng.integers(-2, 3, size=(K, N)).astype(np.float32)
    B[::7, :] = 1.0
    c_ref, _ = check(A, B, e, m, 1, paths=paths_for(e, m))
    exact = A.astype(np.float64) @ B.astype(np.float64)
    assert np.any(c_ref != exact)   # the small accumulator really lost something


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (7, 8), (8, 7)])
@pytest.mark.parametrize("den", [1, 0])
def test_overflow_infinities_nans_and_zeros(e, m, den):
    rng = workloads.rng_for(420 + e, den)
    M, N, K = 40, 36, 50
    big = float(oracle.max_normal(e, m))
    A = quantized(workloads.lognormal_tensor(rng, (M, K), np.log2(big) / 2 - 3, 3.0, p_zero=0.1), e, m, den)
    B = quantized(workloads.lognormal_tensor(rng, (K, N), np.log2(big) / 2 - 3, 3.0, p_zero=0.1), e, m, den)
    A[0, 3], A[1, 4], A[2, 5] = np.inf, -np.inf, np.nan
    B[7, 0], B[8, 1] = np.inf, 0.0
    A[3, :] = 0.0
    A[4, 8] = np.inf        # times B[8, 1] = 0: invalid
    B[:, 5] = -0.0
    check(A, B, e, m, den, paths=paths_for(e, m))


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (1, 1, 8), (1, 1, 9), (2, 3, 0), (0, 5, 4), (4, 0, 4), (3, 5, 7),
                                   (128, 64, 32), (129, 65, 33), (256, 128, 64), (5, 300, 17), (300, 5, 16)])
def test_shapes(M, N, K):
    rng = workloads.rng_for(430, M * 31 + N * 7 + K)
    for e, m in ((5, 10), (6, 9)):
        A = quantized(workloads.lognormal_tensor(rng, (M, K), -4.0, 3.0), e, m, 1)
        B = quantized(workloads.lognormal_tensor(rng, (K, N), -4.0, 3.0), e, m, 1)
        if M == 0 or N == 0:
            c, st = run_gpu(A, B, e, m, 1)
            assert c.shape == (M, N) and int(st.sum()) == 0
            continue
        check(A, B, e, m, 1, paths=paths_for(e, m))


@pytest.mark.parametrize("den", [1, 0])
def test_bfloat16_family_extreme_exponents(den):
    """1/8/7: products far outside fp32's range in both directions (2^-250 .. 2^250), sums that
    overflow fp32 before they are rounded, fp32-denormal accumulator values."""
    rng = workloads.rng_for(445, den)
    M, N, K = 70, 66, 50
    e, m = 8, 7
    A = quantized(workloads.lognormal_tensor(rng, (M, K), 0.0, 40.0, p_zero=0.05), e, m, den)
    B = quantized(workloads.lognormal_tensor(rng, (K, N), 0.0, 40.0, p_zero=0.05), e, m, den)
    A[:, :10] = quantized(workloads.lognormal_tensor(rng, (M, 10), -70.0, 3.0), e, m, den)   # tiny x tiny
    B[:10, :] = quantized(workloads.lognormal_tensor(rng, (10, N), -66.0, 3.0), e, m, den)
    A[:, 10:14] = quantized(workloads.lognormal_tensor(rng, (M, 4), 63.0, 1.0), e, m, den)   # near the top
    B[10:14, :] = quantized(workloads.lognormal_tensor(rng, (4, N), 63.5, 1.0), e, m, den)
    check(A, B, e, m, den, paths=(0, 1, 2))


def test_unaligned_output_and_leading_dimension():
    rng = workloads.rng_for(431)
    A = quantized(workloads.lognormal_tensor(rng, (70, 24), -3.0, 2.0), 6, 9, 1)
    B = quantized(workloads.lognormal_tensor(rng, (24, 37), -3.0, 2.0), 6, 9, 1)
    check(A, B, 6, 9, 1, ldc=41, off=1)
    check(A, B, 6, 9, 1, ldc=40, off=0, want_stats=False)
    A = quantized(A, 5, 10, 1)
    B = quantized(B, 5, 10, 1)
    check(A, B, 5, 10, 1, ldc=44, off=3, paths=(1, 2))


def test_group_boundaries_match_algorithm_1():
    """One large element and many ones: what survives depends on which group of eight each element
    falls into (hand-computed in the oracle's pins); here through the GPU."""
    x = np.array([[2048, 1, 1, 1, 1, 1, 1, 1] + [1] * 8], dtype=np.float32)
    ones = np.ones((16, 1), dtype=np.float32)
    for path in (1, 2):
        c, _ = run_gpu(x, ones, 5, 10, 1, path=path)
        assert c[0, 0] == 2056.0
        c, _ = run_gpu(np.ascontiguousarray(x[:, :8]), ones[:8], 5, 10, 1, path=path)
        assert c[0, 0] == 2048.0


def test_denormal_fraction_of_fmac8_output_binary16():
    """The quantity Table II reports: with small operands most of the 1/5/10 output is denormal
    while 1/6/9 has none; counts come from the kernel's own statistics."""
    rng = workloads.rng_for(440)
    M, N, K = 256, 192, 96
    X = workloads.lognormal_tensor(rng, (M, K), -10.0, 1.0)
    W = workloads.lognormal_tensor(rng, (K, N), -10.0, 1.0)
    frac = {}
    for e, m in ((5, 10), (6, 9)):
        A, B = quantized(X, e, m, 1), quantized(W, e, m, 1)
        _, st_ref = check(A, B, e, m, 1, paths=paths_for(e, m))
        frac[(e, m)] = int(st_ref[oracle.ST_DENORMAL]) / (M * N)
    assert frac[(5, 10)] > 0.5 and frac[(6, 9)] == 0.0


@pytest.mark.parametrize("e,m,path", [(6, 9, 0), (5, 10, 0)])
def test_config3_forward_full_size_sampled(e, m, path):
    """The BERT-base forward product at full size (4096 x 3072 x 768) in the benchmark's launch
    configuration; 8192 sampled outputs, each recomputed by the oracle."""
    cfg = workloads.config3()
    X, W = quantized(cfg["X"], e, m, 1), quantized(cfg["W"], e, m, 1)
    dX, dW = torch.from_numpy(X).to(DEV), torch.from_numpy(W).to(DEV)
    M, N = X.shape[0], W.shape[1]
    dC = torch.empty(M, N, dtype=torch.float32, device=DEV)
    st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    qf.qfmt_gemm_fmac8(qf.make_matrix(dX), qf.make_matrix(dW), dC, N, qf.make_format(e, m, 1), st, 0, path)
    torch.cuda.synchronize()
    c = dC.cpu().numpy()
    rng = np.random.default_rng(450)
    ii = np.concatenate([rng.integers(0, M, size=8188), [0, 0, M - 1, M - 1]])
    jj = np.concatenate([rng.integers(0, N, size=8188), [0, N - 1, 0, N - 1]])
    ref = oracle.fmac8_gemm_sampled(X, W, ii, jj, e, m, 1)
    assert np.array_equal(c[ii, jj].view(np.uint32), ref.view(np.uint32))
    # the statistics describe the tensor that was written: recount it on the CPU
    _, st_c = oracle.quantize_stats(c, e, m, 1, 1.0)
    got = st.cpu().numpy().view(np.uint64)
    assert np.array_equal(got[:256], st_c[:256]) and int(got[oracle.ST_TOTAL]) == M * N
    assert int(got[oracle.ST_DENORMAL]) == int(st_c[oracle.ST_DENORMAL])


def test_errors():
    d = torch.ones(64, dtype=torch.float32, device=DEV)
    a = qf.make_matrix(d.data_ptr(), False, 8, 8, 8)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_gemm_fmac8(a, a, d, 8, qf.make_format(8, 11))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT       # operands of more than 11 significant bits
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_gemm_fmac8(a, a, d, 8, qf.make_format(6, 9), None, 0, 2)
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT       # the native kernel is for 1/5/10 and 1/8/7 only
    b = qf.make_matrix(d.data_ptr(), False, 4, 8, 8)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_gemm_fmac8(a, b, d, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG          # inner dimensions differ
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_gemm_fmac8(a, a, d, 4, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG          # ldc below N
    torch.cuda.synchronize()
    assert torch.all(d == 1.0)
