"""GPU parity of qfmt_gemm_packed16 (the FMACS contraction of Section III-B on packed binary16 /
bfloat16 codes) against the fp64 oracle applied to the oracle's own expansion of the codes.

Bar, as for qfmt_gemm: |c_gpu - c_exact| <= 2^-20 * sum_k |a_ik||b_jk| per element; bit-exact
where every accumulation order is exact; identical bits run to run."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

TOL = 2.0 ** -20
DEV = "cuda:0"
FORMATS = [(5, 10), (8, 7)]


def codes_of(x, e, m):
    """Packed codes of x rounded to 1/e/m and their fp32 containers, both by the oracle."""
    codes, _ = oracle.quantize_stats_pack16(x, e, m, 1, 1.0)
    return codes, oracle.unpack16(codes, e, m)


def gpu_gemm16(cA, cB, e, m, transA=False, transB=True, lda_pad=0, ldb_pad=0, ldc_pad=0, workspace=None):
    """cA, cB are the STORED code matrices; C = op(A) op(B) as float32 [M, N].  The default flags are
    the K-contiguous pair A [M, K], B [N, K]."""
    def stored(c, pad, trans):
        r, k = c.shape
        d = torch.full((max(r, 1), k + pad), 0x7E00, dtype=torch.int16, device=DEV)   # padding holds NaN codes
        if r and k:
            d[:r, :k] = torch.from_numpy(np.ascontiguousarray(c).view(np.int16)).to(DEV)
        return qf.make_matrix(d, trans, rows=r, cols=k, ld=k + pad), d
    a, dA = stored(cA, lda_pad, transA)
    b, dB = stored(cB, ldb_pad, transB)
    M = cA.shape[1] if transA else cA.shape[0]
    N = cB.shape[0] if transB else cB.shape[1]
    ldc = N + ldc_pad
    dC = torch.full((max(M, 1), ldc), float("nan"), dtype=torch.float32, device=DEV)
    wb = qf.qfmt_gemm_packed16_workspace_bytes(a, b) if workspace is None else workspace
    ws = torch.zeros(max(wb, 256), dtype=torch.uint8, device=DEV)
    qf.qfmt_gemm_packed16(a, b, dC, ldc, qf.make_format(e, m), ws, max(wb, 256))
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    torch.cuda.synchronize()
    out = dC.cpu().numpy()[:M]
    if ldc_pad:
        assert np.all(np.isnan(out[:, N:]))
    return out[:, :N]


def worst_ratio(C, A, B, sample=None, seed=0, transA=False, transB=True):
    """A, B: stored fp32 containers; returns the worst error as a multiple of the tolerance."""
    if sample is None:
        ref, T = oracle.gemm(A, B, transA, transB)
        c = C.astype(np.float64)
    else:
        rng = np.random.default_rng(seed)
        M, N = C.shape
        ii = np.concatenate([rng.integers(0, M, size=sample), [0, M - 1, 0, M - 1]])
        jj = np.concatenate([rng.integers(0, N, size=sample), [0, N - 1, N - 1, 0]])
        ref, T = oracle.gemm_sampled(A, B, ii, jj, transA, transB)
        c = C[ii, jj].astype(np.float64)
    err = np.abs(c - ref)
    assert np.all(err <= TOL * T), f"worst {float(np.max(err / np.maximum(T, 1e-300))) / TOL:.3f} x tolerance"
    return float(np.max(err / np.maximum(T, 1e-300))) / TOL


@pytest.mark.parametrize("e,m", FORMATS)
@pytest.mark.parametrize("transA", [False, True])
@pytest.mark.parametrize("transB", [True, False])
@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (5, 3, 16), (64, 128, 64), (128, 256, 64), (256, 256, 128), (300, 260, 200),
                                   (513, 40, 1000), (64, 700, 72), (70, 50, 203), (257, 513, 4104)])
def test_small_integers_are_bit_exact(e, m, M, N, K, transA, transB):
    """Entries in -4..4: every product and partial sum is a small integer, exact in any order, so
    a wrong tile offset, K range, transpose or split shows up as a wrong integer.  All four
    operand layouts (K-contiguous and M- / N-contiguous).  Ragged sizes:
    partial tiles in M and N, K not a multiple of the 64-element stage (the copy engine zero-fills
    past K; the NaN codes in the row padding must never be read as data)."""
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A = rng.integers(-4, 5, size=(K, M) if transA else (M, K)).astype(np.float32)
    B = rng.integers(-4, 5, size=(N, K) if transB else (K, N)).astype(np.float32)
    cA, qA = codes_of(A, e, m)
    cB, qB = codes_of(B, e, m)
    assert np.array_equal(qA, A) and np.array_equal(qB, B)
    pad = lambda c: 8 if c % 8 == 0 else 8 - c % 8      # leading dimensions must be multiples of 8
    C = gpu_gemm16(cA, cB, e, m, transA, transB, lda_pad=pad(A.shape[1]), ldb_pad=pad(B.shape[1]) + 8, ldc_pad=3)
    ref, _ = oracle.gemm(A, B, transA, transB)
    assert np.array_equal(C.astype(np.float64), ref)


@pytest.mark.parametrize("e,m", FORMATS)
def test_operand_order_and_layout(e, m):
    """A one-hot A row picks a row of B: C[i, j] = B[j, k_i] exactly, which fails for a transposed
    or swapped operand; powers of two spread over the format's range keep products exact."""
    rng = np.random.default_rng(5)
    M, N, K = 130, 270, 192
    ks = rng.integers(0, K, size=M)
    A = np.zeros((M, K), np.float32)
    A[np.arange(M), ks] = 2.0
    B = np.ldexp(1.0, rng.integers(-12, 12, size=(N, K))).astype(np.float32) * rng.choice([-1.0, 1.0], size=(N, K))
    cA, _ = codes_of(A, e, m)
    cB, qB = codes_of(B, e, m)
    C = gpu_gemm16(cA, cB, e, m)
    assert np.array_equal(C, 2.0 * qB[:, ks].T)
    # the same product from the transposed copies of both operands (M and N contiguous)
    C = gpu_gemm16(np.ascontiguousarray(cA.T), np.ascontiguousarray(cB.T), e, m, True, False, lda_pad=6, ldb_pad=2)
    assert np.array_equal(C, 2.0 * qB[:, ks].T)


@pytest.mark.parametrize("e,m", FORMATS)
def test_format_values_within_bound_and_reproducible(e, m):
    """Signed weights against heavy-tailed activations, denormal codes included; several tiles, a
    ragged tail and a K long enough for several summation groups."""
    rng = workloads.rng_for(700, e)
    M, N, K = 520, 390, 2600
    X = workloads.lognormal_tensor(rng, (M, K), -3.0, 2.0)
    W = workloads.normal_tensor(rng, (N, K), 0.02)
    if e == 5:
        X[:, ::7] *= 2.0 ** -14   # into binary16's denormal range
    cA, qA = codes_of(X, e, m)
    cB, qB = codes_of(W, e, m)
    C1 = gpu_gemm16(cA, cB, e, m)
    C2 = gpu_gemm16(cA, cB, e, m)
    assert np.array_equal(C1.view(np.uint32), C2.view(np.uint32))
    print("worst", worst_ratio(C1, qA, qB))
    C3 = gpu_gemm16(cA, cB, e, m, workspace=256)   # no room for split K: still within the bound
    worst_ratio(C3, qA, qB)


@pytest.mark.parametrize("e,m", FORMATS)
def test_denormal_codes_are_not_flushed(e, m):
    """Products of the format's denormals with large normals are exact and must arrive."""
    M, N, K = 128, 256, 64
    tiny = 2.0 ** (oracle.min_denormal_log2(e, m))
    A = np.zeros((M, K), np.float32)
    B = np.zeros((N, K), np.float32)
    A[:, 0] = tiny * 3 if e == 5 else tiny   # a denormal code
    B[:, 0] = 2.0 ** 10
    cA, qA = codes_of(A, e, m)
    cB, qB = codes_of(B, e, m)
    assert qA[0, 0] != 0.0
    C = gpu_gemm16(cA, cB, e, m)
    expect = np.float32(np.float64(qA[0, 0]) * 2.0 ** 10)
    assert expect != 0.0 and np.all(C == expect)


@pytest.mark.parametrize("e,m", FORMATS)
def test_config5_ffn_up_forward_full_size(e, m):
    """8192 x 4096 x 1024 (the shape the bench times): 65 536 sampled outputs, each a full
    reduction by the oracle."""
    cfg = workloads.config5_layer(2, 0)
    cA, qA = codes_of(cfg["X"], e, m)
    cB, qB = codes_of(np.ascontiguousarray(cfg["W"].T), e, m)
    C = gpu_gemm16(cA, cB, e, m)
    print("config5 ffn_up", (e, m), worst_ratio(C, qA, qB, sample=65536, seed=9))
    cW, qW = codes_of(cfg["W"], e, m)                     # stored [d_in, d_out]: N contiguous
    C2 = gpu_gemm16(cA, cW, e, m, False, False)
    assert np.array_equal(C.view(np.uint32), C2.view(np.uint32))


@pytest.mark.parametrize("e,m", FORMATS)
def test_long_k_weight_gradient_shape(e, m):
    """1024 x 1024 x 8192: few tiles and a long K, so K is split among CTAs and the parts are added
    by the reduction pass."""
    rng = workloads.rng_for(701, e)
    X = workloads.lognormal_tensor(rng, (8192, 1024), -3.0, 2.0)
    G = workloads.lognormal_tensor(rng, (8192, 1024), -6.0, 3.0)
    cA, qA = codes_of(X, e, m)
    cB, qB = codes_of(G, e, m)
    C = gpu_gemm16(cA, cB, e, m, True, False)           # dW = X^T dY: tokens are K, both operands MN-major
    print("wgrad", (e, m), worst_ratio(C, qA, qB, sample=32768, seed=3, transA=True, transB=False))
    cAt, cBt = np.ascontiguousarray(cA.T), np.ascontiguousarray(cB.T)
    C2 = gpu_gemm16(cAt, cBt, e, m)                      # the same product from K-contiguous copies
    assert np.array_equal(C.view(np.uint32), C2.view(np.uint32))


def test_empty_and_errors():
    fmt = qf.make_format(5, 10)
    d16 = torch.zeros(64 * 64 + 8, dtype=torch.int16, device=DEV)
    dC = torch.full((64, 64), 5.0, dtype=torch.float32, device=DEV)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    mat = lambda rows, cols, ld=64, trans=False, t=d16: qf.make_matrix(t, trans, rows=rows, cols=cols, ld=ld)
    qf.qfmt_gemm_packed16(mat(0, 64), mat(64, 64), dC, 64, fmt, ws, 256)       # M = 0: nothing happens
    qf.qfmt_gemm_packed16(mat(64, 64), mat(64, 0), dC, 64, fmt, ws, 256)       # N = 0
    torch.cuda.synchronize()
    assert torch.all(dC == 5.0)
    qf.qfmt_gemm_packed16(mat(64, 0), mat(0, 64), dC, 64, fmt, ws, 256)        # K = 0: zeros
    torch.cuda.synchronize()
    assert torch.all(dC == 0.0)
    for bad_fmt in ((6, 9), (4, 3), (8, 10)):
        with pytest.raises(qf.QfmtError) as ei:
            qf.qfmt_gemm_packed16(mat(64, 64), mat(64, 64), dC, 64, qf.make_format(*bad_fmt), ws, 256)
        assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT
    for a, b, ldc in ((mat(64, 64, ld=56), mat(64, 64), 64),          # ld below the row length
                      (mat(8, 60, ld=60), mat(60, 64), 64),           # ld not a multiple of 8
                      (mat(8, 64, t=d16[1:]), mat(64, 64), 64),       # base not 16-byte aligned
                      (mat(64, 64), mat(32, 64), 64),                 # K mismatch
                      (mat(64, 64), mat(64, 64), 60),                 # ldc below N
                      (mat(64, 64, t=None), mat(64, 64), 64)):
        with pytest.raises(qf.QfmtError) as ei:
            qf.qfmt_gemm_packed16(a, b, dC, ldc, fmt, ws, 256)
        assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    torch.cuda.synchronize()
