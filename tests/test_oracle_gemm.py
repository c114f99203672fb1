"""Pins for the oracle's contractions (no GPU): hand-computed cases, numpy float64 matmul,
torch float64 conv2d with autograd, and the 1x1-convolution-is-a-GEMM identity."""
import numpy as np
import pytest
import torch

import oracle


def test_hand_computed_2x2x2():
    A = np.array([[1, 2], [3, 4]], dtype=np.float32)
    B = np.array([[5, 6], [7, 8]], dtype=np.float32)
    C, T = oracle.gemm(A, B)
    assert C.tolist() == [[19.0, 22.0], [43.0, 50.0]]
    assert T.tolist() == [[19.0, 22.0], [43.0, 50.0]]
    # transposed reads of the stored matrices: A^T B, A B^T, A^T B^T
    assert oracle.gemm(A, B, transA=True)[0].tolist() == [[26.0, 30.0], [38.0, 44.0]]
    assert oracle.gemm(A, B, transB=True)[0].tolist() == [[17.0, 23.0], [39.0, 53.0]]
    assert oracle.gemm(A, B, transA=True, transB=True)[0].tolist() == [[23.0, 31.0], [34.0, 46.0]]


def test_hand_computed_3x3x4_signed_powers_of_two():
    A = np.array([[1, -2, 0.5, 0], [0, 4, -1, 2], [-8, 0.25, 0, 1]], dtype=np.float32)
    B = np.array([[2, 0, -1], [1, 1, 0], [-4, 2, 8], [0.5, -2, 1]], dtype=np.float32)
    C, T = oracle.gemm(A, B)
    assert C.tolist() == [[-2.0, -1.0, 3.0], [9.0, -2.0, -6.0], [-15.25, -1.75, 9.0]]
    assert T.tolist() == [[6.0, 3.0, 5.0], [9.0, 10.0, 10.0], [16.75, 2.25, 9.0]]


@pytest.mark.parametrize("transA", [False, True])
@pytest.mark.parametrize("transB", [False, True])
def test_matches_numpy_float64(transA, transB):
    rng = np.random.default_rng(3)
    M, N, K = 37, 29, 53
    A = rng.standard_normal((K, M) if transA else (M, K)).astype(np.float32)
    B = rng.standard_normal((N, K) if transB else (K, N)).astype(np.float32)
    C, T = oracle.gemm(A, B, transA, transB)
    a = (A.T if transA else A).astype(np.float64)
    b = (B.T if transB else B).astype(np.float64)
    assert np.allclose(C, a @ b, rtol=0, atol=1e-12)
    assert np.allclose(T, np.abs(a) @ np.abs(b), rtol=1e-14, atol=0)
    ii = rng.integers(0, M, size=50)
    jj = rng.integers(0, N, size=50)
    c, t = oracle.gemm_sampled(A, B, ii, jj, transA, transB)
    assert np.array_equal(c, C[ii, jj]) and np.array_equal(t, T[ii, jj])


GEOMS = [
    (2, 3, 5, 6, 4, 3, 3, 1, 1),
    (1, 4, 7, 7, 2, 1, 1, 0, 0),
    (2, 2, 6, 5, 3, 3, 2, 1, 0),
    (1, 1, 4, 4, 1, 3, 3, 0, 0),
]


@pytest.mark.parametrize("geom", GEOMS)
def test_conv_matches_torch_float64(geom):
    n, ci, h, w, co, r, s, ph, pw = geom
    rng = np.random.default_rng(17)
    X = rng.standard_normal((n, ci, h, w)).astype(np.float32)
    Wt = rng.standard_normal((co, ci, r, s)).astype(np.float32)
    tx = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    tw = torch.tensor(Wt, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(tx, tw, padding=(ph, pw))
    dY = rng.standard_normal(tuple(y.shape)).astype(np.float32)
    gx, gw = torch.autograd.grad(y, (tx, tw), torch.tensor(dY, dtype=torch.float64))
    c, t = oracle.conv(oracle.CONV_FWD, X, Wt, geom)
    assert np.allclose(c, y.detach().numpy().reshape(-1), rtol=0, atol=1e-12)
    ta = torch.nn.functional.conv2d(tx.detach().abs(), tw.detach().abs(), padding=(ph, pw))
    assert np.allclose(t, ta.numpy().reshape(-1), rtol=1e-13, atol=0)
    c, _ = oracle.conv(oracle.CONV_DGRAD, dY, Wt, geom)
    assert np.allclose(c, gx.numpy().reshape(-1), rtol=0, atol=1e-12)
    c, _ = oracle.conv(oracle.CONV_WGRAD, dY, X, geom)
    assert np.allclose(c, gw.numpy().reshape(-1), rtol=0, atol=1e-12)
    idx = rng.integers(0, c.size, size=7)
    cs, _ = oracle.conv(oracle.CONV_WGRAD, dY, X, geom, idx)
    assert np.array_equal(cs, c[idx])


def test_conv_1x1_is_a_gemm():
    n, ci, h, w, co = 2, 5, 3, 4, 6
    rng = np.random.default_rng(19)
    X = rng.standard_normal((n, ci, h, w)).astype(np.float32)
    Wt = rng.standard_normal((co, ci, 1, 1)).astype(np.float32)
    c, t = oracle.conv(oracle.CONV_FWD, X, Wt, (n, ci, h, w, co, 1, 1, 0, 0))
    A = X.transpose(0, 2, 3, 1).reshape(n * h * w, ci)          # [pixels][ci]
    C, T = oracle.gemm(A, Wt.reshape(co, ci), transB=True)       # [pixels][co]
    assert np.array_equal(c.reshape(n, co, h, w).transpose(0, 2, 3, 1).reshape(-1, co), C)
    assert np.array_equal(t.reshape(n, co, h, w).transpose(0, 2, 3, 1).reshape(-1, co), T)


def test_products_of_format_values_are_exact_in_fp64():
    """Significands of at most 11 bits: the product needs 22 bits, far inside fp64's 53, and the
    exponent range of 1/8/m products (down to 2^-272) is inside fp64's, so 'exact product' holds."""
    a = np.float32(2.0 ** -133) * np.float32(127)   # 1/8/7 denormal, largest significand
    b = np.float32((2 - 2.0 ** -10) * 2.0 ** -120)
    C, _ = oracle.gemm(np.array([[a]], dtype=np.float32), np.array([[b]], dtype=np.float32))
    from fractions import Fraction
    assert Fraction(float(C[0, 0])) == Fraction(float(a)) * Fraction(float(b))
