"""Pins for the oracle's single-rounding sums (no GPU): FMAC and Algorithm 1 (FMAC-8), and the
layer formula Y = R(R(acc) + R(B)) of Section IV-A.

Checked against: the host's IEEE fp32 and binary16 additions, exact rational arithmetic with a
nearest-value search over the enumerated format, and hand-computed dot products in which the
format-precision accumulator visibly loses what a wide accumulator would keep.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from test_oracle_format import NearestTable, bits_f32, f32_bits, frac_of_f32_bits


def format_values(e, m, rng, n, lo=None, hi=None):
    """n random finite values of format (e, m) as fp32 words, signs mixed, exponents spread."""
    tab_codes = 1 << (e + m)
    top = ((1 << e) - 1) << m
    codes = rng.integers(0, top, size=n, dtype=np.uint64)
    if lo is not None:
        codes = rng.integers(lo << m, hi << m, size=n, dtype=np.uint64)
    codes |= rng.integers(0, 2, size=n, dtype=np.uint64) << np.uint64(e + m)
    assert tab_codes > 0
    return np.array([oracle.decode_code(int(c), e, m) for c in codes], dtype=np.uint32)


def rational_round(tab: NearestTable, v: Fraction, e, m):
    """fp32 word of the format value nearest to the exact rational v (None for an exact zero)."""
    if v == 0:
        return None
    code = tab.nearest_code(abs(v)) | ((1 if v < 0 else 0) << (e + m))
    return oracle.decode_code(code, e, m)


# ---------------------------------------------------------------------------------------------
# round(a + b)
# ---------------------------------------------------------------------------------------------
def test_add_to_e8_m23_is_the_host_fp32_addition():
    assert np.float32(1e-40) + np.float32(1e-41) != 0, "host flushes denormals; pin not meaningful"
    rng = np.random.default_rng(5)
    n = 60000
    a = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    b = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    # a third with nearby exponents (cancellation, carries), a few exact opposites and zeros
    near = slice(0, n // 3)
    b[near] = (b[near] & np.uint32(0x807FFFFF)) | (((a[near] >> np.uint32(23)) & np.uint32(0xFF)) << np.uint32(23))
    b[n - 50:n - 25] = a[n - 50:n - 25] ^ np.uint32(0x80000000)
    a[n - 25:n - 20] = 0
    b[n - 20:n - 15] = 0x80000000
    a[n - 15:n - 10], b[n - 15:n - 10] = 0x80000000, 0x80000000
    with np.errstate(over="ignore", invalid="ignore"):
        ref = (a.view(np.float32) + b.view(np.float32)).view(np.uint32)
    got = np.array([oracle.add_round_bits(int(x), int(y), 8, 23) for x, y in zip(a, b)], dtype=np.uint32)
    nan = np.isnan(ref.view(np.float32))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all(np.isnan(got[nan].view(np.float32)))


def test_add_binary16_matches_numpy_half_addition():
    rng = np.random.default_rng(6)
    a = format_values(5, 10, rng, 40000)
    b = format_values(5, 10, rng, 40000)
    ah, bh = bits_f32(a).astype(np.float16), bits_f32(b).astype(np.float16)
    with np.errstate(over="ignore"):
        ref = (ah + bh).astype(np.float32).view(np.uint32)
    got = np.array([oracle.add_round_bits(int(x), int(y), 5, 10) for x, y in zip(a, b)], dtype=np.uint32)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("e,m", [(6, 9), (5, 10), (8, 7)])
def test_add_matches_exact_rational_nearest(e, m):
    rng = np.random.default_rng(7)
    tab = NearestTable(e, m)
    n = 6000
    a = format_values(e, m, rng, n)
    b = format_values(e, m, rng, n)
    # adversarial third: a is a power of two and b a negative value near a quarter / half of
    # a's last place, where a sum rounded first to 24 bits could land on a tie it is not on
    k = n // 3
    lo_e, hi_e = 2 * m + 6, (1 << e) - 2
    ea = rng.integers(lo_e, hi_e, size=k)
    a[:k] = [oracle.decode_code(int(E) << m, e, m) for E in ea]
    eb = ea - m - rng.integers(0, 3, size=k)
    fb = rng.integers(0, 4, size=k) * rng.integers(0, 2, size=k)
    b[:k] = [oracle.decode_code((1 << (e + m)) | (int(E) << m) | int(f), e, m) for E, f in zip(eb, fb)]
    for x, y in zip(a.tolist(), b.tolist()):
        want = rational_round(tab, frac_of_f32_bits(x) + frac_of_f32_bits(y), e, m)
        got = oracle.add_round_bits(x, y, e, m)
        if want is None:
            assert got in (0, 0x80000000)
        else:
            assert got == want, (hex(x), hex(y))


def test_add_special_values():
    inf, ninf, nan = 0x7F800000, 0xFF800000, 0x7FC00000
    one = int(f32_bits(1.0))
    assert oracle.add_round_bits(inf, ninf, 6, 9) == nan
    assert oracle.add_round_bits(inf, one, 6, 9) == inf
    assert oracle.add_round_bits(one, ninf, 6, 9) == ninf
    assert oracle.add_round_bits(0xFFC00000, one, 6, 9) == nan      # NaN in, positive quiet NaN out
    assert oracle.add_round_bits(0x80000000, 0x80000000, 6, 9) == 0x80000000
    assert oracle.add_round_bits(0x80000000, 0, 6, 9) == 0
    assert oracle.add_round_bits(one, one ^ 0x80000000, 6, 9) == 0   # exact cancellation gives +0
    big = oracle.decode_code(((1 << 6) - 2) << 9 | 0x1FF, 6, 9)      # largest normal of 1/6/9
    assert oracle.add_round_bits(big, big, 6, 9) == inf
    # denormals: smallest + smallest is exact; with flushing the denormal result becomes zero
    tiny = oracle.decode_code(1, 6, 9)
    assert oracle.add_round_bits(tiny, tiny, 6, 9, 1) == oracle.decode_code(2, 6, 9)
    assert oracle.add_round_bits(tiny, tiny, 6, 9, 0) == 0


# ---------------------------------------------------------------------------------------------
# FMAC: round(a + x*y), one rounding
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("e,m", [(6, 9), (5, 10), (8, 7)])
def test_fmac_matches_exact_rational_nearest(e, m):
    rng = np.random.default_rng(8)
    tab = NearestTable(e, m)
    n = 6000
    b = 2 ** (e - 1) - 1
    # factors around 2^0 +- a quarter of the range so that products stay mostly finite
    lo, hi = max(1, b - b // 2), min((1 << e) - 2, b + b // 2)
    x = format_values(e, m, rng, n, lo, hi)
    y = format_values(e, m, rng, n, lo, hi)
    a = format_values(e, m, rng, n)
    # half of the accumulators close to the product's size: carries, cancellation and ties
    for i in range(0, n, 2):
        p = abs(frac_of_f32_bits(int(x[i])) * frac_of_f32_bits(int(y[i])))
        w = rational_round(tab, p * Fraction(int(rng.integers(1, 9)), 4), e, m)
        if w is not None and w & 0x7FFFFFFF != 0x7F800000:
            a[i] = w | (int(rng.integers(0, 2)) << 31)
    for u, v, w in zip(a.tolist(), x.tolist(), y.tolist()):
        exact = frac_of_f32_bits(u) + frac_of_f32_bits(v) * frac_of_f32_bits(w)
        want = rational_round(tab, exact, e, m)
        got = oracle.fmac_bits(u, v, w, e, m)
        if want is None:
            assert got in (0, 0x80000000)
        else:
            assert got == want, (hex(u), hex(v), hex(w))


def test_fmac_is_fused_not_two_roundings():
    # 1/5/10: x*y = (1 + 2^-10)^2 = 1 + 2^-9 + 2^-20.  Rounding the product first gives 1 + 2^-9,
    # and 1 + 2^-9 minus (1 + 2^-9) is 0; the fused operation keeps the 2^-20.
    x = int(f32_bits(1.0 + 2.0 ** -10))
    a = int(f32_bits(-(1.0 + 2.0 ** -9)))
    assert oracle.fmac_bits(a, x, x, 5, 10) == int(f32_bits(2.0 ** -20))
    # denormals flushed: the same tiny result is below 2^-14 and becomes zero
    assert oracle.fmac_bits(a, x, x, 5, 10, 0) & 0x7FFFFFFF == 0
    assert oracle.fmac_bits(0x7F800000, 0, x, 5, 10) == 0x7F800000   # inf + 0*x
    assert oracle.fmac_bits(0, 0x7F800000, 0, 5, 10) == 0x7FC00000   # inf * 0 is invalid


# ---------------------------------------------------------------------------------------------
# Algorithm 1 (FMAC-8)
# ---------------------------------------------------------------------------------------------
def fmac8_row(x, e, m, denormals=1):
    """FMAC-8 dot product of x with a vector of ones, through the matrix entry point."""
    A = np.asarray(x, dtype=np.float32).reshape(1, -1)
    B = np.ones((A.shape[1], 1), dtype=np.float32)
    return float(oracle.fmac8_gemm(A, B, e, m, denormals)[0, 0])


def test_fmac8_hand_computed_binary16():
    # values up to 2048 have spacing 1 in 1/5/10, from 2048 on spacing 2
    assert fmac8_row([1, 2, 3, 4, 5, 6, 7, 8], 5, 10) == 36.0            # all exact
    # 2048 + 1 is a tie between 2048 and 2050 and goes to the even significand, seven times over
    assert fmac8_row([2048, 1, 1, 1, 1, 1, 1, 1], 5, 10) == 2048.0
    # the ninth element starts a new group: its 8 ones survive in the fp32 master accumulator
    assert fmac8_row([2048, 1, 1, 1, 1, 1, 1, 1] + [1] * 8, 5, 10) == 2056.0
    # moving the large element to position 8 (second group) changes what is lost
    assert fmac8_row([1] * 8 + [2048] + [1] * 7, 5, 10) == 2056.0
    assert fmac8_row([1] * 7 + [2048], 5, 10) == 2056.0                  # 7 + 2048 = 2055 -> tie -> 2056
    # 2048 + 3 = 2051 is a tie between 2050 and 2052; 2052 has the even significand
    assert fmac8_row([2048, 3], 5, 10) == 2052.0
    # master accumulator is fp32: 2048 and 1 in different groups add to 2049 exactly, and only the
    # final rounding to the format makes it 2048
    assert fmac8_row([2048] + [0] * 7 + [1], 5, 10) == 2048.0
    assert fmac8_row([2048] + [0] * 7 + [3], 5, 10) == 2052.0
    # a group total above 65504 + 16 overflows the small accumulator although the sum would fit fp32
    assert fmac8_row([40000, 40000], 5, 10) == float("inf")
    assert fmac8_row([40000] + [0] * 7 + [-40000], 5, 10) == 0.0
    assert fmac8_row([40000, 40000] + [0] * 6 + [-40000], 5, 10) == float("inf")


def test_fmac8_hand_computed_1_6_9():
    # 1/6/9: spacing 1 up to 1024, spacing 2 from 1024 on
    assert fmac8_row([1024, 1, 1, 1], 6, 9) == 1024.0
    assert fmac8_row([1024, 3, 1], 6, 9) == 1028.0   # 1027 -> tie -> 1028; 1029 -> tie -> 1028
    assert fmac8_row([1, 1, 1, 1021], 6, 9) == 1024.0
    # denormal accumulator values: 2^-39 is the smallest denormal; 3 of them are exact, and with
    # flushing every partial sum is flushed as it is produced
    t = 2.0 ** -39
    assert fmac8_row([t, t, t], 6, 9, 1) == 3 * t
    assert fmac8_row([t, t, t], 6, 9, 0) == 0.0


@pytest.mark.parametrize("e,m", [(6, 9), (5, 10)])
@pytest.mark.parametrize("den", [1, 0])
def test_fmac8_matches_rational_model(e, m, den):
    """Algorithm 1 step by step with exact rationals for the small accumulator (nearest-value
    search over the enumerated format) and numpy's fp32 addition for the master accumulator."""
    rng = np.random.default_rng(9 + e)
    tab = NearestTable(e, m)
    b = 2 ** (e - 1) - 1
    M, N, K = 5, 4, 45
    A = bits_f32(format_values(e, m, rng, M * K, b - 8, b + 4)).reshape(M, K)
    B = bits_f32(format_values(e, m, rng, K * N, 1, 12)).reshape(K, N)   # tiny factors: denormal sums
    B[:, 2:] = bits_f32(format_values(e, m, rng, K * 2, b - 3, b + 3)).reshape(K, 2)
    got = oracle.fmac8_gemm(A, B, e, m, den).view(np.uint32)
    min_normal = Fraction(2) ** (1 - b)

    def to_format(v: Fraction) -> Fraction:
        w = rational_round(tab, v, e, m)
        if w is None:
            return Fraction(0)
        r = frac_of_f32_bits(w)   # finite by construction of the inputs
        return Fraction(0) if (not den and abs(r) < min_normal) else r

    for i in range(M):
        for j in range(N):
            master, small = np.float32(0), Fraction(0)
            for k in range(K):
                if k % 8 == 0:
                    master = np.float32(master + np.float32(float(small)))
                    small = Fraction(0)
                small = to_format(small + Fraction(float(A[i, k])) * Fraction(float(B[k, j])))
            master = np.float32(master + np.float32(float(small)))
            want = to_format(Fraction(float(master)))
            assert Fraction(float(bits_f32(got[i, j]))) == want, (i, j)


def test_fmac8_transposes_and_sampling():
    rng = np.random.default_rng(10)
    e, m = 6, 9
    M, N, K = 7, 6, 19
    A = bits_f32(format_values(e, m, rng, M * K, 25, 36)).reshape(M, K)
    B = bits_f32(format_values(e, m, rng, K * N, 25, 36)).reshape(K, N)
    C = oracle.fmac8_gemm(A, B, e, m)
    assert np.array_equal(oracle.fmac8_gemm(np.ascontiguousarray(A.T), B, e, m, transA=True), C)
    assert np.array_equal(oracle.fmac8_gemm(A, np.ascontiguousarray(B.T), e, m, transB=True), C)
    ii, jj = rng.integers(0, M, size=20), rng.integers(0, N, size=20)
    assert np.array_equal(oracle.fmac8_gemm_sampled(A, B, ii, jj, e, m), C[ii, jj])
    with pytest.raises(ValueError):
        oracle.fmac8_gemm(np.full((2, 2), 1.0 + 2.0 ** -20, dtype=np.float32), B[:2], e, m)


# ---------------------------------------------------------------------------------------------
# Y = R(R(acc) + R(B)) with statistics of Y
# ---------------------------------------------------------------------------------------------
def test_layer_output_without_bias_is_quantize_stats():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal((33, 47)) * 2.0 ** rng.integers(-45, 35, size=(33, 47))).astype(np.float32)
    x[0, :5] = [0.0, -0.0, np.inf, -np.inf, np.nan]
    for scale in (1.0, 2.0 ** 8):
        q0, s0 = oracle.quantize_stats(x, 6, 9, 1, scale)
        q1, s1 = oracle.bias_quantize_stats(x, None, 6, 9, 1, scale)
        assert np.array_equal(q0.view(np.uint32), q1.view(np.uint32)) and np.array_equal(s0, s1)


def test_layer_output_binary16_matches_numpy_half_arithmetic():
    rng = np.random.default_rng(12)
    acc = (rng.standard_normal((64, 40)) * 2.0 ** rng.integers(-20, 8, size=(64, 40))).astype(np.float32)
    bias = (rng.standard_normal(40) * 2.0 ** rng.integers(-16, 4, size=40)).astype(np.float32)
    y, st = oracle.bias_quantize_stats(acc, bias, 5, 10, 1, 1.0)
    ref = (acc.astype(np.float16) + bias.astype(np.float16)[None, :]).astype(np.float32)
    assert np.array_equal(y.view(np.uint32), ref.view(np.uint32))
    # recount the histogram from the result with frexp: value = f * 2^ex, 0.5 <= f < 1
    _, ex = np.frexp(ref.astype(np.float64))
    code = np.where(ref == 0, 0, np.clip(ex - 1 + 15, 0, None))
    code = np.where(np.abs(ref) < 2.0 ** -14, 0, code)
    assert np.array_equal(st[:32].astype(np.int64), np.bincount(code.ravel(), minlength=32)[:32])
    assert int(st[oracle.ST_TOTAL]) == acc.size and int(st[:256].sum()) == acc.size
    den = (np.abs(ref) < 2.0 ** -14) & (ref != 0)
    assert int(st[oracle.ST_DENORMAL]) == int(den.sum())


@pytest.mark.parametrize("den", [1, 0])
def test_layer_output_matches_exact_rational_and_invariants(den):
    rng = np.random.default_rng(13)
    e, m = 6, 9
    tab = NearestTable(e, m)
    rows, cols = 48, 24
    acc = (rng.standard_normal((rows, cols)) * 2.0 ** rng.integers(-44, 33, size=(rows, cols))).astype(np.float32)
    bias = (rng.standard_normal(cols) * 2.0 ** rng.integers(-44, 33, size=cols)).astype(np.float32)
    bias[0], acc[:, 1] = 0.0, 0.0
    acc[3, 2] = -bias[2]                       # may cancel exactly once both are rounded
    scale = 4.0
    y, st = oracle.bias_quantize_stats(acc, bias, e, m, den, scale)
    ra, _ = oracle.quantize_stats(acc, e, m, den, scale, want_stats=False)
    rb, _ = oracle.quantize_stats(bias, e, m, den, scale, want_stats=False)
    min_normal = Fraction(2) ** (1 - 31)
    zero_in = under = over = 0
    for i in range(rows):
        for j in range(cols):
            if not (np.isfinite(ra[i, j]) and np.isfinite(rb[j])):
                continue
            s = Fraction(float(ra[i, j])) + Fraction(float(rb[j]))
            w = rational_round(tab, s, e, m)
            got = int(y.view(np.uint32)[i, j])
            if w is None:
                zero_in += 1
                assert got & 0x7FFFFFFF == 0
                continue
            if not den and w & 0x7FFFFFFF != 0x7F800000 and abs(frac_of_f32_bits(w)) < min_normal:
                w &= 0x80000000
            assert got == w, (i, j)
            under += int(w & 0x7FFFFFFF == 0)
            over += int(w & 0x7FFFFFFF == 0x7F800000)
    finite_terms = np.isfinite(ra) & np.isfinite(rb)[None, :]
    if finite_terms.all():
        assert int(st[oracle.ST_ZERO_IN]) == zero_in
        assert int(st[oracle.ST_UNDERFLOW]) == under and int(st[oracle.ST_OVERFLOW]) == over
    n = rows * cols
    assert int(st[:256].sum()) == n == int(st[oracle.ST_TOTAL])
    top = (1 << e) - 1
    assert int(st[top]) == int(st[oracle.ST_OVERFLOW] + st[oracle.ST_INF_IN] + st[oracle.ST_NAN])
    if den:
        assert int(st[0]) == int(st[oracle.ST_ZERO_IN] + st[oracle.ST_UNDERFLOW] + st[oracle.ST_DENORMAL])
        assert int(st[oracle.ST_UNDERFLOW]) == 0   # a sum of two format values is on the denormal grid
    else:
        assert int(st[0]) == int(st[oracle.ST_ZERO_IN] + st[oracle.ST_UNDERFLOW])
        assert int(st[oracle.ST_DENORMAL]) == int(st[oracle.ST_UNDERFLOW])
