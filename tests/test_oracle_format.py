"""Pins for the oracle's format arithmetic (no GPU).

Each test checks the oracle against something other than itself: Table I, the value formula of
Definition III.1 evaluated with Python integers, numpy's IEEE binary16 and torch's bfloat16
conversions, exact rational nearest-value search, and the host's own fp32 multiply.
"""
import bisect
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2103_15940_b200 import workloads

FORMATS16 = [(5, 10), (6, 9), (8, 7)]
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_formats.txt")


def f32_bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def bits_f32(u):
    return np.asarray(u, dtype=np.uint32).view(np.float32)


def frac_of_f32_bits(u: int) -> Fraction:
    """Exact value of a finite fp32 word, from the IEEE-754 definition."""
    s = -1 if u >> 31 else 1
    E, f = (u >> 23) & 0xFF, u & 0x7FFFFF
    assert E != 255
    if E == 0:
        return s * Fraction(f, 1 << 149)
    return s * (Fraction((1 << 23) | f) * Fraction(2) ** (E - 150))


# ---------------------------------------------------------------------------------------------
# Table I
# ---------------------------------------------------------------------------------------------
def test_table1_constants():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for name, e, p, e_min, e_max, min_den in rows:
        e, p = int(e), int(p)
        assert oracle.emin(e) == int(e_min), name
        assert oracle.emax(e) == int(e_max), name
        assert oracle.bias(e) == 2 ** (e - 1) - 1
        if min_den != "-":
            assert oracle.min_denormal_log2(e, p) == int(min_den), name
        assert oracle.max_normal(e, p) == (2 - 2.0 ** -p) * 2.0 ** oracle.bias(e)
    assert oracle.max_normal(5, 10) == 65504.0


# ---------------------------------------------------------------------------------------------
# Packed codes: decode follows Eq. (1); binary16 / bfloat16 agree with the libraries' views.
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("e,m", FORMATS16)
def test_decode_matches_value_formula(e, m):
    b = 2 ** (e - 1) - 1
    for code in range(1 << 16):
        s, E, f = code >> 15, (code >> m) & ((1 << e) - 1), code & ((1 << m) - 1)
        u = oracle.decode_code(code, e, m)
        if E == (1 << e) - 1:
            if f:
                assert (u & 0x7FFFFFFF) > 0x7F800000
            else:
                assert u == (s << 31) | 0x7F800000
            continue
        # Eq. (1): x = M * 2^(E - p + 1) with p = m + 1 significand bits
        if E == 0:
            val = Fraction(f) * Fraction(2) ** (1 - b - m)
        else:
            val = Fraction((1 << m) | f) * Fraction(2) ** (E - b - m)
        if val == 0:
            assert u == s << 31
        else:
            assert frac_of_f32_bits(u) == (-val if s else val)


def test_decode_binary16_matches_numpy():
    codes = np.arange(1 << 16, dtype=np.uint16)
    ref = codes.view(np.float16).astype(np.float32).view(np.uint32)
    got = np.array([oracle.decode_code(int(c), 5, 10) for c in codes], dtype=np.uint32)
    nan = np.isnan(ref.view(np.float32))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all(np.isnan(got[nan].view(np.float32)))


def test_decode_bfloat16_matches_torch():
    codes = torch.arange(1 << 16, dtype=torch.int32).to(torch.int16)
    ref = codes.view(torch.bfloat16).to(torch.float32).numpy().view(np.uint32)
    got = np.array([oracle.decode_code(c, 8, 7) for c in range(1 << 16)], dtype=np.uint32)
    nan = np.isnan(ref.view(np.float32))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all(np.isnan(got[nan].view(np.float32)))


# ---------------------------------------------------------------------------------------------
# Brute force over all 2^16 encodings.
# ---------------------------------------------------------------------------------------------
def finite_positive_codes(e, m):
    return list(range(0, ((1 << e) - 1) << m))  # +0, denormals, normals, ascending in value


@pytest.mark.parametrize("e,m", FORMATS16)
def test_decode_quantize_identity_and_flush(e, m):
    for code in range(1 << 16):
        u = oracle.decode_code(code, e, m)
        E, f = (code >> m) & ((1 << e) - 1), code & ((1 << m) - 1)
        q, den = oracle.quantize_bits(u, e, m, 1)
        if E == (1 << e) - 1 and f:
            assert (q & 0x7FFFFFFF) == 0x7FC00000
            continue
        assert q == u
        assert den == (1 if (E == 0 and f) else 0)
        assert oracle.encode_code(q, e, m) == code
        qn, den_n = oracle.quantize_bits(u, e, m, 0)
        if E == 0:
            assert qn == (u & 0x80000000) and den_n == (1 if f else 0)
        else:
            assert qn == u


@pytest.mark.parametrize("e,m", FORMATS16)
def test_midpoints_tie_to_even_and_neighbours(e, m):
    codes = finite_positive_codes(e, m)
    vals = [oracle.decode_code(c, e, m) for c in codes]
    for sign in (0, 0x80000000):
        for c in range(len(codes) - 1):
            lo, hi = frac_of_f32_bits(vals[c]), frac_of_f32_bits(vals[c + 1])
            mid = (lo + hi) / 2
            # midpoints of adjacent values need m+2 significant bits: exact in fp32 unless it
            # falls below the fp32 denormal grid (only 1/8/7's lowest midpoints)
            mf = np.float32(float(mid))
            if Fraction(float(mf)) != mid:
                continue
            mb = int(f32_bits(mf)) | sign
            even_code = codes[c] if codes[c] % 2 == 0 else codes[c + 1]
            q, _ = oracle.quantize_bits(mb, e, m, 1)
            assert q == (oracle.decode_code(even_code, e, m) | sign), (c, hex(mb))
            below, _ = oracle.quantize_bits(mb - 1, e, m, 1)  # one fp32 ulp towards zero
            above, _ = oracle.quantize_bits(mb + 1, e, m, 1)
            assert below == (vals[c] | sign)
            assert above == (vals[c + 1] | sign)


@pytest.mark.parametrize("e,m", FORMATS16)
def test_overflow_and_underflow_thresholds(e, m):
    b = 2 ** (e - 1) - 1
    if e < 8:
        maxn = np.float32((2 - 2.0 ** -m) * 2.0 ** b)
        thresh = np.float32((2 - 2.0 ** -(m + 1)) * 2.0 ** b)  # max normal + half ulp (a tie)
        tb = int(f32_bits(thresh))
        assert oracle.quantize_bits(tb, e, m, 1)[0] == 0x7F800000
        assert oracle.quantize_bits(tb - 1, e, m, 1)[0] == int(f32_bits(maxn))
        assert oracle.quantize_bits(tb | 0x80000000, e, m, 1)[0] == 0xFF800000
        half_min = int(f32_bits(np.float32(2.0 ** (1 - b - m - 1))))  # tie between 0 and min denormal
        min_den = int(f32_bits(np.float32(2.0 ** (1 - b - m))))
        assert oracle.quantize_bits(half_min, e, m, 1)[0] == 0
        assert oracle.quantize_bits(half_min + 1, e, m, 1) == (min_den, 1)
        assert oracle.quantize_bits(half_min | 0x80000000, e, m, 1)[0] == 0x80000000
    # flush happens after rounding: just below min normal still rounds up to min normal
    min_norm = int(f32_bits(np.float32(2.0 ** (1 - b))))
    assert oracle.quantize_bits(min_norm - 1, e, m, 0) == (min_norm, 0)


@pytest.mark.parametrize("e,m", FORMATS16)
@pytest.mark.parametrize("den", [1, 0])
def test_monotone(e, m, den):
    rng = np.random.default_rng(7)
    u = np.concatenate([rng.integers(0, 0x7F800000, size=200000, dtype=np.uint32),
                        workloads.edge_bit_patterns()])
    u = u[(u & 0x7FFFFFFF) <= 0x7F800000]
    x = np.sort(u.view(np.float32))
    q, _ = oracle.quantize_stats(x, e, m, den, 1.0, want_stats=False)
    assert np.all(q[1:] >= q[:-1])


# ---------------------------------------------------------------------------------------------
# Library conversions: IEEE binary16 (numpy) and bfloat16 (torch CPU), round-to-nearest-even.
# ---------------------------------------------------------------------------------------------
def random_patterns(n, seed):
    rng = np.random.default_rng(seed)
    return np.concatenate([rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32),
                           workloads.edge_bit_patterns()])


def test_binary16_matches_numpy_conversion():
    u = random_patterns(1 << 22, 11)
    # concentrate a second batch in binary16's own range, denormals included
    rng = np.random.default_rng(12)
    near = (rng.integers(0x30000000, 0x48000000, size=1 << 22, dtype=np.uint64).astype(np.uint32)
            | (rng.integers(0, 2, size=1 << 22, dtype=np.uint64).astype(np.uint32) << np.uint32(31)))
    u = np.concatenate([u, near])
    x = u.view(np.float32)
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).astype(np.float32)
    q, _ = oracle.quantize_stats(x, 5, 10, 1, 1.0, want_stats=False)
    nan = np.isnan(ref)
    assert np.array_equal(q.view(np.uint32)[~nan], ref.view(np.uint32)[~nan])
    assert np.all(np.isnan(q[nan]))


def test_bfloat16_matches_torch_conversion():
    u = random_patterns(1 << 22, 13)
    rng = np.random.default_rng(14)
    tiny = rng.integers(0, 0x01000000, size=1 << 20, dtype=np.uint64).astype(np.uint32)  # fp32 denormals
    u = np.concatenate([u, tiny, tiny | np.uint32(0x80000000)])
    x = u.view(np.float32)
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    q, _ = oracle.quantize_stats(x, 8, 7, 1, 1.0, want_stats=False)
    nan = np.isnan(ref)
    assert np.array_equal(q.view(np.uint32)[~nan], ref.view(np.uint32)[~nan])
    assert np.all(np.isnan(q[nan]))


def test_e8_m23_is_identity():
    u = random_patterns(1 << 20, 15)
    x = u.view(np.float32)
    q, st = oracle.quantize_stats(x, 8, 23, 1, 1.0)
    nan = np.isnan(x)
    assert np.array_equal(q.view(np.uint32)[~nan], u[~nan])
    assert int(st[oracle.ST_UNDERFLOW]) == 0 and int(st[oracle.ST_OVERFLOW]) == 0


# ---------------------------------------------------------------------------------------------
# 1/6/9 has no library: "nearest representable", taken literally, by exact rational search.
# ---------------------------------------------------------------------------------------------
class NearestTable:
    """All finite non-negative values of a format as exact integers on a common grid."""

    def __init__(self, e, m):
        self.e, self.m = e, m
        self.codes = finite_positive_codes(e, m)
        self.unit = 1 - (2 ** (e - 1) - 1) - m  # log2 of the smallest denormal
        b = 2 ** (e - 1) - 1
        vals = []
        for c in self.codes:
            E, f = c >> m, c & ((1 << m) - 1)
            vals.append(f if E == 0 else ((1 << m) | f) << (E - 1))
        self.vals = vals  # value = vals[i] * 2^unit
        self.over = (1 << m) << ((1 << e) - 2)  # 2^(Emax+1) on the same grid: code E = 2^e-1, f = 0

    def nearest_code(self, mag: Fraction):
        """Packed code (without sign) of the nearest value; ties to the even code; inf code on
        reaching max + half ulp."""
        grid = mag / (Fraction(2) ** self.unit)
        i = bisect.bisect_right(self.vals, grid) - 1  # vals[i] <= grid
        lo = self.vals[i]
        hi = self.vals[i + 1] if i + 1 < len(self.vals) else self.over
        d_lo, d_hi = grid - lo, hi - grid
        if d_lo < d_hi:
            pick = i
        elif d_hi < d_lo:
            pick = i + 1
        else:
            pick = i if self.codes[i] % 2 == 0 else i + 1
        if pick == len(self.vals):
            return ((1 << self.e) - 1) << self.m
        return self.codes[pick]


def nearest_check(e, m, x_bits, scale_log2=0, scale=1.0):
    tab = NearestTable(e, m)
    x = x_bits.view(np.float32)
    q, _ = oracle.quantize_stats(x, e, m, 1, scale, want_stats=False)
    qb = q.view(np.uint32)
    for u, got in zip(x_bits.tolist(), qb.tolist()):
        mag = abs(frac_of_f32_bits(u)) * Fraction(2) ** scale_log2
        code = tab.nearest_code(mag) | ((u >> 31) << 15)
        assert got == oracle.decode_code(code, e, m), hex(u)


@pytest.mark.parametrize("e,m", [(6, 9), (5, 10)])
def test_nearest_by_exact_rational_search(e, m):
    rng = np.random.default_rng(21)
    b = 2 ** (e - 1) - 1
    lo_exp, hi_exp = 127 + (1 - b - m) - 3, 127 + b + 2
    ex = rng.integers(lo_exp, hi_exp, size=120000, dtype=np.uint64).astype(np.uint32)
    fr = rng.integers(0, 1 << 23, size=120000, dtype=np.uint64).astype(np.uint32)
    # half of the fractions get only a few high bits so that exact ties are common
    fr[::2] &= np.uint32(0x7FF000)
    sg = rng.integers(0, 2, size=120000, dtype=np.uint64).astype(np.uint32) << np.uint32(31)
    nearest_check(e, m, (sg | (ex << np.uint32(23)) | fr).astype(np.uint32))


# ---------------------------------------------------------------------------------------------
# Loss scale: the host's IEEE single-precision multiply; powers of two give one exact rounding.
# ---------------------------------------------------------------------------------------------
def test_scale_matches_host_multiply():
    assert np.float32(1e-40) * np.float32(0.5) != 0, "host flushes denormals; pin not meaningful"
    rng = np.random.default_rng(31)
    x = random_patterns(200000, 32)
    scales = np.concatenate([
        np.array([1.0, 2.0 ** 8, 2.0 ** 15, 2.0 ** 16, 2.0 ** -20, 3.0, 0.1, 1000.0, 65535.0, 1e-30, 1e30],
                 dtype=np.float32),
        rng.integers(0x00000001, 0x7F800000, size=40, dtype=np.uint64).astype(np.uint32).view(np.float32)])
    for s in scales:
        sb = int(f32_bits(s))
        sub = x[rng.integers(0, x.size, size=6000)]
        with np.errstate(over="ignore", under="ignore", invalid="ignore"):
            ref = (sub.view(np.float32) * s).view(np.uint32)
        got = np.array([oracle.scale_bits(int(u), sb) for u in sub], dtype=np.uint32)
        nan = np.isnan(ref.view(np.float32))
        assert np.array_equal(got[~nan], ref[~nan]), float(s)
        assert np.all(np.isnan(got[nan].view(np.float32)))


@pytest.mark.parametrize("k", [8, 15, -5])
def test_power_of_two_scale_is_single_exact_rounding(k):
    rng = np.random.default_rng(41)
    e, m = 6, 9
    ex = rng.integers(127 - 45 - k, 127 + 33 - k, size=40000, dtype=np.uint64).astype(np.uint32)
    fr = rng.integers(0, 1 << 23, size=40000, dtype=np.uint64).astype(np.uint32)
    fr[::2] &= np.uint32(0x7FE000)
    nearest_check(e, m, ((ex << np.uint32(23)) | fr).astype(np.uint32), scale_log2=k, scale=2.0 ** k)
