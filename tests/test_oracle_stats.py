"""Pins for the oracle's range statistics (no GPU).

Counts are checked against closed forms on enumerated inputs, against the invariants that tie
the histogram to the counters, against an independent recount with numpy's frexp, and against
the normal-distribution closed form for the log-normal synthetic tensors (which also shows the
paper's qualitative claim, Section V-A: 1/6/9 cuts the denormal fraction sharply versus 1/5/10
and loss scaling cuts it further).
"""
import math

import numpy as np
import pytest

import oracle
from paper_2103_15940_b200 import workloads

FORMATS16 = [(5, 10), (6, 9), (8, 7)]


def all_finite_values(e, m):
    codes = [c for c in range(1 << 16) if ((c >> m) & ((1 << e) - 1)) != (1 << e) - 1]
    return np.array([oracle.decode_code(c, e, m) for c in codes], dtype=np.uint32).view(np.float32)


@pytest.mark.parametrize("e,m", FORMATS16)
def test_enumerated_inputs_closed_form(e, m):
    x = all_finite_values(e, m)  # every finite code once, both signs
    q, st = oracle.quantize_stats(x, e, m, 1, 1.0)
    assert np.array_equal(q.view(np.uint32), x.view(np.uint32))
    nb = 1 << e
    assert int(st[0]) == 2 * (1 << m)                      # +-0 and the 2^m - 1 denormals per sign
    assert all(int(st[c]) == 2 * (1 << m) for c in range(1, nb - 1))
    assert int(st[nb - 1]) == 0 and int(st[nb:256].sum()) == 0
    assert int(st[oracle.ST_DENORMAL]) == 2 * ((1 << m) - 1)
    assert int(st[oracle.ST_ZERO_IN]) == 2
    assert int(st[oracle.ST_TOTAL]) == x.size
    assert int(st[oracle.ST_UNDERFLOW]) == 0 and int(st[oracle.ST_OVERFLOW]) == 0
    # flushed variant: the same denormals are counted, and they all become underflows
    qn, sn = oracle.quantize_stats(x, e, m, 0, 1.0)
    assert int(sn[oracle.ST_DENORMAL]) == 2 * ((1 << m) - 1)
    assert int(sn[oracle.ST_UNDERFLOW]) == 2 * ((1 << m) - 1)
    assert int(sn[0]) == 2 * (1 << m)
    assert np.count_nonzero(qn) == x.size - 2 * (1 << m)


def check_invariants(st, e, den):
    nb = 1 << e
    assert int(st[:256].sum()) == int(st[oracle.ST_TOTAL])
    assert int(st[nb:256].sum()) == 0
    z, u, d = int(st[oracle.ST_ZERO_IN]), int(st[oracle.ST_UNDERFLOW]), int(st[oracle.ST_DENORMAL])
    if den:
        assert int(st[0]) == z + u + d
    else:
        assert int(st[0]) == z + u and d <= u
    assert int(st[nb - 1]) == int(st[oracle.ST_OVERFLOW]) + int(st[oracle.ST_INF_IN]) + int(st[oracle.ST_NAN])


@pytest.mark.parametrize("e,m", FORMATS16 + [(4, 3), (8, 23), (2, 1)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("scale", [1.0, 2.0 ** 15, 3.0e-3])
def test_invariants_on_arbitrary_bit_patterns(e, m, den, scale):
    rng = np.random.default_rng(5)
    u = np.concatenate([rng.integers(0, 1 << 32, size=300000, dtype=np.uint64).astype(np.uint32),
                        workloads.edge_bit_patterns()])
    _, st = oracle.quantize_stats(u.view(np.float32), e, m, den, scale, want_q=False)
    check_invariants(st, e, den)
    x = u.view(np.float32)
    assert int(st[oracle.ST_NAN]) == int(np.isnan(x).sum())
    assert int(st[oracle.ST_INF_IN]) == int(np.isinf(x).sum())
    assert int(st[oracle.ST_ZERO_IN]) == int((x == 0).sum())


@pytest.mark.parametrize("e,m", FORMATS16)
@pytest.mark.parametrize("den", [1, 0])
def test_recount_with_frexp(e, m, den):
    """Histogram and counters recomputed from (x, q) with library routines only."""
    x = workloads.lognormal_tensor(workloads.rng_for(9), (400000,), -16.0, 9.0, p_zero=0.01)
    x[:5] = [np.inf, -np.inf, np.nan, 1e38, -1e38]
    scale = 2.0 ** 4
    q, st = oracle.quantize_stats(x, e, m, den, scale)
    b = 2 ** (e - 1) - 1
    mant, ex = np.frexp(q.astype(np.float64))  # |q| = mant * 2^ex, mant in [0.5, 1)
    lg = ex - 1
    code = np.where(q == 0, 0, np.where(~np.isfinite(q), (1 << e) - 1,
                                         np.where(lg < 1 - b, 0, lg + b))).astype(np.int64)
    hist = np.bincount(code, minlength=256)
    assert np.array_equal(hist, st[:256].astype(np.int64))
    finite_in = np.isfinite(x)
    assert int(st[oracle.ST_UNDERFLOW]) == int((finite_in & (x != 0) & (q == 0)).sum())
    assert int(st[oracle.ST_OVERFLOW]) == int((finite_in & np.isinf(q)).sum())
    if den:
        assert int(st[oracle.ST_DENORMAL]) == int(((q != 0) & np.isfinite(q) & (lg < 1 - b)).sum())
    else:
        # flushed elements are exactly those the denormal-keeping variant leaves denormal
        qd, sd = oracle.quantize_stats(x, e, m, 1, scale)
        assert int(st[oracle.ST_DENORMAL]) == int(sd[oracle.ST_DENORMAL])
        assert np.array_equal(q.view(np.uint32) != qd.view(np.uint32), (qd != 0) & (np.abs(qd.astype(np.float64)) < 2.0 ** (1 - b)))


def phi(z):
    return 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))


@pytest.mark.parametrize("e,m", FORMATS16[:2])
@pytest.mark.parametrize("k", [0, 8, 15])
def test_lognormal_closed_form_fractions(e, m, k):
    """log2|x| ~ N(mu, sigma): P(denormal) = (1-p0) [Phi((Emin-mu')/s) - Phi((Emin-m-1-mu')/s)],
    P(underflow) = (1-p0) Phi((Emin-m-1-mu')/s), mu' = mu + log2 S, up to rounding at the two
    edges (a sliver of one part in 2^(m+1) of a binade)."""
    n, mu, sigma, p0 = 1 << 22, -18.0, 8.0, 0.005
    x = workloads.config2_tensor(seed=1, n=n)
    _, st = oracle.quantize_stats(x, e, m, 1, 2.0 ** k, want_q=False)
    b = 2 ** (e - 1) - 1
    emin, mu2 = 1 - b, mu + k
    p_den = (1 - p0) * (phi((emin - mu2) / sigma) - phi((emin - m - 1 - mu2) / sigma))
    p_und = (1 - p0) * phi((emin - m - 1 - mu2) / sigma)
    for p, got in ((p_den, int(st[oracle.ST_DENORMAL])), (p_und, int(st[oracle.ST_UNDERFLOW]))):
        sd = math.sqrt(n * p * (1 - p))
        assert abs(got - n * p) <= 5 * sd + 2e-3 * n * p + 3, (p, got / n)
    assert abs(int(st[oracle.ST_ZERO_IN]) - n * p0) <= 5 * math.sqrt(n * p0)


def test_paper_qualitative_claim_on_synthetic_gradients():
    """Denormal fraction: 1/5/10 >> 1/6/9, and a loss scale lowers both (Tables II and III)."""
    x = workloads.lognormal_tensor(workloads.rng_for(2), (1 << 20,), -20.0, 4.0)
    frac = {}
    for e, m in FORMATS16[:2]:
        for k in (0, 10):
            _, st = oracle.quantize_stats(x, e, m, 1, 2.0 ** k, want_q=False)
            frac[(e, k)] = int(st[oracle.ST_DENORMAL]) / x.size
    assert frac[(5, 0)] > 0.5 and frac[(6, 0)] < 0.02
    assert frac[(5, 10)] < frac[(5, 0)] and frac[(6, 10)] <= frac[(6, 0)]


def test_empty_and_stats_only():
    q, st = oracle.quantize_stats(np.zeros(0, dtype=np.float32), 6, 9)
    assert q.size == 0 and int(st.sum()) == 0
    x = np.array([1.0, 0.0, -0.0, 2.0 ** -35], dtype=np.float32)
    q, st = oracle.quantize_stats(x, 6, 9, want_q=False)
    assert q is None and int(st[oracle.ST_TOTAL]) == 4 and int(st[oracle.ST_DENORMAL]) == 1


@pytest.mark.parametrize("threads", [2, 3, 16])
def test_pieces_in_parallel_equal_the_single_pass(threads):
    """The all-cores form used for timing (pieces with records of their own, summed) gives the same
    tensor and the same record as the one-element-at-a-time pass, ragged piece sizes included."""
    x = workloads.lognormal_tensor(workloads.rng_for(77), (100003,), -25.0, 8.0, p_zero=0.01)
    x[::977] = np.inf
    x[5::1013] = np.nan
    for e, m, den, scale in ((6, 9, 1, 1.0), (5, 10, 0, 2.0 ** 8), (8, 7, 1, 3.0e-5)):
        q1, s1 = oracle.quantize_stats(x, e, m, den, scale)
        qt, stt = oracle.quantize_stats(x, e, m, den, scale, threads=threads)
        assert np.array_equal(q1.view(np.uint32), qt.view(np.uint32))
        assert np.array_equal(s1, stt)
    _, s0 = oracle.quantize_stats(x[:5], 6, 9, threads=threads)  # fewer elements than pieces
    assert int(s0[oracle.ST_TOTAL]) == 5
