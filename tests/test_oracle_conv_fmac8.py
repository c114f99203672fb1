"""Pins for the oracle's FMAC-8 convolution (no GPU): Algorithm 1 applied to the sums of a
convolution layer (Section IV-A), in the order of reduction the oracle's header states.

Checked against: the already pinned FMAC-8 matrix product (a 1 x 1 filter is one), the exact
convolution where every partial sum is representable (small integers: pins taps, padding and
index order), and a step-by-step rational model of Algorithm 1 fed with the reduction sequence
built here in plain loops (pins the order of the reduction, the place a padding term keeps in its
run, and the run boundaries).
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from test_oracle_format import NearestTable, bits_f32, frac_of_f32_bits
from test_oracle_fmac import format_values, rational_round


def fmt_tensor(rng, shape, e, m, lo, hi):
    n = int(np.prod(shape))
    return bits_f32(format_values(e, m, rng, n, lo, hi)).reshape(shape)


# ---------------------------------------------------------------------------------------------
# 1 x 1 filter, no padding: each of the three products is an FMAC-8 matrix product
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("e,m", [(6, 9), (5, 10)])
def test_pointwise_filter_is_the_fmac8_matrix_product(e, m):
    rng = np.random.default_rng(21 + e)
    n, ci, h, w, co = 2, 19, 3, 4, 5      # 19 channels: a run of eight, another, a run of three
    geom = (n, ci, h, w, co, 1, 1, 0, 0)
    b = 2 ** (e - 1) - 1
    X = fmt_tensor(rng, (n, ci, h, w), e, m, b - 4, b + 3)
    Wt = fmt_tensor(rng, (co, ci, 1, 1), e, m, b - 4, b + 3)
    dY = fmt_tensor(rng, (n, co, h, w), e, m, b - 4, b + 3)
    pix = n * h * w
    Xm = np.ascontiguousarray(X.transpose(0, 2, 3, 1).reshape(pix, ci))      # [pixel][ci]
    dYm = np.ascontiguousarray(dY.transpose(0, 2, 3, 1).reshape(pix, co))    # [pixel][co]
    Wm = np.ascontiguousarray(Wt.reshape(co, ci))
    # forward: Y[pixel][co] = sum_ci X[pixel][ci] W[co][ci]
    Y = oracle.conv_fmac8(oracle.CONV_FWD, X, Wt, geom, e, m).reshape(n, co, h, w)
    want = oracle.fmac8_gemm(Xm, Wm, e, m, transB=True).reshape(n, h, w, co).transpose(0, 3, 1, 2)
    assert np.array_equal(Y.view(np.uint32), np.ascontiguousarray(want).view(np.uint32))
    # data gradient: dX[pixel][ci] = sum_co dY[pixel][co] W[co][ci]
    dX = oracle.conv_fmac8(oracle.CONV_DGRAD, dY, Wt, geom, e, m).reshape(n, ci, h, w)
    want = oracle.fmac8_gemm(dYm, Wm, e, m).reshape(n, h, w, ci).transpose(0, 3, 1, 2)
    assert np.array_equal(dX.view(np.uint32), np.ascontiguousarray(want).view(np.uint32))
    # filter gradient: dW[co][ci] = sum_pixel dY[pixel][co] X[pixel][ci], pixels in (n, oh, ow) order
    dW = oracle.conv_fmac8(oracle.CONV_WGRAD, dY, X, geom, e, m).reshape(co, ci)
    want = oracle.fmac8_gemm(dYm, Xm, e, m, transA=True)
    assert np.array_equal(dW.view(np.uint32), want.view(np.uint32))


# ---------------------------------------------------------------------------------------------
# small integers: nothing is ever rounded before the end, so the result is R(exact convolution)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("geom", [(2, 8, 5, 6, 3, 3, 3, 1, 1), (1, 5, 4, 4, 2, 3, 2, 0, 1), (2, 3, 6, 3, 4, 2, 3, 1, 0)])
def test_small_integers_give_the_rounded_exact_convolution(geom):
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    rng = np.random.default_rng(sum(geom))
    X = rng.integers(-2, 3, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(co, ci, r, s)).astype(np.float32)
    dY = rng.integers(-2, 3, size=(n, co, oh, ow)).astype(np.float32)
    for which, P, Q in ((oracle.CONV_FWD, X, Wt), (oracle.CONV_DGRAD, dY, Wt), (oracle.CONV_WGRAD, dY, X)):
        exact, _ = oracle.conv(which, P, Q, geom)
        assert np.max(np.abs(exact)) < 1024            # every partial sum is a value of 1/6/9
        got = oracle.conv_fmac8(which, P, Q, geom, 6, 9)
        assert np.array_equal(got.astype(np.float64), exact)
        ii = rng.integers(0, exact.size, size=17)
        assert np.array_equal(oracle.conv_fmac8(which, P, Q, geom, 6, 9, idx=ii), got[ii])


# ---------------------------------------------------------------------------------------------
# the order of the reduction, padding terms and run boundaries: Algorithm 1 step by step
# ---------------------------------------------------------------------------------------------
def sequences(which, P, Q, geom, channel_major=False):
    """For every output, in the flat order of ``oracle.conv``: the list of (x, y) factor pairs of
    its sum in the oracle's stated order (or, channel_major, with the channel index outermost: an
    order the oracle does not use).  Padding positions appear as x = 0 (or y = 0)."""
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1

    def taps_then_channels(nc):
        if channel_major:
            return [(rr, ss, c) for c in range(nc) for rr in range(r) for ss in range(s)]
        return [(rr, ss, c) for rr in range(r) for ss in range(s) for c in range(nc)]

    out = []
    if which == oracle.CONV_FWD:
        for b in range(n):
            for o in range(co):
                for y0 in range(oh):
                    for x0 in range(ow):
                        seq = []
                        for rr, ss, c in taps_then_channels(ci):
                            ih, iw = y0 + rr - ph, x0 + ss - pw
                            xin = float(P[b, c, ih, iw]) if 0 <= ih < h and 0 <= iw < w else 0.0
                            seq.append((xin, float(Q[o, c, rr, ss])))
                        out.append(seq)
    elif which == oracle.CONV_DGRAD:
        for b in range(n):
            for c in range(ci):
                for y0 in range(h):
                    for x0 in range(w):
                        seq = []
                        for rr, ss, o in taps_then_channels(co):
                            yy, xx = y0 - rr + ph, x0 - ss + pw
                            g = float(P[b, o, yy, xx]) if 0 <= yy < oh and 0 <= xx < ow else 0.0
                            seq.append((g, float(Q[o, c, rr, ss])))
                        out.append(seq)
    else:
        for o in range(co):
            for c in range(ci):
                for rr in range(r):
                    for ss in range(s):
                        seq = []
                        for b in range(n):
                            for yy in range(oh):
                                for xx in range(ow):
                                    ih, iw = yy + rr - ph, xx + ss - pw
                                    xin = float(Q[b, c, ih, iw]) if 0 <= ih < h and 0 <= iw < w else 0.0
                                    seq.append((float(P[b, o, yy, xx]), xin))
                        out.append(seq)
    return out


def algorithm1(seq, tab, e, m, den):
    b = 2 ** (e - 1) - 1
    min_normal = Fraction(2) ** (1 - b)

    def to_format(v):
        wd = rational_round(tab, v, e, m)
        if wd is None:
            return Fraction(0)
        rr = frac_of_f32_bits(wd)
        return Fraction(0) if (not den and abs(rr) < min_normal) else rr

    master, small = np.float32(0), Fraction(0)
    for k, (x, y) in enumerate(seq):
        if k % 8 == 0:
            master = np.float32(master + np.float32(float(small)))
            small = Fraction(0)
        small = to_format(small + Fraction(x) * Fraction(y))
    master = np.float32(master + np.float32(float(small)))
    return to_format(Fraction(float(master)))


@pytest.mark.parametrize("den", [1, 0])
def test_matches_algorithm_1_on_the_stated_order(den):
    e, m = 6, 9
    tab = NearestTable(e, m)
    b = 2 ** (e - 1) - 1
    geom = (2, 12, 4, 3, 3, 3, 3, 1, 1)    # twelve channels: runs of eight straddle the taps, padding included
    n, ci, h, w, co, r, s, ph, pw = geom
    rng = np.random.default_rng(77)
    X = fmt_tensor(rng, (n, ci, h, w), e, m, b - 6, b + 3)
    Wt = fmt_tensor(rng, (co, ci, r, s), e, m, b - 6, b + 3)
    dY = fmt_tensor(rng, (n, co, h, w), e, m, 1, 14)          # small gradients: denormal sums
    differs_from_other_order = 0
    for which, P, Q in ((oracle.CONV_FWD, X, Wt), (oracle.CONV_DGRAD, dY, Wt), (oracle.CONV_WGRAD, dY, X)):
        got = oracle.conv_fmac8(which, P, Q, geom, e, m, den).view(np.uint32)
        seqs = sequences(which, P, Q, geom)
        assert len(seqs) == got.size
        pick = rng.choice(got.size, size=min(got.size, 60), replace=False)
        other = sequences(which, P, Q, geom, channel_major=True) if which != oracle.CONV_WGRAD else None
        for f in pick:
            want = algorithm1(seqs[f], tab, e, m, den)
            assert Fraction(float(bits_f32(got[f]))) == want, (which, int(f))
            if other is not None and algorithm1(other[f], tab, e, m, den) != want:
                differs_from_other_order += 1
    # the check can tell the stated order from another one
    assert differs_from_other_order > 0
