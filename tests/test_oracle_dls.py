"""Pins for the oracle's dynamic-loss-scale controller (no GPU).  The paper uses dynamic loss
scaling (Sections II and V) without stating the rule; the rule taken is written out in the oracle
and checked here against traces worked out by hand."""
import numpy as np

import oracle


def record(overflow=0, nan=0, inf_in=0):
    st = np.zeros(oracle.STATS_WORDS, dtype=np.uint64)
    st[oracle.ST_OVERFLOW], st[oracle.ST_NAN], st[oracle.ST_INF_IN] = overflow, nan, inf_in
    st[oracle.ST_TOTAL] = 1000
    st[5] = 1000 - overflow - nan - inf_in
    return st


def make(scale=2.0 ** 16, growth=2.0, backoff=0.5, interval=3, lo=1.0, hi=2.0 ** 24):
    return oracle.DlsState(scale, growth, backoff, lo, hi, interval, 0, 0, 0, 0, 0)


def test_hand_computed_trace():
    s = make()
    clean, bad = [record(), record()], [record(), record(overflow=2)]
    # step:   1      2      3 (grows)  4 (overflow)  5      6      7 (grows)  8 (NaN)  9 (inf in)
    steps = [clean, clean, clean, bad, clean, clean, clean, [record(nan=1)], [record(inf_in=7)]]
    want_scale = [2.0 ** 16, 2.0 ** 16, 2.0 ** 17, 2.0 ** 16, 2.0 ** 16, 2.0 ** 16, 2.0 ** 17, 2.0 ** 16, 2.0 ** 15]
    want_skip = [0, 0, 0, 1, 0, 0, 0, 1, 1]
    want_clean = [1, 2, 0, 0, 1, 2, 0, 0, 0]
    for i, recs in enumerate(steps):
        oracle.dls_update(s, np.stack(recs))
        assert (s.scale, s.skip, s.clean_steps) == (want_scale[i], want_skip[i], want_clean[i]), i
    assert (s.n_steps, s.n_skipped) == (9, 3)


def test_limits_and_counters_that_do_not_matter():
    s = make(scale=2.0, interval=1, lo=1.0, hi=4.0)
    # underflow and denormal counts never trigger a skip: only non-finite gradients do
    st = record()
    st[oracle.ST_UNDERFLOW], st[oracle.ST_DENORMAL] = 500, 400
    oracle.dls_update(s, st)
    assert (s.scale, s.skip) == (4.0, 0)
    oracle.dls_update(s, st)
    assert s.scale == 4.0                       # capped at max_scale
    for want in (2.0, 1.0, 1.0):                # floored at min_scale
        oracle.dls_update(s, record(overflow=1))
        assert (s.scale, s.skip) == (want, 1)
    oracle.dls_update(s, np.zeros((0, oracle.STATS_WORDS), dtype=np.uint64))   # no records: a clean step
    assert (s.scale, s.skip) == (2.0, 0)


def test_non_power_of_two_factors_are_fp32_products():
    s = make(scale=1000.0, growth=1.7, backoff=0.3, interval=1)
    oracle.dls_update(s, record())
    assert s.scale == float(np.float32(1000.0) * np.float32(1.7))
    prev = np.float32(s.scale)
    oracle.dls_update(s, record(nan=3))
    assert s.scale == float(prev * np.float32(0.3))
