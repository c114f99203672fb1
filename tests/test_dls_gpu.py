"""GPU parity of the device-resident dynamic-loss-scale controller and of the rounding pass that
reads its scale from device memory, against the CPU oracle (bit-exact)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def to_device(state: qf.qfmt_dls_t):
    raw = np.frombuffer(bytes(state), dtype=np.uint8).copy()
    return torch.from_numpy(raw).to(DEV)


def from_device(t) -> qf.qfmt_dls_t:
    return qf.qfmt_dls_t.from_buffer_copy(t.cpu().numpy().tobytes())


def same(a, b):
    fields = [f[0] for f in qf.qfmt_dls_t._fields_]
    return all(getattr(a, f) == getattr(b, f) for f in fields)


def test_struct_layout_matches_the_header():
    assert ctypes.sizeof(qf.qfmt_dls_t) == 56 and ctypes.sizeof(oracle.DlsState) == 56


def test_controller_trace_matches_oracle():
    rng = np.random.default_rng(500)
    for growth, backoff, interval in ((2.0, 0.5, 3), (1.7, 0.3, 1), (2.0, 0.5, 5)):
        ref = oracle.DlsState(2.0 ** 12, growth, backoff, 2.0 ** -4, 2.0 ** 16, interval, 0, 0, 0, 0, 0)
        d_state = to_device(qf.qfmt_dls_t(2.0 ** 12, growth, backoff, 2.0 ** -4, 2.0 ** 16, interval, 0, 0, 0, 0, 0))
        for step in range(60):
            n_rec = int(rng.integers(0, 600))            # also more records than the block has threads
            recs = np.zeros((n_rec, qf.STATS_WORDS), dtype=np.uint64)
            recs[:, oracle.ST_TOTAL] = 100
            recs[:, oracle.ST_UNDERFLOW] = rng.integers(0, 50, size=n_rec)   # must not matter
            if n_rec and rng.random() < 0.3:
                col = [oracle.ST_OVERFLOW, oracle.ST_NAN, oracle.ST_INF_IN][int(rng.integers(0, 3))]
                recs[int(rng.integers(0, n_rec)), col] = int(rng.integers(1, 1 << 40))
            d_recs = torch.from_numpy(recs.view(np.int64)).to(DEV)
            qf.qfmt_dls_update(d_state, d_recs, n_rec)
            oracle.dls_update(ref, recs)
            assert same(from_device(d_state), ref), (growth, step)


def test_scale_search_on_a_gradient_tensor():
    """Gradients that overflow 1/5/10 at the starting scale: the loop quantizes with the device
    scale, updates the controller, and never reads anything back until the end of each step (only
    to compare).  The oracle runs the same loop on the CPU."""
    n = 200003
    g = workloads.lognormal_tensor(workloads.rng_for(510), (n,), -6.0, 3.0, p_zero=0.01)
    e, m = 5, 10
    ref = oracle.DlsState(2.0 ** 24, 2.0, 0.5, 1.0, 2.0 ** 24, 4, 0, 0, 0, 0, 0)
    d_state = to_device(qf.qfmt_dls_t(2.0 ** 24, 2.0, 0.5, 1.0, 2.0 ** 24, 4, 0, 0, 0, 0, 0))
    d_g = torch.from_numpy(g).to(DEV)
    d_q = torch.empty_like(d_g)
    d_st = torch.zeros(1, qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    fmt = qf.make_format(e, m, 1, 123.0)   # the scale in the descriptor is ignored by the _dls call
    skipped = 0
    for step in range(24):
        qf.qfmt_quantize_stats_dls(d_g, d_q, n, fmt, d_state, d_st[0])
        qf.qfmt_dls_update(d_state, d_st, 1)
        q_ref, st_ref = oracle.quantize_stats(g, e, m, 1, ref.scale)
        oracle.dls_update(ref, st_ref)
        torch.cuda.synchronize()
        assert np.array_equal(d_q.cpu().numpy().view(np.uint32), q_ref.view(np.uint32)), step
        assert np.array_equal(d_st.cpu().numpy().view(np.uint64)[0], st_ref), step
        assert same(from_device(d_state), ref), step
        skipped += ref.skip
    assert 0 < skipped < 24 and ref.scale < 2.0 ** 24   # it backed off, then ran clean steps


def test_errors():
    d = torch.zeros(64, dtype=torch.uint8, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_dls_update(None, d, 0)
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_dls_update(d, None, 3)
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_quantize_stats_dls(d, d, 4, qf.make_format(6, 9), None)
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
