"""GPU parity of qfmt_quantize_stats against the CPU oracle: rounded tensors and every count
must match bit for bit (integer work; no tolerance)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

FORMATS = [(5, 10), (6, 9), (8, 7)]


def run_gpu(x_np, e, m, den, scale, *, want_out=True, want_stats=True, in_place=False, in_off=0, out_off=0,
            accumulate=0, stats_t=None):
    """Runs the library on a device copy of x_np placed in_off floats past a 256-byte boundary."""
    n = x_np.size
    dev = torch.device("cuda:0")
    buf_in = torch.zeros(n + 64, dtype=torch.float32, device=dev)
    d_in = buf_in[in_off:in_off + n]
    d_in.copy_(torch.from_numpy(x_np.reshape(-1)))
    if in_place:
        d_out = d_in
    elif want_out:
        buf_out = torch.full((n + 64,), 7.0, dtype=torch.float32, device=dev)
        d_out = buf_out[out_off:out_off + n]
    else:
        d_out = None
    if want_stats and stats_t is None:
        stats_t = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=dev)  # dirty on purpose
    fmt = qf.make_format(e, m, den, scale)
    qf.qfmt_quantize_stats(d_in, d_out, n, fmt, stats_t if want_stats else None, accumulate)
    torch.cuda.synchronize()
    q = d_out.cpu().numpy() if d_out is not None else None
    if want_out and not in_place:
        # canaries around the output stay untouched
        assert torch.all(buf_out[:out_off] == 7.0) and torch.all(buf_out[out_off + n:] == 7.0)
    st = stats_t.cpu().numpy().view(np.uint64) if want_stats else None
    return q, st


def assert_same(q, st, q_ref, st_ref):
    if q is not None:
        assert np.array_equal(q.view(np.uint32).reshape(-1), q_ref.view(np.uint32).reshape(-1))
    if st is not None:
        assert np.array_equal(st, st_ref), (st[np.nonzero(st != st_ref)], st_ref[np.nonzero(st != st_ref)])


@pytest.mark.parametrize("e,m", FORMATS + [(8, 23), (2, 1), (4, 3), (7, 8), (5, 2)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("scale", [1.0, 2.0 ** 8, 3.0e-5, 1.0e30])
def test_arbitrary_bit_patterns(e, m, den, scale):
    rng = np.random.default_rng(100 + e * 31 + m)
    u = np.concatenate([rng.integers(0, 1 << 32, size=70001, dtype=np.uint64).astype(np.uint32),
                        workloads.edge_bit_patterns()])
    x = u.view(np.float32)
    q_ref, st_ref = oracle.quantize_stats(x, e, m, den, scale)
    q, st = run_gpu(x, e, m, den, scale)
    nan = np.isnan(q_ref)
    assert_same(q, st, q_ref, st_ref)
    assert np.all(np.isnan(q[nan]))


@pytest.mark.parametrize("e,m", FORMATS)
def test_all_codes_and_all_midpoints(e, m):
    """Every finite value of the format, every midpoint between neighbours and its two fp32
    neighbours: several tiles, with the ties that separate RNE from other roundings."""
    codes = np.array([c for c in range(1 << 16) if ((c >> m) & ((1 << e) - 1)) != (1 << e) - 1])
    vals = np.array([oracle.decode_code(int(c), e, m) for c in codes], dtype=np.uint32).view(np.float32)
    pos = np.sort(vals[vals >= 0].astype(np.float64))
    mids = ((pos[1:] + pos[:-1]) / 2).astype(np.float32)
    mb = mids.view(np.uint32)
    x = np.concatenate([vals, mids, (mb + 1).view(np.float32), (mb[mb > 0] - 1).view(np.float32), -mids])
    for den in (1, 0):
        q_ref, st_ref = oracle.quantize_stats(x, e, m, den, 1.0)
        q, st = run_gpu(x, e, m, den, 1.0)
        assert_same(q, st, q_ref, st_ref)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 127, 128, 129, 1023, 1024, 1025, 4099, 262147])
def test_sizes_and_ragged_tails(n):
    x = workloads.lognormal_tensor(workloads.rng_for(50, n), (n,), -20.0, 9.0, p_zero=0.02)
    q_ref, st_ref = oracle.quantize_stats(x, 6, 9, 1, 2.0 ** 3)
    q, st = run_gpu(x, 6, 9, 1, 2.0 ** 3)
    assert_same(q, st, q_ref, st_ref)


@pytest.mark.parametrize("in_off,out_off", [(0, 0), (1, 1), (3, 3), (2, 2), (1, 0), (0, 3), (2, 1)])
def test_unaligned_pointers(in_off, out_off):
    n = 10007
    x = workloads.lognormal_tensor(workloads.rng_for(51), (n,), -14.0, 6.0, p_zero=0.01)
    q_ref, st_ref = oracle.quantize_stats(x, 5, 10, 1, 1.0)
    q, st = run_gpu(x, 5, 10, 1, 1.0, in_off=in_off, out_off=out_off)
    assert_same(q, st, q_ref, st_ref)


def test_in_place_stats_only_no_stats_and_accumulate():
    n = 300001
    x = workloads.lognormal_tensor(workloads.rng_for(52), (n,), -30.0, 6.0, p_zero=0.01)
    q_ref, st_ref = oracle.quantize_stats(x, 6, 9, 0, 1.0)
    q, st = run_gpu(x, 6, 9, 0, 1.0, in_place=True)
    assert_same(q, st, q_ref, st_ref)
    q, st = run_gpu(x, 6, 9, 0, 1.0, want_out=False)
    assert q is None
    assert_same(None, st, None, st_ref)
    q, st = run_gpu(x, 6, 9, 0, 1.0, want_stats=False)
    assert_same(q, None, q_ref, None)
    # accumulate = 1 adds to the record, accumulate = 0 clears it first
    stats_t = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device="cuda:0")
    run_gpu(x, 6, 9, 0, 1.0, stats_t=stats_t)
    _, st2 = run_gpu(x, 6, 9, 0, 1.0, stats_t=stats_t, accumulate=1)
    assert np.array_equal(st2, 2 * st_ref)
    _, st3 = run_gpu(x, 6, 9, 0, 1.0, stats_t=stats_t, accumulate=0)
    assert np.array_equal(st3, st_ref)


def test_concentrated_values_do_not_break_counting():
    """Weights ~ N(0, 0.02) fall into three or four binades: the worst case for a histogram."""
    w = workloads.normal_tensor(workloads.rng_for(53), (1 << 20,), 0.02)
    for e, m in FORMATS:
        q_ref, st_ref = oracle.quantize_stats(w, e, m, 1, 1.0)
        q, st = run_gpu(w, e, m, 1, 1.0)
        assert_same(q, st, q_ref, st_ref)
    ones = np.full(1 << 18, 1.0, dtype=np.float32)
    q_ref, st_ref = oracle.quantize_stats(ones, 6, 9, 1, 1.0)
    q, st = run_gpu(ones, 6, 9, 1, 1.0)
    assert_same(q, st, q_ref, st_ref)


def test_config1_tensors():
    cfg = workloads.config1()
    e, m = cfg["fmt"]
    for name in ("A", "B"):
        q_ref, st_ref = oracle.quantize_stats(cfg[name], e, m, cfg["denormals"], cfg["loss_scale"])
        q, st = run_gpu(cfg[name], e, m, cfg["denormals"], cfg["loss_scale"])
        assert_same(q, st, q_ref, st_ref)
        assert int(st[:64].sum()) == cfg[name].size  # the 64-bin histogram covers every element


def test_config2_full_size_all_18_runs():
    """The benchmark's own workload and launch configuration: 64 Mi elements, all 18 runs.
    Counts are compared in full; rounded values in full as well (the oracle needs ~1 s per run)."""
    x = workloads.config2_tensor()
    d_in = torch.from_numpy(x).to("cuda:0")
    d_out = torch.empty_like(d_in)
    d_st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device="cuda:0")
    for name, e, m, den, scale in workloads.config2_runs():
        qf.qfmt_quantize_stats(d_in, d_out, x.size, qf.make_format(e, m, den, scale), d_st, 0)
        torch.cuda.synchronize()
        q_ref, st_ref = oracle.quantize_stats(x, e, m, den, scale)
        assert np.array_equal(d_st.cpu().numpy().view(np.uint64), st_ref), name
        assert np.array_equal(d_out.cpu().numpy().view(np.uint32), q_ref.view(np.uint32)), name


def test_host_buffer_entry_point():
    n = 100003
    x = workloads.lognormal_tensor(workloads.rng_for(54), (n,), -18.0, 8.0, p_zero=0.005)
    q_ref, st_ref = oracle.quantize_stats(x, 6, 9, 1, 2.0 ** 8)
    h_in = torch.from_numpy(x).pin_memory()
    h_out = torch.empty(n, dtype=torch.float32).pin_memory()
    h_st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64).pin_memory()
    wb = qf.qfmt_quantize_stats_host_work_bytes(n)
    d_work = torch.empty(wb, dtype=torch.uint8, device="cuda:0")
    qf.qfmt_quantize_stats_host(h_in, h_out, n, qf.make_format(6, 9, 1, 2.0 ** 8), h_st, d_work, wb)
    assert np.array_equal(h_out.numpy().view(np.uint32), q_ref.view(np.uint32))
    assert np.array_equal(h_st.numpy().view(np.uint64), st_ref)


def test_host_buffer_entry_point_pipelined_pieces():
    """More than 2 Mi elements: the tensor crosses the link in pieces on the library's own streams
    while earlier pieces are rounded and returned; values and the accumulated statistics are those
    of one pass.  Also without an output tensor (statistics only) and twice in a row."""
    n = (20 << 20) + 3
    x = workloads.lognormal_tensor(workloads.rng_for(55), (n,), -18.0, 8.0, p_zero=0.005)
    q_ref, st_ref = oracle.quantize_stats(x, 5, 10, 0, 2.0 ** 8)
    h_in = torch.from_numpy(x).pin_memory()
    h_out = torch.empty(n, dtype=torch.float32).pin_memory()
    h_st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64).pin_memory()
    wb = qf.qfmt_quantize_stats_host_work_bytes(n)
    d_work = torch.empty(wb, dtype=torch.uint8, device="cuda:0")
    fmt = qf.make_format(5, 10, 0, 2.0 ** 8)
    for _ in range(2):
        h_out.zero_()
        qf.qfmt_quantize_stats_host(h_in, h_out, n, fmt, h_st, d_work, wb)
        assert np.array_equal(h_out.numpy().view(np.uint32), q_ref.view(np.uint32))
        assert np.array_equal(h_st.numpy().view(np.uint64), st_ref)
    h_st.zero_()
    qf.qfmt_quantize_stats_host(h_in, None, n, fmt, h_st, d_work, wb)
    assert np.array_equal(h_st.numpy().view(np.uint64), st_ref)
    # on a side stream, after work that is already queued there
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        h_out.zero_()
        qf.qfmt_quantize_stats_host(h_in, h_out, n, fmt, None, d_work, wb, stream=side)
    assert np.array_equal(h_out.numpy().view(np.uint32), q_ref.view(np.uint32))


def test_errors_leave_outputs_untouched():
    d = torch.ones(16, dtype=torch.float32, device="cuda:0")
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_quantize_stats(d, d, 16, qf.make_format(9, 3))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_quantize_stats(d.data_ptr() + 2, d, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    torch.cuda.synchronize()
    assert torch.all(d == 1.0)


@pytest.mark.parametrize("batch,rows,cols", [(1, 1, 1), (2, 3, 5), (3, 32, 32), (2, 33, 65), (4, 64, 196),
                                             (5, 256, 9), (1, 100, 1), (7, 1, 50),
                                             # rows and cols multiples of 4: the 128-bit kernel, ragged tiles
                                             (1, 4, 4), (2, 68, 36), (3, 128, 100), (5, 256, 12), (2, 60, 200)])
@pytest.mark.parametrize("e,m,den,scale", [(6, 9, 1, 1.0), (5, 10, 0, 2.0 ** 10), (8, 7, 1, 1.0)])
def test_transposing_variant(batch, rows, cols, e, m, den, scale):
    """[batch][rows][cols] -> [batch][cols][rows]: same bits as the oracle's values, permuted; same counts."""
    x = workloads.lognormal_tensor(workloads.rng_for(70, batch * rows + cols), (batch, rows, cols), -15.0, 7.0, 0.02)
    q_ref, st_ref = oracle.quantize_stats(x, e, m, den, scale)
    d_in = torch.from_numpy(x).to("cuda:0")
    d_out = torch.full((batch * rows * cols + 8,), 7.0, dtype=torch.float32, device="cuda:0")
    st = torch.full((qf.STATS_WORDS,), 5, dtype=torch.int64, device="cuda:0")
    qf.qfmt_quantize_stats_transpose(d_in, d_out, batch, rows, cols, qf.make_format(e, m, den, scale), st, 0)
    torch.cuda.synchronize()
    got = d_out.cpu().numpy()
    assert np.all(got[batch * rows * cols:] == 7.0)
    want = np.ascontiguousarray(q_ref.transpose(0, 2, 1))
    assert np.array_equal(got[:batch * rows * cols].view(np.uint32), want.reshape(-1).view(np.uint32))
    assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref)
