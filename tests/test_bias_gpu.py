"""GPU parity of qfmt_bias_quantize_stats (Y = R(R(acc) + R(B)), Section IV-A) against the CPU
oracle: rounded outputs and every count must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def run_gpu(acc, bias, e, m, den, scale, *, ld_acc=None, ld_out=None, in_place=False, off=0, want_stats=True,
            accumulate=0, stats_t=None):
    rows, cols = acc.shape
    ld_acc = ld_acc or cols
    ld_out = ld_acc if in_place else (ld_out or cols)
    buf_a = torch.full((rows * ld_acc + 64,), 3.0, dtype=torch.float32, device=DEV)
    d_acc = buf_a[off:off + rows * ld_acc]
    d_acc.view(rows, ld_acc)[:, :cols].copy_(torch.from_numpy(acc))
    buf_b = torch.zeros(cols + 64, dtype=torch.float32, device=DEV)
    d_bias = buf_b[off:off + cols]
    d_bias.copy_(torch.from_numpy(bias))
    if in_place:
        buf_o, d_out = buf_a, d_acc
    else:
        buf_o = torch.full((rows * ld_out + 64,), 7.0, dtype=torch.float32, device=DEV)
        d_out = buf_o[off:off + rows * ld_out]
    if want_stats and stats_t is None:
        stats_t = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV)  # dirty on purpose
    qf.qfmt_bias_quantize_stats(d_acc, ld_acc, d_bias, d_out, ld_out, rows, cols, qf.make_format(e, m, den, scale),
                                stats_t if want_stats else None, accumulate)
    torch.cuda.synchronize()
    full = d_out.view(rows, ld_out).cpu().numpy() if rows else np.zeros((0, ld_out), np.float32)
    fill = 3.0 if in_place else 7.0
    assert np.all(full[:, cols:] == fill)                       # padding columns untouched
    assert torch.all(buf_o[:off] == fill) and torch.all(buf_o[off + rows * ld_out:] == fill)
    st = stats_t.cpu().numpy().view(np.uint64) if want_stats else None
    return np.ascontiguousarray(full[:, :cols]), st


def check(acc, bias, e, m, den, scale, **kw):
    y_ref, st_ref = oracle.bias_quantize_stats(acc, bias, e, m, den, scale)
    y, st = run_gpu(acc, bias, e, m, den, scale, **kw)
    assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))
    if st is not None and not kw.get("accumulate"):
        assert np.array_equal(st, st_ref), (st[np.nonzero(st != st_ref)], st_ref[np.nonzero(st != st_ref)])
    return st, st_ref


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7), (4, 3), (7, 8)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("scale", [1.0, 2.0 ** 8, 3.0e-5])
def test_arbitrary_bit_patterns(e, m, den, scale):
    """Random fp32 words (NaN, inf, denormals, both zeros included) in both terms, several tiles
    and a ragged last one."""
    rng = np.random.default_rng(300 + e * 31 + m)
    rows, cols = 531, 132
    acc = rng.integers(0, 1 << 32, size=rows * cols, dtype=np.uint64).astype(np.uint32)
    edge = workloads.edge_bit_patterns()
    acc[:edge.size] = edge
    bias = rng.integers(0, 1 << 32, size=cols, dtype=np.uint64).astype(np.uint32)
    bias[:40] = edge[:40]
    check(acc.view(np.float32).reshape(rows, cols), bias.view(np.float32), e, m, den, scale)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7)])
def test_sums_near_ties_and_cancellation(e, m):
    """Terms of comparable and of very different size: powers of two minus values near a quarter
    and half of the last place, exact opposites, carries into the next binade, sums that overflow,
    denormal sums."""
    rng = np.random.default_rng(310 + e)
    top = ((1 << e) - 1) << m
    cols = 256
    bias_codes = rng.integers(0, top, size=cols, dtype=np.uint64)
    bias_codes[:64] = (rng.integers(m + 3, (1 << e) - 1, size=64, dtype=np.uint64) << np.uint64(m))  # powers of two
    bias_codes[64:72] = top - 1                                                              # largest normal
    bias_codes[72:80] = rng.integers(1, 1 << m, size=8, dtype=np.uint64)                        # denormals
    bias = np.array([oracle.decode_code(int(c), e, m) for c in bias_codes], dtype=np.uint32)
    rows = 96
    acc = np.empty((rows, cols), dtype=np.uint32)
    for j in range(cols):
        E = int(bias_codes[j]) >> m
        lo = max(1, E - m - 3)
        near = rng.integers(lo << m, min(top, (E + 2) << m), size=rows, dtype=np.uint64)
        near |= rng.integers(0, 2, size=rows, dtype=np.uint64) << np.uint64(e + m)
        acc[:, j] = [oracle.decode_code(int(c), e, m) for c in near]
    acc[0, :] = bias ^ np.uint32(0x80000000)                    # exact cancellation
    acc[1, :] = bias                                            # doubling (overflow for the largest)
    # also feed values that still need the first rounding: add low mantissa bits
    acc[2:40, :] |= rng.integers(0, 1 << 13, size=(38, cols), dtype=np.uint64).astype(np.uint32)
    for den in (1, 0):
        check(acc.view(np.float32), bias.view(np.float32), e, m, den, 1.0)


@pytest.mark.parametrize("rows,cols", [(0, 8), (5, 0), (1, 1), (1, 4), (3, 5), (7, 12), (129, 36), (1000, 1024),
                                       (2, 20000), (64, 3072)])
def test_shapes(rows, cols):
    rng = workloads.rng_for(320, rows * 7 + cols)
    acc = workloads.lognormal_tensor(rng, (rows, cols), -6.0, 5.0, p_zero=0.02)
    bias = workloads.lognormal_tensor(rng, (cols,), -7.0, 4.0, p_zero=0.05)
    check(acc, bias, 6, 9, 1, 1.0)


@pytest.mark.parametrize("off,ld_acc,ld_out", [(0, 40, 44), (0, 37, 36), (1, 36, 36), (2, 48, 36), (0, 36, 39)])
def test_leading_dimensions_and_alignment(off, ld_acc, ld_out):
    rng = workloads.rng_for(321, off + ld_acc)
    acc = workloads.lognormal_tensor(rng, (211, 36), -10.0, 6.0, p_zero=0.02)
    bias = workloads.lognormal_tensor(rng, (36,), -10.0, 6.0)
    check(acc, bias, 5, 10, 0, 4.0, off=off, ld_acc=ld_acc, ld_out=ld_out)


def test_in_place_no_stats_and_accumulate():
    rng = workloads.rng_for(322)
    acc = workloads.lognormal_tensor(rng, (777, 64), -28.0, 5.0, p_zero=0.01)
    bias = workloads.lognormal_tensor(rng, (64,), -30.0, 4.0)
    check(acc, bias, 6, 9, 1, 1.0, in_place=True, ld_acc=72)
    check(acc, bias, 6, 9, 0, 1.0, want_stats=False)
    stats_t = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    _, st_ref = check(acc, bias, 6, 9, 0, 1.0, stats_t=stats_t)
    st2, _ = check(acc, bias, 6, 9, 0, 1.0, stats_t=stats_t, accumulate=1)
    assert np.array_equal(st2, 2 * st_ref)


def test_linear_layer_forward_config3_and_config5_shapes():
    """The whole forward formula on the library's own product: Y = R(R(R(X) R(W)) + R(B)) for the
    BERT-base layer (K = 768) and one BERT-large layer (K = 1024); the epilogue is compared bit
    for bit on the GPU's own accumulator values."""
    for cfg, bias_seed in ((workloads.config3(), 330), (workloads.config5_layer(1, 0), 331)):
        X, W = cfg["X"], cfg["W"]
        e, m = 6, 9
        fmt = qf.make_format(e, m, 1, 1.0)
        dX, dW = torch.from_numpy(X).to(DEV), torch.from_numpy(W).to(DEV)
        qf.qfmt_quantize_stats(dX, dX, dX.numel(), fmt)
        qf.qfmt_quantize_stats(dW, dW, dW.numel(), fmt)
        M, N = X.shape[0], W.shape[1]
        acc = torch.empty(M, N, dtype=torch.float32, device=DEV)
        a, b = qf.make_matrix(dX), qf.make_matrix(dW)
        ws = torch.zeros(max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=DEV)
        qf.qfmt_gemm(a, b, acc, N, fmt, ws, ws.numel())
        assert qf.qfmt_device_status(ws) == qf.QFMT_OK
        bias = workloads.normal_tensor(workloads.rng_for(bias_seed), (N,), 0.02)
        d_bias = torch.from_numpy(bias).to(DEV)
        st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=DEV)
        y = torch.empty_like(acc)
        qf.qfmt_bias_quantize_stats(acc, N, d_bias, y, N, M, N, fmt, st)
        torch.cuda.synchronize()
        y_ref, st_ref = oracle.bias_quantize_stats(acc.cpu().numpy(), bias, e, m, 1, 1.0)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))
        assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref)


def run_gpu_pack(acc, bias, e, m, den, scale, *, ld_acc=None, ld_codes=None, off=0, want_stats=True):
    rows, cols = acc.shape
    ld_acc, ld_codes = ld_acc or cols, ld_codes or cols
    buf_a = torch.full((rows * ld_acc + 64,), 3.0, dtype=torch.float32, device=DEV)
    d_acc = buf_a[off:off + rows * ld_acc]
    d_acc.view(rows, ld_acc)[:, :cols].copy_(torch.from_numpy(acc))
    buf_b = torch.zeros(cols + 64, dtype=torch.float32, device=DEV)
    d_bias = buf_b[off:off + cols]
    d_bias.copy_(torch.from_numpy(bias))
    buf_o = torch.full((rows * ld_codes + 64,), 0x1234, dtype=torch.int16, device=DEV)
    d_codes = buf_o[off:off + rows * ld_codes]
    stats_t = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV) if want_stats else None
    qf.qfmt_bias_quantize_stats_pack16(d_acc, ld_acc, d_bias, d_codes, ld_codes, rows, cols, qf.make_format(e, m, den, scale),
                                       stats_t)
    torch.cuda.synchronize()
    full = d_codes.view(rows, ld_codes).cpu().numpy().view(np.uint16)
    assert np.all(full[:, cols:] == 0x1234)                     # padding untouched
    assert torch.all(buf_o[:off] == 0x1234) and torch.all(buf_o[off + rows * ld_codes:] == 0x1234)
    return np.ascontiguousarray(full[:, :cols]), (stats_t.cpu().numpy().view(np.uint64) if want_stats else None)


def check_pack(acc, bias, e, m, den, scale, **kw):
    """Codes must be the encoding of the containers the oracle's layer formula gives (packing a
    tensor that is already rounded loses nothing); the statistics are those of the container pass."""
    y_ref, st_ref = oracle.bias_quantize_stats(acc, bias, e, m, den, scale)
    codes_ref, _ = oracle.quantize_stats_pack16(y_ref, e, m, 1, 1.0)
    codes, st = run_gpu_pack(acc, bias, e, m, den, scale, **kw)
    assert np.array_equal(codes, codes_ref.reshape(codes.shape))
    if st is not None:
        assert np.array_equal(st, st_ref)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7), (4, 3), (7, 8)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("scale", [1.0, 2.0 ** 8])
def test_pack16_arbitrary_bit_patterns(e, m, den, scale):
    rng = np.random.default_rng(340 + e * 31 + m)
    rows, cols = 531, 132
    acc = rng.integers(0, 1 << 32, size=rows * cols, dtype=np.uint64).astype(np.uint32)
    edge = workloads.edge_bit_patterns()
    acc[:edge.size] = edge
    bias = rng.integers(0, 1 << 32, size=cols, dtype=np.uint64).astype(np.uint32)
    bias[:40] = edge[:40]
    check_pack(acc.view(np.float32).reshape(rows, cols), bias.view(np.float32), e, m, den, scale)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7)])
def test_pack16_all_codes_come_back(e, m):
    """acc runs over every finite container of the format with a zero bias: the codes written must
    be the codes the containers came from."""
    all_codes = np.arange(1 << 16, dtype=np.uint16)
    vals = oracle.unpack16(all_codes, e, m)
    keep = np.isfinite(vals)
    acc = np.zeros(1 << 16, np.float32)
    acc[keep] = vals[keep]
    codes, _ = run_gpu_pack(acc.reshape(256, 256), np.zeros(256, np.float32), e, m, 1, 1.0)
    got = codes.reshape(-1)
    neg_zero = all_codes == 0x8000            # -0 + (+0) = +0 in round-to-nearest
    assert np.array_equal(got[keep & ~neg_zero], all_codes[keep & ~neg_zero])
    assert got[0x8000] == 0


@pytest.mark.parametrize("rows,cols,off,ld_acc,ld_codes", [(0, 8, 0, 8, 8), (5, 0, 0, 4, 4), (1, 1, 0, 1, 1), (3, 5, 0, 5, 7),
                                                          (129, 36, 0, 36, 36), (129, 36, 0, 40, 44), (129, 36, 1, 36, 36),
                                                          (129, 36, 2, 36, 38), (1000, 1024, 0, 1024, 1024),
                                                          (2, 20000, 0, 20000, 20000), (64, 3072, 4, 3072, 3072)])
def test_pack16_shapes_and_alignment(rows, cols, off, ld_acc, ld_codes):
    rng = workloads.rng_for(341, rows * 7 + cols + off)
    acc = workloads.lognormal_tensor(rng, (rows, cols), -6.0, 5.0, p_zero=0.02)
    bias = workloads.lognormal_tensor(rng, (cols,), -7.0, 4.0, p_zero=0.05)
    check_pack(acc, bias, 6, 9, 1, 1.0, off=off, ld_acc=ld_acc, ld_codes=ld_codes)
    check_pack(acc, bias, 8, 7, 0, 1.0, off=off, ld_acc=ld_acc, ld_codes=ld_codes, want_stats=False)


def test_pack16_errors():
    d = torch.ones(64, dtype=torch.float32, device=DEV)
    c = torch.zeros(64, dtype=torch.int16, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats_pack16(d, 8, d, c, 8, 8, 8, qf.make_format(8, 8))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT          # 1 + 8 + 8 bits do not fit
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats_pack16(d, 8, d, c, 4, 8, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats_pack16(d, 8, d, None, 8, 8, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    torch.cuda.synchronize()
    assert torch.all(c == 0)


def test_errors():
    d = torch.ones(64, dtype=torch.float32, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats(d, 8, d, d, 8, 8, 8, qf.make_format(8, 11))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT          # m > 10: the one-add sum is not exact enough
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats(d, 4, d, d, 8, 8, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG             # leading dimension below cols
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_bias_quantize_stats(d, 8, None, d, 8, 8, 8, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    torch.cuda.synchronize()
    assert torch.all(d == 1.0)
