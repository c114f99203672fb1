"""GPU parity of qfmt_conv_fmac8 (FMAC-8 accumulation in convolution layers, Section IV-A) against the
CPU oracle.  Algorithm 1 and the stated order of the reduction fix every rounding, so outputs and
statistics must match bit for bit, on the general kernel and on the native 16-bit one."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def quantized(x, e, m, den):
    return oracle.quantize_stats(x, e, m, den, 1.0, want_stats=False)[0]


def channels_last(t):
    """[n][c][h][w] -> [n][h][w][c] (filters [co][ci][r][s] -> [co][r][s][ci])."""
    return np.ascontiguousarray(t.transpose(0, 2, 3, 1))


def run_gpu(op, geom, P_cl, Q_cl, out_shape_cl, e, m, den, path, want_stats=True):
    n, ci, h, w, co, r, s, ph, pw = geom
    g = qf.qfmt_conv_t(n, ci, h, w, co, r, s, ph, pw)
    dP, dQ = torch.from_numpy(P_cl).to(DEV), torch.from_numpy(Q_cl).to(DEV)
    numel = int(np.prod(out_shape_cl))
    buf = torch.full((numel + 8,), 7.0, dtype=torch.float32, device=DEV)
    st = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV) if want_stats else None
    qf.qfmt_conv_fmac8(op, g, dP, dQ, buf[4:4 + numel], qf.make_format(e, m, den), st, 0, path)
    torch.cuda.synchronize()
    assert torch.all(buf[:4] == 7.0) and torch.all(buf[4 + numel:] == 7.0)
    out = buf[4:4 + numel].view(*out_shape_cl).permute(0, 3, 1, 2).contiguous().cpu().numpy()
    return out, (st.cpu().numpy().view(np.uint64) if want_stats else None)


def check_all_three(geom, X, Wt, dY, e, m, den, paths):
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    Xc, Wc, Gc = channels_last(X), channels_last(Wt), channels_last(dY)
    cases = ((qf.QFMT_CONV_FWD, oracle.CONV_FWD, X, Wt, Xc, Wc, (n, oh, ow, co)),
             (qf.QFMT_CONV_DGRAD, oracle.CONV_DGRAD, dY, Wt, Gc, Wc, (n, h, w, ci)),
             (qf.QFMT_CONV_WGRAD, oracle.CONV_WGRAD, dY, X, Gc, Xc, (co, r, s, ci)))
    for op, which, P, Q, Pc, Qc, shape_cl in cases:
        ref, master = oracle.conv_fmac8(which, P, Q, geom, e, m, den, want_master=True)
        _, st_ref = oracle.quantize_stats(master, e, m, den, 1.0)
        for path in paths:
            got, st = run_gpu(op, geom, Pc, Qc, shape_cl, e, m, den, path)
            g = got.reshape(-1).view(np.uint32)
            bad = np.nonzero(g != ref.view(np.uint32))[0]
            assert bad.size == 0, (op, path, bad[:5], got.reshape(-1)[bad[:5]], ref[bad[:5]])
            assert np.array_equal(st, st_ref), (op, path)


def paths_for(e, m):
    return (0, 1, 2) if (e, m) in ((5, 10), (8, 7)) else (0, 1)


GEOMS = [
    (2, 12, 5, 6, 7, 3, 3, 1, 1),      # twelve and seven channels: runs of eight straddle taps and padding
    (1, 8, 9, 9, 16, 3, 3, 0, 0),      # no padding, output smaller than input
    (3, 5, 4, 7, 9, 2, 3, 1, 0),       # asymmetric filter and padding
    (2, 40, 6, 5, 70, 1, 1, 0, 0),     # 1 x 1: a plain FMAC-8 matrix product, two column tiles of the general kernel
    (2, 16, 11, 10, 24, 5, 5, 2, 2),   # 5 x 5 filter: 220 output pixels, four row tiles
]


@pytest.mark.parametrize("geom", GEOMS)
@pytest.mark.parametrize("e,m", [(6, 9), (5, 10), (8, 7)])
@pytest.mark.parametrize("den", [1, 0])
def test_random_tensors_match_the_oracle_bit_for_bit(geom, e, m, den):
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    rng = workloads.rng_for(700 + e, sum(geom))
    X = quantized(workloads.lognormal_tensor(rng, (n, ci, h, w), -2.0, 2.0, p_zero=0.3), e, m, den)      # post-ReLU like
    Wt = quantized(workloads.lognormal_tensor(rng, (co, ci, r, s), -4.0, 1.5, p_zero=0.0), e, m, den)
    dY = quantized(workloads.lognormal_tensor(rng, (n, co, oh, ow), -11.0, 3.0, p_zero=0.02), e, m, den)  # small gradients
    check_all_three(geom, X, Wt, dY, e, m, den, paths_for(e, m))


def test_small_integers_give_the_rounded_exact_convolution():
    """Nothing rounds before the end: the result is the exact convolution (all sums below 2^10)."""
    geom = (2, 8, 6, 6, 8, 3, 3, 1, 1)
    n, ci, h, w, co, r, s, ph, pw = geom
    rng = np.random.default_rng(5)
    X = rng.integers(-2, 3, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(co, ci, r, s)).astype(np.float32)
    dY = rng.integers(-2, 3, size=(n, co, h, w)).astype(np.float32)
    Xc, Wc, Gc = channels_last(X), channels_last(Wt), channels_last(dY)
    for op, which, P, Q, Pc, Qc, shape in ((qf.QFMT_CONV_FWD, oracle.CONV_FWD, X, Wt, Xc, Wc, (n, h, w, co)),
                                           (qf.QFMT_CONV_DGRAD, oracle.CONV_DGRAD, dY, Wt, Gc, Wc, (n, h, w, ci)),
                                           (qf.QFMT_CONV_WGRAD, oracle.CONV_WGRAD, dY, X, Gc, Xc, (co, r, s, ci))):
        exact, _ = oracle.conv(which, P, Q, geom)
        got, _ = run_gpu(op, geom, Pc, Qc, shape, 6, 9, 1, 0)
        assert np.array_equal(got.reshape(-1).astype(np.float64), exact)


def test_config4_shaped_layer_sampled():
    """The 3 x 3 layer of the ResNet-50-shaped workload at a reduced batch (4 images of 256 channels at
    14 x 14): forward and data gradient on sampled outputs, binary16 on the native kernel."""
    geom = (4, 256, 14, 14, 256, 3, 3, 1, 1)
    n, ci, h, w, co, r, s, ph, pw = geom
    e, m, den = 5, 10, 1
    rng = workloads.rng_for(733)
    X = quantized(workloads.lognormal_tensor(rng, (n, ci, h, w), -2.0, 2.0, p_zero=0.5), e, m, den)
    Wt = quantized((rng.standard_normal((co, ci, r, s)) * np.sqrt(2.0 / (ci * r * s))).astype(np.float32), e, m, den)
    dY = quantized(workloads.lognormal_tensor(rng, (n, co, h, w), -12.0, 3.0, p_zero=0.0), e, m, den)
    Xc, Wc, Gc = channels_last(X), channels_last(Wt), channels_last(dY)
    for op, which, P, Q, Pc, Qc, shape in ((qf.QFMT_CONV_FWD, oracle.CONV_FWD, X, Wt, Xc, Wc, (n, h, w, co)),
                                           (qf.QFMT_CONV_DGRAD, oracle.CONV_DGRAD, dY, Wt, Gc, Wc, (n, h, w, ci))):
        got, _ = run_gpu(op, geom, Pc, Qc, shape, e, m, den, 2, want_stats=False)
        idx = np.concatenate([rng.integers(0, got.size, size=3000), [0, got.size - 1]])
        ref = oracle.conv_fmac8(which, P, Q, geom, e, m, den, idx=idx)
        assert np.array_equal(got.reshape(-1)[idx].view(np.uint32), ref.view(np.uint32))


def test_argument_errors():
    g = qf.qfmt_conv_t(1, 8, 4, 4, 8, 3, 3, 1, 1)
    x = torch.zeros(1 * 4 * 4 * 8, dtype=torch.float32, device=DEV)
    wt = torch.zeros(8 * 9 * 8, dtype=torch.float32, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_conv_fmac8(qf.QFMT_CONV_FWD, g, x, wt, x, qf.make_format(5, 11))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT          # operands of more than 11 significant bits
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_conv_fmac8(qf.QFMT_CONV_FWD, g, x, wt, x, qf.make_format(6, 9), None, 0, 2)
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT          # the native kernel is for 1/5/10 and 1/8/7 only
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_conv_fmac8(7, g, x, wt, x, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_conv_fmac8(qf.QFMT_CONV_FWD, qf.qfmt_conv_t(1, 8, 2, 2, 8, 5, 5, 0, 0), x, wt, x, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG             # filter larger than the padded image
