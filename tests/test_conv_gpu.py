"""GPU parity of qfmt_conv (and of the transposing rounding pass that feeds it) against the
oracle's direct NCHW definitions of the forward, data-gradient and filter-gradient products."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 2.0 ** -20


def to_channels_last(x_nchw_np, fmt):
    """NCHW (or KCRS) numpy -> rounded channels-last device tensor via the library's own pass."""
    b, c, h, w = x_nchw_np.shape
    d_in = torch.from_numpy(np.ascontiguousarray(x_nchw_np)).to(DEV)
    d_out = torch.empty(b * h * w * c, dtype=torch.float32, device=DEV)
    qf.qfmt_quantize_stats_transpose(d_in, d_out, b, c, h * w, fmt)
    return d_out.view(b, h, w, c)


def run_conv(op, geom, d_p, d_q, out_shape, fmt):
    g = qf.qfmt_conv_t(*geom)
    wb = qf.qfmt_conv_workspace_bytes(op, g)
    assert wb > 0
    ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
    d_out = torch.full(out_shape, float("nan"), dtype=torch.float32, device=DEV)
    qf.qfmt_conv(op, g, d_p, d_q, d_out, fmt, ws, wb)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    return d_out


def all_three(geom, X, Wt, dY, e=6, m=9, grad_scale=1.0, exact=False, sample=None, seed=0):
    """Runs fwd/dgrad/wgrad on the GPU and checks them; returns worst error / tolerance per product."""
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    fmt = qf.make_format(e, m, 1)
    dX = to_channels_last(X, fmt)
    dW = to_channels_last(Wt, fmt)
    dG = to_channels_last(dY, qf.make_format(e, m, 1, grad_scale))
    qX, _ = oracle.quantize_stats(X, e, m, 1, 1.0, want_stats=False)
    qW, _ = oracle.quantize_stats(Wt, e, m, 1, 1.0, want_stats=False)
    qG, _ = oracle.quantize_stats(dY, e, m, 1, grad_scale, want_stats=False)
    assert np.array_equal(dX.cpu().numpy().view(np.uint32), qX.transpose(0, 2, 3, 1).view(np.uint32))
    assert np.array_equal(dW.cpu().numpy().view(np.uint32), qW.transpose(0, 2, 3, 1).view(np.uint32))
    Y = run_conv(qf.QFMT_CONV_FWD, geom, dX, dW, (n, oh, ow, co), fmt).permute(0, 3, 1, 2).contiguous().cpu().numpy()
    gX = run_conv(qf.QFMT_CONV_DGRAD, geom, dG, dW, (n, h, w, ci), fmt).permute(0, 3, 1, 2).contiguous().cpu().numpy()
    gW = run_conv(qf.QFMT_CONV_WGRAD, geom, dG, dX, (co, r, s, ci), fmt).permute(0, 3, 1, 2).contiguous().cpu().numpy()
    worst = {}
    rng = np.random.default_rng(seed)
    for name, which, P, Q, got in (("fwd", oracle.CONV_FWD, qX, qW, Y), ("dgrad", oracle.CONV_DGRAD, qG, qW, gX),
                                   ("wgrad", oracle.CONV_WGRAD, qG, qX, gW)):
        flat = got.reshape(-1).astype(np.float64)
        if sample is None or sample >= flat.size:
            idx = None
            ref, T = oracle.conv(which, P, Q, geom)
        else:
            idx = np.concatenate([rng.integers(0, flat.size, size=sample), [0, flat.size - 1]])
            ref, T = oracle.conv(which, P, Q, geom, idx)
            flat = flat[idx]
        if exact:
            assert np.array_equal(flat, ref), name
        err = np.abs(flat - ref)
        assert np.all(err <= TOL * T), f"{name}: worst {float(np.max(err / np.maximum(T, 1e-300)) / TOL):.3f} x tolerance"
        worst[name] = float(np.max(err / np.maximum(T, 1e-300)) / TOL)
    return worst


SMALL = [
    (2, 32, 5, 6, 32, 3, 3, 1, 1),
    (3, 64, 14, 14, 96, 3, 3, 1, 1),      # 42 image rows: four complete 9-row tiles and a partial one
    (1, 32, 7, 7, 288, 1, 1, 0, 0),       # more than one 256-column tile
    (2, 32, 8, 10, 32, 3, 2, 1, 0),       # asymmetric filter and padding, output smaller than input
    (2, 32, 4, 32, 64, 3, 3, 1, 1),       # 32-pixel rows: one image row per filter-gradient stage
    (9, 32, 14, 14, 32, 3, 3, 1, 1),      # 126 image rows: split-K in the filter gradient
    (2, 96, 6, 5, 32, 5, 5, 2, 2),        # 25 taps
    (1, 32, 3, 3, 32, 3, 3, 0, 0),        # single output pixel
    (3, 256, 8, 7, 64, 3, 3, 1, 1),       # filter gradient with padded stages: 7-pixel rows take 8 K rows
    (2, 256, 10, 9, 32, 3, 3, 0, 0),      # the same without zero padding: the pad rows of B hold real pixels
    (2, 512, 4, 14, 32, 1, 1, 0, 0),      # padded stages, two 256-column tiles per tap
    (64, 32, 3, 3, 64, 3, 3, 1, 1),       # 42 three-pixel rows per M-tile: fourteen images (copies) per tile and stage
    (2, 256, 4, 7, 256, 3, 3, 1, 1),      # filter gradient on CTA pairs: padded stages and 256 output channels
    (1, 256, 8, 8, 320, 3, 3, 1, 1),      # the same with a second, incomplete row of pair tiles (320 output channels)
    (1, 64, 5, 40, 32, 3, 3, 1, 1),       # 40-pixel rows: two filter-gradient stages per row, the second 8 pixels and zeros
    (2, 64, 6, 56, 64, 3, 3, 1, 1),       # 56-pixel rows (the first stage of a ResNet-50-shaped network), split K
    (1, 32, 3, 70, 32, 1, 3, 0, 0),       # 68-pixel output rows without padding: three stages per row, the last 4 pixels
]


@pytest.fixture(params=[0, 1, 2, 3], ids=["automatic", "single_cta", "pairs_whole_tiles", "pairs_balanced"])
def conv_kernel(request):
    """Forward and data gradient on both kernels and both schedules of the pair kernel."""
    qf.qfmt_conv_tile_policy(request.param)
    yield request.param
    qf.qfmt_conv_tile_policy(0)


@pytest.mark.parametrize("geom", SMALL)
def test_small_integer_convolutions_are_exact(geom, conv_kernel):
    """Entries in -3..3: all sums are small integers, exact in any accumulation order, so a wrong
    tap offset, padding, channel block, transpose or split shows up as a wrong integer."""
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    rng = np.random.default_rng(sum(geom))
    X = rng.integers(-3, 4, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-3, 4, size=(co, ci, r, s)).astype(np.float32)
    dY = rng.integers(-3, 4, size=(n, co, oh, ow)).astype(np.float32)
    all_three(geom, X, Wt, dY, exact=True)


def test_balanced_schedule_is_exact(conv_kernel):
    """163 four-row tiles (the last one three rows) of 27 chunks each: forward and data gradient deal
    the K chunks out in equal ranges (among 148 CTAs on the single-CTA kernel, among 74 pairs of two
    tiles on the pair kernel), so most of them finish one tile and begin another, and the pieces that
    begin inside a tile are added to what another CTA or pair stored.  Small integers keep every
    order of summation exact; outputs are sampled because the oracle is slow at this size."""
    geom = (21, 192, 31, 32, 192, 3, 3, 1, 1)
    n, ci, h, w, co, r, s, ph, pw = geom
    rng = np.random.default_rng(11)
    X = rng.integers(-2, 3, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(co, ci, r, s)).astype(np.float32)
    dY = rng.integers(-2, 3, size=(n, co, h, w)).astype(np.float32)
    all_three(geom, X, Wt, dY, exact=True, sample=30000, seed=5)


@pytest.mark.parametrize("geom", SMALL[:3])
def test_format_values_within_bound(geom):
    n, ci, h, w, co, r, s, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s + 1
    rng = workloads.rng_for(80, sum(geom))
    X = workloads.lognormal_tensor(rng, (n, ci, h, w), -2.0, 2.0, p_zero=0.5, positive=True)
    Wt = workloads.normal_tensor(rng, (co, ci, r, s), 0.05)
    dY = workloads.lognormal_tensor(rng, (n, co, oh, ow), -20.0, 4.0)
    all_three(geom, X, Wt, dY, grad_scale=2.0 ** 10)


def test_pair_schedule_on_config4_shape_is_exact_and_reproducible():
    """The 3 x 3 layer of the ResNet-50-shaped workload (batch 128, 256 -> 256 channels, 14 x 14): 100
    pair tiles of 36 chunks on 74 pairs, the last conv tile incomplete.  Integers: exact; then real
    values twice: identical bits."""
    sh = workloads.CONV3X3
    geom = (sh.n, sh.c_in, sh.h, sh.w, sh.c_out, sh.r, sh.s, sh.pad, sh.pad)
    rng = np.random.default_rng(17)
    X = rng.integers(-2, 3, size=(sh.n, sh.c_in, sh.h, sh.w)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(sh.c_out, sh.c_in, sh.r, sh.s)).astype(np.float32)
    dY = rng.integers(-2, 3, size=(sh.n, sh.c_out, sh.h, sh.w)).astype(np.float32)
    all_three(geom, X, Wt, dY, exact=True, sample=30000, seed=6)
    cfg = workloads.config4(sh)
    fmt = qf.make_format(6, 9, 1)
    dX, dW = to_channels_last(cfg["X"], fmt), to_channels_last(cfg["W"], fmt)
    outs = [run_conv(qf.QFMT_CONV_FWD, geom, dX, dW, (sh.n, sh.h, sh.w, sh.c_out), fmt).cpu().numpy() for _ in range(3)]
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))
    assert np.array_equal(outs[0].view(np.uint32), outs[2].view(np.uint32))


@pytest.mark.parametrize("shape", [workloads.CONV3X3, workloads.CONV1X1], ids=["3x3", "1x1"])
def test_config4_resnet50_shaped_layers(shape):
    """Full-size layers (batch 128, 14x14): 65 536 sampled outputs per product, each a full
    reduction by the oracle's direct definition."""
    cfg = workloads.config4(shape)
    geom = (shape.n, shape.c_in, shape.h, shape.w, shape.c_out, shape.r, shape.s, shape.pad, shape.pad)
    e, m = cfg["fmt"]
    worst = all_three(geom, cfg["X"], cfg["W"], cfg["dY"], e, m, cfg["grad_scale"], sample=65536, seed=40 + shape.r)
    print("config4", shape.r, worst)


def test_56x56_stage_sampled():
    """A layer shaped like the first stage of a ResNet-50 (64 -> 64 channels at 56 x 56, 3 x 3, batch 8):
    the filter gradient runs two 32-pixel stages per output row over 448 rows and splits K; forward and data
    gradient have two image rows per tile.  Integers first (exact), then values of the format within the bound,
    on sampled outputs."""
    geom = (8, 64, 56, 56, 64, 3, 3, 1, 1)
    n, ci, h, w, co, r, s, ph, pw = geom
    rng = np.random.default_rng(56)
    X = rng.integers(-2, 3, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(co, ci, r, s)).astype(np.float32)
    dY = rng.integers(-1, 2, size=(n, co, h, w)).astype(np.float32)
    all_three(geom, X, Wt, dY, exact=True, sample=20000, seed=7)
    rng = workloads.rng_for(56, 3)
    X = workloads.lognormal_tensor(rng, (n, ci, h, w), -2.0, 2.0, p_zero=0.5, positive=True)
    Wt = workloads.normal_tensor(rng, (co, ci, r, s), 0.05)
    dY = workloads.lognormal_tensor(rng, (n, co, h, w), -20.0, 4.0)
    all_three(geom, X, Wt, dY, grad_scale=2.0 ** 10, sample=20000, seed=8)


def test_unsupported_geometries_are_refused():
    d = torch.zeros(1 << 16, dtype=torch.float32, device=DEV)
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    fmt = qf.make_format(6, 9)
    for geom, op in (((1, 30, 8, 8, 32, 3, 3, 1, 1), qf.QFMT_CONV_FWD),     # channels not a multiple of 32
                     ((1, 32, 8, 200, 32, 3, 3, 1, 1), qf.QFMT_CONV_FWD),    # rows longer than an M-tile
                     ((1, 32, 8, 200, 32, 3, 3, 1, 1), qf.QFMT_CONV_DGRAD),  # the same for the data gradient
                     ((1, 32, 2, 2, 32, 5, 5, 0, 0), qf.QFMT_CONV_FWD)):     # empty output
        g = qf.qfmt_conv_t(*geom)
        assert qf.qfmt_conv_workspace_bytes(op, g) == 0
        with pytest.raises(qf.QfmtError) as ei:
            qf.qfmt_conv(op, g, d, d, d, fmt, ws, ws.numel())
        assert ei.value.status == qf.QFMT_ERR_BAD_ARG
