"""Seeded random shapes, alignments, formats and options through every entry point, each checked
against the oracle: the parity tests proper fix their shapes by hand, this one looks for the
combination nobody thought of (odd leading dimensions, tiny and ragged tiles, transposes, flushing
with a loss scale, ...).  Integer work must match bit for bit; qfmt_gemm within its bound."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads
from test_conv_gpu import all_three

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
FORMATS = [(5, 10), (6, 9), (8, 7), (4, 3), (7, 8), (5, 2), (3, 4)]


def rand_tensor(rng, shape, e, m):
    """Values spread over the format's whole range and a little beyond, with zeros and specials."""
    b = 2 ** (e - 1) - 1
    x = workloads.lognormal_tensor(workloads.rng_for(int(rng.integers(1 << 30))), shape,
                                   float(rng.uniform(-b - m, b - 4)), float(rng.uniform(0.5, 6.0)),
                                   p_zero=float(rng.choice([0.0, 0.02, 0.5])))
    flat = x.reshape(-1)
    if flat.size >= 8 and rng.random() < 0.5:
        pos = rng.integers(0, flat.size, size=4)
        flat[pos] = [np.inf, -np.inf, np.nan, -0.0]
    return x


@pytest.mark.parametrize("seed", range(24))
def test_rounding_entry_points(seed):
    rng = np.random.default_rng(9000 + seed)
    for _ in range(6):
        e, m = FORMATS[int(rng.integers(len(FORMATS)))]
        den = int(rng.integers(2))
        scale = float(rng.choice([1.0, 2.0 ** 8, 2.0 ** -6, 3.0, 1.0e-3]))
        n = int(rng.choice([1, 5, 33, 1000, 4097, 70001, 300007]))
        x = rand_tensor(rng, (n,), e, m)
        q_ref, st_ref = oracle.quantize_stats(x, e, m, den, scale)
        off_in, off_out = int(rng.integers(4)), int(rng.integers(4))
        buf_in = torch.zeros(n + 8, dtype=torch.float32, device=DEV)
        buf_out = torch.full((n + 8,), 7.0, dtype=torch.float32, device=DEV)
        d_in, d_out = buf_in[off_in:off_in + n], buf_out[off_out:off_out + n]
        d_in.copy_(torch.from_numpy(x))
        st = torch.full((qf.STATS_WORDS,), 5, dtype=torch.int64, device=DEV)
        fmt = qf.make_format(e, m, den, scale)
        qf.qfmt_quantize_stats(d_in, d_out, n, fmt, st)
        torch.cuda.synchronize()
        got = d_out.cpu().numpy()
        nan = np.isnan(q_ref)
        assert np.array_equal(got.view(np.uint32)[~nan], q_ref.view(np.uint32)[~nan]), (e, m, den, scale, n)
        assert np.array_equal(got.view(np.uint32)[nan], q_ref.view(np.uint32)[nan])
        assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref)
        assert torch.all(buf_out[:off_out] == 7.0) and torch.all(buf_out[off_out + n:] == 7.0)
        if e + m <= 15:
            c_ref, _ = oracle.quantize_stats_pack16(x, e, m, den, scale)
            codes = torch.zeros(n + 16, dtype=torch.int16, device=DEV)
            d_codes = codes[off_out:off_out + n]
            qf.qfmt_quantize_stats_pack16(d_in, d_codes, n, fmt, st)
            back = torch.empty(n, dtype=torch.float32, device=DEV)
            qf.qfmt_unpack16(d_codes, back, n, fmt)
            torch.cuda.synchronize()
            assert np.array_equal(d_codes.cpu().numpy().view(np.uint16), c_ref), (e, m, den, scale, n)
            assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref)
            assert np.array_equal(back.cpu().numpy().view(np.uint32), oracle.unpack16(c_ref, e, m).view(np.uint32))


@pytest.mark.parametrize("seed", range(20))
def test_layer_output(seed):
    rng = np.random.default_rng(9100 + seed)
    for _ in range(5):
        e, m = [(5, 10), (6, 9), (8, 7), (4, 3), (7, 8)][int(rng.integers(5))]
        den = int(rng.integers(2))
        scale = float(rng.choice([1.0, 4.0, 2.0 ** -5]))
        rows, cols = int(rng.integers(1, 400)), int(rng.choice([1, 3, 4, 36, 100, 513, 2048]))
        ld_a, ld_o = cols + int(rng.choice([0, 0, 1, 4, 12])), cols + int(rng.choice([0, 0, 3, 4]))
        off = int(rng.choice([0, 0, 1, 2]))
        acc, bias = rand_tensor(rng, (rows, cols), e, m), rand_tensor(rng, (cols,), e, m)
        y_ref, st_ref = oracle.bias_quantize_stats(acc, bias, e, m, den, scale)
        buf_a = torch.zeros(rows * ld_a + 8, dtype=torch.float32, device=DEV)
        d_acc = buf_a[off:off + rows * ld_a].view(rows, ld_a)
        d_acc[:, :cols].copy_(torch.from_numpy(acc))
        d_bias = torch.zeros(cols + 8, dtype=torch.float32, device=DEV)[off:off + cols]
        d_bias.copy_(torch.from_numpy(bias))
        buf_o = torch.full((rows * ld_o + 8,), 7.0, dtype=torch.float32, device=DEV)
        d_out = buf_o[off:off + rows * ld_o].view(rows, ld_o)
        st = torch.full((qf.STATS_WORDS,), 5, dtype=torch.int64, device=DEV)
        qf.qfmt_bias_quantize_stats(d_acc, ld_a, d_bias, d_out, ld_o, rows, cols, qf.make_format(e, m, den, scale), st)
        torch.cuda.synchronize()
        got = d_out[:, :cols].cpu().numpy()
        assert np.array_equal(got.view(np.uint32), y_ref.view(np.uint32)), (e, m, den, scale, rows, cols, ld_a, ld_o, off)
        assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref)
        assert torch.all(d_out[:, cols:] == 7.0)


@pytest.mark.parametrize("seed", range(20))
def test_fmac8_product(seed):
    rng = np.random.default_rng(9200 + seed)
    for _ in range(3):
        e, m = [(5, 10), (6, 9), (7, 10), (4, 3), (6, 5), (8, 7)][int(rng.integers(6))]
        den = int(rng.integers(2))
        M, N, K = int(rng.integers(1, 150)), int(rng.integers(1, 150)), int(rng.integers(0, 90))
        tA, tB = bool(rng.integers(2)), bool(rng.integers(2))
        b = 2 ** (e - 1) - 1
        mu = float(rng.uniform(-b / 2 - 2, b / 2 - 2))
        A = oracle.quantize_stats(workloads.lognormal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                             (K, M) if tA else (M, K), mu, 2.0, p_zero=0.05),
                                  e, m, den, 1.0, want_stats=False)[0]
        B = oracle.quantize_stats(workloads.lognormal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                             (N, K) if tB else (K, N), mu, 2.0, p_zero=0.05),
                                  e, m, den, 1.0, want_stats=False)[0]
        c_ref, master = oracle.fmac8_gemm(A, B, e, m, den, tA, tB, want_master=True)
        _, st_ref = oracle.quantize_stats(master, e, m, den, 1.0)
        dA = torch.from_numpy(A).to(DEV) if A.size else torch.zeros(1, device=DEV)
        dB = torch.from_numpy(B).to(DEV) if B.size else torch.zeros(1, device=DEV)
        ldc = N + int(rng.choice([0, 0, 1, 4]))
        dC = torch.full((M, ldc), 7.0, dtype=torch.float32, device=DEV)
        st = torch.full((qf.STATS_WORDS,), 5, dtype=torch.int64, device=DEV)
        a = qf.make_matrix(dA.data_ptr(), tA, A.shape[0], A.shape[1], A.shape[1])
        bm = qf.make_matrix(dB.data_ptr(), tB, B.shape[0], B.shape[1], B.shape[1])
        paths = (0, 1, 2) if (e, m) in ((5, 10), (8, 7)) else (0,)
        for path in paths:
            qf.qfmt_gemm_fmac8(a, bm, dC, ldc, qf.make_format(e, m, den), st, 0, path)
            torch.cuda.synchronize()
            got = dC[:, :N].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), c_ref.view(np.uint32)), (e, m, den, M, N, K, tA, tB, path)
            assert np.array_equal(st.cpu().numpy().view(np.uint64), st_ref), (e, m, den, M, N, K, tA, tB, path)
            assert torch.all(dC[:, N:] == 7.0)


@pytest.mark.parametrize("seed", range(16))
def test_fmacs_product(seed):
    rng = np.random.default_rng(9300 + seed)
    for _ in range(3):
        e, m = [(5, 10), (6, 9), (8, 7)][int(rng.integers(3))]
        M, N = 4 * int(rng.integers(1, 120)), 4 * int(rng.integers(1, 160))
        K = 4 * int(rng.integers(1, 700))
        tA, tB = bool(rng.integers(2)), bool(rng.integers(2))
        qf.qfmt_gemm_tile_policy(int(rng.integers(3)))
        try:
            A = oracle.quantize_stats(workloads.lognormal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                                 (K, M) if tA else (M, K), -3.0, 2.0, p_zero=0.02),
                                      e, m, 1, 1.0, want_stats=False)[0]
            B = oracle.quantize_stats(workloads.normal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                              (N, K) if tB else (K, N), 0.05),
                                      e, m, 1, 1.0, want_stats=False)[0]
            dA, dB = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
            a, bm = qf.make_matrix(dA, tA), qf.make_matrix(dB, tB)
            ldc = N + 4 * int(rng.integers(0, 3))
            dC = torch.full((M, ldc), 7.0, dtype=torch.float32, device=DEV)
            wb = max(256, qf.qfmt_gemm_workspace_bytes(a, bm))
            ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
            qf.qfmt_gemm(a, bm, dC, ldc, qf.make_format(e, m), ws, wb)
            assert qf.qfmt_device_status(ws) == qf.QFMT_OK
            ref, T = oracle.gemm(A, B, tA, tB)
            err = np.abs(dC[:, :N].cpu().numpy().astype(np.float64) - ref)
            assert np.all(err <= 2.0 ** -20 * T), (e, m, M, N, K, tA, tB, float(np.max(err / np.maximum(T, 1e-300))) * 2 ** 20)
            assert torch.all(dC[:, N:] == 7.0)
        finally:
            qf.qfmt_gemm_tile_policy(0)


@pytest.mark.parametrize("seed", range(16))
def test_fmacs_product_on_packed_codes(seed):
    """qfmt_gemm_packed16 on random shapes (any M, N, K; stored row lengths padded to multiples of
    8), layouts and the two formats; against the oracle's expansion of the same codes."""
    rng = np.random.default_rng(9500 + seed)
    for _ in range(3):
        e, m = [(5, 10), (8, 7)][int(rng.integers(2))]
        M, N, K = int(rng.integers(1, 480)), int(rng.integers(1, 640)), int(rng.integers(1, 2800))
        tA, tB = bool(rng.integers(2)), bool(rng.integers(2))
        cA, _ = oracle.quantize_stats_pack16(workloads.lognormal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                                        (K, M) if tA else (M, K), -3.0, 2.0, p_zero=0.02),
                                             e, m, 1, 1.0)
        cB, _ = oracle.quantize_stats_pack16(workloads.normal_tensor(workloads.rng_for(int(rng.integers(1 << 30))),
                                                                     (N, K) if tB else (K, N), 0.05), e, m, 1, 1.0)
        A, B = oracle.unpack16(cA, e, m), oracle.unpack16(cB, e, m)
        mats = []
        for c, t in ((cA, tA), (cB, tB)):
            ld = (c.shape[1] + 7) // 8 * 8 + 8 * int(rng.integers(0, 2))
            d = torch.full((c.shape[0], ld), 0x7C00, dtype=torch.int16, device=DEV)   # padding: binary16 infinity
            d[:, :c.shape[1]] = torch.from_numpy(c.view(np.int16)).to(DEV)
            mats.append((qf.make_matrix(d, t, rows=c.shape[0], cols=c.shape[1], ld=ld), d))
        ldc = N + int(rng.integers(0, 3))
        dC = torch.full((M, ldc), 7.0, dtype=torch.float32, device=DEV)
        wb = max(256, qf.qfmt_gemm_packed16_workspace_bytes(mats[0][0], mats[1][0]))
        ws = torch.zeros(wb, dtype=torch.uint8, device=DEV)
        qf.qfmt_gemm_packed16(mats[0][0], mats[1][0], dC, ldc, qf.make_format(e, m), ws, wb)
        assert qf.qfmt_device_status(ws) == qf.QFMT_OK
        ref, T = oracle.gemm(A, B, tA, tB)
        err = np.abs(dC[:, :N].cpu().numpy().astype(np.float64) - ref)
        assert np.all(err <= 2.0 ** -20 * T), (e, m, M, N, K, tA, tB, float(np.max(err / np.maximum(T, 1e-300))) * 2 ** 20)
        assert torch.all(dC[:, N:] == 7.0)


@pytest.mark.parametrize("seed", range(12))
def test_convolution_products(seed):
    """Random small geometries with small-integer tensors: every order of summation is exact, so the
    three products must equal the oracle's direct definitions exactly."""
    rng = np.random.default_rng(9400 + seed)
    r, s_ = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    ph, pw = int(rng.integers(0, r)), int(rng.integers(0, s_))
    w = int(rng.integers(max(s_ - 2 * pw, 1), 20))
    h = int(rng.integers(max(r - 2 * ph, 1), 12))
    geom = (int(rng.integers(1, 5)), 32 * int(rng.integers(1, 4)), h, w, 32 * int(rng.integers(1, 10)), r, s_, ph, pw)
    n, ci, h, w, co, r, s_, ph, pw = geom
    oh, ow = h + 2 * ph - r + 1, w + 2 * pw - s_ + 1
    X = rng.integers(-3, 4, size=(n, ci, h, w)).astype(np.float32)
    Wt = rng.integers(-3, 4, size=(co, ci, r, s_)).astype(np.float32)
    dY = rng.integers(-3, 4, size=(n, co, oh, ow)).astype(np.float32)
    all_three(geom, X, Wt, dY, exact=True)
