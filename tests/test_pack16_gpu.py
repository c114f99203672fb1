"""GPU parity of the 16-bit storage entry points against the CPU oracle: packed codes, the
statistics taken while packing, and the expansion back to fp32 containers, all bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import workloads

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def pack_gpu(x, e, m, den, scale, in_off=0, out_off=0, want_stats=True):
    n = x.size
    buf_in = torch.zeros(n + 16, dtype=torch.float32, device=DEV)
    d_in = buf_in[in_off:in_off + n]
    d_in.copy_(torch.from_numpy(x.reshape(-1)))
    buf = torch.full((n + 32,), 0x7777, dtype=torch.int16, device=DEV)
    d_codes = buf[out_off:out_off + n]
    st = torch.full((qf.STATS_WORDS,), 99, dtype=torch.int64, device=DEV) if want_stats else None
    qf.qfmt_quantize_stats_pack16(d_in, d_codes, n, qf.make_format(e, m, den, scale), st)
    torch.cuda.synchronize()
    assert torch.all(buf[:out_off] == 0x7777) and torch.all(buf[out_off + n:] == 0x7777)
    return d_codes, (st.cpu().numpy().view(np.uint64) if want_stats else None)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7), (4, 3), (5, 2), (7, 8)])
@pytest.mark.parametrize("den", [1, 0])
@pytest.mark.parametrize("scale", [1.0, 2.0 ** 8, 3.0e-5])
def test_codes_and_stats_on_arbitrary_bit_patterns(e, m, den, scale):
    rng = np.random.default_rng(700 + e * 31 + m)
    u = np.concatenate([rng.integers(0, 1 << 32, size=70003, dtype=np.uint64).astype(np.uint32),
                        workloads.edge_bit_patterns()])
    x = u.view(np.float32)
    c_ref, st_ref = oracle.quantize_stats_pack16(x, e, m, den, scale)
    d_codes, st = pack_gpu(x, e, m, den, scale)
    got = d_codes.cpu().numpy().view(np.uint16)
    bad = np.nonzero(got != c_ref)[0]
    assert bad.size == 0, (bad[:5], got[bad[:5]], c_ref[bad[:5]], u[bad[:5]])
    assert np.array_equal(st, st_ref)
    # expansion of the GPU's codes on the GPU equals the oracle's decoding
    d_out = torch.full((x.size + 8,), 7.0, dtype=torch.float32, device=DEV)
    qf.qfmt_unpack16(d_codes, d_out, x.size, qf.make_format(e, m, den))
    torch.cuda.synchronize()
    back = d_out[:x.size].cpu().numpy()
    ref = oracle.unpack16(c_ref, e, m)
    assert np.array_equal(back.view(np.uint32), ref.view(np.uint32))
    assert torch.all(d_out[x.size:] == 7.0)


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7)])
def test_every_code_unpacks_and_packs_back(e, m):
    codes = np.arange(1 << 16, dtype=np.uint16)
    d_codes = torch.from_numpy(codes.view(np.int16)).to(DEV)
    d_out = torch.empty(codes.size, dtype=torch.float32, device=DEV)
    qf.qfmt_unpack16(d_codes, d_out, codes.size, qf.make_format(e, m))
    torch.cuda.synchronize()
    vals = d_out.cpu().numpy()
    ref = oracle.unpack16(codes, e, m)
    assert np.array_equal(vals.view(np.uint32), ref.view(np.uint32))
    again, _ = pack_gpu(vals, e, m, 1, 1.0, want_stats=False)
    got = again.cpu().numpy().view(np.uint16)
    fin = ((codes >> m) & ((1 << e) - 1)) != (1 << e) - 1
    assert np.array_equal(got[fin], codes[fin])
    infs = ~fin & ((codes & ((1 << m) - 1)) == 0)
    assert np.array_equal(got[infs], codes[infs])


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 15, 16, 17, 1023, 4099, 262147])
@pytest.mark.parametrize("in_off,out_off", [(0, 0), (1, 0), (0, 3), (2, 5)])
def test_sizes_tails_and_alignment(n, in_off, out_off):
    x = workloads.lognormal_tensor(workloads.rng_for(710, n), (n,), -18.0, 8.0, p_zero=0.02)
    c_ref, st_ref = oracle.quantize_stats_pack16(x, 6, 9, 1, 4.0)
    d_codes, st = pack_gpu(x, 6, 9, 1, 4.0, in_off, out_off)
    assert np.array_equal(d_codes.cpu().numpy().view(np.uint16), c_ref) and np.array_equal(st, st_ref)


def test_binary16_and_bfloat16_codes_are_the_native_types():
    """For 1/5/10 and 1/8/7 the packed tensor can be handed to code that expects the hardware's
    own half and bfloat16 types."""
    x = workloads.lognormal_tensor(workloads.rng_for(720), (100003,), -10.0, 6.0, p_zero=0.01)
    d_codes, _ = pack_gpu(x, 5, 10, 1, 1.0)
    assert torch.equal(d_codes.view(torch.float16), torch.from_numpy(x).to(DEV).to(torch.float16))
    d_codes, _ = pack_gpu(x, 8, 7, 1, 1.0)
    assert torch.equal(d_codes.view(torch.bfloat16), torch.from_numpy(x).to(DEV).to(torch.bfloat16))


def test_config2_full_size_pack_and_unpack_feed_the_same_values():
    """64 Mi elements (the benchmark's tensor): unpack(pack(x)) equals the fp32-container pass."""
    x = workloads.config2_tensor()
    d_in = torch.from_numpy(x).to(DEV)
    n = x.size
    d_codes = torch.empty(n, dtype=torch.int16, device=DEV)
    d_q = torch.empty_like(d_in)
    d_ref = torch.empty_like(d_in)
    st = torch.zeros(2, qf.STATS_WORDS, dtype=torch.int64, device=DEV)
    for e, m, den, scale in ((6, 9, 1, 1.0), (5, 10, 0, 2.0 ** 8), (8, 7, 1, 2.0 ** 15)):
        fmt = qf.make_format(e, m, den, scale)
        qf.qfmt_quantize_stats_pack16(d_in, d_codes, n, fmt, st[0])
        qf.qfmt_unpack16(d_codes, d_q, n, fmt)
        qf.qfmt_quantize_stats(d_in, d_ref, n, fmt, st[1])
        torch.cuda.synchronize()
        assert torch.equal(d_q.view(torch.int32), d_ref.view(torch.int32)) and torch.equal(st[0], st[1])
        c_ref, _ = oracle.quantize_stats_pack16(x[:1 << 20], e, m, den, scale)
        assert np.array_equal(d_codes[:1 << 20].cpu().numpy().view(np.uint16), c_ref)


def test_errors():
    d = torch.ones(64, dtype=torch.float32, device=DEV)
    c = torch.zeros(64, dtype=torch.int16, device=DEV)
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_quantize_stats_pack16(d, c, 64, qf.make_format(8, 10))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT        # 1 + 8 + 10 bits do not fit a 16-bit word
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_unpack16(c, d, 64, qf.make_format(6, 12))
    assert ei.value.status == qf.QFMT_ERR_BAD_FORMAT
    with pytest.raises(qf.QfmtError) as ei:
        qf.qfmt_quantize_stats_pack16(d, None, 64, qf.make_format(6, 9))
    assert ei.value.status == qf.QFMT_ERR_BAD_ARG
