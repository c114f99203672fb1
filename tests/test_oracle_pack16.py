"""Pins for the oracle's 16-bit storage (no GPU): packed codes against the host's IEEE binary16 and
bfloat16 conversions, and the pack/unpack round trip against the rounding itself."""
import numpy as np
import pytest
import torch

import oracle
from paper_2103_15940_b200 import workloads


def patterns(n, seed):
    rng = np.random.default_rng(seed)
    u = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    return np.concatenate([u, workloads.edge_bit_patterns()]).view(np.float32)


def test_binary16_codes_are_numpy_half_bits():
    x = patterns(200000, 1)
    codes, _ = oracle.quantize_stats_pack16(x, 5, 10)
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    nan = np.isnan(x)
    assert np.array_equal(codes[~nan], ref[~nan])
    assert np.all((codes[nan] & 0x7C00) == 0x7C00) and np.all((codes[nan] & 0x03FF) != 0)


def test_bfloat16_codes_are_torch_bfloat16_bits():
    x = patterns(200000, 2)
    codes, _ = oracle.quantize_stats_pack16(x, 8, 7)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(x)
    assert np.array_equal(codes[~nan], ref[~nan])


@pytest.mark.parametrize("e,m", [(5, 10), (6, 9), (8, 7), (4, 3), (5, 2)])
@pytest.mark.parametrize("den", [1, 0])
def test_round_trip_is_the_rounding(e, m, den):
    x = patterns(60000, 3 + e)
    q, st = oracle.quantize_stats(x, e, m, den, 4.0)
    codes, st2 = oracle.quantize_stats_pack16(x, e, m, den, 4.0)
    assert np.array_equal(st, st2)
    assert int(codes.max()) < (1 << (1 + e + m))
    back = oracle.unpack16(codes, e, m)
    nan = np.isnan(q)
    assert np.array_equal(back.view(np.uint32)[~nan], q.view(np.uint32)[~nan])
    assert np.all(np.isnan(back[nan]))
    # every code decodes and encodes back to itself (finite codes, all of them)
    allc = np.arange(1 << (1 + e + m), dtype=np.uint16)
    fin = ((allc >> m) & ((1 << e) - 1)) != (1 << e) - 1
    vals = oracle.unpack16(allc[fin], e, m)
    again, _ = oracle.quantize_stats_pack16(vals, e, m, 1, 1.0)
    assert np.array_equal(again, allc[fin])
