"""Host logic of the balanced schedule of the CTA-pair kernels (no GPU): the pieces of all 74 pairs
cover every K chunk of every tile exactly once, a tile has at most two pieces, and the order in
which a pair runs its pieces is the one the hand-over between pairs relies on."""
import pytest

import paper_2103_15940_b200 as qf
from paper_2103_15940_b200 import build as qbuild

PAIRS = 74


@pytest.fixture(scope="module", autouse=True)
def _lib():
    qbuild.build()


def pieces_of(tiles, cpt, pair):
    out, j = [], 0
    n_slots = qf.qfmt_selftest_pair_schedule(tiles, cpt, pair, 0)[5]
    for j in range(n_slots):
        tile, first, n, partial, head, _ = qf.qfmt_selftest_pair_schedule(tiles, cpt, pair, j)
        if n > 0:
            out.append((tile, first, n, partial, head))
    return out, n_slots


@pytest.mark.parametrize("tiles,cpt", [(74, 1), (74, 16), (75, 16), (98, 16), (100, 36), (128, 16), (147, 5), (148, 12),
                                       (192, 12), (384, 16), (512, 16), (1000, 3), (2047, 7), (4500, 1), (333, 64)])
def test_every_chunk_once_and_two_pieces_per_tile(tiles, cpt):
    seen = {}
    per_tile = {}
    for pair in range(PAIRS):
        pcs, n_slots = pieces_of(tiles, cpt, pair)
        assert len(pcs) <= n_slots
        total = sum(n for _, _, n, _, _ in pcs)
        assert abs(total - tiles * cpt / PAIRS) < 1.0 + 1e-9          # equal ranges
        assert total >= cpt                                            # at least a tile long
        for i, (tile, first, n, partial, head) in enumerate(pcs):
            assert 0 <= tile < tiles and first >= 0 and first + n <= cpt
            assert partial == (1 if first > 0 else 0)
            assert head == (1 if first + n < cpt else 0)
            # the order the hand-over relies on: a head piece runs first, a partial piece last
            if head:
                assert i == 0
            if partial:
                assert i == len(pcs) - 1
            assert not (head and partial)
            for c in range(first, first + n):
                assert (tile, c) not in seen
                seen[(tile, c)] = pair
            per_tile.setdefault(tile, []).append((pair, first, n, partial, head))
    assert len(seen) == tiles * cpt
    for tile, pcs in per_tile.items():
        assert len(pcs) <= 2
        if len(pcs) == 2:
            (p0, f0, n0, part0, head0), (p1, f1, n1, part1, head1) = sorted(pcs, key=lambda x: x[1])
            assert p1 == p0 + 1 and head0 == 1 and part0 == 0 and part1 == 1 and head1 == 0 and f1 == f0 + n0


def test_head_is_stored_before_the_next_pair_needs_it():
    """Timing argument in chunk units (all pairs start together and run at the same rate): pair u's head
    piece ends at its length; pair u+1 first needs it when it has run everything but its partial piece plus
    that piece's first summation group (16 chunks)."""
    for tiles, cpt in [(98, 16), (100, 36), (192, 12), (384, 16), (128, 64), (75, 200)]:
        sched = [pieces_of(tiles, cpt, pair)[0] for pair in range(PAIRS)]
        for u in range(PAIRS - 1):
            heads = [pc for pc in sched[u] if pc[4]]
            parts = [pc for pc in sched[u + 1] if pc[3]]
            if not heads:
                continue
            assert len(heads) == 1 and len(parts) == 1 and heads[0][0] == parts[0][0]
            head_done = heads[0][2]
            total_next = sum(n for _, _, n, _, _ in sched[u + 1])
            needed_at = total_next - parts[0][2] + min(16, parts[0][2])
            assert needed_at >= head_done + 1


def test_rejects_what_the_schedule_does_not_take():
    with pytest.raises(qf.QfmtError):
        qf.qfmt_selftest_pair_schedule(73, 16, 0, 0)       # fewer tiles than pairs
    with pytest.raises(qf.QfmtError):
        qf.qfmt_selftest_pair_schedule(100, 16, 74, 0)     # no such pair
    with pytest.raises(qf.QfmtError):
        qf.qfmt_selftest_pair_schedule(10 ** 6, 2, 0, 0)   # more pieces per pair than the kernel's table holds
