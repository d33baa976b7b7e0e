"""The sweep's schedule, checked on the host (no GPU): qf_plan_pieces returns the pieces the kernels cut the
stage-unit space into.  The pieces must tile the space exactly and in order, whatever the total; the drawn
chunks must come in rounds of halving size, each at most a 1/n_ctas share of what is still undrawn."""
import numpy as np
import pytest

from paper_2608_15473_b200 import binding as qf
from paper_2608_15473_b200 import build as qf_build


@pytest.fixture(scope="module", autouse=True)
def built():
    qf_build.build()


def check_tiling(pieces, total, n_ctas):
    assert len(pieces) >= n_ctas
    pos = 0
    for i, (b, e) in enumerate(pieces):
        assert b == min(pos, total) or (b == pos), (i, b, e, pos)
        assert e >= b
        if i >= n_ctas:
            assert e > b, "a drawn chunk is never empty"
        pos = e
    assert pos == total
    # static slices are equal except possibly the last non-empty one
    static = [e - b for b, e in pieces[:n_ctas]]
    nz = [x for x in static if x > 0]
    if nz:
        assert max(nz[:-1], default=nz[0]) == nz[0] and nz[-1] <= nz[0]


@pytest.mark.parametrize("n_ctas", [1, 2, 7, 132, 148, 160])
def test_pieces_tile_the_unit_space_for_every_total(n_ctas):
    rng = np.random.default_rng(n_ctas)
    totals = list(range(0, 3 * n_ctas + 3)) + [112 * n_ctas - 1, 112 * n_ctas, 112 * n_ctas + 1] + \
        [int(x) for x in rng.integers(1, 3_000_000, size=60)] + [2**31 - 1 - 160]
    for total in totals:
        for always in (False, True):
            pieces = qf.plan_pieces(total, n_ctas, always)
            check_tiling(pieces, total, n_ctas)
            drawn = pieces[n_ctas:]
            if total < (2 if always else 112) * n_ctas:
                assert not drawn, "short sweeps stay static"
            assert len(drawn) <= 3 * 160


def test_drawn_share_and_halving_rounds():
    n = 148
    for total in (112 * n, 30_916, 65_536, 131_171, 1_000_003):
        pieces = qf.plan_pieces(total, n)
        static, drawn = pieces[:n], pieces[n:]
        static_end = static[-1][1]
        share = total - static_end
        assert total // 10 <= share < total // 10 + n          # a tenth, rounded up to whole slices
        sizes = [e - b for b, e in drawn]
        # rounds: half of the share, half of the rest, then the rest; within a round the chunks are equal
        # (the round's last one may be shorter) and there are at most n of them
        r0 = (share + 1) // 2
        r1 = (share - r0 + 1) // 2
        rounds, k = [], 0
        for quota in (r0, r1, share - r0 - r1):
            got, first = 0, k
            while got < quota:
                got += sizes[k]
                k += 1
            assert got == quota, "a chunk never straddles two rounds"
            rounds.append(sizes[first:k])
        assert k == len(sizes)
        left = share
        for r, chunk_sizes in enumerate(rounds):
            assert 1 <= len(chunk_sizes) <= n
            assert all(x == chunk_sizes[0] for x in chunk_sizes[:-1]) and chunk_sizes[-1] <= chunk_sizes[0]
            if r < 2:   # never more than a 1/n share of what is still undrawn (or the 3-unit minimum)
                for x in chunk_sizes:
                    assert x <= max(3, -(-left // n)), (total, r, x, left)
                    left -= x
        assert rounds[0][0] >= rounds[1][0] >= rounds[2][0] >= 3 or share < 12 * n
        assert rounds[2][0] <= max(3, -(-rounds[0][0] // 2) + 1)


def test_bad_arguments():
    with pytest.raises(qf.QFError):
        qf.plan_pieces(-1, 148)
    with pytest.raises(qf.QFError):
        qf.plan_pieces(100, 0)
    with pytest.raises(qf.QFError):
        qf.plan_pieces(100, 161)
