"""Work list of the split-K down projection (srm_k_gemm_splitk_plan: pure host arithmetic, the function the
kernel evaluates on the device). Every (tile, k-block) exactly once; a pair's pieces are one contiguous run;
no tile is cut more than once; the upper part of a cut tile is the FIRST piece of its pair (it is finished
early, so the lower part, the LAST piece of the previous pair, never waits for it); the load is even."""
import ctypes as C

import numpy as np
import pytest

import paper_2605_08696_b200 as P


def _pieces(M, N, K, pairs, pair):
    lib = P.load_library()
    n = lib.srm_k_gemm_splitk_plan(M, N, K, pairs, pair, None, 0)
    if n < 0:
        return n
    buf = (C.c_int64 * (4 * max(n, 1)))()
    assert lib.srm_k_gemm_splitk_plan(M, N, K, pairs, pair, buf, n) == n
    return np.array(buf[: 4 * n], dtype=np.int64).reshape(n, 4)


@pytest.mark.parametrize("M,N,K,pairs", [
    (4096, 1024, 4096, 74),      # 64 tiles for 74 pairs: groups of 6 or 7 tiles for 7 or 8 pairs
    (8192, 1024, 4096, 74),      # 128 tiles: 1.73 tiles per pair
    (8192, 1536, 6144, 74),      # rollout model: 192 tiles of 96 k-blocks
    (3000, 1024, 4096, 74),      # 48 tiles, ragged rows
    (4096, 1024, 4096, 70),      # six extra pairs: groups of 10 or 11 tiles
    (16384, 1024, 4096, 74),     # 256 tiles: 3.46 per pair
])
def test_split_covers_every_k_block_once_with_at_most_one_cut_per_tile(M, N, K, pairs):
    m_tiles, n_tiles, kb = -(-M // 256), -(-N // 256), K // 64
    seen = np.zeros((m_tiles, n_tiles, kb), dtype=np.int64)
    work, cuts = [], np.zeros((m_tiles, n_tiles), dtype=np.int64)
    first_piece_upper = []
    for c in range(pairs):
        pcs = _pieces(M, N, K, pairs, c)
        assert not isinstance(pcs, int), "this shape should be split"
        flat = []
        for i, (tm, tn, k0, k1) in enumerate(pcs):
            assert 0 <= k0 < k1 <= kb
            seen[tm, tn, k0:k1] += 1
            flat.append(((tn * m_tiles + tm) * kb + k0, (tn * m_tiles + tm) * kb + k1))
            if k0 > 0:
                cuts[tm, tn] += 1
                first_piece_upper.append(i == 0)       # an upper part always opens its pair's range
            if k1 < kb:
                assert i == len(pcs) - 1               # a lower part always closes its pair's range
        for (a0, a1), (b0, b1) in zip(flat, flat[1:]):
            assert a1 == b0
        work.append(sum(k1 - k0 for _, _, k0, k1 in pcs))
    assert (seen == 1).all()
    assert cuts.max() <= 1
    assert all(first_piece_upper)
    total = m_tiles * n_tiles * kb
    assert sum(work) == total
    whole_rounds = -(-m_tiles * n_tiles // pairs) * kb
    assert max(work) <= total / pairs + 13         # even: within the 12 k-blocks a group's last pair is spared ...
    assert max(work) < 0.95 * whole_rounds         # ... and clearly below whole tiles per pair


def test_last_pair_of_a_group_finishes_early():
    """64 tiles on 74 pairs: a group's last pair holds one piece, the upper part of the group's last tile; the
    piece that must be added after it closes the previous pair's range, so the last pair gets 12 k-blocks less."""
    loads = []
    for c in range(74):
        pcs = _pieces(4096, 1024, 4096, 74, c)
        loads.append(int(sum(k1 - k0 for _, _, k0, k1 in pcs)))
    short = [c for c in range(74) if loads[c] < 50]
    assert len(short) == 10                             # one per group
    for c in short:
        pcs = _pieces(4096, 1024, 4096, 74, c)
        assert len(pcs) == 1 and pcs[0][3] == 64 and pcs[0][2] > 0
        assert max(loads) - loads[c] >= 12


@pytest.mark.parametrize("M,N,K,pairs", [(75776, 1024, 4096, 74),                 # 1184 tiles = 16 whole rounds
                                         (256, 1024, 4096, 74),                   # 4 tiles: far fewer than pairs
                                         (4096, 1024, 4096, 66),                  # two spare pairs: 3 % to gain, not worth it
                                         (4096, 1024, 256, 74)])                  # 4 k-blocks: nothing to share out
def test_shapes_that_are_not_split(M, N, K, pairs):
    assert _pieces(M, N, K, pairs, 0) == -2
