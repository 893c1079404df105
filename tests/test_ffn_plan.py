"""Work lists of the fused feed-forward kernel (srm_k_ffn_plan: pure host arithmetic; the lists travel to the kernel
as a launch parameter). Every tile of both projections exactly once (an up tile possibly as its two 256 x 128 halves:
item kinds 0 = up tile, 1 = down tile, 2 / 3 = first / second half of an up tile); the lists cannot block one another (a down tile
waits for the up tiles of its row block, which other pairs hold further down their own lists); under the planner's
cost model the plan ends close to the even share of all work and never later than two launches in whole rounds."""
import pytest

import paper_2605_08696_b200 as P

SHAPES = [
    (4096, 1024, 4096, 74),      # mid model, one pass: 256 up tiles, 64 down tiles of 64 k-blocks
    (2048, 1024, 4096, 74),      # fewer down tiles than half the pairs
    (256, 1024, 4096, 74),       # one row block
    (100, 512, 2048, 74),        # ragged single row block, small model
    (3000, 1024, 4096, 74),      # ragged rows
    (8192, 1536, 6144, 74),      # rollout model pass: 768 + 192 tiles, several down tiles per pair
    (10240, 1024, 4096, 74),
    (16384, 1536, 6144, 74),     # 1920 tiles: near the plan's capacity
    (4096, 1024, 4096, 66),      # fewer resident pairs
    (4096, 1024, 4096, 2),
    (512, 2048, 8192, 74),       # widest shape
]


def _run_lists(lists, Rb, Cu, Cd):
    """Executes the lists with the STRICTEST reading of the dependency (a down tile cannot finish before every up
    tile of its row block has): returns the number of sweeps, or None when the lists block one another."""
    up_done = [[0] * Cu for _ in range(Rb)]          # bit 0: columns 0..127 done, bit 1: columns 128..255
    pos = [0] * len(lists)
    left = sum(len(l) for l in lists)
    sweeps = 0
    while left:
        progress = False
        for c, l in enumerate(lists):
            while pos[c] < len(l):
                kind, rb, cb = l[pos[c]]
                if kind == 1 and not all(v == 3 for v in up_done[rb]):
                    break
                if kind != 1:
                    up_done[rb][cb] |= {0: 3, 2: 1, 3: 2}[kind]
                pos[c] += 1
                left -= 1
                progress = True
        if not progress:
            return None
        sweeps += 1
    return sweeps


@pytest.mark.parametrize("M,d,F,pairs", SHAPES)
def test_plan_holds_every_tile_once_and_cannot_block(M, d, F, pairs):
    lists, makespan, ideal = P.k_ffn_plan(M, d, F, pairs)
    Rb, Cu, Cd = -(-M // 256), F // 256, d // 256
    assert len(lists) == pairs
    ups = [(rb, cb) for l in lists for (kind, rb, cb) in l if kind == 0]
    first = [(rb, cb) for l in lists for (kind, rb, cb) in l if kind == 2]
    second = [(rb, cb) for l in lists for (kind, rb, cb) in l if kind == 3]
    downs = [(rb, cb) for l in lists for (kind, rb, cb) in l if kind == 1]
    assert sorted(first) == sorted(second) and len(set(first)) == len(first) and 2 * len(first) <= pairs
    assert sorted(ups + first) == [(rb, cb) for rb in range(Rb) for cb in range(Cu)]
    assert sorted(downs) == [(rb, cb) for rb in range(Rb) for cb in range(Cd)]
    assert _run_lists(lists, Rb, Cu, Cd) is not None
    assert makespan > 0 and ideal > 0


@pytest.mark.parametrize("M,d,F,pairs", SHAPES)
def test_plan_length_under_the_cost_model(M, d, F, pairs):
    _, makespan, ideal = P.k_ffn_plan(M, d, F, pairs)
    Rb, Cu, Cd, ku, kd = -(-M // 256), F // 256, d // 256, d // 64, F // 64
    up, dn = ku * 1.0 + 3.1, kd * 0.96 + 1.5                   # the planner's tile costs
    two_launches = -(-Rb * Cu // pairs) * up + -(-Rb * Cd // pairs) * dn
    assert makespan >= ideal - 1e-9
    # never later than whole rounds of two launches (plus the model's lag between an up tile's end and its
    # visibility to other pairs, which the two-launch figure leaves out)
    assert makespan <= two_launches + 16.5 + 0.1 * up
    if Rb * (Cu + Cd) >= 4 * pairs:
        assert makespan <= 1.17 * ideal                         # within one up tile or so of the even share


def test_within_a_row_block_up_tiles_come_in_column_order():
    """A down tile consumes H column tile after column tile: the up tiles of a row block that one pair computes
    must come in ascending column order, or the consumer would wait for a tile queued behind a later one."""
    lists, _, _ = P.k_ffn_plan(4096, 1024, 4096, 74)
    for l in lists:
        last = {}
        for kind, rb, cb in l:
            if kind != 1:
                assert last.get(rb, -1) < cb
                last[rb] = cb


def test_last_round_of_up_tiles_goes_out_as_halves():
    """Mid model, 4096 rows on 74 pairs: 64 pairs take three up tiles and a down tile, ten pairs up tiles only; the
    four tiles left over would give four pairs a fourth up tile: they go out as eight halves instead."""
    lists, makespan, ideal = P.k_ffn_plan(4096, 1024, 4096, 74)
    halves = [(c, it) for c, l in enumerate(lists) for it in l if it[0] in (2, 3)]
    assert len(halves) == 8 and len({c for c, _ in halves}) == 8
    assert all(l.index(it) == 0 for c, it in halves for l in [lists[c]])        # the first item of their pairs
    assert makespan < 1.13 * ideal


def test_unsupported_shapes_are_refused():
    for M, d, F in [(4096, 1000, 4000), (4096, 320, 1280), (20000, 1024, 4096), (16384, 2048, 8192)]:
        with pytest.raises(P.SRMError) as e:
            P.k_ffn_plan(M, d, F, 74)
        assert e.value.code == P.ERR_UNSUPPORTED
