"""Host arithmetic of the matmul tail split (no GPU): the plan dvm_launch would use, walked the way the kernel walks
it -- every k block of every tile of the last wave is computed exactly once, parts of a tile belong to consecutive
units starting at its owner, a unit's pieces come in the order end-of-tile then start-of-next (so an owner only
ever waits for units that do not wait), and the limits of the exchange (parts per tile, workspace) hold."""
import itertools

import pytest

import paper_2603_24239_b200 as dvm


def _walk(plan, k_blocks, n_units):
    """The pieces (tile, kb0, kb1, part, parts) of every unit, from the kernel's formulas."""
    W, P, r = plan["kb_per_unit"], plan["tile_pitch"], plan["r"]
    gend = (r - 1) * P + k_blocks
    out = {}
    for unit in range(n_units):
        pieces = []
        for q in itertools.count():
            g0 = unit * W
            if g0 >= gend:
                break
            g1 = min(g0 + W, gend)
            a = g0 // P + q
            if a >= r:
                break
            s0, s1 = max(g0, a * P), min(g1, a * P + k_blocks)
            if s0 >= s1:
                break
            owner = (a * P) // W
            parts = (a * P + k_blocks - 1) // W - owner + 1
            pieces.append((a, s0 - a * P, s1 - a * P, unit - owner, parts))
        out[unit] = pieces
    return out


@pytest.mark.parametrize("units,nr", [(148, 1), (74, 2), (132, 1), (66, 2)])
def test_every_k_block_once(units, nr):
    dvm.set_matmul_tail_split(True)
    n_split = 0
    for k_blocks in (16, 17, 25, 64, 80, 128, 214, 448):
        for tiles in list(range(1, units)) + [units + 1, 3 * units + 37, 7 * units + units - 1]:
            plan = dvm.matmul_tail_plan(tiles, units, k_blocks, nr)
            if plan is None:
                continue
            n_split += 1
            r = plan["r"]
            assert plan["first"] == tiles - r and r == tiles % units and 0 < r < units
            assert 2 <= plan["parts_max"] <= 4 and plan["units_used"] <= units
            assert r * (plan["parts_max"] - 1) * nr <= 200          # partial accumulators the workspace holds
            pieces = _walk(plan, k_blocks, units)
            assert all(not pieces[u] for u in range(plan["units_used"], units))
            assert all(pieces[u] for u in range(plan["units_used"]))
            cover = {a: [] for a in range(r)}
            for u, ps in pieces.items():
                assert len(ps) <= 2
                for i, (a, kb0, kb1, part, parts) in enumerate(ps):
                    assert 0 <= kb0 < kb1 <= k_blocks and 0 <= part < parts <= plan["parts_max"]
                    cover[a].append((kb0, kb1, part, parts, u))
                    if i == 1:   # a unit's second piece starts a tile (it owns it); its first was not one that waits
                        assert part == 0 and kb0 == 0 and (ps[0][3] > 0 or ps[0][4] == 1)
            for a, segs in cover.items():
                segs.sort()
                assert segs[0][0] == 0 and segs[-1][1] == k_blocks
                assert all(x[1] == y[0] for x, y in zip(segs, segs[1:]))      # no gap, no overlap
                assert [x[2] for x in segs] == list(range(len(segs)))         # parts 0, 1, .. in k order
                assert all(x[3] == len(segs) for x in segs)
                assert [x[4] for x in segs] == list(range(segs[0][4], segs[0][4] + len(segs)))   # consecutive units
    assert n_split > 100


def test_no_split_cases():
    dvm.set_matmul_tail_split(True)
    assert dvm.matmul_tail_plan(148 * 5, 148, 64) is None       # whole waves
    assert dvm.matmul_tail_plan(100, 148, 8) is None            # too few k blocks to share
    assert dvm.matmul_tail_plan(147, 148, 64) is None           # nothing to gain
    dvm.set_matmul_tail_split(False)
    try:
        assert dvm.matmul_tail_plan(10, 148, 64) is None
    finally:
        dvm.set_matmul_tail_split(True)
    with pytest.raises(dvm.DvmError):
        dvm.matmul_tail_plan(10, 0, 64)
