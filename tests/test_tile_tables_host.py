"""The tile tables of the Newton-Schulz products, checked on the host (no GPU):
every output block that has to be stored is stored exactly once, nothing
outside the matrix is stored, and every tile obeys the rules the kernel's
operand layouts impose.

A tile is a CTA pair's work: 128 rows from each CTA (row blocks i[0], i[1] of
matrices dm[0], dm[1] of the unit) against one or two column blocks j.  One
instruction reads the operand tiles of both CTAs in one layout, and a symmetric
operand kept as its upper blocks changes layout at the diagonal, so for such
operands the two row blocks (and the two column blocks) of a tile must be equal
or neighbours.  A tile whose CTAs work on different matrices computes two cross
blocks that mean nothing; they must not be stored.  A half-height tile is one
row block, 64 rows per CTA.  The tables exist in four modes
(muon_debug_set_tile_mode); all are checked.
"""

import pytest

from paper_2502_16982_b200 import binding as b

SHAPES = [(1408, 2048), (2048, 1408), (2048, 2048), (128, 256), (100, 300), (129, 257), (640, 256), (1536, 1536),
          (1792, 4608), (2304, 6016), (6656, 2560), (576, 2048), (512, 4096), (16, 65536), (384, 384), (3200, 3300)]


def blocks(v):
    return -(-v // 128)


@pytest.fixture(params=[0, 1, 2, 3])
def tile_mode(request):
    prev = b.muon_debug_set_tile_mode(request.param)
    yield request.param
    b.muon_debug_set_tile_mode(prev)


def stored_blocks(t):
    """(matrix, row block, column block) of every block a tile stores."""
    out = []
    if t["half"]:
        assert t["i"][0] == t["i"][1] and t["dm"][0] == t["dm"][1] and t["keep"][1] == 0
        for h in range(t["nbw"]):
            if (t["keep"][0] >> h) & 1:
                out.append((t["dm"][0], t["i"][0], t["j"][h]))
        return out
    for rank in (0, 1):
        for h in range(t["nbw"]):
            if (t["keep"][rank] >> h) & 1:
                # with the full width the B rows of half h come from CTA h's matrix
                if t["nbw"] == 2:
                    assert t["dm"][h] == t["dm"][rank], t
                out.append((t["dm"][rank], t["i"][rank], t["j"][h]))
    return out


@pytest.mark.parametrize("rows,cols", SHAPES)
def test_symmetric_product_tables_cover_the_upper_triangle_once(rows, cols, tile_mode):
    m = min(rows, cols)
    nb = blocks(m)
    for which in (0, 1):
        tiles, unit = b.muon_debug_tile_table(rows, cols, which)
        if which == 1:
            assert unit == 1
            if not tiles:  # single-matrix units need no table for a last matrix alone
                assert b.muon_debug_tile_table(rows, cols, 0)[1] == 1
                continue
            unit_here = 1
        else:
            # matrices pair up only to share their lone diagonal blocks: an odd number of row blocks
            assert unit == (2 if nb % 2 == 1 and not tile_mode & 2 else 1) and tiles
            unit_here = unit
        seen = {}
        for t in tiles:
            assert t["nbw"] in (1, 2)
            assert bool(t["half"]) <= bool(tile_mode & 2)
            # layout rule for symmetric operands: neighbours or equal, on both sides
            assert abs(t["i"][0] - t["i"][1]) <= 1
            if t["nbw"] == 2:
                assert abs(t["j"][0] - t["j"][1]) <= 1
            assert all(k >> t["nbw"] == 0 for k in t["keep"]), t
            for (d, i, j) in stored_blocks(t):
                assert 0 <= d < unit_here
                if i >= nb:
                    continue  # rows beyond the matrix: the kernel stores nothing for them
                assert j < nb and i <= j, t  # on or above the diagonal, inside the matrix
                seen[(d, i, j)] = seen.get((d, i, j), 0) + 1
        want = {(d, i, j) for d in range(unit_here) for i in range(nb) for j in range(i, nb)}
        assert set(seen) == want
        assert all(c == 1 for c in seen.values())


@pytest.mark.parametrize("rows,cols", SHAPES)
def test_combine_tables_cover_the_output_once(rows, cols, tile_mode):
    m, n = min(rows, cols), max(rows, cols)
    for which, out_rows, out_cols in ((2, m, n), (3, n, m)):
        tiles, unit = b.muon_debug_tile_table(rows, cols, which)
        assert unit == 1
        rb, cb = blocks(out_rows), blocks(out_cols)
        seen = {}
        for t in tiles:
            assert t["dm"] == (0, 0)
            if t["half"]:
                assert tile_mode & 1 and t["i"][0] == rb - 1 and rb % 2 == 1  # only the row block without a partner
            else:
                assert t["i"][1] == t["i"][0] + 1  # the symmetric operand's rows (or X^T's): neighbours
                assert not (tile_mode & 1 and t["i"][1] >= rb)
            assert len(stored_blocks(t)) == (1 if t["half"] else 2) * t["nbw"]
            for (d, i, j) in stored_blocks(t):
                assert j < cb
                if i < rb:
                    seen[(i, j)] = seen.get((i, j), 0) + 1
        assert set(seen) == {(i, j) for i in range(rb) for j in range(cb)}
        assert all(c == 1 for c in seen.values())
    assert len(b.muon_debug_tile_table(rows, cols, 2)[0]) == len(b.muon_debug_tile_table(rows, cols, 3)[0])


def test_executed_work_follows_the_tables():
    """muon_plan_work: planned FLOPs add up to muon_plan_flops' figure, executed
    FLOPs are the tiles' (256 rows x 128 or 256 columns x the contraction length
    in whole 64-element stages)."""
    shapes = [(1408, 2048, 7), (2048, 2048, 3), (100, 300, 5)]
    for ns in (1, 5, 10):
        planned, executed = b.muon_plan_work(shapes, ns)
        alg, planned_total = b.muon_plan_flops(shapes, ns)
        assert abs(sum(planned.values()) - planned_total) <= 1e-9 * planned_total
        for kind in ("gram", "poly", "comb"):
            assert executed[kind] >= planned[kind] > 0
        assert executed["momentum"] == executed["norm"] == executed["update"] == 0
    # one expert-shaped bucket of 7 matrices, by hand from the tables
    prev = b.muon_debug_set_tile_mode(0)
    try:
        for mode in (0, 3):
            b.muon_debug_set_tile_mode(mode)
            planned, executed = b.muon_plan_work([(1408, 2048, 7)], 1)
            unit, mats = b.muon_debug_tile_table(1408, 2048, 0)
            tail, _ = b.muon_debug_tile_table(1408, 2048, 1)
            comb, _ = b.muon_debug_tile_table(1408, 2048, 2)
            per = lambda tiles, k: sum(2.0 * (128 if t["half"] else 256) * 128 * t["nbw"] * k for t in tiles)
            units, left = divmod(7, mats)
            assert executed["gram"] == units * per(unit, 2048) + left * per(tail, 2048)
            assert executed["poly"] == units * per(unit, 1408) + left * per(tail, 1408)
            assert executed["comb"] == 7 * per(comb, 1408)
            assert planned["gram"] == 7 * 1408.0 ** 2 * 2048 and planned["comb"] == 2 * planned["gram"]
            if mode == 3:  # nothing computed in vain but the lower halves of the diagonal blocks
                assert executed["comb"] == planned["comb"]
                assert abs(executed["gram"] / planned["gram"] - 66 / 60.5) < 1e-12
    finally:
        b.muon_debug_set_tile_mode(prev)


def test_expert_shape_tables_have_the_expected_sizes():
    """1408 rows are 11 row blocks: 15 full tiles per matrix and six diagonal
    blocks.  Default (mode 1): the six pair up with the neighbour matrix's (36
    tiles per two matrices; a matrix alone takes them as six half-width tiles),
    and the combine's eleventh row block is eight half-height tiles.  Mode 3:
    each of the six is a half-height, half-width tile of its own matrix."""
    assert b.muon_debug_set_tile_mode(-1) == 1  # query only
    unit, mats = b.muon_debug_tile_table(2048, 1408, 0)
    assert mats == 2 and len(unit) == 36 and all(t["nbw"] == 2 and not t["half"] for t in unit)
    shared = [t for t in unit if t["dm"] == (0, 1)]
    assert len(shared) == 6 and all(t["i"][0] == t["i"][1] == t["j"][0] == t["j"][1] for t in shared)
    assert all(t["keep"] == (1, 2) for t in shared)
    tail, _ = b.muon_debug_tile_table(2048, 1408, 1)
    assert len(tail) == 21 and sum(1 for t in tail if t["nbw"] == 1) == 6
    comb, _ = b.muon_debug_tile_table(2048, 1408, 2)
    assert len(comb) == 48 and sum(1 for t in comb if t["half"]) == 8
    prev = b.muon_debug_set_tile_mode(3)
    try:
        unit, mats = b.muon_debug_tile_table(2048, 1408, 0)
        assert mats == 1 and len(unit) == 21
        assert sum(1 for t in unit if t["half"]) == 6 and all(t["nbw"] == 1 for t in unit if t["half"])
    finally:
        b.muon_debug_set_tile_mode(prev)


def test_an_even_number_of_row_blocks_needs_no_lone_tiles():
    """2048 rows = 16 row blocks: 36 full tiles, eight of which hold a block
    under the diagonal that is dropped; single-matrix units."""
    tiles, mats = b.muon_debug_tile_table(2048, 2048, 0)
    assert mats == 1 and len(tiles) == 36 and all(t["nbw"] == 2 and not t["half"] for t in tiles)
    assert sum(1 for t in tiles if t["keep"] == (3, 2)) == 8


@pytest.mark.parametrize("rows,cols,count,expect_tiles,width", [(1024, 1024, 1, 36, 1), (2048, 2048, 1, 72, 2),
                                                                 (512, 512, 1, 10, 1), (1408, 2048, 1, 66, 1)])
def test_few_small_matrices_are_cut_into_finer_tiles(rows, cols, count, expect_tiles, width):
    """A launch with fewer full tiles than the GPU has CTA pairs would leave SMs
    idle: the symmetric products of such a bucket take every row block on its
    own at half height, or block by block; coverage stays exact, and the same
    shapes in a large bucket keep full tiles."""
    nb = blocks(min(rows, cols))
    tiles, mats = b.muon_debug_tile_table(rows, cols, 0, count)
    assert mats == 1 and len(tiles) == expect_tiles and all(t["half"] for t in tiles)
    assert max(t["nbw"] for t in tiles) == width
    seen = sorted((i, j) for t in tiles for (_, i, j) in stored_blocks(t))
    assert seen == [(i, j) for i in range(nb) for j in range(i, nb)]
    for t in tiles:
        assert t["nbw"] == 1 or t["j"][1] == t["j"][0] + 1
    big, _ = b.muon_debug_tile_table(rows, cols, 0, 512)
    assert not any(t["half"] for t in big)
    prev = b.muon_debug_set_tile_mode(1 | 4)  # the finer cut switched off
    try:
        coarse, _ = b.muon_debug_tile_table(rows, cols, 1 if nb % 2 else 0, count)
        assert not any(t["half"] for t in coarse)
    finally:
        b.muon_debug_set_tile_mode(prev)
