"""Host-side work decomposition of the tensor-core kernels, checked without a GPU.

Whatever tile shapes and splits the planners choose, the work items must cover every
(matrix, 128-row tile, 64-column step) of the compression and every (matrix, 128-row tile, column slab) of the
decompression exactly once, stay inside the matrices, respect the hardware limits the kernels rely on
(tensor-memory columns, shared memory, cluster size) and carry a consistent ownership flag.
"""
import collections

import pytest

from paper_2402_03293_b200 import binding as fb
from paper_2402_03293_b200 import workloads as wl

SMEM_LIMIT = 227 * 1024
SHAPE_SETS = {
    "gpt2_small_set": wl.WORKLOADS["gpt2_small_set"].shapes,
    "t5_large_set": wl.WORKLOADS["t5_large_set"].shapes,
    "single": wl.WORKLOADS["single_bf16_4096x11008"].shapes,
    "gpt2_xl_block": wl.WORKLOADS["gpt2_xl_set"].shapes[:8],
    "ragged": ((130, 70), (1000, 515), (257, 4097), (128, 64), (4000, 129)),
    "many": tuple((128 + 128 * (i % 3), 64 + 64 * (i % 5)) for i in range(460)),     # more matrices than one launch carries seeds for
}
RANKS = (8, 32, 64, 100, 128, 192, 256)


def tiles_of(n):
    return (n + 127) // 128


@pytest.mark.parametrize("name", sorted(SHAPE_SETS))
@pytest.mark.parametrize("r", RANKS)
def test_compression_items_cover_every_tile_and_step_once(name, r):
    shapes = SHAPE_SETS[name]
    items, (T, S, gstages, astages, gen_warps, teams, launches, smem) = fb.flora_debug_plan(shapes, r, "compress")
    # accumulator columns: r rounded up to 16, or to 64 for the ranks that run on CTA pairs
    r_pad = (r + 15) // 16 * 16 if r <= 64 else (r + 63) // 64 * 64
    assert 1 <= T and T * r_pad <= 512                         # accumulators fit tensor memory
    assert S in (1, 2, 4, 8) and r_pad % (8 * S) == 0          # portable cluster sizes; whole 8-row groups per CTA
    assert r <= 64 or S >= 2                                   # pairs
    assert gstages >= 1 and astages >= 1 and smem <= SMEM_LIMIT
    assert 1 <= teams <= astages and gen_warps % teams == 0
    assert launches == (len(shapes) + 447) // 448
    assert len(items) % S == 0
    seen = collections.Counter()
    split = collections.defaultdict(set)
    for g0 in range(0, len(items), S):
        group = items[g0:g0 + S]
        mat, _, _, k0, ks, direct = group[0]
        n, m = shapes[mat]
        steps = (m + 63) // 64
        assert ks >= 1 and 0 <= k0 and k0 + ks <= steps
        split[mat].add((k0, ks))
        row = group[0][1]
        for (mt, row0, tl, kk0, kks, dr) in group:             # the CTAs of a cluster: same matrix and columns, consecutive rows
            assert (mt, kk0, kks, dr) == (mat, k0, ks, direct)
            assert 0 <= tl <= T and row0 % 128 == 0
            assert row0 == row or tl == 0
            row += tl * 128
            for t in range(tl):
                assert row0 // 128 + t < tiles_of(n)
                for k in range(k0, k0 + ks):
                    seen[(mat, row0 // 128 + t, k)] += 1
        assert any(tl > 0 for (_, _, tl, _, _, _) in group)
    expected = sum(tiles_of(n) * ((m + 63) // 64) for n, m in shapes)
    assert len(seen) == expected and all(v == 1 for v in seen.values())
    for (mat, _, _, k0, ks, direct) in items:                  # an item owns its rows iff the matrix is not cut along the columns
        assert direct == (1 if len(split[mat]) == 1 else 0)


@pytest.mark.parametrize("name", sorted(SHAPE_SETS))
@pytest.mark.parametrize("r", RANKS)
def test_persistent_compression_slots_partition_the_units(name, r):
    """Ranks above 64: every launch lists, per cluster slot, a contiguous non-empty range of its units; together the
    ranges cover the launch's units once, and no launch asks for more clusters than 148 SMs could hold."""
    shapes = SHAPE_SETS[name]
    items, (T, S, *_rest, launches, _smem) = fb.flora_debug_plan(shapes, r, "compress")
    table, _ = fb.flora_debug_plan(shapes, r, "compress_slots")
    table = [t[0] for t in table]
    if r <= 64:
        assert table == []
        return
    units_total = len(items) // S
    covered, pos = 0, 0
    for _ in range(launches):
        assert table[pos] == 0
        end = pos + 1
        while end < len(table) and table[end] > table[end - 1]:
            end += 1
        begins = table[pos:end]
        assert len(begins) >= 2 and len(begins) - 1 <= 148 // S
        covered += begins[-1]
        pos = end
    assert pos == len(table) and covered == units_total


@pytest.mark.parametrize("name", sorted(SHAPE_SETS))
@pytest.mark.parametrize("r", RANKS)
def test_decompression_items_cover_every_tile_of_every_slab_once(name, r):
    shapes = SHAPE_SETS[name]
    items, (bn, slots, cstages, nslabs, gen_warps, bf16, launches, smem) = fb.flora_debug_plan(shapes, r, "decompress")
    assert bn in (64, 128) and slots >= 1 and cstages >= 1 and nslabs in (1, 2) and smem <= SMEM_LIMIT
    assert bf16 == (1 if r > 64 else 0)
    assert launches == (len(shapes) + 447) // 448
    seen = collections.Counter()
    for (mat, col0, row0, tl) in items:
        n, m = shapes[mat]
        assert col0 % bn == 0 and 0 <= col0 < m and row0 % 128 == 0 and tl >= 0      # (tl == 0: padding of a CTA's list)
        for t in range(tl):
            assert row0 // 128 + t < tiles_of(n)
            seen[(mat, row0 // 128 + t, col0 // bn)] += 1
    expected = sum(tiles_of(n) * ((m + bn - 1) // bn) for n, m in shapes)
    assert len(seen) == expected and all(v == 1 for v in seen.values())


def test_launches_hold_consecutive_matrices():
    """Seeds travel per launch as a table of 448: a launch's items must stay inside one window of 448 matrices."""
    shapes = SHAPE_SETS["many"]
    for which in ("compress", "decompress"):
        items, _ = fb.flora_debug_plan(shapes, 32, which)
        mats = [it[0] for it in items]
        cut = next(i for i, mt in enumerate(mats) if mt >= 448)
        assert all(mt < 448 for mt in mats[:cut]) and all(mt >= 448 for mt in mats[cut:])


def test_plan_rejects_bad_arguments():
    with pytest.raises(RuntimeError):
        fb.flora_debug_plan([(128, 64)], 0, "compress")
    with pytest.raises(RuntimeError):
        fb.flora_debug_plan([(128, 64)], 257, "decompress")
    items, _ = fb.flora_debug_plan([], 8, "compress")
    assert items == []
