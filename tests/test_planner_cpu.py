"""Host logic of the tensor-core kernel's static schedule, checked without a GPU.

The schedule decides which CTA computes which (token rows x vocabulary rows) tile; a hole or an
overlap in it would silently drop or double-count logits.  The library exposes the schedule it
would use (the same function the device code calls) and these tests check its invariants."""
import numpy as np
import pytest

import paper_2504_07878_b200 as P

SHAPES = [(1, 151936), (16, 151936), (64, 128256), (128, 151936), (129, 151936), (256, 151936), (300, 3001),
          (512, 128256), (4096, 151936), (8192, 151936), (16384, 128256), (7, 5), (200, 33), (1000, 17), (256, 257)]


@pytest.mark.parametrize("n,V", SHAPES)
def test_tiles_cover_every_logit_exactly_once(n, V):
    tiles, plan = P.tlr_debug_plan_tiles(n, V, 148)
    g = plan.reserved
    cta = 2 if n > 128 else 1
    assert g % (16 * cta) == 0
    assert plan.grid <= 148 and plan.grid % cta == 0 and 1 <= plan.vocab_chunks <= 192
    rows_per_unit = 128 * cta
    assert plan.row_units == -(-n // rows_per_unit)
    assert np.all(tiles[:, 4] > 0) and np.all(tiles[:, 4] <= 256) and np.all(tiles[:, 4] % g == 0)
    assert np.all(tiles[:, 3] % 16 == 0)
    # per row unit, the tiles' vocabulary ranges tile [0, ceil(V/g)*g) with no gap and no overlap
    for ru in range(plan.row_units):
        sel = tiles[tiles[:, 2] == ru * rows_per_unit]
        order = np.argsort(sel[:, 3])
        v0, rows = sel[order, 3], sel[order, 4]
        assert v0[0] == 0
        assert np.array_equal(v0[1:], (v0 + rows)[:-1])
        end = v0[-1] + rows[-1]
        assert V <= end < V + g
    # a unit belongs to one worker, and a worker walks a unit's tiles in ascending vocabulary order
    for unit in np.unique(tiles[:, 1]):
        sel = tiles[tiles[:, 1] == unit]
        assert len(np.unique(sel[:, 0])) == 1
        assert np.all(np.diff(sel[:, 3]) > 0)
    # units of one chunk are consecutive numbers (chunk-major order)
    assert np.array_equal(np.unique(tiles[:, 1]), np.arange(plan.vocab_chunks * plan.row_units))


def test_decode_plans_are_balanced_and_use_full_tiles_in_pair_mode():
    tiles, plan = P.tlr_debug_plan_tiles(256, 151936, 148)
    per_worker = np.bincount(tiles[:, 0], weights=tiles[:, 4])
    assert per_worker.max() <= 1.02 * per_worker.mean()          # rows per worker within 2 %
    counts = np.bincount(tiles[:, 0])
    assert counts.max() - counts.min() <= 1
    assert (tiles[:, 4] == 256).mean() > 0.95                    # full-width tiles, plus a few remainders
    tiles, plan = P.tlr_debug_plan_tiles(16, 151936, 148)
    per_worker = np.bincount(tiles[:, 0], weights=tiles[:, 4])
    assert plan.grid >= 146 and per_worker.max() <= 1.02 * per_worker.mean()
    assert len(set(np.bincount(tiles[:, 0]).tolist())) == 1      # every worker walks the same number of tiles


def test_plan_argument_errors():
    import ctypes
    lib = P.load_library()
    c = ctypes.c_int32(0)
    assert lib.tlr_debug_plan_tiles(0, 100, 148, 0, None, 0, ctypes.byref(c), None) == 1
    assert lib.tlr_debug_plan_tiles(10, 100, 148, 0, None, 5, ctypes.byref(c), None) == 1
    assert lib.tlr_debug_plan_tiles(10, 100, 148, -1, None, 0, ctypes.byref(c), None) == 1


@pytest.mark.parametrize("n,V,hidden", [(16, 151936, 256), (256, 151936, 256), (300, 3001, 96), (8192, 151936, 256),
                                        (64, 128256, 1000), (129, 5000, 40), (4096, 151936, 1024)])
def test_learned_router_units_follow_the_vocabulary_units(n, V, hidden):
    """With a learned router inside the launch its first layer's rows (reported as vocabulary rows V ..) are
    walked once per row unit, by units numbered after all vocabulary units, and the vocabulary is still
    covered exactly once."""
    tiles, plan = P.tlr_debug_plan_tiles(n, V, 148, hidden)
    g = plan.reserved
    cta = 2 if n > 128 else 1
    rows_per_unit = 128 * cta
    vocab_units = plan.vocab_chunks * plan.row_units
    assert np.array_equal(np.unique(tiles[:, 1]), np.arange(vocab_units + plan.row_units))
    router = tiles[tiles[:, 1] >= vocab_units]
    vocab = tiles[tiles[:, 1] < vocab_units]
    assert np.all(vocab[:, 3] + vocab[:, 4] <= -(-V // g) * g) and np.all(router[:, 3] >= V)
    padded = -(-hidden // (16 * cta)) * (16 * cta)
    for ru in range(plan.row_units):
        sel = router[router[:, 2] == ru * rows_per_unit]
        assert len(np.unique(sel[:, 1])) == 1                      # one unit per row unit
        order = np.argsort(sel[:, 3])
        v0, rows = sel[order, 3] - V, sel[order, 4]
        assert v0[0] == 0 and np.array_equal(v0[1:], (v0 + rows)[:-1]) and v0[-1] + rows[-1] == padded
        assert np.all(rows % (16 * cta) == 0) and np.all(rows <= 256)
        sel = vocab[vocab[:, 2] == ru * rows_per_unit]
        order = np.argsort(sel[:, 3])
        v0, rows = sel[order, 3], sel[order, 4]
        assert v0[0] == 0 and np.array_equal(v0[1:], (v0 + rows)[:-1]) and V <= v0[-1] + rows[-1] < V + g
    assert plan.grid <= 148


def test_learned_router_costs_the_decode_plans_little():
    """The busiest worker of the decode plans carries at most 3 % more rows with a 256-wide router inside."""
    for n in (16, 256):
        plain, _ = P.tlr_debug_plan_tiles(n, 151936, 148)
        fused, _ = P.tlr_debug_plan_tiles(n, 151936, 148, 256)
        a = np.bincount(plain[:, 0], weights=plain[:, 4]).max()
        b = np.bincount(fused[:, 0], weights=fused[:, 4]).max()
        assert b <= 1.03 * a


@pytest.mark.parametrize("n,V", [(256, 151936), (512, 128256), (1024, 151936), (4096, 151936), (8192, 151936),
                                 (4096, 128256), (16384, 128256)])
def test_pair_mode_minimises_the_busiest_workers_tile_passes(n, V):
    """With a CTA pair per worker a tile costs a pass over h whatever its width, so the plan must give the busiest
    worker as few tiles as any chunk count (up to the 192 partials a row may have) allows."""
    tiles, plan = P.tlr_debug_plan_tiles(n, V, 148)
    workers, g = plan.grid // 2, plan.reserved
    busiest = np.bincount(tiles[:, 0]).max()
    row_units, granules = -(-n // 256), -(-V // g)
    fewest = min(-(-row_units * c // 74) * -(-(-(-granules // c) * g) // 256) for c in range(1, 193))
    assert workers <= 74 and busiest == fewest
