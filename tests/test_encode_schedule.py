"""The encode launch's work units (host arithmetic of the library, no GPU): every 256-column tile of every 256-token row
tile of every item is covered exactly once, pieces of one row tile go to distinct candidate lists, the pairs' modelled
loads are even, and the scratch bound that callers size their workspace with holds the schedule at any shorter length."""
import numpy as np
import pytest

import paper_2601_17702_b200.binding as B

PAIRS = 74          # a 148-SM device


def _tiles(T, d_sae):
    return (T + 255) // 256, (d_sae + 255) // 256


def _check_cover(items, units, slots):
    for i, (T, d_in, d_sae, k) in enumerate(items):
        n_rows, nct = _tiles(T, d_sae)
        cover = np.zeros((n_rows, nct), dtype=np.int32)
        seen = set()
        for pr, it, mt, lo, hi, slot in units[units[:, 1] == i].tolist():
            assert 0 <= lo < hi <= nct and 0 <= mt < n_rows and hi - lo <= 255
            cover[mt, lo:hi] += 1
            assert (mt, slot) not in seen and 0 <= slot < slots[i]
            seen.add((mt, slot))
        assert (cover == 1).all()


def _tile_cost(items, d_in, k):
    # the library's model of a 256-column tile, in SM cycles: its MMAs or its Top-k filter (two epilogue groups when no
    # encoder of the launch is wider than 1024), whichever takes longer
    return max(600.0 * ((d_in + 63) // 64), (12000.0 + 100.0 * k) / (1.5 if max(x[1] for x in items) <= 1024 else 1.0))


def _loads(items, units, n_pairs):
    load = np.zeros(n_pairs)
    for pr, it, mt, lo, hi, slot in units.tolist():
        d_in, k = items[it][1], items[it][3]
        load[pr] += 5000.0 + 100.0 * k + (hi - lo) * _tile_cost(items, d_in, k)
    return load


@pytest.mark.parametrize("items", [
    [(8192, 1024, 16384, 32)],                                   # one key encoder, one chunk: 32 row tiles on 74 pairs
    [(8192, 1024, 16384, 32)] * 4,                               # the four layers' key encoders in one launch
    [(16384, 1024, 16384, 64)],                                  # retrieval queries through the key encoder
    [(16384, 512, 8192, 16)] * 3,                                # three narrow layers: 192 row tiles, 2.6 per pair
    [(4096, 1024, 16384, 32)],
    [(8000, 1024, 16384, 32), (300, 512, 8192, 16), (8192, 128, 16384, 32)],     # unequal items, ragged row tiles
    [(2048, 1024, 16384, 32)],                                   # eight row tiles: seven tiles per pair
    [(65536, 128, 16384, 32)],
])
def test_balanced_units_cover_every_tile_once_and_load_the_pairs_evenly(items):
    units, slots = B.s3_encode_schedule_describe(items, PAIRS)
    assert units is not None
    _check_cover(items, units, slots)
    assert (np.diff(units[:, 0]) >= 0).all()                     # stored pair by pair
    load = _loads(items, units, PAIRS)
    busy = load[load > 0]
    total_tiles = sum(_tiles(T, d)[0] * _tiles(T, d)[1] for T, _, d, _ in items)
    if total_tiles >= 8 * PAIRS:
        assert len(busy) == PAIRS
        tile = max(_tile_cost(items, d_in, k) for _, d_in, _, k in items)
        assert busy.max() <= max(1.08 * busy.mean(), busy.mean() + 3.0 * tile), (busy.max(), busy.mean())   # whole tiles, whole pieces
    for i, (T, d_in, d_sae, k) in enumerate(items):
        assert slots[i] <= min(16, 4 + -(-PAIRS // _tiles(T, d_sae)[0]))


def test_wide_encoder_walks_bands_of_row_tiles_with_its_slices_in_step():
    # 4096 -> 32768: 268 MB of weights, far more than L2. Its row tiles are not cut at shares; bands of row tiles are swept
    # by uniform column slices, one unit per pair, so the pairs of a slice read the same weight tiles at the same time
    # and a band's token tiles (18 x 2 MB) stay in L2. Each band has its own slice count.
    item = (8192, 4096, 32768, 64)
    units, slots = B.s3_encode_schedule_describe([item], PAIRS)
    assert units is not None and slots[0] == 5 and len(units) == 18 * 4 + 14 * 5
    _check_cover([item], units, slots)
    first, second = units[units[:, 2] < 18], units[units[:, 2] >= 18]
    assert set((lo, hi) for _, _, _, lo, hi, _ in first.tolist()) == {(0, 32), (32, 64), (64, 96), (96, 128)}      # 18 row tiles x 4 slices
    assert len(set((lo, hi) for _, _, _, lo, hi, _ in second.tolist())) == 5 and (second[:, 4] - second[:, 3]).max() == 26
    assert len(np.unique(first[:, 0])) == 72 and len(np.unique(second[:, 0])) == 70            # one unit per pair and band
    tiles = np.bincount(units[:, 0], weights=units[:, 4] - units[:, 3], minlength=PAIRS)
    assert tiles.max() == 58 and (tiles > 0).all()                                             # 64 with two bands of 16 x 4
    for pr in range(PAIRS):
        mine = units[units[:, 0] == pr]
        assert len(mine) <= 2 and (np.diff(mine[:, 2]) > 0).all()                              # band 0's unit first
    # 37 row tiles: two slices over all of them keep every pair busy (74 units of 64 tiles); bands of four slices would take 96
    units, slots = B.s3_encode_schedule_describe([(9472, 4096, 32768, 64)], PAIRS)
    assert slots[0] == 2 and len(units) == 74 and np.bincount(units[:, 0]).max() == 1
    # few row tiles: more slices, one band
    units, slots = B.s3_encode_schedule_describe([(2048, 4096, 32768, 64)], PAIRS)
    assert slots[0] == 9 and len(units) == 72
    # two wide items in one launch: uniform slices, dealt out by table
    both = [(8192, 4096, 32768, 64), (4096, 4096, 32768, 64)]
    units, slots = B.s3_encode_schedule_describe(both, PAIRS)
    assert units is not None
    _check_cover(both, units, slots)
    for i in (0, 1):
        mine = units[units[:, 1] == i]
        assert len(set((lo, hi) for _, _, _, lo, hi, _ in mine.tolist())) == slots[i]      # the same slices in every row tile


def test_whole_row_tiles_that_fill_the_waves_are_not_cut():
    # 8 layers x 64 row tiles = 512 units in 7 waves of 74 (98.8 % full): every unit is a whole row tile, dealt by table
    items = [(16384, 512, 8192, 16)] * 8
    units, slots = B.s3_encode_schedule_describe(items, PAIRS)
    assert units is not None and len(units) == 512 and (slots == 1).all()
    _check_cover(items, units, slots)
    assert ((units[:, 3] == 0) & (units[:, 4] == 32)).all()
    per_pair = np.bincount(units[:, 0], minlength=PAIRS)
    assert per_pair.max() == 7 and per_pair.min() == 6


def test_one_row_tile_falls_back_to_sixteen_uniform_slices():
    # 64 column tiles cannot be cut into 74 pieces of at least three within 16 lists per row
    units, slots = B.s3_encode_schedule_describe([(256, 1024, 16384, 32)], PAIRS)
    assert units is None and slots[0] == 16


def test_few_pairs_and_invalid_queries():
    units, slots = B.s3_encode_schedule_describe([(8192, 1024, 16384, 32)], 10)
    _check_cover([(8192, 1024, 16384, 32)], units, slots)
    assert units[:, 0].max() == 9
    units, slots = B.s3_encode_schedule_describe([(100, 128, 256, 4)], PAIRS)            # a single tile
    assert len(units) == 1 and units[0].tolist() == [0, 0, 0, 0, 1, 0]
    with pytest.raises(ValueError):
        B.s3_encode_schedule_describe([(0, 128, 256, 4)], PAIRS)
    with pytest.raises(ValueError):
        B.s3_encode_schedule_describe([(100, 128, 256, 4)], 0)


def test_lists_of_a_shorter_chunk_fit_the_bound_of_the_full_chunk():
    # T * slots(T) stays within 5 T + 256 pairs (capped at 16 T), which grows with T
    for d_in, d_sae, k in [(1024, 16384, 32), (512, 8192, 16), (128, 16384, 32)]:
        for T_full in (4096, 8192, 16384):
            bound = min(16 * T_full, 5 * T_full + 256 * PAIRS)
            for T in (1, 255, 256, 257, 1000, 2048, 3000, T_full // 2 + 1, T_full - 1, T_full):
                _, slots = B.s3_encode_schedule_describe([(T, d_in, d_sae, k)], PAIRS)
                assert T * int(slots[0]) <= bound, (T, slots, bound)
