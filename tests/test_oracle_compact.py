"""Pins of the oracle's compact (block-delta, bit-packed) index encoding (Sec. 3.4: contiguous integer arrays with
delta encoding and optional stop-feature pruning): a hand-packed example, closed-form sizes, the round trip through the
independently written decoder, and pruning against a direct filter."""
import numpy as np

import oracle as O


def _csr(lists):
    rp = np.cumsum([0] + [len(l) for l in lists]).astype(np.uint64)
    pos = np.array([p for l in lists for p in l], dtype=np.int32)
    return rp, pos


def test_hand_packed_example():
    # feature 0: positions 5, 6, 9, 20: gaps-1 = 0, 2, 10 -> width 4, bits 0000 | 0010<<4 | 1010<<8 = 0xA20, one word
    # feature 1: empty;  feature 2: a single posting 7 -> width 0, no payload
    c = O.compact_encode(*_csr([[5, 6, 9, 20], [], [7]]))
    assert c["row_ptr"].tolist() == [0, 4, 4, 5]
    assert c["blk_ptr"].tolist() == [0, 1, 1, 2]
    assert c["blk_first"].tolist() == [5, 7]
    assert c["blk_desc"].tolist() == [(0 << 6) | 4, (1 << 6) | 0]
    assert c["payload"].tolist() == [0xA20, 0]


def test_value_straddling_a_word():
    # 12 postings with gaps-1 = 1, 2, ..., 11 at width 4 -> 44 bits: value 9 (index 8) sits in bits 32..35
    p = np.cumsum([0] + [g + 1 for g in range(1, 12)]).tolist()
    c = O.compact_encode(*_csr([p]))
    assert c["blk_desc"].tolist() == [4]
    want = sum(g << (4 * i) for i, g in enumerate(range(1, 12)))
    assert c["payload"].tolist() == [want & 0xFFFFFFFF, want >> 32, 0]


def test_closed_form_sizes():
    # 100 consecutive positions: gaps-1 all zero -> width 0 in 4 blocks, no payload words
    c = O.compact_encode(*_csr([list(range(1000, 1100))]))
    assert c["blk_ptr"].tolist() == [0, 4] and (c["blk_desc"] == 0).all() and c["payload"].tolist() == [0]
    assert c["blk_first"].tolist() == [1000, 1032, 1064, 1096]
    # constant gap g: width = bit length of g - 1; a full block stores 31 values
    for g, w in [(2, 1), (3, 2), (512, 9), (513, 10)]:
        c = O.compact_encode(*_csr([list(range(0, 64 * g, g))]))
        assert [int(d) & 63 for d in c["blk_desc"]] == [w, w]
        assert len(c["payload"]) - 1 == 2 * ((31 * w + 31) // 32)
        assert int(c["blk_desc"][1]) >> 6 == (31 * w + 31) // 32
    # the gap between blocks is not stored: a huge jump across a block border costs nothing
    c = O.compact_encode(*_csr([list(range(32)) + [2**31 - 1]]))
    assert [int(d) & 63 for d in c["blk_desc"]] == [0, 0] and c["blk_first"].tolist() == [0, 2**31 - 1]
    # the widest value: positions 0 and 2^31 - 1 inside one block -> width 31
    c = O.compact_encode(*_csr([[0, 2**31 - 1]]))
    assert c["blk_desc"].tolist() == [31] and c["payload"].tolist() == [2**31 - 2, 0]


def test_round_trip_and_pruning():
    rng = np.random.default_rng(3)
    lists = []
    for f in range(60):
        n = int(rng.choice([0, 1, 2, 31, 32, 33, 64, 65, 200]))
        lists.append(np.sort(rng.choice(1 << int(rng.integers(8, 22)), size=n, replace=False)).tolist())
    rp, pos = _csr(lists)
    for stop in (0, 40):
        c = O.compact_encode(rp, pos, stop)
        want_rp, want_pos = O.prune_stop_features(rp, pos, stop)
        got_rp, got_pos = O.compact_decode(c)
        np.testing.assert_array_equal(got_rp, want_rp)
        np.testing.assert_array_equal(got_pos, want_pos)
    kept = [l if len(l) <= 40 else [] for l in lists]                  # direct filter
    np.testing.assert_array_equal(O.prune_stop_features(rp, pos, 40)[1], _csr(kept)[1])
    assert c["payload"][-1] == 0 and len(c["blk_first"]) == sum((len(l) + 31) // 32 for l in kept)
