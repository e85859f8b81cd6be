"""Pins of the oracle's head aggregation (sum of a feature's activations over the heads, then Top-k): a hand example,
one head as the identity, and exactly representable sums against a dense scatter-add + full sort."""
import numpy as np

import oracle as O


def test_hand_example():
    # two heads, k = 3. feature 5: 1.0 + 2.0 = 3.0; feature 2: 2.5; feature 9: 0.5 + 0.25 = 0.75; feature 7: 3.0
    ids = np.array([[[5, 2, 9], [7, 5, 9]]], np.int32)
    vals = np.array([[[1.0, 2.5, 0.5], [3.0, 2.0, 0.25]]], np.float32)
    oi, ov = O.head_aggregate(ids, vals, 3)
    assert oi.tolist() == [[5, 7, 2]]            # 3.0 (id 5) before 3.0 (id 7): equal sums, lower id first; then 2.5
    assert ov.tolist() == [[3.0, 3.0, 2.5]]
    oi, ov = O.head_aggregate(ids, vals, 6)
    assert oi.tolist() == [[5, 7, 2, 9, -1, -1]] and ov.tolist() == [[3.0, 3.0, 2.5, 0.75, 0.0, 0.0]]


def test_single_head_is_the_identity_on_sorted_rows():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, 16)).astype(np.float32)
    W = rng.standard_normal((16, 40)).astype(np.float32)
    ids, vals = O.encode_topk(x, W, np.zeros(40, np.float32), np.zeros(16, np.float32), 5)
    oi, ov = O.head_aggregate(ids[:, None, :], vals[:, None, :], 5)
    np.testing.assert_array_equal(oi, ids)
    np.testing.assert_array_equal(ov, vals)
    oi3, _ = O.head_aggregate(ids[:, None, :], vals[:, None, :], 3)
    np.testing.assert_array_equal(oi3, ids[:, :3])


def test_against_dense_scatter_add_and_sort():
    rng = np.random.default_rng(1)
    T, H, k, D, k_out = 20, 8, 6, 30, 10
    ids = np.stack([np.stack([rng.permutation(D)[:k] for _ in range(H)]) for _ in range(T)]).astype(np.int32)
    vals = rng.integers(1, 64, size=(T, H, k)).astype(np.float32) / 8      # multiples of 1/8: every sum is exact
    ids[0, 0, 3:] = -1
    oi, ov = O.head_aggregate(ids, vals, k_out)
    for t in range(T):
        dense = np.zeros(D)
        for h in range(H):
            for j in range(k):
                if ids[t, h, j] >= 0:
                    dense[ids[t, h, j]] += vals[t, h, j]
        order = np.lexsort((np.arange(D), -dense))                        # by sum descending, then id ascending
        order = [f for f in order if dense[f] > 0][:k_out]
        assert oi[t, :len(order)].tolist() == order
        assert ov[t, :len(order)].tolist() == [dense[f] for f in order]
        assert (oi[t, len(order):] == -1).all()
