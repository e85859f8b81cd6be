"""Pins of the oracle's index-set union (Sec. 3.6, Eq. 7: M_S3 U M_BM25 U M_Bias): a hand-worked example,
closed-form sizes for disjoint and fully overlapping parts, and invariants."""
import numpy as np

import oracle as O


def test_hand_example():
    # L = 40, window 6 around centres 10 and 13 ([7,13) U [10,16) = 7..15), lexical {3, 14, 39, 50(ignored), -1(pad)},
    # lead 2 (0, 1), tail 3 (37, 38, 39)
    got = O.fuse_index_sets([[10, 13, -1]], 6, [[3, 14, 39, 50, -1]], 2, 3, 40)
    assert got[0].tolist() == [0, 1, 3, 7, 8, 9, 10, 11, 12, 13, 14, 15, 37, 38, 39]


def test_closed_form_sizes():
    L, w = 1000, 10
    centers = np.array([[100, 200, 300, 400]])           # disjoint windows, away from the borders
    lex = np.array([[50, 60, 70]])                       # disjoint from everything else
    got = O.fuse_index_sets(centers, w, lex, 5, 7, L)[0]
    assert len(got) == 4 * w + 3 + 5 + 7
    same = O.fuse_index_sets(np.array([[100, 100, 100]]), w, np.array([[100, 101]]), 0, 0, L)[0]
    assert same.tolist() == list(range(95, 105))         # identical windows and lexical hits inside them add nothing
    assert O.fuse_index_sets(np.array([[-1, -1]]), w, None, 0, 0, L)[0].size == 0
    assert O.fuse_index_sets(np.array([[-1]]), w, None, 600, 600, L)[0].tolist() == list(range(L))   # lead and tail overlap


def test_windows_are_clipped_and_results_sorted_unique():
    rng = np.random.default_rng(0)
    L, w = 257, 48
    centers = rng.integers(-1, L, size=(5, 40))
    lex = rng.integers(-1, L + 20, size=(5, 30))
    for q, got in enumerate(O.fuse_index_sets(centers, w, lex, 16, 16, L)):
        assert (np.diff(got) > 0).all() and got.min() >= 0 and got.max() < L
        member = np.zeros(L, bool)
        member[got] = True
        assert member[:16].all() and member[-16:].all()
        for c in centers[q]:
            if c >= 0:
                assert member[max(0, c - w // 2): min(L, c - w // 2 + w)].all()
        assert member[lex[q][(lex[q] >= 0) & (lex[q] < L)]].all()
        # nothing else: every member is explained by one of the three parts
        explained = np.zeros(L, bool)
        explained[:16] = explained[-16:] = True
        explained[lex[q][(lex[q] >= 0) & (lex[q] < L)]] = True
        for c in centers[q]:
            if c >= 0:
                explained[max(0, c - w // 2): min(L, c - w // 2 + w)] = True
        assert (member == explained).all()
