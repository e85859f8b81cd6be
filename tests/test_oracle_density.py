"""Pins of the oracle's per-position relevance / density / NMS routine (Sec. 3.5, Eq. 6 and "Adaptive
Granularity"; Alg. 1 Phase 2) against things other than itself: a hand-computed example, numpy's convolution,
the span-sum identity with the weighted span score, closed forms and invariants, plus planted mistakes."""
import os

import numpy as np
import pytest

import oracle as O
from conftest import read_golden

RNG = np.random.default_rng(77)
SCALE = 2.0 ** 24


def _rand_sets(T, k, D, rng, hot=0):
    keys = rng.random((T, D))
    if hot:
        keys[:, :hot] *= 0.1
    return np.argsort(keys, axis=1)[:, :k].astype(np.int32)


def test_hand_example(golden_dir):
    g = read_golden(os.path.join(golden_dir, "position_density_hand_example.txt"))
    toks = np.array(g["tokens"], np.int32).reshape(1, -1, 2)
    q = np.array(g["query"], np.int32).reshape(1, 1, -1, 2)
    qv = np.array(g["query_vals"], np.float32).reshape(1, 1, -1, 2)
    S, D, c, dens = O.position_density(toks, q, qv, 8, 3, 1, 3)
    w1, w5, w7 = (float(g[n][0]) for n in ("w1", "w5", "w7"))
    np.testing.assert_allclose(S[0], [w1, w1 + w5, w5, w1, w7, w5 + w7, w5, w5], atol=2e-7)
    np.testing.assert_allclose(D[0], [float(v) for v in g["D"]], atol=2e-6)
    assert D[0][1] == D[0][2]                       # an exact tie in fixed point: the lower position is taken
    assert c[0].tolist() == [int(v) for v in g["centers"]]
    np.testing.assert_allclose(dens[0], D[0][c[0]], rtol=1e-7)


def test_single_posting_closed_form():
    # one context token holds the query's only feature: S is w * IDF(1) = w / (ln 2 + 1) there and 0 elsewhere
    L, D = 50, 16
    ctx = np.full((1, L, 2), -1, np.int32)
    ctx[0, :, 0] = 3
    ctx[0, 20, 1] = 9
    q = np.array([9, -1], np.int32).reshape(1, 1, 1, 2)
    qv = np.array([2.5, 7.0], np.float32).reshape(1, 1, 1, 2)
    S, Dn, c, dens = O.position_density(ctx, q, qv, D, 5, 2, 2)
    expect = 2.5 / (np.log(2.0) + 1.0)
    assert abs(S[0, 20] - expect) < 1e-7 and np.count_nonzero(S[0]) == 1
    assert np.flatnonzero(Dn[0]).tolist() == [18, 19, 20, 21, 22]            # box of 5 centred on 20
    assert c[0].tolist() == [18, 21] and abs(dens[0, 0] - expect) < 1e-6      # flat top: lowest position, then beyond radius 2


@pytest.mark.parametrize("K", [1, 2, 8, 48])
def test_density_is_numpy_box_convolution(K):
    L, D, k = 300, 40, 4
    ctx = np.stack([_rand_sets(L, k, D, RNG, hot=2) for _ in range(2)])
    q = np.stack([_rand_sets(3 * 5, 3, D, RNG).reshape(3, 5, 3) for _ in range(2)])
    qv = (RNG.random(q.shape) * 2).astype(np.float32)
    S, Dn, _, _ = O.position_density(ctx, q, qv, D, K, 4, 4)
    for qi in range(3):
        full = np.convolve(S[qi], np.ones(K))                        # index j = sum S[j-K+1 .. j]
        ref = full[K - 1 - K // 2: K - 1 - K // 2 + L]               # window starting at t - K//2
        np.testing.assert_allclose(Dn[qi], ref, rtol=0, atol=1e-9)


def test_span_sums_of_S_equal_the_weighted_span_score():
    # Eq. 6 summed over a span: the weighted mode of the span scorer, up to the 2^-24 weight quantisation
    L, D, k, W = 256, 64, 4, 32
    ctx = np.stack([_rand_sets(L, k, D, RNG, hot=3)])
    q = np.stack([_rand_sets(2 * 6, 4, D, RNG).reshape(2, 6, 4)])
    qv = (RNG.random(q.shape) * 3).astype(np.float32)
    S, _, _, _ = O.position_density(ctx, q, qv, D, 8, 4, 4)
    ws = O.score_spans(ctx, q, qv, D, W, W, 1)
    spans = S.reshape(2, L // W, W).sum(axis=2)
    np.testing.assert_allclose(spans, ws, rtol=1e-5, atol=W * k * 2.0 ** -24)


def test_nms_invariants_and_brute_force():
    L, D, k, K, R, N = 400, 32, 4, 8, 10, 12
    ctx = np.stack([_rand_sets(L, k, D, RNG, hot=2)])
    q = np.stack([_rand_sets(4 * 3, 4, D, RNG).reshape(4, 3, 4)])
    qv = RNG.random(q.shape).astype(np.float32)
    _, Dn, c, dens = O.position_density(ctx, q, qv, D, K, R, N)
    for qi in range(4):
        fix = np.rint(Dn[qi] * SCALE).astype(np.int64)
        alive = np.ones(L, bool)
        for i in range(N):                                   # greedy reference in numpy
            cand = np.flatnonzero(alive & (fix > 0))
            if len(cand) == 0:
                assert c[qi, i] == -1 and dens[qi, i] == 0
                continue
            best = cand[np.argmax(fix[cand])]                # argmax returns the first (lowest) maximum
            assert c[qi, i] == best
            alive[max(0, best - R): best + R + 1] = False
        got = c[qi][c[qi] >= 0]
        assert (np.abs(got[:, None] - got[None, :])[~np.eye(len(got), dtype=bool)] > R).all()
        assert (np.diff(dens[qi][: len(got)]) <= 0).all()


def test_stop_features_and_empty_query():
    L, D, k = 120, 16, 3
    ctx = np.stack([_rand_sets(L, k, D, RNG, hot=1)])        # feature 0 in almost every token
    q = np.array([0, 5, 6], np.int32).reshape(1, 1, 1, 3)
    qv = np.ones(q.shape, np.float32)
    S_all, _, _, _ = O.position_density(ctx, q, qv, D, 4, 2, 3)
    S_stop, _, _, _ = O.position_density(ctx, q, qv, D, 4, 2, 3, stop_freq=60)
    has0 = (ctx[0] == 0).any(axis=1)
    assert has0.sum() > 60
    idf0 = 1.0 / (np.log(1.0 + has0.sum()) + 1.0)
    np.testing.assert_allclose(S_all[0] - S_stop[0], has0 * idf0, atol=2e-7)
    qe = np.full((1, 1, 2, 3), -1, np.int32)
    S, Dn, c, dens = O.position_density(ctx, qe, np.ones(qe.shape, np.float32), D, 4, 2, 3)
    assert not S.any() and not Dn.any() and (c == -1).all() and (dens == 0).all()


def test_planted_mistakes_are_caught():
    # an off-centre window, a missing IDF and a max-instead-of-sum aggregation all change the hand example
    g = {"tokens": [1, 3, 1, 5, 3, 5, 1, 2, 0, 7, 5, 7, 5, 6, 2, 5], "query": [1, 5, 1, 7], "vals": [0.5, 2.0, 1.5, 1.0]}
    toks = np.array(g["tokens"], np.int32).reshape(1, -1, 2)
    q = np.array(g["query"], np.int32).reshape(1, 1, -1, 2)
    qv = np.array(g["vals"], np.float32).reshape(1, 1, -1, 2)
    S, D, c, _ = O.position_density(toks, q, qv, 8, 3, 1, 3)
    w = {1: 2.0 / (np.log(4) + 1), 5: 2.0 / (np.log(6) + 1), 7: 1.0 / (np.log(3) + 1)}
    sets = toks[0]
    S_ref = np.array([sum(w.get(int(f), 0.0) for f in row) for row in sets])
    assert np.allclose(S[0], S_ref, atol=2e-7)
    no_idf = np.array([sum({1: 2.0, 5: 2.0, 7: 1.0}.get(int(f), 0.0) for f in row) for row in sets])
    max_agg = np.array([sum({1: 1.5 / (np.log(4) + 1), 5: w[5], 7: w[7]}.get(int(f), 0.0) for f in row) for row in sets])
    assert not np.allclose(S[0], no_idf, atol=1e-3) and not np.allclose(S[0], max_agg, atol=1e-3)
    left_window = np.array([S_ref[max(0, t - 2): t + 1].sum() for t in range(8)])     # window ending at t
    assert not np.allclose(D[0], left_window, atol=1e-3)
