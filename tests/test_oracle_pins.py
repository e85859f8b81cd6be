"""Pins the CPU oracle to things other than itself: library routines, brute force, closed forms,
the paper's printed index-size instance and a hand-worked co-activation example."""
import os

import numpy as np
import pytest

import oracle as O
from conftest import read_golden

RNG = np.random.default_rng(1234)


def _rand_sae(T, d_in, d_sae, rng=RNG):
    x = rng.standard_normal((T, d_in)).astype(np.float32)
    W = rng.standard_normal((d_in, d_sae)).astype(np.float32)
    W /= np.linalg.norm(W, axis=0, keepdims=True)
    b_enc = (0.1 * rng.standard_normal(d_sae)).astype(np.float32)
    b_dec = (0.05 * rng.standard_normal(d_in)).astype(np.float32)
    return x, W, b_enc, b_dec


# ---------------------------------------------------------------- encode (Eq. 1)

def test_preact_matches_blas_fp64():
    # non-square shapes so a transposed operand cannot pass
    x, W, b_enc, b_dec = _rand_sae(37, 24, 200)
    ref = (x.astype(np.float64) - b_dec.astype(np.float64)) @ W.astype(np.float64) + b_enc.astype(np.float64)
    got = O.preact(x, W, b_enc, b_dec)
    assert got.shape == (37, 200)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_preact_identity_sae_is_x():
    d = 16
    x = RNG.standard_normal((9, d)).astype(np.float32)
    W = np.eye(d, dtype=np.float32)
    z = O.preact(x, W, np.zeros(d, np.float32), np.zeros(d, np.float32))
    np.testing.assert_array_equal(z, x.astype(np.float64))
    ids, vals = O.topk(z, 3)
    for t in range(9):
        order = sorted([(-(x[t, f]), f) for f in range(d) if x[t, f] > 0])[:3]
        assert [f for _, f in order] == [i for i in ids[t] if i >= 0]


def test_preact_x_equals_bdec_gives_benc():
    x, W, b_enc, b_dec = _rand_sae(5, 12, 40)
    x = np.tile(b_dec, (5, 1))
    z = O.preact(x, W, b_enc, b_dec)
    np.testing.assert_array_equal(z, np.tile(b_enc.astype(np.float64), (5, 1)))


def test_preact_one_hot_closed_form():
    _, W, b_enc, b_dec = _rand_sae(1, 10, 30)
    for i in (0, 3, 9):
        x = np.zeros((1, 10), np.float32)
        x[0, i] = 1.0
        z = O.preact(x, W, b_enc, b_dec)[0]
        for f in (0, 7, 29):
            want = float(W[i, f]) - sum(float(W[j, f]) * float(b_dec[j]) for j in range(10)) + float(b_enc[f])
            assert abs(z[f] - want) < 1e-12


def test_preact_bias_signs():
    # b_dec is subtracted from x, b_enc is added: single-element case with exact values
    W = np.array([[2.0]], np.float32)
    z = O.preact(np.array([[3.0]], np.float32), W, np.array([0.5], np.float32), np.array([1.0], np.float32))
    assert z[0, 0] == 2.0 * (3.0 - 1.0) + 0.5


# ---------------------------------------------------------------- ReLU + Top-k (Eq. 1-3)

def _brute_topk(z, k):
    T, D = z.shape
    ids = -np.ones((T, k), np.int32)
    vals = np.zeros((T, k), np.float32)
    for t in range(T):
        c = [(float(z[t, f]), f) for f in range(D) if z[t, f] > 0]
        c.sort(key=lambda p: (-p[0], p[1]))
        for j, (v, f) in enumerate(c[:k]):
            ids[t, j] = f
            vals[t, j] = np.float32(v)
    return ids, vals


@pytest.mark.parametrize("k", [1, 4, 8, 17])
def test_topk_vs_full_sort(k):
    z = RNG.standard_normal((50, 64))
    z[3] = -np.abs(z[3])            # no positive entry at all
    z[4, 5:] = -1.0                 # fewer than k positives
    z[5, :] = 0.0                   # zeros are not selected
    z[6, :] = 1.0                   # all tied: ids 0..k-1
    z[7, ::2] = 2.5                 # duplicated values
    ids, vals = O.topk(z, k)
    bi, bv = _brute_topk(z, k)
    np.testing.assert_array_equal(ids, bi)
    np.testing.assert_array_equal(vals, bv)
    assert (ids[3] == -1).all() and (ids[5] == -1).all()
    assert list(ids[6]) == list(range(k))


def test_topk_invariants():
    k = 8
    z = RNG.standard_normal((200, 96))
    ids, vals = O.topk(z, k)
    for t in range(200):
        npos = int((z[t] > 0).sum())
        sel = ids[t][ids[t] >= 0]
        assert len(sel) == min(k, npos)
        assert len(set(sel.tolist())) == len(sel)
        assert (np.diff(vals[t][: len(sel)]) <= 0).all()
        rest = np.setdiff1d(np.arange(96), sel)
        if len(sel) == k:
            assert z[t, rest].max() <= z[t, sel].min()
        assert (vals[t][len(sel):] == 0).all()


# ---------------------------------------------------------------- postings (Eq. 4)

def _rand_ids(T, k, d_sae, rng=RNG, short_rows=True):
    ids = np.stack([rng.choice(d_sae, size=k, replace=False) for _ in range(T)]).astype(np.int32)
    if short_rows and T > 4:
        ids[2, k // 2:] = -1
        ids[4, :] = -1
    return ids


def test_postings_brute_force_and_inversion():
    T, k, D, base = 60, 5, 40, 1000
    ids = _rand_ids(T, k, D)
    row_ptr, pos, _ = O.postings(ids, D, base)
    assert row_ptr[0] == 0 and row_ptr[-1] == (ids >= 0).sum() == len(pos)
    for f in range(D):
        want = [base + t for t in range(T) if f in ids[t]]
        got = pos[row_ptr[f]:row_ptr[f + 1]].tolist()
        assert got == want                      # ascending absolute positions
    # inverting the index gives back every token's id set
    back = [set() for _ in range(T)]
    for f in range(D):
        for p in pos[row_ptr[f]:row_ptr[f + 1]]:
            back[p - base].add(f)
    for t in range(T):
        assert back[t] == set(ids[t][ids[t] >= 0].tolist())


def test_postings_values_travel_with_positions():
    T, k, D = 20, 3, 16
    ids = _rand_ids(T, k, D, short_rows=False)
    vals = RNG.random((T, k)).astype(np.float32)
    row_ptr, pos, pval = O.postings(ids, D, 0, vals)
    for f in range(D):
        for p, v in zip(pos[row_ptr[f]:row_ptr[f + 1]], pval[row_ptr[f]:row_ptr[f + 1]]):
            j = list(ids[p]).index(f)
            assert v == vals[p, j]


def test_postings_total_matches_index_size_formula(golden_dir):
    g = read_golden(os.path.join(golden_dir, "index_size_instance.txt"))
    L, nl, k = int(g["L"][0]), int(g["layers"][0]), int(g["k"][0])
    assert L * nl * k * int(g["bytes_per_posting"][0]) == int(g["mib"][0]) * 1024 * 1024
    # scaled-down instance: every token carries exactly k ids => P = L * layers * k
    Ls, ks, D = 512, 8, 64
    total = 0
    for layer in range(nl):
        ids = _rand_ids(Ls, ks, D, np.random.default_rng(layer), short_rows=False)
        row_ptr, pos, _ = O.postings(ids, D, 0)
        total += int(row_ptr[-1])
    assert total == Ls * nl * ks


def test_index_merge_equals_single_chunk_build():
    T, k, D = 96, 4, 32
    ids = _rand_ids(T, k, D)
    whole_rp, whole_pos, _ = O.postings(ids, D, 0)
    chunks = []
    for c0 in (0, 40, 64):
        c1 = {0: 40, 40: 64, 64: 96}[c0]
        rp, ps, _ = O.postings(ids[c0:c1], D, c0)
        chunks.append((rp, ps))
    rp, ps = O.index_merge(chunks, D)
    np.testing.assert_array_equal(rp, whole_rp.astype(np.uint64))
    np.testing.assert_array_equal(ps, whole_pos)


def test_postings_empty_and_single():
    rp, pos, _ = O.postings(np.zeros((0, 4), np.int32), 8, 0)
    assert (rp == 0).all() and len(pos) == 0
    rp, pos, _ = O.postings(np.array([[3]], np.int32), 8, 77)
    assert rp.tolist() == [0, 0, 0, 0, 1, 1, 1, 1, 1] and pos.tolist() == [77]


# ---------------------------------------------------------------- IDF (appendix)

def test_idf_closed_forms(golden_dir):
    g = read_golden(os.path.join(golden_dir, "idf_points.txt"))
    for fr, want in zip(g["freq"], g["idf"]):
        assert abs(O.idf(float(fr)) - float(want)) < 1e-14
    xs = [O.idf(n) for n in range(0, 100)]
    assert all(a > b for a, b in zip(xs, xs[1:]))   # strictly decreasing in freq


# ---------------------------------------------------------------- span scoring + fusion

def test_hand_example(golden_dir):
    g = read_golden(os.path.join(golden_dir, "coactivation_hand_example.txt"))
    D, k, W, S = int(g["d_sae"][0]), int(g["k"][0]), int(g["width"][0]), int(g["stride"][0])
    toks = np.array(g["tokens"], np.int32).reshape(-1, k)
    rp, pos, _ = O.postings(toks, D, 0)
    assert rp.tolist() == [int(v) for v in g["row_ptr"]]
    assert pos.tolist() == [int(v) for v in g["pos"]]
    q = np.array(g["query"], np.int32).reshape(1, 1, -1, k)
    qv = np.ones(q.shape, np.float32)
    co = O.score_spans(toks[None], q, qv, D, W, S, mode=0)
    assert co.tolist() == [[int(v) for v in g["coact"]]]
    bm = np.array([[float(v) for v in g["bm25"]]], np.float32)
    ti, ts, alls = O.fuse_select(co, bm, float(g["alpha"][0]), float(g["beta"][0]), 2)
    assert alls[0].tolist() == [float(v) for v in g["fused"]]
    assert ti[0].tolist() == [int(v) for v in g["top_order"]]
    assert ts[0].tolist() == [3.0, 2.0]
    # without the lexical term the order flips back
    ti0, _, _ = O.fuse_select(co, None, 1.0, 0.0, 2)
    assert ti0[0].tolist() == [0, 1]
    ws = O.score_spans(toks[None], q, qv, D, W, S, mode=1)
    tol = float(g["weighted_tol"][0])
    for got, want in zip(ws[0], g["weighted"]):
        assert abs(got - float(want)) < tol


def _score_from_postings(ctx_ids, q_ids, q_vals, D, W, S, mode, stop_freq=0):
    """Independent route: through the inverted index (python loops), for tiny inputs."""
    nl, L, k = ctx_ids.shape
    _, Q, nq, kq = q_ids.shape
    ns = (L - W) // S + 1 if L >= W else 0
    out = np.zeros((Q, ns), np.float64)
    for l in range(nl):
        rp, pos, _ = O.postings(ctx_ids[l], D, 0)
        for q in range(Q):
            cQ, aQ = {}, {}
            for u in range(nq):
                for j in range(kq):
                    f = int(q_ids[l, q, u, j])
                    if f >= 0:
                        cQ[f] = cQ.get(f, 0) + 1
                        aQ[f] = aQ.get(f, 0.0) + float(q_vals[l, q, u, j])
            for f in sorted(cQ):
                lst = pos[rp[f]:rp[f + 1]]
                freq = len(lst)
                if mode == 1 and stop_freq > 0 and freq > stop_freq:
                    continue
                for s in range(ns):
                    cS = int(((lst >= s * S) & (lst < s * S + W)).sum())
                    if mode == 0:
                        out[q, s] += min(cQ[f], cS)
                    else:
                        out[q, s] += aQ[f] * (1.0 / (np.log(1.0 + freq) + 1.0)) * cS
    return out


@pytest.mark.parametrize("W,S", [(8, 8), (8, 2), (6, 4), (5, 7)])
@pytest.mark.parametrize("mode", [0, 1])
def test_scoring_dense_vs_postings_route(W, S, mode):
    rng = np.random.default_rng(7 + W * 10 + S)
    nl, L, k, D, Q, nq, kq = 2, 50, 3, 12, 3, 4, 3
    ctx = np.stack([_rand_ids(L, k, D, rng) for _ in range(nl)])
    q = np.stack([np.stack([_rand_ids(nq, kq, D, rng, short_rows=False) for _ in range(Q)]) for _ in range(nl)])
    q[0, 0, 1, 2] = -1
    qv = rng.random(q.shape).astype(np.float32)
    got = O.score_spans(ctx, q, qv, D, W, S, mode=mode, stop_freq=(14 if mode else 0))
    want = _score_from_postings(ctx, q, qv, D, W, S, mode, stop_freq=(14 if mode else 0))
    if mode == 0:
        np.testing.assert_array_equal(got, want.astype(np.int64))
    else:
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_scoring_saturated_query_counts_postings():
    # with cQ >= width for every query feature, min(cQ, cS) = cS, so the score is the number of
    # postings of the query's features inside the span, and over a tiling it sums to sum_f freq(f)
    rng = np.random.default_rng(5)
    L, k, D, W = 64, 4, 20, 8
    ctx = _rand_ids(L, k, D, rng, short_rows=False)[None]
    feats = np.array([1, 5, 9], np.int32)
    q = np.tile(feats, (1, 1, W, 1)).astype(np.int32)     # W identical query tokens
    co = O.score_spans(ctx, q, np.ones(q.shape, np.float32), D, W, W, mode=0)
    freq = sum(int((ctx[0] == f).sum()) for f in feats)
    assert int(co.sum()) == freq
    for s in range(L // W):
        want = sum(int((ctx[0, s * W:(s + 1) * W] == f).sum()) for f in feats)
        assert co[0, s] == want
    # bounds 0 <= coact <= min(nq*kq, W*k)
    assert co.min() >= 0 and co.max() <= min(W * 3, W * k)


def test_fuse_select_reductions_and_rounding():
    rng = np.random.default_rng(11)
    co = rng.integers(0, 50, size=(4, 37)).astype(np.int64)
    bm = rng.gamma(2.0, 1.0, size=(4, 37)).astype(np.float32)
    ti, ts, alls = O.fuse_select(co, bm, 0.3, 0.7, 5)
    want = (np.float32(0.3) * co.astype(np.float32)).astype(np.float32) + (np.float32(0.7) * bm).astype(np.float32)
    np.testing.assert_array_equal(alls, want.astype(np.float32))
    for q in range(4):
        order = sorted(range(37), key=lambda j: (-float(want[q, j]), j))[:5]
        assert ti[q].tolist() == order
        np.testing.assert_array_equal(ts[q], want[q, order])
    # alpha = 0: the top-s of the lexical vector alone
    ti, _, _ = O.fuse_select(co, bm, 0.0, 1.0, 5)
    for q in range(4):
        assert ti[q].tolist() == sorted(range(37), key=lambda j: (-float(bm[q, j]), j))[:5]
    # ties broken by lower span index; s larger than n_spans pads with -1
    ti, ts, _ = O.fuse_select(np.array([[2, 7, 7, 1]], np.int64), None, 1.0, 0.0, 6)
    assert ti[0].tolist() == [1, 2, 0, 3, -1, -1] and ts[0].tolist() == [7, 7, 2, 1, 0, 0]


def test_end_to_end_tiny_chain_consistency():
    # encode -> top-k -> postings -> score, on a tiny SAE, against the python route above
    x, W, b_enc, b_dec = _rand_sae(48, 8, 32, np.random.default_rng(3))
    ids, vals = O.encode_topk(x, W, b_enc, b_dec, 4)
    xq = np.random.default_rng(4).standard_normal((6, 8)).astype(np.float32)
    qi, qv = O.encode_topk(xq, W, b_enc, b_dec, 4)
    q = qi.reshape(1, 2, 3, 4)
    qvv = qv.reshape(1, 2, 3, 4)
    for mode in (0, 1):
        got = O.score_spans(ids[None], q, qvv, 32, 8, 4, mode=mode)
        want = _score_from_postings(ids[None], q, qvv, 32, 8, 4, mode)
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
