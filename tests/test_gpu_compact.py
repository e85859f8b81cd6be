"""GPU parity of the compact (block-delta, bit-packed) index: the device build against the oracle's encoder, bit for
bit on all five arrays, and span scoring on the compact form against the oracle's scores of the pruned context
(Sec. 3.4 memory analysis: delta encoding and stop-feature pruning; Sec. 3.5 for the scores)."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from workloads import configs as C
from workloads import generators as G

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def _csr(lists):
    rp = np.cumsum([0] + [len(l) for l in lists]).astype(np.uint64)
    pos = np.array([p for l in lists for p in l], dtype=np.int32)
    return rp, pos


def gpu_build(rp, pos, stop=0, **kw):
    d = _dev()
    D = len(rp) - 1
    pos_t = torch.as_tensor(pos if len(pos) else np.zeros(1, np.int32)).to(d)[: len(pos)]
    return S.s3_compact_build(torch.as_tensor(rp.astype(np.int64)).to(d), pos_t, D, stop, **kw)


def assert_same(c, want):
    np.testing.assert_array_equal(c.row_ptr.cpu().numpy().astype(np.uint64), want["row_ptr"])
    np.testing.assert_array_equal(c.blk_ptr.cpu().numpy().astype(np.uint32), want["blk_ptr"])
    np.testing.assert_array_equal(c.blk_first.cpu().numpy(), want["blk_first"])
    np.testing.assert_array_equal(c.blk_desc.cpu().numpy().astype(np.uint64), want["blk_desc"])
    np.testing.assert_array_equal(c.payload.cpu().numpy().astype(np.uint32), want["payload"])


def test_build_hand_example():
    c = gpu_build(*_csr([[5, 6, 9, 20], [], [7]]))
    assert c.blk_first.tolist() == [5, 7] and c.blk_desc.tolist() == [4, 64] and c.payload.tolist() == [0xA20, 0]


@pytest.mark.parametrize("seed,D,max_pos_bits,stop", [
    (1, 70, 12, 0),          # short gaps
    (2, 300, 24, 0),         # wide gaps, many ragged blocks
    (3, 300, 31, 0),         # the widest values (width up to 31)
    (4, 64, 16, 100),        # stop-feature pruning at build time
    (5, 2500, 20, 0),        # more lists than one scan tile
])
def test_build_matches_oracle_encoder(seed, D, max_pos_bits, stop):
    rng = np.random.default_rng(seed)
    lists = []
    for f in range(D):
        n = int(rng.choice([0, 0, 1, 2, 31, 32, 33, 63, 64, 65, 150, 400]))
        hi = 1 << int(rng.integers(min(10, max_pos_bits), max_pos_bits + 1))
        n = min(n, hi)
        if hi > (1 << 24):                                   # sampling without replacement from a huge range
            p = np.unique(rng.integers(0, hi - 1, size=n))
        else:
            p = np.sort(rng.choice(hi - 1, size=n, replace=False))
        lists.append(p.tolist())
    lists[0] = list(range(1000, 1100))                        # consecutive positions: width 0
    lists[1] = [0, 2**31 - 1]                                 # gap - 1 = 2^31 - 2: width 31
    rp, pos = _csr(lists)
    assert_same(gpu_build(rp, pos, stop), O.compact_encode(rp, pos, stop))


def test_build_on_scan_sized_index():
    # 4096 lists of about 128 random positions out of 32K: half a million postings, 18K blocks (several scan tiles)
    rng = np.random.default_rng(3)
    lists = [np.sort(rng.choice(32768, size=int(rng.poisson(128)), replace=False)).tolist() for _ in range(4096)]
    rp, pos = _csr(lists)
    c = gpu_build(rp, pos, 0)
    assert_same(c, O.compact_encode(rp, pos, 0))
    assert c.nbytes() < 0.6 * (pos.nbytes + rp.nbytes)        # gaps of about 8 bits plus headers: well under 4 B per posting


def test_expand_is_the_inverse_of_build():
    rng = np.random.default_rng(9)
    lists = [np.sort(rng.choice(1 << 20, size=int(rng.choice([0, 1, 31, 32, 33, 100, 700])), replace=False)).tolist()
             for _ in range(400)]
    lists[3] = [0, 2**31 - 1]
    rp, pos = _csr(lists)
    for stop in (0, 90):
        c = gpu_build(rp, pos, stop)
        want_rp, want_pos = O.compact_decode(O.compact_encode(rp, pos, stop))          # the oracle's own decoder
        got_rp, got_pos = S.s3_compact_expand(c, len(rp) - 1)
        np.testing.assert_array_equal(got_rp.cpu().numpy().astype(np.uint64), want_rp)
        np.testing.assert_array_equal(got_pos.cpu().numpy(), want_pos)
        np.testing.assert_array_equal(want_pos, O.prune_stop_features(rp, pos, stop)[1])
    d = _dev()
    view = c.view()
    ws = torch.zeros(64, dtype=torch.uint8, device=d)
    small = torch.empty(4, dtype=torch.int32, device=d)
    S.binding._check(S.binding.lib().s3_compact_expand(S.binding.C.byref(view), len(rp) - 1, small.data_ptr(), 4, ws.data_ptr(), 64,
                                                       S.binding._stream()))
    with pytest.raises(S.S3Error):
        S.s3_workspace_status(ws)


def test_empty_index_and_capacity_error():
    c = gpu_build(np.zeros(9, np.uint64), np.zeros(0, np.int32))
    assert c.blk_first.numel() == 0 and c.payload.tolist() == [0] and c.row_ptr.tolist() == [0] * 9
    rp, pos = _csr([list(range(0, 6400, 2))] * 3)
    with pytest.raises(S.S3Error):
        gpu_build(rp, pos, cap_blocks=10)
    with pytest.raises(S.S3Error):
        gpu_build(rp, pos, cap_words=5)
    d = _dev()
    with pytest.raises(S.S3Error):
        S.s3_compact_build(torch.zeros(9, dtype=torch.int64, device=d), torch.zeros(4, dtype=torch.int32, device=d), 8, -1)


# ------------------------------------------------------------------------------------------------ scoring
def _rand_ids(T, k, d_sae, seed, hot=None):
    rng = np.random.default_rng(seed)
    keys = rng.random((T, d_sae))
    if hot:
        keys[:, :hot] *= 0.15
    return np.argsort(keys, axis=1)[:, :k].astype(np.int32)


def gpu_score_compact(ctx, q, qv, d_sae, width, stride, s, alpha, beta, bm25, mode, build_stop, score_stop=0):
    d = _dev()
    n_layers, L, k = ctx.shape
    layers = []
    for l in range(n_layers):
        rp, pos, _ = O.postings(ctx[l], d_sae, 0)
        layers.append(gpu_build(rp.astype(np.uint64), pos, build_stop))
    ns = C.n_spans(L, width, stride)
    Q = q.shape[1]
    alls = torch.zeros((Q, max(ns, 1)), dtype=torch.float32, device=d)
    # odd list totals: the full workspace, so that each query is cut over many thread blocks; even ones: one block per query
    split = int(layers[0].row_ptr[-1]) % 2 == 1
    ws = S.new_workspace(S.s3_score_workspace_bytes(Q, q.shape[2], q.shape[3], n_layers, ns, s) if split else 64)
    bm = None if bm25 is None else torch.as_tensor(bm25).to(d).contiguous()
    ti, ts = S.s3_coactivation_score_topspans_compact(layers, d_sae, L, torch.as_tensor(q).to(d).contiguous(),
                                                      torch.as_tensor(qv).to(d).contiguous(), width, stride, s, alpha, beta,
                                                      ws, bm, mode, score_stop, all_scores=alls)
    assert S.s3_workspace_status(ws) == 0
    return ti.cpu().numpy(), ts.cpu().numpy(), alls.cpu().numpy()[:, :ns], layers


def _pruned_ctx(ctx, d_sae, stop):
    if stop <= 0:
        return ctx
    out = ctx.copy()
    for l in range(ctx.shape[0]):
        freq = np.bincount(ctx[l].ravel(), minlength=d_sae)
        out[l][np.isin(ctx[l], np.nonzero(freq > stop)[0])] = -1
    return out


@pytest.mark.parametrize("L,k,d_sae,n_layers,Q,nq,kq,width,stride,s,stop", [
    (8, 2, 8, 1, 1, 2, 2, 4, 4, 2, 0),
    (2048, 8, 1024, 1, 1, 16, 8, 64, 64, 4, 0),
    (1000, 8, 256, 3, 5, 7, 8, 64, 16, 16, 0),
    (12000, 4, 32, 1, 2, 5, 4, 64, 16, 8, 0),       # lists of hundreds of blocks
    (9000, 4, 16, 2, 2, 3, 4, 50, 30, 8, 0),        # stride not a power of two
    (5000, 8, 16, 1, 2, 40, 8, 64, 8, 8, 0),        # cQ up to 40: the earlier posting lies one or two blocks back
    (6000, 8, 16, 1, 2, 64, 8, 64, 16, 8, 0),       # cQ up to 64: exactly two blocks back as well
    (3000, 8, 64, 2, 3, 7, 8, 64, 16, 8, 500),      # hot features pruned when the index is built
    (30, 4, 64, 1, 2, 3, 4, 64, 16, 4, 0),          # no full span at all
])
def test_score_mincount_on_compact_index(L, k, d_sae, n_layers, Q, nq, kq, width, stride, s, stop):
    ctx = np.stack([_rand_ids(L, k, d_sae, 50 + l, hot=3) for l in range(n_layers)])
    q = np.stack([_rand_ids(Q * nq, kq, d_sae, 80 + l, hot=3).reshape(Q, nq, kq) for l in range(n_layers)])
    q[0, 0, 0, -1] = -1
    qv = np.random.default_rng(9).random(q.shape).astype(np.float32)
    ns = C.n_spans(L, width, stride)
    bm = G.gamma21(4, Q, max(ns, 1)).numpy()[:, :ns] if ns else None
    co = O.score_spans(_pruned_ctx(ctx, d_sae, stop), q, qv, d_sae, width, stride, 0)
    oi, os_, oall = O.fuse_select(co, bm, 0.5, 0.5, s)
    ti, ts, alls, layers = gpu_score_compact(ctx, q, qv, d_sae, width, stride, s, 0.5, 0.5, bm, 0, stop)
    np.testing.assert_array_equal(alls, oall)
    np.testing.assert_array_equal(ti, oi)
    np.testing.assert_array_equal(ts, os_)
    if stop:
        assert any(int(c.row_ptr[-1]) < L * k for c in layers)      # something was pruned


def test_score_weighted_on_compact_index():
    L, k, d_sae, n_layers, Q, nq, kq, width, stride, s = 600, 8, 128, 2, 4, 6, 8, 64, 16, 8
    ctx = np.stack([_rand_ids(L, k, d_sae, 150 + l, hot=3) for l in range(n_layers)])
    q = np.stack([_rand_ids(Q * nq, kq, d_sae, 180 + l, hot=3).reshape(Q, nq, kq) for l in range(n_layers)])
    qv = (np.random.default_rng(19).random(q.shape) * 3).astype(np.float32)
    for build_stop, score_stop in ((0, 0), (400, 0), (0, 400)):
        # pruning at build time removes the same features as the scorer's own threshold and leaves the IDF of the
        # kept features untouched
        w = O.score_spans(ctx, q, qv, d_sae, width, stride, 1, max(build_stop, score_stop))
        _, _, oall = O.fuse_select(w, None, 1.0, 0.0, s)
        ti, ts, alls, _ = gpu_score_compact(ctx, q, qv, d_sae, width, stride, s, 1.0, 0.0, None, 1, build_stop, score_stop)
        np.testing.assert_allclose(alls, oall, rtol=1e-5, atol=1e-6)
        for qi in range(Q):
            order = sorted(range(alls.shape[1]), key=lambda j: (-float(alls[qi, j]), j))[:s]
            assert ti[qi].tolist() == order


def test_saved_index_scores_the_same(tmp_path):
    L, k, d_sae = 4000, 8, 128
    ctx = np.stack([_rand_ids(L, k, d_sae, 7, hot=3)])
    q = _rand_ids(2 * 5, 8, d_sae, 8, hot=3).reshape(1, 2, 5, 8)
    qv = np.ones(q.shape, np.float32)
    ti, ts, alls, layers = gpu_score_compact(ctx, q, qv, d_sae, 64, 16, 8, 1.0, 0.0, None, 0, 0)
    path = str(tmp_path / "ctx.s3c")
    S.s3_compact_save(path, [c.to("cpu") for c in layers], d_sae)
    back, _ = S.s3_compact_load(path)
    d = _dev()
    ws = S.new_workspace(64)
    ti2, ts2 = S.s3_coactivation_score_topspans_compact([c.to(d) for c in back], d_sae, L, torch.as_tensor(q).to(d),
                                                        torch.as_tensor(qv).to(d), 64, 16, 8, 1.0, 0.0, ws)
    np.testing.assert_array_equal(ti2.cpu().numpy(), ti)
    np.testing.assert_array_equal(ts2.cpu().numpy(), ts)
    co = O.score_spans(ctx, q, qv, d_sae, 64, 16, 0)
    oi, _, _ = O.fuse_select(co, None, 1.0, 0.0, 8)
    np.testing.assert_array_equal(ti, oi)
