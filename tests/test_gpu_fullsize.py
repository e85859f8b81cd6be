"""GPU parity at the benchmark's full sizes and in its launch configuration (a whole 8192-token chunk of the
128K-token workload per call, the batched postings build of all layers and both SAEs, the 256-query retrieval
over a 32K-token index), checked on sampled outputs the CPU oracle can compute one by one and on properties
that hold at any size. Integer results bit-exact; encode within the bf16 tolerance (see test_gpu_parity.py)."""
import gc

import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from paper_2601_17702_b200.scan import SaeSlot, ScanPipeline, stage_index_on_device
from parity import assert_tight, check_topk_against_preact, csr_equal
from workloads import configs as C, generators as G

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def _sample_rows(T, n=48):
    return np.unique(np.concatenate([np.arange(0, n), np.arange(T // 2 - n // 2, T // 2 + n // 2), np.arange(T - n, T),
                                     np.arange(255, 258), np.arange(127, 130)]))


# one chunk per call as the scan does it (the query SAE's launch walks two bands of 16 row tiles with four column slices
# each; the key SAE's row tiles are cut at the thread-block pairs' shares), and two chunks of the query SAE in one call
# (four bands)
@pytest.mark.parametrize("which,layer,chunk_idx,n_chunks", [("key", 0, 0, 1), ("key", 3, 15, 1), ("query", 2, 7, 1), ("query", 0, 2, 2)])
def test_cfg3_full_chunk_encode_sampled_rows(which, layer, chunk_idx, n_chunks):
    cfg = C.CFG3
    shp = cfg.key if which == "key" else cfg.query
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae(which, layer)
    T = n_chunks * cfg.chunk
    x = inp.x(which, layer, chunk_idx * cfg.chunk, T)
    d = _dev()
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    ws = S.new_workspace(sae.encode_workspace_bytes(T, shp.k))
    ids = torch.full((T, shp.k), -7, dtype=torch.int32, device=d)
    vals = torch.full((T, shp.k), -7.0, dtype=torch.float32, device=d)
    S.s3_sae_encode_topk(sae, x.to(d), shp.k, ids, vals, ws)
    assert S.s3_workspace_status(ws) == 0
    ids, vals = ids.cpu().numpy(), vals.cpu().numpy()
    rows = _sample_rows(T)
    pre = O.preact(x[rows].float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    stats = {}
    check_topk_against_preact(pre, ids[rows], vals[rows], shp.k, TOL_BF16, stats)
    assert_tight(stats)            # nearly every sampled row IS the oracle's Top-k, values at fp32-accumulation accuracy
    # properties of every row: k distinct ids in range, values positive and descending
    assert (ids >= 0).all() and (ids < shp.d_sae).all()
    assert (np.sort(ids, axis=1)[:, 1:] != np.sort(ids, axis=1)[:, :-1]).all()
    assert (vals > 0).all() and (np.diff(vals, axis=1) <= 0).all()


def test_cfg3_batched_postings_and_index_full_chunk():
    """All 8 chunk-layers of one benchmark step through the batched postings build and the host index; two
    chunks, so that the merged CSR spans a chunk boundary. Bit-exact against the oracle on the same ids."""
    cfg = C.CFG3
    d = _dev()
    T = cfg.chunk
    rng = np.random.default_rng(5)
    shapes = [(cfg.key.k, cfg.key.d_sae)] * 4 + [(cfg.query.k, cfg.query.d_sae)] * 4
    indexes = [S.Index(1, D, 8 << 20) for _, D in shapes]
    bufs = [(torch.zeros(D + 1, dtype=torch.int32, device=d), torch.zeros(T * k, dtype=torch.int32, device=d)) for k, D in shapes]
    ws = S.new_workspace(sum(S.s3_postings_workspace_bytes(T, k, D) for k, D in shapes))
    ref = [[] for _ in shapes]
    for c in range(2):
        ids_h = []
        for k, D in shapes:      # k distinct ids per token: random start + distinct strides modulo D
            start = rng.integers(0, D, size=(T, 1))
            ids_h.append(((start + np.arange(k)[None, :] * 257) % D).astype(np.int32))
        ids_d = [torch.as_tensor(a).to(d) for a in ids_h]
        for ix in indexes:
            ix.stream_wait()
        items = [S.make_postings_item(ids_d[i], D, c * T, bufs[i][0], bufs[i][1]) for i, (k, D) in enumerate(shapes)]
        S.s3_postings_build_batched(items, ws)
        for i, (k, D) in enumerate(shapes):
            indexes[i].append(0, bufs[i][0], bufs[i][1], T, k, c * T)
            ref[i].append(O.postings(ids_h[i], D, c * T)[:2])
    assert S.s3_workspace_status(ws) == 0
    for i, (k, D) in enumerate(shapes):
        rp, ps, _ = indexes[i].export_csr(0)
        orp, opos = O.index_merge(ref[i], D)
        csr_equal(rp.numpy(), ps.numpy(), orp, opos)
        assert indexes[i].stats()["n_postings"] == 2 * T * k      # P = L * layers * k (Sec. 3.4)
        indexes[i].close()


def test_cfg4_retrieval_sampled_queries():
    """The benchmark's retrieval call (256 queries x 64 tokens, k 64, 2045 overlapping spans over a 32K-token
    index, 0.5/0.5 fusion, top 16): every output of 12 sampled queries against the oracle, bit-exact."""
    r = C.CFG4
    d = _dev()
    L, k, D = r.scan.L, r.scan.key.k, r.scan.key.d_sae
    rng = np.random.default_rng(11)
    start = rng.integers(0, D, size=(L, 1))
    start[rng.random((L, 1)) < 0.3] = 7                  # feature 7 is popular: a posting list of ~10K entries
    ctx = ((start + np.arange(k)[None, :] * 131) % D).astype(np.int32)      # k distinct ids per token
    qs = rng.integers(0, D, size=(r.Q * r.nq, 1))
    qs[::r.nq] = 7                                       # every query has the popular feature in its first token
    q = ((qs + np.arange(r.kq)[None, :] * 67) % D).astype(np.int32).reshape(1, r.Q, r.nq, r.kq)
    qv = rng.random(q.shape).astype(np.float32)
    ns = C.n_spans(L, r.width, r.stride)
    bm = G.gamma21(r.bm25_seed, r.Q, ns)
    rp, pos, _ = O.postings(ctx, D, 0)
    layers = [(torch.as_tensor(rp.astype(np.int64)).to(d), torch.as_tensor(pos).to(d))]
    alls = torch.zeros((r.Q, ns), dtype=torch.float32, device=d)
    ws = S.new_workspace(64)
    ti, ts = S.s3_coactivation_score_topspans(layers, D, L, torch.as_tensor(q).to(d), torch.as_tensor(qv).to(d), r.width, r.stride,
                                              r.s, r.alpha, r.beta, ws, bm.to(d), all_scores=alls)
    assert S.s3_workspace_status(ws) == 0
    ti, ts, alls = ti.cpu().numpy(), ts.cpu().numpy(), alls.cpu().numpy()
    sample = [0, 1, 2, 63, 64, 127, 128, 200, 253, 254, 255, 100]
    co = O.score_spans(ctx[None], q[:, sample], qv[:, sample], D, r.width, r.stride, 0)
    oi, os_, oall = O.fuse_select(co, bm.numpy()[sample], r.alpha, r.beta, r.s)
    np.testing.assert_array_equal(alls[sample], oall)
    np.testing.assert_array_equal(ti[sample], oi)
    np.testing.assert_array_equal(ts[sample], os_)
    # every query: the selected spans are the best of its own scores, in order
    for qi in range(r.Q):
        order = np.lexsort((np.arange(ns), -alls[qi]))[:r.s]
        assert ti[qi].tolist() == order.tolist()


def _cfg4_inputs():
    r = C.CFG4
    L, k, D = r.scan.L, r.scan.key.k, r.scan.key.d_sae
    rng = np.random.default_rng(11)
    start = rng.integers(0, D, size=(L, 1))
    start[rng.random((L, 1)) < 0.3] = 7                  # feature 7 is popular: a posting list of ~10K entries
    ctx = ((start + np.arange(k)[None, :] * 131) % D).astype(np.int32)      # k distinct ids per token
    qs = rng.integers(0, D, size=(r.Q * r.nq, 1))
    qs[::r.nq] = 7                                       # every query has the popular feature in its first token
    q = ((qs + np.arange(r.kq)[None, :] * 67) % D).astype(np.int32).reshape(1, r.Q, r.nq, r.kq)
    qv = rng.random(q.shape).astype(np.float32)
    return r, L, k, D, ctx, q, qv


def test_cfg4_compact_index_scores_like_the_raw_one():
    """The retrieval call of the benchmark on the compact form of its index: all 256 queries give the very spans and
    scores of the raw CSR, sampled queries match the oracle, and with the popular feature pruned at build time the
    sampled queries match the oracle on the context without it."""
    r, L, k, D, ctx, q, qv = _cfg4_inputs()
    d = _dev()
    ns = C.n_spans(L, r.width, r.stride)
    bm = G.gamma21(r.bm25_seed, r.Q, ns)
    rp, pos, _ = O.postings(ctx, D, 0)
    rp_t, pos_t = torch.as_tensor(rp.astype(np.int64)).to(d), torch.as_tensor(pos).to(d)
    qi_t, qv_t = torch.as_tensor(q).to(d), torch.as_tensor(qv).to(d)
    ws = S.new_workspace(64)
    ti0, ts0 = S.s3_coactivation_score_topspans([(rp_t, pos_t)], D, L, qi_t, qv_t, r.width, r.stride, r.s, r.alpha, r.beta, ws, bm.to(d))
    comp = S.s3_compact_build(rp_t, pos_t, D)
    assert comp.nbytes() < 0.75 * (pos_t.numel() * 4 + rp_t.numel() * 8)
    ti1, ts1 = S.s3_coactivation_score_topspans_compact([comp], D, L, qi_t, qv_t, r.width, r.stride, r.s, r.alpha, r.beta, ws, bm.to(d))
    assert torch.equal(ti0, ti1) and torch.equal(ts0, ts1)
    stop = 5000                                          # the appendix's hard threshold: drops feature 7's ~10K postings
    pruned = S.s3_compact_build(rp_t, pos_t, D, stop)
    assert int(pruned.row_ptr[-1]) < pos_t.numel()
    alls = torch.zeros((r.Q, ns), dtype=torch.float32, device=d)
    ti2, ts2 = S.s3_coactivation_score_topspans_compact([pruned], D, L, qi_t, qv_t, r.width, r.stride, r.s, r.alpha, r.beta, ws,
                                                        bm.to(d), all_scores=alls)
    assert S.s3_workspace_status(ws) == 0
    sample = [0, 1, 64, 128, 255]
    freq = np.bincount(ctx.ravel(), minlength=D)
    ctx_p = ctx.copy()
    ctx_p[np.isin(ctx, np.nonzero(freq > stop)[0])] = -1
    co = O.score_spans(ctx_p[None], q[:, sample], qv[:, sample], D, r.width, r.stride, 0)
    oi, os_, oall = O.fuse_select(co, bm.numpy()[sample], r.alpha, r.beta, r.s)
    np.testing.assert_array_equal(alls.cpu().numpy()[sample], oall)
    np.testing.assert_array_equal(ti2.cpu().numpy()[sample], oi)
    np.testing.assert_array_equal(ts2.cpu().numpy()[sample], os_)


def test_cfg4_position_density_sampled_queries():
    """The paper's Phase 2 tail at the retrieval workload's size (256 queries, 32K positions, 48 taps, 40 centres):
    relevance, density and centres of sampled queries against the oracle, exactly; every query's centres are valid
    (distinct, at least the radius apart, densities descending)."""
    r, L, k, D, ctx, q, qv = _cfg4_inputs()
    d = _dev()
    K, R, N = 48, 24, 40
    rp, pos, _ = O.postings(ctx, D, 0)
    layers = [(torch.as_tensor(rp.astype(np.int64)).to(d), torch.as_tensor(pos).to(d))]
    ws = S.new_workspace(S.s3_density_workspace_bytes(r.Q, L, 1, D, r.nq, r.kq))
    S_out = torch.empty((r.Q, L), dtype=torch.float32, device=d)
    D_out = torch.empty((r.Q, L), dtype=torch.float32, device=d)
    c, dens = S.s3_position_density_topcenters(layers, D, L, torch.as_tensor(q).to(d), torch.as_tensor(qv).to(d), K, R, N, ws, 5000,
                                               S_out, D_out)
    assert S.s3_workspace_status(ws) == 0
    c, dens = c.cpu().numpy(), dens.cpu().numpy()
    sample = [0, 1, 127, 128, 255]
    oS, oD, oc, odens = O.position_density(ctx[None], q[:, sample], qv[:, sample], D, K, R, N, 5000)
    np.testing.assert_array_equal(S_out.cpu().numpy()[sample], oS.astype(np.float32))
    np.testing.assert_array_equal(D_out.cpu().numpy()[sample], oD.astype(np.float32))
    np.testing.assert_array_equal(c[sample], oc)
    np.testing.assert_array_equal(dens[sample], odens)
    for qi in range(r.Q):
        got = c[qi][c[qi] >= 0]
        assert len(set(got.tolist())) == len(got)
        if len(got) > 1:
            assert np.abs(got[:, None] - got[None, :])[~np.eye(len(got), dtype=bool)].min() > R
        assert (np.diff(dens[qi][: len(got)]) <= 0).all()
    idx, cnt = S.s3_fuse_index_sets(torch.as_tensor(c[sample]).to(d), 256, None, 64, 64, L, N * 256 + 128,
                                    S.new_workspace(S.s3_fuse_workspace_bytes(len(sample), L)))
    want = O.fuse_index_sets(oc, 256, None, 64, 64, L)
    for i, m in enumerate(want):
        assert int(cnt[i]) == len(m)
        np.testing.assert_array_equal(idx[i, : len(m)].cpu().numpy(), m)


def test_scan_device_memory_is_flat_across_chunks():
    """Sec. 3.4 / memory-complexity proposition: device memory is bounded by the chunk, not by the context.
    After the first chunk, scanning more chunks allocates nothing on the device; the index grows on the host."""
    cfg = C.CFG2
    d = _dev()
    inp = C.ScanInputs(cfg, device=d)
    sae = S.Sae(*inp.sae("key", 0))
    pipe = ScanPipeline([SaeSlot("key", [sae], cfg.key.k, cfg.chunk)])
    pipe.reserve_index(cfg.L)
    xs = [inp.x("key", 0, c * cfg.chunk, cfg.chunk) for c in range(2)]
    pipe.scan_chunk(0, {"key": [xs[0]]})
    torch.cuda.synchronize()
    gc.collect()                                         # tensors of earlier tests must not be freed in mid-measurement
    base = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    for c in range(1, cfg.n_chunks):
        pipe.scan_chunk(c * cfg.chunk, {"key": [xs[c % 2]]})
    pipe.finish()
    assert torch.cuda.max_memory_allocated() <= base and torch.cuda.memory_allocated() <= base      # nothing was allocated
    st = pipe.slots[0].index.stats()
    assert st["n_postings"] == cfg.L * cfg.key.k and st["n_positions"] == cfg.L
    csr = stage_index_on_device(pipe.slots[0].index, d)
    assert int(csr[0][0][-1].item()) == cfg.L * cfg.key.k
    pipe.close()
