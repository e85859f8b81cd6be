"""The benchmark configurations as chains, on the GPU, against the CPU oracle.

  * the Llama-3-8B-shaped key scan (32K tokens in chunks of 4096, lognormal channel scales with outlier channels,
    1024 -> 16384, k = 32) through the streaming pipeline, every row of every chunk against the oracle's
    pre-activations, the merged index against the oracle's postings of the same ids; then the retrieval workload on
    THAT index: 256 queries x 64 vectors of the same distribution through the same SAE at k = 64, min-count scores
    of 64-token spans at stride 16 and at stride 64, fused 0.5/0.5 with Gamma(2,1) lexical scores, top 16;
  * the 1M-token Qwen2.5-7B-shaped scan (512 -> 8192, k = 16, 8 layers, chunks of 16384, Zipf(1.1) popularity):
    16 of its 64 chunks through the pipeline with device memory flat from chunk 2 on, the postings total and the
    popularity slope of the longest lists.
Integer results bit-exact; encode within the bf16 tolerance and, much tighter, nearly every row equal to the
oracle's Top-k with values at fp32-accumulation accuracy."""
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


def test_cfg2_scan_full_parity_then_cfg4_retrieval_on_its_index():
    cfg = C.CFG2
    d = _dev()
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("key", 0)
    Wf, be, bd = W.float().numpy(), b_enc.numpy(), b_dec.numpy()
    k, D, chunk = cfg.key.k, cfg.key.d_sae, cfg.chunk
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    pipe = ScanPipeline([SaeSlot("key", [sae], k, chunk)])
    pipe.reserve_index(cfg.L)
    slot = pipe.slots[0]

    # ---- scan: all 8 chunks, every row against the oracle
    stats = {}
    ctx_ids, chunk_refs = [], []
    for c in range(cfg.n_chunks):
        x = inp.x("key", 0, c * chunk, chunk)
        pipe.scan_chunk(c * chunk, {"key": [x.to(d)]})
        ids = slot.ids[0].cpu().numpy().copy()
        vals = slot.vals[0].cpu().numpy().copy()
        pre = O.preact(x.float().numpy(), Wf, be, bd)
        check_topk_against_preact(pre, ids, vals, k, TOL_BF16, stats)
        del pre
        ctx_ids.append(ids)
        chunk_refs.append(O.postings(ids, D, c * chunk)[:2])          # the GPU's own ids through the oracle's step
    pipe.finish()
    assert stats["rows"] == cfg.L
    assert_tight(stats)
    ctx_ids = np.concatenate(ctx_ids)
    assert (ctx_ids >= 0).all()

    # ---- index: the merged CSR of the host index, bit-exact; P = L * k (Sec. 3.4)
    rp, ps, _ = slot.index.export_csr(0)
    orp, opos = O.index_merge(chunk_refs, D)
    csr_equal(rp.numpy(), ps.numpy(), orp, opos)
    assert slot.index.stats()["n_postings"] == cfg.L * k
    csr = stage_index_on_device(slot.index, d)

    # ---- retrieval: the queries go through the same SAE (the shared codebook) at k = 64
    r = C.CFG4
    xq = inp.retrieval_queries(0, r.Q, r.nq)
    q_ids = torch.empty((r.Q * r.nq, r.kq), dtype=torch.int32, device=d)
    q_vals = torch.empty((r.Q * r.nq, r.kq), dtype=torch.float32, device=d)
    ws = S.new_workspace(sae.encode_workspace_bytes(r.Q * r.nq, r.kq))
    S.s3_sae_encode_topk(sae, xq.to(d), r.kq, q_ids, q_vals, ws)
    assert S.s3_workspace_status(ws) == 0
    qi_h, qv_h = q_ids.cpu().numpy(), q_vals.cpu().numpy()
    rows = np.unique(np.concatenate([np.arange(0, 512), np.arange(8000, 8256), np.arange(r.Q * r.nq - 256, r.Q * r.nq)]))
    qstats = {}
    pre = O.preact(xq[rows].float().numpy(), Wf, be, bd)
    check_topk_against_preact(pre, qi_h[rows], qv_h[rows], r.kq, TOL_BF16, qstats)
    assert_tight(qstats)
    qi4 = qi_h.reshape(1, r.Q, r.nq, r.kq)
    qv4 = qv_h.reshape(1, r.Q, r.nq, r.kq)

    sample = [0, 1, 2, 3, 31, 32, 63, 64, 65, 100, 127, 128, 129, 191, 200, 222, 253, 254, 255, 77]
    sws = S.new_workspace(64)
    for rc in (C.CFG4, C.CFG4_S64):
        ns = C.n_spans(cfg.L, rc.width, rc.stride)
        assert ns == (2045 if rc.stride == 16 else 512)
        bm = G.gamma21(rc.bm25_seed, rc.Q, ns)
        alls = torch.zeros((rc.Q, ns), dtype=torch.float32, device=d)
        ti, ts = S.s3_coactivation_score_topspans(csr, D, cfg.L, q_ids.view(1, rc.Q, rc.nq, rc.kq), q_vals.view(1, rc.Q, rc.nq, rc.kq),
                                                  rc.width, rc.stride, rc.s, rc.alpha, rc.beta, sws, bm.to(d), all_scores=alls)
        assert S.s3_workspace_status(sws) == 0
        ti, ts, alls = ti.cpu().numpy(), ts.cpu().numpy(), alls.cpu().numpy()
        co = O.score_spans(ctx_ids[None], qi4[:, sample], qv4[:, sample], D, rc.width, rc.stride, 0)
        oi, os_, oall = O.fuse_select(co, bm.numpy()[sample], rc.alpha, rc.beta, rc.s)
        np.testing.assert_array_equal(alls[sample], oall)
        np.testing.assert_array_equal(ti[sample], oi)
        np.testing.assert_array_equal(ts[sample], os_)
        for qi in range(rc.Q):                           # every query: its spans are the best of its own scores, in order
            order = np.lexsort((np.arange(ns), -alls[qi]))[:rc.s]
            assert ti[qi].tolist() == order.tolist()
            np.testing.assert_array_equal(ts[qi], alls[qi][order])
    pipe.close()


def test_cfg5_scan_16_chunks_flat_memory_and_zipf_lists():
    cfg = C.CFG5
    d = _dev()
    n_chunks = 16
    k, D, chunk, nl = cfg.key.k, cfg.key.d_sae, cfg.chunk, cfg.n_layers
    inp = C.ScanInputs(cfg, device=d)
    saes = [S.Sae(*inp.sae("key", l)) for l in range(nl)]
    pipe = ScanPipeline([SaeSlot("key", saes, k, chunk)])
    pipe.reserve_index(n_chunks * chunk)
    xs = [[inp.x("key", l, c * chunk, chunk) for l in range(nl)] for c in range(n_chunks)]      # 2 GB, made up front
    torch.cuda.synchronize()
    gc.collect()

    marks = {}
    for c in range(n_chunks):
        pipe.scan_chunk(c * chunk, {"key": xs[c]})
        if c == 1:
            torch.cuda.synchronize()
            marks["alloc"] = torch.cuda.memory_allocated()
            marks["free"] = torch.cuda.mem_get_info()[0]          # cudaMemGetInfo: what the driver itself has handed out
            torch.cuda.reset_peak_memory_stats()
    pipe.finish()
    torch.cuda.synchronize()
    # Sec. 3.4 / memory-complexity proposition: bounded by the chunk, independent of the tokens scanned
    assert torch.cuda.max_memory_allocated() <= marks["alloc"]
    assert torch.cuda.memory_allocated() <= marks["alloc"]
    assert torch.cuda.mem_get_info()[0] >= marks["free"]

    L_scanned = n_chunks * chunk
    st = pipe.slots[0].index.stats()
    assert st["n_postings"] == L_scanned * k * nl                 # P = L * layers * k
    assert st["n_positions"] == L_scanned
    for l in (0, nl - 1):
        rp, ps, _ = pipe.slots[0].index.export_csr(l)
        rp = rp.numpy().astype(np.int64)
        lens = np.sort(np.diff(rp))[::-1].astype(np.float64)
        assert int(rp[-1]) == L_scanned * k
        # every list ascending
        pos = ps.numpy()
        starts = rp[:-1][np.diff(rp) > 0]
        d1 = np.diff(pos.astype(np.int64))
        d1[starts[1:] - 1] = 1
        assert (d1 > 0).all()
        # the popular features' lists fall off like rank^-1.1 over the chance level of an unpopular feature
        chance = np.median(lens)
        top = lens[:32] - chance
        slope = np.polyfit(np.log(np.arange(1, 33)), np.log(top), 1)[0]
        assert abs(slope + cfg.zipf_exponent) <= 0.15, slope
    pipe.close()
