"""GPU parity: every kernel of the path, called through the C ABI, against the CPU oracle on the same
seeded inputs. Integer results (postings, co-activation counts, selected spans) must be bit-exact;
encode values must satisfy max |dz| / (|z| + 1) <= 2e-2 (bf16 inputs, fp32 accumulate) or <= 1e-5 (fp32
inputs), and Top-k id sets must agree outside the near-tie band of the same width."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from parity import assert_tight, check_topk_against_preact, csr_equal
from workloads import configs as C, generators as G

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-5


def dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def gpu_encode(W, b_enc, b_dec, x, k, n_slices=0, max_ctas=0):
    d = dev()
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    sae.set_schedule(n_slices, max_ctas)
    T = x.shape[0]
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k))
    ids = torch.full((T, k), -7, dtype=torch.int32, device=d)
    vals = torch.full((T, k), -7.0, dtype=torch.float32, device=d)
    S.s3_sae_encode_topk(sae, x.to(d), k, ids, vals, ws)
    assert S.s3_workspace_status(ws) == 0
    return ids.cpu().numpy(), vals.cpu().numpy()


def gpu_postings(ids, d_sae, pos_base=0, vals=None):
    d = dev()
    T, k = ids.shape
    ids_d = torch.as_tensor(ids, dtype=torch.int32).to(d).contiguous()
    row_ptr = torch.full((d_sae + 1,), -1, dtype=torch.int32, device=d)
    pos = torch.full((max(T * k, 1),), -1, dtype=torch.int32, device=d)
    vals_d = pval = None
    if vals is not None:
        vals_d = torch.as_tensor(vals, dtype=torch.float32).to(d).contiguous()
        pval = torch.zeros(max(T * k, 1), dtype=torch.float32, device=d)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(T, k, d_sae))
    S.s3_postings_build(ids_d, d_sae, pos_base, row_ptr, pos, ws, vals_d, pval)
    assert S.s3_workspace_status(ws) == 0
    rp = row_ptr.cpu().numpy().astype(np.int64)
    n = int(rp[-1])
    return rp, pos.cpu().numpy()[:n], (None if pval is None else pval.cpu().numpy()[:n])


# ------------------------------------------------------------------------------------ encode, fp32 path

def test_cfg1_encode_fp32_full():
    cfg = C.CFG1
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("key", 0)
    x = inp.x("key", 0, 0, cfg.L)
    pre = O.preact(x.numpy(), W.numpy(), b_enc.numpy(), b_dec.numpy())
    for n_slices in (0, 1, 3):
        ids, vals = gpu_encode(W, b_enc, b_dec, x, cfg.key.k, n_slices)
        check_topk_against_preact(pre, ids, vals, cfg.key.k, TOL_F32)
    oi, ov = O.topk(pre, cfg.key.k)
    ids, vals = gpu_encode(W, b_enc, b_dec, x, cfg.key.k)
    assert (ids == oi).mean() > 0.999          # fp32 vs fp64: practically always the very same ids


@pytest.mark.parametrize("T,d_in,d_sae,k", [(1, 8, 16, 1), (130, 24, 200, 5), (257, 100, 1000, 64), (64, 128, 129, 17),
                                            (100, 32, 600, 128)])
def test_encode_fp32_shapes(T, d_in, d_sae, k):
    rng = np.random.default_rng(T + d_in)
    x = torch.from_numpy(rng.standard_normal((T, d_in)).astype(np.float32))
    W, b_enc, b_dec = G.sae_weights(T, 0, d_in, d_sae, torch.float32)
    pre = O.preact(x.numpy(), W.numpy(), b_enc.numpy(), b_dec.numpy())
    ids, vals = gpu_encode(W, b_enc, b_dec, x, k)
    check_topk_against_preact(pre, ids, vals, k, TOL_F32)


def test_encode_fp32_degenerate_rows():
    # identity SAE: pre = x. Rows with no / few positives, zeros, ties.
    D = 64
    x = torch.zeros(6, D)
    x[0] = -1.0                                   # nothing positive
    x[1, :3] = torch.tensor([3.0, 1.0, 2.0])      # three positives, rest zero
    x[2] = 1.0                                    # all tied
    x[3] = torch.arange(D, dtype=torch.float32) - 10.0
    x[4, 5::7] = 2.5                              # duplicated values
    x[5, 63] = 1e-30                              # tiny but strictly positive
    W = torch.eye(D)
    z = torch.zeros(D)
    ids, vals = gpu_encode(W, z, z, x, 8)
    oi, ov = O.encode_topk(x.numpy(), W.numpy(), z.numpy(), z.numpy(), 8)
    np.testing.assert_array_equal(ids, oi)
    np.testing.assert_array_equal(vals, ov)
    assert (ids[0] == -1).all() and ids[1].tolist() == [0, 2, 1, -1, -1, -1, -1, -1]
    assert ids[2].tolist() == list(range(8))


# ------------------------------------------------------------------------------------ encode, tensor-core path

@pytest.mark.parametrize("T,d_in,d_sae,k,n_slices", [
    (128, 64, 256, 8, 0),          # one tile, one k-block
    (300, 128, 1024, 8, 0),        # ragged row tile
    (300, 192, 1000, 16, 2),       # ragged K (192 = 3 k-blocks) and ragged column tile
    (1000, 1024, 4096, 32, 0),
    (640, 512, 8192, 16, 5),
    (257, 256, 2048, 64, 3),
    (96, 72, 264, 1, 0),           # smaller than every tile; d_in, d_sae only multiples of 8
    (300, 128, 16384, 128, 0),     # the paper's per-head SAE: d_head 128, expansion 128, k = 128
    (260, 256, 4096, 128, 3),      # k = 128, the largest supported, over several slices
    (64, 64, 136, 128, 0),         # k close to d_sae
    (300, 128, 16384, 128, 16),    # sixteen short lists of k = 128 survivors each: far more candidates than the merge's buffer
    (200, 128, 16384, 96, 11),
])
def test_encode_bf16_shapes(T, d_in, d_sae, k, n_slices):
    x = G.activations(11, 0, 0, T, d_in, torch.bfloat16)
    W, b_enc, b_dec = G.sae_weights(T + d_sae, 0, d_in, d_sae, torch.bfloat16)
    pre = O.preact(x.float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    ids, vals = gpu_encode(W, b_enc, b_dec, x, k, n_slices)
    check_topk_against_preact(pre, ids, vals, k, TOL_BF16)
    # tighter than the acceptance bound: fp32 accumulation of exact bf16 products
    oi, ov = O.topk(pre, k)
    same = ids == oi
    assert same.mean() > 0.98
    assert np.abs(vals[same] - ov[same]).max() < 2e-3


def test_encode_bf16_degenerate_rows():
    """Rows that defeat the streaming bound on the tensor-core path: every feature tied (the candidate lists overflow
    and fall back to the exact cut), no positive value, fewer positives than k, a plateau of ties around the k-th value.
    Exactly representable values, so ids and values must equal the oracle's."""
    d_in, D, k = 64, 4096, 32
    W = torch.zeros((d_in, D))
    W[0, :] = 1.0                                         # pre[t, f] = x[t, 0] + b_enc[f]
    W[1, 100:140] = 1.0                                   # features 100..139 also see x[t, 1]
    b_enc = torch.zeros(D)
    b_enc[2000:2100] = 0.5                                # a plateau of 100 tied features above the rest
    x = torch.zeros((6, d_in))
    x[0, 0] = 1.0                                         # all 4096 tied at 1.0, plateau at 1.5
    x[1, 0] = -1.0                                        # plateau at -0.5: nothing positive
    x[2, 0] = -0.25                                       # only the plateau (0.25) is positive: 100 ties, k = 32 of them
    x[3, 0] = -1.0
    x[3, 1] = 1.25                                        # 40 positives (0.25) only through the second input
    x[4, 0] = 2.0
    x[4, 1] = -1.0                                        # 40 features one below the rest
    # row 5: all zero -> pre = b_enc: plateau 0.5, rest 0 (not positive)
    for n_slices in (0, 1, 4):
        ids, vals = gpu_encode(W.to(torch.bfloat16), b_enc, torch.zeros(d_in), x.to(torch.bfloat16), k, n_slices)
        oi, ov = O.encode_topk(x.numpy(), W.numpy(), b_enc.numpy(), np.zeros(d_in, np.float32), k)
        np.testing.assert_array_equal(ids, oi)
        np.testing.assert_array_equal(vals, ov)
    assert ids[0].tolist() == list(range(2000, 2032)) and (ids[1] == -1).all()
    assert ids[3].tolist() == list(range(100, 132)) and ids[5].tolist() == list(range(2000, 2032))


def test_encode_bf16_result_independent_of_schedule():
    T, d_in, d_sae, k = 512, 256, 4096, 32
    x = G.activations(12, 0, 0, T, d_in, torch.bfloat16)
    W, b_enc, b_dec = G.sae_weights(77, 0, d_in, d_sae, torch.bfloat16)
    ref = gpu_encode(W, b_enc, b_dec, x, k, 1)
    for n_slices, max_ctas in ((2, 0), (7, 0), (16, 0), (4, 3), (0, 1)):
        got = gpu_encode(W, b_enc, b_dec, x, k, n_slices, max_ctas)
        np.testing.assert_array_equal(got[0], ref[0])
        np.testing.assert_array_equal(got[1], ref[1])


def test_encode_bf16_strided_input_and_ties():
    # x given as a column slice of a wider matrix (row pitch > d_in); identity-like SAE makes exact ties
    T, d_in, d_sae, k = 200, 64, 128, 8
    wide = G.activations(13, 0, 0, T, 2 * d_in, torch.bfloat16)
    W = torch.zeros(d_in, d_sae)
    W[:, :d_in] = torch.eye(d_in)
    W[:, d_in:] = torch.eye(d_in)              # feature f and f+64 always tie
    W = W.to(torch.bfloat16)
    z = torch.zeros(d_sae)
    zi = torch.zeros(d_in)
    d = dev()
    sae = S.Sae(W.to(d), z.to(d), zi.to(d))
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k))
    ids = torch.empty((T, k), dtype=torch.int32, device=d)
    vals = torch.empty((T, k), dtype=torch.float32, device=d)
    xs = wide.to(d)[:, :d_in]
    assert xs.stride(0) == 2 * d_in
    S.s3_sae_encode_topk(sae, xs, k, ids, vals, ws)
    assert S.s3_workspace_status(ws) == 0
    oi, ov = O.encode_topk(wide[:, :d_in].float().numpy(), W.float().numpy(), z.numpy(), zi.numpy(), k)
    np.testing.assert_array_equal(ids.cpu().numpy(), oi)     # exact products: ties resolved by lower id
    np.testing.assert_array_equal(vals.cpu().numpy(), ov)


def test_cfg2_chunk_encode_sampled_rows():
    cfg = C.CFG2
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("key", 0)
    chunk = 5                                   # one chunk out of the middle of the 32K context
    x = inp.x("key", 0, chunk * cfg.chunk, cfg.chunk)
    ids, vals = gpu_encode(W, b_enc, b_dec, x, cfg.key.k)
    rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(2000, 2064), np.arange(cfg.chunk - 62, cfg.chunk)]))
    pre = O.preact(x[rows].float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    stats = {}
    check_topk_against_preact(pre, ids[rows], vals[rows], cfg.key.k, TOL_BF16, stats)
    assert_tight(stats)
    assert (ids >= 0).all()


def test_cfg3_query_sae_sampled_rows():
    cfg = C.CFG3
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("query", 1)
    T = 1024
    x = inp.x("query", 1, 3 * cfg.chunk, T)
    ids, vals = gpu_encode(W, b_enc, b_dec, x, cfg.query.k)
    rows = np.concatenate([np.arange(0, 40), np.arange(500, 540), np.arange(T - 40, T)])
    pre = O.preact(x[rows].float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    stats = {}
    check_topk_against_preact(pre, ids[rows], vals[rows], cfg.query.k, TOL_BF16, stats)
    assert_tight(stats)


def test_cfg5_zipf_chunk_sampled_rows():
    cfg = C.CFG5
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("key", 2)
    x = inp.x("key", 2, 7 * cfg.chunk, cfg.chunk)
    ids, vals = gpu_encode(W, b_enc, b_dec, x, cfg.key.k)
    rows = np.concatenate([np.arange(0, 128), np.arange(8000, 8128), np.arange(cfg.chunk - 128, cfg.chunk)])
    pre = O.preact(x[rows].float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    stats = {}
    check_topk_against_preact(pre, ids[rows], vals[rows], cfg.key.k, TOL_BF16, stats)
    assert_tight(stats)
    # full-size postings of the skewed chunk, bit-exact against the oracle on the GPU's own ids
    rp, pos, _ = gpu_postings(ids, cfg.key.d_sae, 7 * cfg.chunk)
    orp, opos, _ = O.postings(ids, cfg.key.d_sae, 7 * cfg.chunk)
    csr_equal(rp, pos, orp, opos)
    lens = np.diff(rp)
    assert lens.max() > 20 * lens.mean()        # the popular features really are popular


# ------------------------------------------------------------------------------------ postings

def _rand_ids(T, k, d_sae, seed, hot=None):
    rng = np.random.default_rng(seed)
    keys = rng.random((T, d_sae)) if d_sae <= 4096 else None
    if keys is not None:
        if hot is not None:
            keys[:, :hot] *= 0.05
        ids = np.argsort(keys, axis=1)[:, :k].astype(np.int32)
    else:
        ids = np.stack([rng.choice(d_sae, size=k, replace=False) for _ in range(T)]).astype(np.int32)
    return ids


@pytest.mark.parametrize("T,k,d_sae,base", [
    (1, 1, 1, 0), (7, 3, 10, 5), (2048, 8, 1024, 0), (4096, 32, 16384, 12288), (1000, 64, 32768, 999),
    (5000, 1, 49152, 0), (513, 16, 8192, 2**31 - 1 - 513),
])
def test_postings_random(T, k, d_sae, base):
    ids = _rand_ids(T, k, d_sae, T * k + d_sae)
    if T > 4:
        ids[1, k // 2:] = -1
        ids[3, :] = -1
    rp, pos, _ = gpu_postings(ids, d_sae, base)
    orp, opos, _ = O.postings(ids, d_sae, base)
    csr_equal(rp, pos, orp, opos)


def test_postings_skewed_and_giant_list():
    T, k, d_sae = 3000, 8, 512
    ids = _rand_ids(T, k, d_sae, 3, hot=4)      # 4 features present in most tokens
    ids[:, 0] = 7                               # one feature in every token: a list of T entries
    for t in range(T):                          # keep ids distinct within a token
        dup = np.flatnonzero(ids[t, 1:] == 7)
        for j in dup:
            ids[t, 1 + j] = -1
    vals = np.random.default_rng(4).random((T, k)).astype(np.float32)
    rp, pos, pval = gpu_postings(ids, d_sae, 100, vals)
    orp, opos, opval = O.postings(ids, d_sae, 100, vals)
    csr_equal(rp, pos, orp, opos)
    np.testing.assert_array_equal(pval, opval)
    assert rp[8] - rp[7] == T


def test_postings_list_longer_than_one_sort_and_values():
    # 64 features, one per bucket: feature 5 sits in every token (a list of 20000 entries, longer than what one
    # shared-memory sort holds), the others are short; values travel with the positions
    T, k, d_sae = 20000, 4, 64
    rng = np.random.default_rng(11)
    ids = np.stack([rng.choice(np.delete(np.arange(d_sae), 5), size=k, replace=False) for _ in range(T)]).astype(np.int32)
    ids[:, 2] = 5
    ids[17, 3] = -1
    vals = rng.random((T, k)).astype(np.float32)
    rp, pos, pval = gpu_postings(ids, d_sae, 4096, vals)
    orp, opos, opval = O.postings(ids, d_sae, 4096, vals)
    csr_equal(rp, pos, orp, opos)
    np.testing.assert_array_equal(pval, opval)
    assert rp[6] - rp[5] == T


def test_postings_skewed_buckets_need_several_sweeps():
    # 24 hot features inside one bucket of 256, each in a third of the tokens: the bucket holds many times what one
    # shared-memory sort takes and is sorted by ranges of its features
    T, k, d_sae = 6000, 16, 4096
    rng = np.random.default_rng(12)
    ids = np.full((T, k), -1, np.int32)
    for t in range(T):
        hot = 256 + rng.choice(24, size=8, replace=False)
        cold = rng.choice(np.concatenate([np.arange(256), np.arange(512, d_sae)]), size=8, replace=False)
        ids[t] = rng.permutation(np.concatenate([hot, cold]))
    rp, pos, _ = gpu_postings(ids, d_sae, 77)
    orp, opos, _ = O.postings(ids, d_sae, 77)
    csr_equal(rp, pos, orp, opos)


def test_postings_more_runs_than_the_segment_table():
    # 17.6 M pairs in one item: more token runs than a bucket block keeps in shared memory
    T, k, d_sae = 1_100_000, 16, 8192
    t = np.arange(T, dtype=np.int64)[:, None]
    j = np.arange(k, dtype=np.int64)[None, :]
    ids = ((t * 7 + (t // 1000) * 3 + j * 131) % d_sae).astype(np.int32)       # distinct within a token: 131 j < d_sae
    rp, pos, _ = gpu_postings(ids, d_sae, 5)
    orp, opos, _ = O.postings(ids, d_sae, 5)
    csr_equal(rp, pos, orp, opos)


def test_postings_repeated_id_in_a_token_is_reported():
    d = dev()
    ids = torch.tensor([[3, 3], [1, 2]], dtype=torch.int32, device=d)
    rp = torch.zeros(9, dtype=torch.int32, device=d)
    ps = torch.zeros(4, dtype=torch.int32, device=d)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(2, 2, 8))
    S.s3_postings_build(ids, 8, 0, rp, ps, ws)
    with pytest.raises(S.binding.S3Error) as e:
        S.s3_workspace_status(ws)
    assert e.value.code == S.binding.S3_ERR_INVALID_ARG
    assert rp.cpu().tolist()[-1] == 4          # nothing is dropped and nothing is written out of range


def test_postings_empty_inputs():
    rp, pos, _ = gpu_postings(np.zeros((0, 4), np.int32), 64, 0)
    assert (rp == 0).all() and len(pos) == 0
    rp, pos, _ = gpu_postings(-np.ones((50, 4), np.int32), 64, 0)
    assert (rp == 0).all() and len(pos) == 0


def test_postings_batched_and_deterministic():
    d = dev()
    items, outs, refs = [], [], []
    shapes = [(512, 32, 16384), (300, 64, 32768), (0, 8, 128), (2000, 16, 8192), (700, 8, 40000)]
    for i, (T, k, d_sae) in enumerate(shapes):
        ids = _rand_ids(T, k, d_sae, 100 + i) if T else np.zeros((0, k), np.int32)
        ids_d = torch.as_tensor(ids).to(d)
        rp = torch.zeros(d_sae + 1, dtype=torch.int32, device=d)
        ps = torch.zeros(max(T * k, 1), dtype=torch.int32, device=d)
        items.append(S.make_postings_item(ids_d, d_sae, 1000 * i, rp, ps))
        outs.append((ids_d, rp, ps))
        refs.append(O.postings(ids, d_sae, 1000 * i))
    ws = S.new_workspace(sum(S.s3_postings_workspace_bytes(T, k, D) for T, k, D in shapes))
    S.s3_postings_build_batched(items, ws)
    first = [(rp.cpu().numpy().copy(), ps.cpu().numpy().copy()) for _, rp, ps in outs]
    for (rp, ps), (orp, opos, _) in zip(first, refs):
        csr_equal(rp, ps, orp, opos)
    S.s3_postings_build_batched(items, ws)      # run-to-run identical bits
    for (rp0, ps0), (_, rp, ps) in zip(first, outs):
        np.testing.assert_array_equal(rp0, rp.cpu().numpy())
        np.testing.assert_array_equal(ps0, ps.cpu().numpy())
    assert S.s3_workspace_status(ws) == 0


def test_postings_bad_feature_id_is_reported_not_written():
    d = dev()
    ids = torch.tensor([[1, 2], [3, 99]], dtype=torch.int32, device=d)
    rp = torch.zeros(9, dtype=torch.int32, device=d)
    ps = torch.zeros(4, dtype=torch.int32, device=d)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(2, 2, 8))
    S.s3_postings_build(ids, 8, 0, rp, ps, ws)
    with pytest.raises(S.binding.S3Error) as e:
        S.s3_workspace_status(ws)
    assert e.value.code == S.binding.S3_ERR_INVALID_ARG
    assert rp.cpu().tolist()[-1] == 3


# ------------------------------------------------------------------------------------ index

def test_index_append_export_matches_oracle_merge():
    d = dev()
    d_sae, k, n_layers = 2048, 8, 2
    chunks = [(0, 700), (700, 300), (1000, 1024), (2024, 1)]
    ix = S.Index(n_layers, d_sae, pinned_slab_bytes=1 << 20)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(1024, k, d_sae))
    ref = {l: [] for l in range(n_layers)}
    row_ptr = torch.zeros(d_sae + 1, dtype=torch.int32, device=d)
    pos = torch.zeros(1024 * k, dtype=torch.int32, device=d)
    for ci, (base, T) in enumerate(chunks):
        for l in range(n_layers):
            ids = _rand_ids(T, k, d_sae, 1000 * l + ci)
            ref[l].append(O.postings(ids, d_sae, base)[:2])
            ix.stream_wait()                               # the copy of the previous chunk must be done
            S.s3_postings_build(torch.as_tensor(ids).to(d), d_sae, base, row_ptr, pos, ws)
            ix.append(l, row_ptr, pos, T, k, base)
    ix.sync()
    st = ix.stats()
    assert st["n_chunks"] == len(chunks) * n_layers and st["n_positions"] == 2025
    assert st["n_postings"] == sum(int(r[0][-1]) for l in ref for r in ref[l])
    for l in range(n_layers):
        rp, ps, _ = ix.export_csr(l)
        orp, opos = O.index_merge(ref[l], d_sae)
        csr_equal(rp.numpy(), ps.numpy(), orp, opos)
    with pytest.raises(S.binding.S3Error) as e:            # a chunk that goes back in position
        ix.append(0, row_ptr, pos, 10, k, 5)
    assert e.value.code == S.binding.S3_ERR_STATE
    ix.close()


# ------------------------------------------------------------------------------------ scoring

def gpu_score(ctx_ids, q_ids, q_vals, d_sae, width, stride, s, alpha, beta, bm25=None, mode=0, stop_freq=0, split=False):
    """split: give the call the full workspace, so that the few queries of these tests are cut over many blocks each."""
    d = dev()
    n_layers, L, k = ctx_ids.shape
    layers = []
    for l in range(n_layers):
        rp, pos, _ = O.postings(ctx_ids[l], d_sae, 0)      # identical id sets on both sides
        pos = pos if len(pos) else np.zeros(1, np.int32)
        layers.append((torch.as_tensor(rp.astype(np.int64)).to(d), torch.as_tensor(pos).to(d)))
    ns = C.n_spans(L, width, stride)
    Q = q_ids.shape[1]
    alls = torch.zeros((Q, max(ns, 1)), dtype=torch.float32, device=d)
    ws = S.new_workspace(S.s3_score_workspace_bytes(Q, q_ids.shape[2], q_ids.shape[3], n_layers, ns, s) if split else 64)
    ws[64:] = 0xA5                              # whatever an earlier call left there must not matter
    bm = None if bm25 is None else torch.as_tensor(bm25).to(d).contiguous()
    ti, ts = S.s3_coactivation_score_topspans(layers, d_sae, L, torch.as_tensor(q_ids).to(d).contiguous(),
                                              torch.as_tensor(q_vals).to(d).contiguous(), width, stride, s, alpha, beta,
                                              ws, bm, mode, stop_freq, all_scores=alls)
    assert S.s3_workspace_status(ws) == 0
    return ti.cpu().numpy(), ts.cpu().numpy(), alls.cpu().numpy()[:, :ns]


@pytest.mark.parametrize("L,k,d_sae,n_layers,Q,nq,kq,width,stride,s", [
    (8, 2, 8, 1, 1, 2, 2, 4, 4, 2),
    (2048, 8, 1024, 1, 1, 16, 8, 64, 64, 4),
    (1000, 8, 256, 3, 5, 7, 8, 64, 16, 16),
    (777, 4, 64, 2, 3, 5, 4, 48, 20, 8),       # width not a multiple of stride
    (500, 4, 64, 1, 2, 3, 4, 10, 25, 64),      # gaps between spans; s larger than n_spans
    (30, 4, 64, 1, 2, 3, 4, 64, 16, 4),        # no full span at all
    (12000, 4, 32, 1, 2, 5, 4, 64, 16, 8),     # hot features with lists longer than one warp's share
    (9000, 4, 16, 2, 2, 3, 4, 50, 30, 8),      # long lists, stride not a power of two, width not a multiple
    (5000, 8, 16, 1, 2, 40, 8, 64, 8, 8),      # features shared by many query tokens (large cQ), 8 spans per position
])
def test_score_mincount_exact(L, k, d_sae, n_layers, Q, nq, kq, width, stride, s):
    ctx = np.stack([_rand_ids(L, k, d_sae, 50 + l, hot=3) for l in range(n_layers)])
    q = np.stack([_rand_ids(Q * nq, kq, d_sae, 80 + l, hot=3).reshape(Q, nq, kq) for l in range(n_layers)])
    q[0, 0, 0, -1] = -1
    qv = np.random.default_rng(9).random(q.shape).astype(np.float32)
    ns = C.n_spans(L, width, stride)
    bm = G.gamma21(4, Q, max(ns, 1)).numpy()[:, :ns] if ns else None
    co = O.score_spans(ctx, q, qv, d_sae, width, stride, 0)
    for alpha, beta, b in ((1.0, 0.0, None), (0.5, 0.5, bm)):
        if ns == 0:
            b = None
        oi, os_, oall = O.fuse_select(co, b, alpha, beta, s)
        for split in (False, True):
            ti, ts, alls = gpu_score(ctx, q, qv, d_sae, width, stride, s, alpha, beta, b, split=split)
            np.testing.assert_array_equal(alls, oall)
            np.testing.assert_array_equal(ti, oi)
            np.testing.assert_array_equal(ts, os_)


def test_score_weighted_mode():
    L, k, d_sae, n_layers, Q, nq, kq, width, stride, s = 600, 8, 128, 2, 4, 6, 8, 64, 16, 8
    ctx = np.stack([_rand_ids(L, k, d_sae, 150 + l, hot=3) for l in range(n_layers)])
    q = np.stack([_rand_ids(Q * nq, kq, d_sae, 180 + l, hot=3).reshape(Q, nq, kq) for l in range(n_layers)])
    qv = (np.random.default_rng(19).random(q.shape) * 3).astype(np.float32)
    for stop in (0, 400):
        w = O.score_spans(ctx, q, qv, d_sae, width, stride, 1, stop)
        _, _, oall = O.fuse_select(w, None, 1.0, 0.0, s)
        ti, ts, alls = gpu_score(ctx, q, qv, d_sae, width, stride, s, 1.0, 0.0, None, 1, stop)
        np.testing.assert_allclose(alls, oall, rtol=1e-5, atol=1e-6)
        for qi in range(Q):                       # the selected spans are the best ones of the GPU's own scores
            order = sorted(range(alls.shape[1]), key=lambda j: (-float(alls[qi, j]), j))[:s]
            assert ti[qi].tolist() == order
        # the weights are summed as fixed-point integers: the same bits from run to run and however the query is
        # cut over thread blocks
        for split in (False, True, True):
            ti2, ts2, alls2 = gpu_score(ctx, q, qv, d_sae, width, stride, s, 1.0, 0.0, None, 1, stop, split=split)
            np.testing.assert_array_equal(alls2, alls)
            np.testing.assert_array_equal(ti2, ti)
            np.testing.assert_array_equal(ts2, ts)


def test_score_weighted_wide_weight_range():
    """Activations spread over five decades: spans that hold a large weight agree with the fp64 sum to 1e-5; the fixed-point
    grid lies 2^-40 below the query's largest weight."""
    L, k, d_sae, Q, nq, kq, width, stride, s = 3000, 8, 256, 2, 6, 8, 64, 16, 8
    ctx = _rand_ids(L, k, d_sae, 250)[None]
    q = _rand_ids(Q * nq, kq, d_sae, 251).reshape(1, Q, nq, kq)
    qv = (10.0 ** np.random.default_rng(29).uniform(-3, 2, q.shape)).astype(np.float32)
    w = O.score_spans(ctx, q, qv, d_sae, width, stride, 1, 0)
    _, _, oall = O.fuse_select(w, None, 1.0, 0.0, s)
    _, _, alls = gpu_score(ctx, q, qv, d_sae, width, stride, s, 1.0, 0.0, None, 1, 0)
    np.testing.assert_allclose(alls, oall, rtol=1e-5, atol=0)


def test_hand_example_on_gpu(golden_dir):
    import os
    from conftest import read_golden
    g = read_golden(os.path.join(golden_dir, "coactivation_hand_example.txt"))
    toks = np.array(g["tokens"], np.int32).reshape(1, -1, 2)
    q = np.array(g["query"], np.int32).reshape(1, 1, -1, 2)
    bm = np.array([[float(v) for v in g["bm25"]]], np.float32)
    ti, ts, alls = gpu_score(toks, q, np.ones(q.shape, np.float32), 8, 4, 4, 2, 0.5, 0.5, bm)
    assert alls[0].tolist() == [2.0, 3.0] and ti[0].tolist() == [1, 0] and ts[0].tolist() == [3.0, 2.0]
    rp, pos, _ = gpu_postings(toks[0], 8, 0)
    assert rp.tolist() == [int(v) for v in g["row_ptr"]] and pos.tolist() == [int(v) for v in g["pos"]]


# ------------------------------------------------------------------------------------ whole scan, config 1

def test_cfg1_scan_and_retrieval_end_to_end():
    cfg, r = C.CFG1, C.CFG1_RETR
    d = dev()
    inp = C.ScanInputs(cfg)
    W, b_enc, b_dec = inp.sae("key", 0)
    x = inp.x("key", 0, 0, cfg.L)
    xq = inp.retrieval_queries(0, r.Q, r.nq)
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    k, D = cfg.key.k, cfg.key.d_sae
    ws = S.new_workspace(sae.encode_workspace_bytes(cfg.L, k))
    ids = torch.empty((cfg.L, k), dtype=torch.int32, device=d)
    vals = torch.empty((cfg.L, k), dtype=torch.float32, device=d)
    S.s3_sae_encode_topk(sae, x.to(d), k, ids, vals, ws)
    row_ptr = torch.zeros(D + 1, dtype=torch.int32, device=d)
    pos = torch.zeros(cfg.L * k, dtype=torch.int32, device=d)
    S.s3_postings_build(ids, D, 0, row_ptr, pos, S.new_workspace(S.s3_postings_workspace_bytes(cfg.L, k, D)))
    ix = S.Index(1, D, 1 << 20)
    ix.append(0, row_ptr, pos, cfg.L, k, 0)
    rp, ps, _ = ix.export_csr(0)
    assert ix.stats()["n_postings"] == cfg.L * k        # P = L * layers * k
    qi = torch.empty((r.Q * r.nq, r.kq), dtype=torch.int32, device=d)
    qv = torch.empty((r.Q * r.nq, r.kq), dtype=torch.float32, device=d)
    S.s3_sae_encode_topk(sae, xq.to(d), r.kq, qi, qv, ws)   # queries go through the key SAE (shared codebook)
    ti, ts = S.s3_coactivation_score_topspans([(rp.to(d), ps.to(d))], D, cfg.L, qi.view(1, r.Q, r.nq, r.kq),
                                              qv.view(1, r.Q, r.nq, r.kq), r.width, r.stride, r.s, r.alpha, r.beta, ws)
    assert S.s3_workspace_status(ws) == 0
    # oracle chain on the GPU's own ids (identical id sets => bit-exact downstream)
    ids_h, qi_h, qv_h = ids.cpu().numpy(), qi.cpu().numpy(), qv.cpu().numpy()
    orp, opos, _ = O.postings(ids_h, D, 0)
    csr_equal(rp.numpy(), ps.numpy(), orp, opos)
    co = O.score_spans(ids_h[None], qi_h.reshape(1, r.Q, r.nq, r.kq), qv_h.reshape(1, r.Q, r.nq, r.kq), D, r.width, r.stride, 0)
    oi, os_, _ = O.fuse_select(co, None, r.alpha, r.beta, r.s)
    np.testing.assert_array_equal(ti.cpu().numpy(), oi)
    np.testing.assert_array_equal(ts.cpu().numpy(), os_)
    # and the oracle's own ids agree with the GPU's on this fp32 config
    pre = O.preact(x.numpy(), W.numpy(), b_enc.numpy(), b_dec.numpy())
    check_topk_against_preact(pre, ids_h, vals.cpu().numpy(), k, TOL_F32)
    ix.close()


# ------------------------------------------------------------------------------------ grouped encode

def test_grouped_encode_equals_the_single_calls_bit_for_bit():
    """Several encoders of unequal shape, input length and k in one grouped launch (Alg. 1 Phase 1: the layers'
    SAEs of one chunk): every item's ids and values are those of its own s3_sae_encode_topk call, and those match
    the oracle. An empty item is skipped."""
    d = dev()
    shapes = [(700, 256, 4096, 32), (300, 1024, 8192, 64), (513, 128, 2048, 8), (0, 64, 512, 4), (1000, 512, 16384, 16),
              (260, 64, 1024, 128), (90, 192, 1000, 16)]
    saes, xs, xs_d, outs, items = [], [], [], [], []
    for i, (T, d_in, d_sae, k) in enumerate(shapes):
        W, b_enc, b_dec = G.sae_weights(300 + i, 0, d_in, d_sae, torch.bfloat16)
        x = G.activations(400 + i, 0, 0, max(T, 1), d_in, torch.bfloat16)[:T]
        sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
        ids = torch.full((T, k), -5, dtype=torch.int32, device=d)
        vals = torch.full((T, k), -5.0, dtype=torch.float32, device=d)
        saes.append((sae, W, b_enc, b_dec))
        xs.append(x)
        outs.append((ids, vals))
        xs_d.append(x.to(d))
        items.append(S.make_encode_item(sae, xs_d[-1], k, ids, vals))
    ws = S.new_workspace(S.s3_sae_encode_grouped_workspace_bytes(items))
    S.s3_sae_encode_topk_grouped(items, ws)
    assert S.s3_workspace_status(ws) == 0
    for (T, d_in, d_sae, k), (sae, W, b_enc, b_dec), x, (ids, vals) in zip(shapes, saes, xs, outs):
        if T == 0:
            continue
        ids1, vals1 = gpu_encode(W, b_enc, b_dec, x, k)
        np.testing.assert_array_equal(ids.cpu().numpy(), ids1)
        np.testing.assert_array_equal(vals.cpu().numpy(), vals1)
        pre = O.preact(x.float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
        check_topk_against_preact(pre, ids.cpu().numpy(), vals.cpu().numpy(), k, TOL_BF16)
    # a second launch over the leftovers of the first, limited to a few thread blocks, gives the same bits
    for ids, vals in outs:
        ids.fill_(-9)
    S.s3_sae_encode_topk_grouped(items, ws, max_ctas=20)
    for (T, d_in, d_sae, k), (sae, W, b_enc, b_dec), x, (ids, vals) in zip(shapes, saes, xs, outs):
        if T:
            np.testing.assert_array_equal(ids.cpu().numpy(), gpu_encode(W, b_enc, b_dec, x, k)[0])
