"""GPU parity of the head aggregation (sum of a feature's activations over a token's heads in fp32, head order, then
Top-k) against the CPU oracle: both sides add in the same precision and order, so ids and values agree exactly."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def gpu(ids, vals, D, k_out):
    d = _dev()
    oi, ov = S.s3_head_aggregate_topk(torch.as_tensor(ids).to(d).contiguous(), torch.as_tensor(vals).to(d).contiguous(), D, k_out)
    torch.cuda.synchronize()
    return oi.cpu().numpy(), ov.cpu().numpy()


def test_hand_example():
    ids = np.array([[[5, 2, 9], [7, 5, 9]]], np.int32)
    vals = np.array([[[1.0, 2.5, 0.5], [3.0, 2.0, 0.25]]], np.float32)
    oi, ov = gpu(ids, vals, 16, 6)
    assert oi.tolist() == [[5, 7, 2, 9, -1, -1]] and ov.tolist() == [[3.0, 3.0, 2.5, 0.75, 0.0, 0.0]]


@pytest.mark.parametrize("T,H,k,D,k_out", [
    (50, 8, 32, 16384, 32),       # 8 KV heads, the key SAE's k
    (20, 32, 64, 32768, 64),      # 32 query heads at k = 64: 2048 entries per token
    (33, 3, 5, 40, 7),            # entry count not a power of two, heavy overlap between heads
    (10, 1, 16, 100, 16),         # one head: identity
    (7, 4, 8, 64, 40),            # more outputs wanted than unique features
    (300, 8, 128, 16384, 128),    # the paper's k = 128 per head: 1024 entries per token
    (300, 4, 128, 16384, 128),    # 512 entries per token, the largest one warp takes
])
def test_parity(T, H, k, D, k_out):
    rng = np.random.default_rng(T + H)
    hot = max(2 * k, D // 50)      # the heads agree on a small set of features most of the time
    ids = np.empty((T, H, k), np.int32)
    for t in range(T):
        for h in range(H):
            pool = np.concatenate([rng.permutation(hot)[: (3 * k) // 4], hot + rng.permutation(D - hot)[: k - (3 * k) // 4]])
            ids[t, h] = pool
    vals = (rng.random((T, H, k)) * 4).astype(np.float32)
    ids[0, 0, k // 2:] = -1
    ids[1 % T] = -1                                                       # a token without any feature
    want_i, want_v = O.head_aggregate(ids, vals, k_out)
    got_i, got_v = gpu(ids, vals, D, k_out)
    np.testing.assert_array_equal(got_i, want_i)
    np.testing.assert_array_equal(got_v, want_v)


def test_feeds_the_postings_builder():
    d = _dev()
    rng = np.random.default_rng(3)
    T, H, k, D = 64, 4, 8, 256
    ids = np.stack([np.stack([rng.permutation(D)[:k] for _ in range(H)]) for _ in range(T)]).astype(np.int32)
    vals = rng.random((T, H, k)).astype(np.float32)
    oi, _ = S.s3_head_aggregate_topk(torch.as_tensor(ids).to(d), torch.as_tensor(vals).to(d), D, k)
    rp = torch.zeros(D + 1, dtype=torch.int32, device=d)
    pos = torch.zeros(T * k, dtype=torch.int32, device=d)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(T, k, D), d)
    S.s3_postings_build(oi, D, 0, rp, pos, ws)
    want_i, _ = O.head_aggregate(ids, vals, k)
    orp, opos, _ = O.postings(want_i, D, 0)
    np.testing.assert_array_equal(rp.cpu().numpy(), orp)
    np.testing.assert_array_equal(pos.cpu().numpy()[: len(opos)], opos)


def test_error_paths():
    d = _dev()
    ids = torch.zeros((2, 65, 64), dtype=torch.int32, device=d)            # H*k = 4160 > 4096
    with pytest.raises(S.S3Error):
        S.s3_head_aggregate_topk(ids, torch.zeros(ids.shape, device=d), 100, 8)
    ids = torch.zeros((2, 2, 4), dtype=torch.int32, device=d)
    with pytest.raises(S.S3Error):
        S.s3_head_aggregate_topk(ids, torch.zeros(ids.shape, device=d), 100, 0)
