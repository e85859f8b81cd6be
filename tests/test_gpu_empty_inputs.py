"""Empty and minimal inputs of the calls beside the benchmark path: every one of them is a no-op or a well-defined
smallest case, never an error or a stray write."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def test_zero_token_calls_are_no_ops():
    d = _dev()
    W = torch.zeros((16, 8), dtype=torch.bfloat16, device=d)
    b = torch.zeros(8, device=d)
    ids = torch.empty((0, 4), dtype=torch.int32, device=d)
    vals = torch.empty((0, 4), device=d)
    xh, err = S.s3_sae_decode(W, b, ids, vals, torch.empty((0, 8), dtype=torch.bfloat16, device=d))
    assert xh.shape == (0, 8) and err.shape == (0,)
    oi, ov = S.s3_head_aggregate_topk(torch.empty((0, 2, 4), dtype=torch.int32, device=d), torch.empty((0, 2, 4), device=d), 16, 4)
    assert oi.shape == (0, 4) and ov.shape == (0, 4)
    We = torch.zeros((8, 16), dtype=torch.bfloat16, device=d)
    sae = S.Sae(We, torch.zeros(16, device=d), torch.zeros(8, device=d))
    out = S.s3_sae_preact(sae, torch.empty((0, 8), dtype=torch.bfloat16, device=d))
    assert out.shape == (0, 16)
    idx, cnt = S.s3_fuse_index_sets(torch.empty((0, 3), dtype=torch.int32, device=d), 8, None, 1, 1, 100, 4,
                                    torch.zeros(256, dtype=torch.uint8, device=d))
    assert idx.shape == (0, 4) and cnt.shape == (0,)
    torch.cuda.synchronize()


def test_smallest_shapes():
    d = _dev()
    # one feature, one posting: a compact index of one block without payload
    c = S.s3_compact_build(torch.tensor([0, 1], dtype=torch.int64, device=d), torch.tensor([5], dtype=torch.int32, device=d), 1)
    assert c.blk_first.tolist() == [5] and c.blk_desc.tolist() == [0] and c.payload.tolist() == [0]
    rp, pos = S.s3_compact_expand(c, 1)
    assert rp.tolist() == [0, 1] and pos.tolist() == [5]
    # one token, one head, one feature
    oi, ov = S.s3_head_aggregate_topk(torch.tensor([[[3]]], dtype=torch.int32, device=d), torch.tensor([[[2.5]]], device=d), 8, 2)
    assert oi.tolist() == [[3, -1]] and ov.tolist() == [[2.5, 0.0]]
    # one position, everything selected
    idx, cnt = S.s3_fuse_index_sets(torch.tensor([[0]], dtype=torch.int32, device=d), 1, None, 0, 0, 1, 2,
                                    torch.zeros(S.s3_fuse_workspace_bytes(1, 1), dtype=torch.uint8, device=d))
    assert idx.tolist() == [[0, -1]] and cnt.tolist() == [1]
    # Adam on an empty tensor
    e = torch.empty(0, device=d)
    S.s3_adam_update(e, e.clone(), e.clone(), e.clone(), 1e-3, 0.9, 0.999, 1e-8, 1)
    # training gradients of a single token with a single active feature against the oracle
    W_enc = torch.tensor([[1.0, 0.5], [0.0, 2.0]], device=d)                  # d_in 2, d_sae 2
    W_dec = torch.tensor([[0.5, 0.0], [0.0, 0.25]], device=d)
    b_dec = torch.tensor([0.1, -0.1], device=d)
    b_enc = torch.tensor([0.2, 0.3], device=d)
    x = torch.tensor([[1.0, 2.0]], device=d)
    ids = torch.tensor([[1]], dtype=torch.int32, device=d)
    loss, gWe, gbe, gWd, gbd = S.s3_sae_backward(W_enc, W_dec, b_dec, x, ids, None, b_enc=b_enc)
    want = O.sae_loss_and_grads(x.cpu().numpy(), W_enc.cpu().numpy(), b_enc.cpu().numpy(), W_dec.cpu().numpy(), b_dec.cpu().numpy(),
                                ids.cpu().numpy())
    np.testing.assert_allclose(float(loss), want[0], rtol=1e-6)
    for got, w in zip((gWe, gbe, gWd, gbd), want[1:]):
        np.testing.assert_allclose(got.cpu().numpy(), w, rtol=1e-5, atol=1e-6)
