"""The encode entry point for callers that cannot allocate device memory (s3_sae_encode_topk_static).

Such callers (a serving loop with a frozen memory pool, a plugin that only receives its input and output
buffers) cannot give the library a workspace, so this entry point keeps its scratch in a fixed array that
is part of the library. The test calls it through the C ABI twice in a row, with different inputs and
sizes so that the second call runs over the first call's leftovers in the shared array, and checks both
results against the regular entry point (same kernels, so ids must be identical and values must agree
within the encode tolerance the other GPU tests use). It also checks that an input too large for the
array is refused with a capacity error instead of being run.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import gc

import numpy as np
import pytest
import torch

import paper_2601_17702_b200 as S
from paper_2601_17702_b200 import binding as B
from workloads import generators as G

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _regular(sae, x, k):
    T = x.shape[0]
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k))
    ids = torch.full((T, k), -7, dtype=torch.int32, device=x.device)
    vals = torch.full((T, k), -7.0, dtype=torch.float32, device=x.device)
    S.s3_sae_encode_topk(sae, x, k, ids, vals, ws)
    assert S.s3_workspace_status(ws) == 0
    return ids.cpu().numpy(), vals.cpu().numpy()


def _static(sae, x, k):
    T = x.shape[0]
    ids = torch.full((T, k), -9, dtype=torch.int32, device=x.device)
    vals = torch.full((T, k), -9.0, dtype=torch.float32, device=x.device)
    status = torch.full((1,), 77, dtype=torch.int32, device=x.device)
    gc.collect()                                            # no tensor of an earlier test is freed inside the window
    before = torch.cuda.memory_allocated()
    S.s3_sae_encode_topk_static(sae, x, k, ids, vals, status)
    assert torch.cuda.memory_allocated() <= before          # nothing was allocated through torch either
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return ids.cpu().numpy(), vals.cpu().numpy()


def test_static_scratch_encode_matches_regular_entry_point_twice_in_a_row():
    assert torch.cuda.is_available()
    d = torch.device("cuda:0")
    d_in, d_sae = 256, 4096
    W, b_enc, b_dec = G.sae_weights(31, 0, d_in, d_sae, torch.bfloat16)
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    # first call: 200 tokens at k = 32 (two row blocks, the second ragged); second call: fewer tokens, another k,
    # other data
    for seed, T, k in ((41, 200, 32), (42, 100, 8)):
        x = G.activations(seed, 0, 0, T, d_in, torch.bfloat16).to(d)
        got_ids, got_vals = _static(sae, x, k)
        ref_ids, ref_vals = _regular(sae, x, k)
        np.testing.assert_array_equal(got_ids, ref_ids)
        err = np.abs(got_vals.astype(np.float64) - ref_vals) / (np.abs(ref_vals.astype(np.float64)) + 1.0)
        assert err.max() <= TOL_BF16


def test_static_scratch_refuses_what_does_not_fit():
    assert torch.cuda.is_available()
    d = torch.device("cuda:0")
    d_in, d_sae, k = 64, 4096, 64
    W, b_enc, b_dec = G.sae_weights(33, 0, d_in, d_sae, torch.bfloat16)
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    T = 1
    while sae.encode_workspace_bytes(T, k) <= B.S3_STATIC_SCRATCH_BYTES:
        T *= 2
    x = torch.zeros((T, d_in), dtype=torch.bfloat16, device=d)
    ids = torch.empty((T, k), dtype=torch.int32, device=d)
    vals = torch.empty((T, k), dtype=torch.float32, device=d)
    with pytest.raises(S.S3Error) as e:
        S.s3_sae_encode_topk_static(sae, x, k, ids, vals)
    assert e.value.code == B.S3_ERR_CAPACITY
    assert "built-in" in str(e.value)
