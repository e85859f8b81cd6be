"""GPU parity of the dense pre-activation / projection call (Eq. 1 before the ReLU; with zero biases the key projection
K = W_K h) against the fp64 oracle: the bf16 tolerance of the encode (fp32 accumulation of exact bf16 products), and the
bf16 output equal to the fp32 output rounded to nearest even."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from workloads import generators as G

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


@pytest.mark.parametrize("T,d_in,d_sae,n_slices", [
    (128, 64, 256, 0),
    (300, 192, 1000, 2),          # ragged rows, ragged K, ragged last column tile
    (1000, 1024, 4096, 0),
    (96, 72, 264, 0),             # smaller than every tile
    (513, 4096, 1024, 3),         # the key projection's shape (d_model 4096 -> 8 heads x 128)
])
def test_preact_matches_oracle(T, d_in, d_sae, n_slices):
    d = _dev()
    x = G.activations(21, 0, 0, T, d_in, torch.bfloat16)
    W, b_enc, b_dec = G.sae_weights(T + d_sae, 0, d_in, d_sae, torch.bfloat16)
    pre = O.preact(x.float().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    sae.set_schedule(n_slices, 0)
    full = torch.full((T, d_sae + 8), -777.0, dtype=torch.float32, device=d)
    out32 = full[:, :d_sae]                                                                     # pitched output
    S.s3_sae_preact(sae, x.to(d), torch.float32, out32)
    out16 = S.s3_sae_preact(sae, x.to(d), torch.bfloat16)
    torch.cuda.synchronize()
    got = out32.cpu().numpy().astype(np.float64)
    assert (np.abs(got - pre) / (np.abs(pre) + 1.0)).max() <= TOL_BF16
    assert (np.abs(got - pre) / (np.abs(pre) + 1.0)).max() < 2e-3                               # in fact far inside it
    assert torch.equal(out16, out32.to(torch.bfloat16))
    assert float(full[:, d_sae:].min()) == -777.0 == float(full[:, d_sae:].max())               # nothing beyond d_sae


def test_projection_then_encode_chain():
    """K = h W_K (zero biases) written as bf16, then the SAE encode of K on the same stream: ids and values equal the
    encode of the same bf16 K computed separately (the chain adds nothing of its own)."""
    d = _dev()
    T, d_model, d_k, D, k = 700, 512, 256, 2048, 16
    h = G.activations(31, 0, 0, T, d_model, torch.bfloat16).to(d)
    Wk, _, _ = G.sae_weights(5, 0, d_model, d_k, torch.bfloat16)
    proj = S.Sae(Wk.to(d), torch.zeros(d_k, device=d), torch.zeros(d_model, device=d))
    W, b_enc, b_dec = G.sae_weights(6, 1, d_k, D, torch.bfloat16)
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    K = S.s3_sae_preact(proj, h, torch.bfloat16)
    ids = torch.empty((T, k), dtype=torch.int32, device=d)
    vals = torch.empty((T, k), dtype=torch.float32, device=d)
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k), d)
    S.s3_sae_encode_topk(sae, K, k, ids, vals, ws)
    torch.cuda.synchronize()
    want = O.preact(h.float().cpu().numpy(), Wk.float().numpy(), np.zeros(d_k, np.float32), np.zeros(d_model, np.float32))
    assert (np.abs(K.float().cpu().numpy() - want) / (np.abs(want) + 1.0)).max() <= TOL_BF16
    pre = O.preact(K.float().cpu().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    oi, ov = O.topk(pre, k)
    assert (ids.cpu().numpy() == oi).mean() > 0.98


def test_preact_error_paths():
    d = _dev()
    W, b_enc, b_dec = G.sae_weights(1, 0, 16, 64, torch.float32)
    sae32 = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    with pytest.raises(S.S3Error):
        S.s3_sae_preact(sae32, torch.zeros((4, 16), device=d))                                   # fp32 encoder
    W, b_enc, b_dec = G.sae_weights(1, 0, 16, 64, torch.bfloat16)
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    out = torch.empty((4, 70), dtype=torch.float32, device=d)[:, :64]                            # pitch 70 is not a multiple of 4
    with pytest.raises(S.S3Error):
        S.s3_sae_preact(sae, torch.zeros((4, 16), dtype=torch.bfloat16, device=d), torch.float32, out)
