"""The upstream projection fused with the per-head encode (K = h W_K for one head kept on the SM as the encode GEMM's
token operand) against the chain it replaces: s3_sae_preact with bf16 output, then s3_sae_encode_topk on the
[T * heads, 128] view. Both chains round K to bf16 from the same fp32 sums, so ids and values agree bit for bit; the
codes are also checked against the CPU oracle's pre-activations of the projected rows."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from parity import check_topk_against_preact
from workloads import generators as G

pytestmark = pytest.mark.gpu
TOL_BF16 = 2e-2


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


@pytest.mark.parametrize("T,d_model,H,d_sae,k", [
    (200, 128, 1, 512, 8),            # one head, one row tile, two column tiles
    (700, 512, 4, 2048, 16),          # ragged last row tile
    (1000, 1024, 8, 16384, 32),       # Llama-3-8B-like: 8 KV heads of 128, expansion 128
    (300, 4096, 2, 16384, 128),       # the paper's per-head SAE: k = 128
])
def test_fused_projection_encode_equals_projection_then_encode(T, d_model, H, d_sae, k):
    d = _dev()
    g = torch.Generator().manual_seed(T + d_model)
    Wp = (torch.randn((d_model, H * 128), generator=g) / d_model ** 0.5).to(torch.bfloat16)
    bp = (torch.randn(H * 128, generator=g) * 0.1).float()
    W, b_enc, b_dec = G.sae_weights(900 + H, 0, 128, d_sae, torch.bfloat16)
    h = G.activations(901, 0, 0, T, d_model, torch.bfloat16)
    proj = S.Sae(Wp.to(d), bp.to(d), torch.zeros(d_model, device=d))
    sae = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))
    h_d = h.to(d)

    # the chain: projection written out as bf16, then the encode reads it head by head
    x = S.s3_sae_preact(proj, h_d, torch.bfloat16)
    rows = x.view(T * H, 128)
    ids1 = torch.full((T * H, k), -7, dtype=torch.int32, device=d)
    vals1 = torch.full((T * H, k), -7.0, dtype=torch.float32, device=d)
    ws1 = S.new_workspace(sae.encode_workspace_bytes(T * H, k))
    S.s3_sae_encode_topk(sae, rows, k, ids1, vals1, ws1)
    assert S.s3_workspace_status(ws1) == 0

    # fused
    ids2 = torch.full((T, H, k), -9, dtype=torch.int32, device=d)
    vals2 = torch.full((T, H, k), -9.0, dtype=torch.float32, device=d)
    ws2 = S.new_workspace(S.s3_sae_project_encode_workspace_bytes(sae, T, H, k))
    for _ in range(2):                                   # the second launch runs over the first one's leftovers
        S.s3_sae_project_encode_topk(proj, sae, h_d, H, k, ids2, vals2, ws2)
        assert S.s3_workspace_status(ws2) == 0
        np.testing.assert_array_equal(ids2.view(T * H, k).cpu().numpy(), ids1.cpu().numpy())
        np.testing.assert_array_equal(vals2.view(T * H, k).cpu().numpy(), vals1.cpu().numpy())

    # against the oracle: the encoder's pre-activations of sampled projected rows
    sample = np.unique(np.concatenate([np.arange(0, min(64, T * H)), np.arange(T * H - min(64, T * H), T * H),
                                       np.arange(T * H // 2, min(T * H // 2 + 32, T * H))]))
    pre = O.preact(rows[sample].float().cpu().numpy(), W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    check_topk_against_preact(pre, ids2.view(T * H, k).cpu().numpy()[sample], vals2.view(T * H, k).cpu().numpy()[sample], k, TOL_BF16)
    # and the projection itself against the oracle (bf16 rounding of an fp32 sum)
    hs = np.unique(np.concatenate([np.arange(0, min(16, T)), np.arange(T - min(16, T), T)]))
    ref = O.preact(h[hs].float().numpy(), Wp.float().numpy(), bp.numpy(), np.zeros(d_model, np.float32))
    got = x[hs].float().cpu().numpy()
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1.0)) <= 1e-2


def test_fused_projection_encode_argument_checks():
    d = _dev()
    W, b_enc, b_dec = G.sae_weights(5, 0, 64, 256, torch.bfloat16)
    narrow = S.Sae(W.to(d), b_enc.to(d), b_dec.to(d))                     # d_in = 64: not a 128-wide head
    Wp = torch.zeros((128, 128), dtype=torch.bfloat16, device=d)
    proj = S.Sae(Wp, torch.zeros(128, device=d), torch.zeros(128, device=d))
    h = torch.zeros((8, 128), dtype=torch.bfloat16, device=d)
    ids = torch.empty((8, 1, 4), dtype=torch.int32, device=d)
    vals = torch.empty((8, 1, 4), dtype=torch.float32, device=d)
    with pytest.raises(S.S3Error) as e:
        S.s3_sae_project_encode_topk(proj, narrow, h, 1, 4, ids, vals, S.new_workspace(1 << 20))
    assert e.value.code == S.binding.S3_ERR_UNSUPPORTED
