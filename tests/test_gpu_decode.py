"""GPU parity of the SAE decode (Sec. 3.3: x_hat = z_hat W_dec + b_dec) and the per-token reconstruction error against
the fp64 oracle on the same (id, value) pairs. Tolerance: k <= 64 fp32 FMAs per output, so |error| <= 1e-5 of the
sum of the terms' magnitudes (k * 2^-24 = 4e-6 at k = 64); the squared error, a sum of d_in fp32 squares, 1e-4 relative
(plus the same bound applied to the differences)."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def _case(T, k, D, d, dtype, seed, pad=True):
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn((D, d), generator=g) / d ** 0.5).to(dtype)
    b = torch.randn(d, generator=g) * 0.1
    x = torch.randn((T, d), generator=g).to(dtype)
    ids = torch.rand((T, D), generator=g).topk(k, dim=1).indices.to(torch.int32)
    vals = torch.rand((T, k), generator=g) * 3
    if pad and T > 2:
        ids[1, k // 2:] = -1
        vals[1, k // 2:] = 0
        ids[2, :] = -1
    return W, b, x, ids, vals


def check(T, k, D, d, dtype, seed=0):
    W, b, x, ids, vals = _case(T, k, D, d, dtype, seed)
    dev = _dev()
    xh, err = S.s3_sae_decode(W.to(dev), b.to(dev), ids.to(dev), vals.to(dev), x.to(dev))
    torch.cuda.synchronize()
    Wn, xn = W.float().numpy(), x.float().numpy()
    oxh, oerr = O.decode(ids.numpy(), vals.numpy(), Wn, b.numpy(), xn)
    z = np.zeros((T, D))
    for t in range(T):
        for j in range(k):
            if ids[t, j] >= 0:
                z[t, ids[t, j]] = vals[t, j]
    scale = np.abs(z) @ np.abs(Wn).astype(np.float64) + np.abs(b.numpy())
    assert (np.abs(xh.cpu().numpy() - oxh) <= 1e-5 * scale + 1e-30).all()
    diff_bound = 2 * np.abs(xn - oxh) * 1e-5 * scale
    np.testing.assert_allclose(err.cpu().numpy(), oerr, rtol=1e-4, atol=float(diff_bound.sum(axis=1).max()) + 1e-12)
    only_err = S.s3_sae_decode(W.to(dev), b.to(dev), ids.to(dev), vals.to(dev), x.to(dev), want_xhat=False)
    assert only_err[0] is None and torch.equal(only_err[1], err)


@pytest.mark.parametrize("T,k,D,d,dtype", [
    (5, 2, 16, 8, torch.bfloat16),
    (300, 32, 2048, 1024, torch.bfloat16),      # the key SAE's width and k
    (70, 64, 4096, 4096, torch.bfloat16),       # the query SAE's width and k: several column passes
    (33, 7, 100, 72, torch.bfloat16),           # k not a multiple of the unroll, ragged column pass
    (40, 8, 64, 24, torch.float32),
    (9, 64, 512, 1028, torch.float32),
])
def test_decode_parity(T, k, D, d, dtype):
    check(T, k, D, d, dtype)


def test_decode_hand_example():
    dev = _dev()
    W = torch.tensor([[1, 0, 2, 0], [0, 1, -1, 0], [3, 3, 3, 0], [0.5, 0, 0, 0]], dtype=torch.float32, device=dev)
    b = torch.tensor([10, 20, 30, 0], dtype=torch.float32, device=dev)
    ids = torch.tensor([[2, 0], [1, -1]], dtype=torch.int32, device=dev)
    vals = torch.tensor([[2.0, 0.5], [4.0, 0.0]], dtype=torch.float32, device=dev)
    x = torch.tensor([[16.5, 26, 36, 0], [10, 24, 26, 0]], dtype=torch.float32, device=dev)
    xh, err = S.s3_sae_decode(W, b, ids, vals, x)
    assert xh.cpu().tolist() == [[16.5, 26.0, 37.0, 0.0], [10.0, 24.0, 26.0, 0.0]]
    assert err.cpu().tolist() == [1.0, 0.0]


def test_encode_then_decode_reconstructs_an_orthonormal_dictionary():
    # W_enc = [Q, -Q], W_dec = W_enc^T: the code of x keeps at most d positive coefficients and decodes back to x
    dev = _dev()
    d = 64
    g = torch.Generator().manual_seed(5)
    Q, _ = torch.linalg.qr(torch.randn((d, d), generator=g, dtype=torch.float64))
    W_enc = torch.cat([Q, -Q], dim=1).float().contiguous()
    x = torch.randn((50, d), generator=g)
    sae = S.Sae(W_enc.to(dev), torch.zeros(2 * d, device=dev), torch.zeros(d, device=dev))
    ids = torch.empty((50, 64), dtype=torch.int32, device=dev)
    vals = torch.empty((50, 64), dtype=torch.float32, device=dev)
    ws = S.new_workspace(sae.encode_workspace_bytes(50, 64), dev)
    S.s3_sae_encode_topk(sae, x.to(dev), 64, ids, vals, ws)
    xh, err = S.s3_sae_decode(W_enc.t().contiguous().to(dev), torch.zeros(d, device=dev), ids, vals, x.to(dev))
    assert float((xh.cpu() - x).abs().max()) < 1e-4 and float(err.max()) < 1e-6


def test_decode_error_paths():
    dev = _dev()
    W = torch.zeros((16, 12), dtype=torch.bfloat16, device=dev)       # d_in not a multiple of 8
    b = torch.zeros(12, device=dev)
    ids = torch.zeros((2, 2), dtype=torch.int32, device=dev)
    vals = torch.zeros((2, 2), device=dev)
    with pytest.raises(S.S3Error):
        S.s3_sae_decode(W, b, ids, vals)
    W = torch.zeros((16, 16), dtype=torch.bfloat16, device=dev)
    b = torch.zeros(16, device=dev)
    with pytest.raises(S.S3Error):
        S.s3_sae_decode(W, b, ids, vals, None, want_xhat=False)         # nothing wanted
    big = torch.zeros((2, 129), dtype=torch.int32, device=dev)
    with pytest.raises(S.S3Error):
        S.s3_sae_decode(W, b, big, torch.zeros((2, 129), device=dev))
