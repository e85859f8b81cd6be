"""GPU parity of the SAE training step (fp32): gradients of the batch-mean squared reconstruction error through the Top-k
code against the fp64 oracle on the same active set, the Adam update, and two full steps (encode -> backward -> Adam) whose
parameters stay with the oracle's. Tolerances: the gradients are sums of up to T*k fp32 products added by atomics in no
fixed order, compared at 1e-4 of the sum of the terms' magnitudes (bounded here by a multiple of the largest entry); Adam is
elementwise fp32, 1e-6 relative."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S

pytestmark = pytest.mark.gpu


# the hyper-parameters as the fp32 values the library receives, so that both sides compute with the same numbers
LR, B1, B2, EPS = (float(np.float32(v)) for v in (1e-3, 0.9, 0.999, 1e-8))


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def _params(seed, d_in, d_sae):
    g = torch.Generator().manual_seed(seed)
    W_enc = torch.randn((d_in, d_sae), generator=g) / d_in ** 0.5
    W_enc = W_enc / W_enc.norm(dim=0, keepdim=True)
    b_enc = torch.randn(d_sae, generator=g) * 0.05
    W_dec = W_enc.t().contiguous() + torch.randn((d_sae, d_in), generator=g) * 0.02
    b_dec = torch.randn(d_in, generator=g) * 0.05
    return [W_enc.contiguous(), b_enc, W_dec, b_dec]


def gpu_encode(params, x, k):
    d = _dev()
    W_enc, b_enc, _, b_dec = params
    sae = S.Sae(W_enc, b_enc, b_dec)
    T = x.shape[0]
    ids = torch.empty((T, k), dtype=torch.int32, device=d)
    vals = torch.empty((T, k), dtype=torch.float32, device=d)
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k), d)
    S.s3_sae_encode_topk(sae, x, k, ids, vals, ws)
    torch.cuda.synchronize()
    sae.close()
    return ids, vals


def close(got, want, rel):
    got, want = got.cpu().numpy().astype(np.float64), np.asarray(want)
    bound = rel * (np.abs(want).max() + 1e-12) * 8
    assert np.abs(got - want).max() <= bound, (np.abs(got - want).max(), bound)


@pytest.mark.parametrize("T,d_in,d_sae,k", [(64, 32, 256, 8), (300, 128, 1024, 32), (130, 72, 500, 5), (40, 512, 2048, 64)])
def test_backward_matches_oracle(T, d_in, d_sae, k):
    d = _dev()
    params = [p.to(d) for p in _params(T, d_in, d_sae)]
    x = torch.randn((T, d_in), generator=torch.Generator().manual_seed(T + 1)).to(d)
    ids, vals = gpu_encode(params, x, k)
    loss, gWe, gbe, gWd, gbd = S.s3_sae_backward(params[0], params[2], params[3], x, ids, vals)
    torch.cuda.synchronize()
    want = O.sae_loss_and_grads(x.cpu().numpy(), *[p.cpu().numpy() for p in params], ids.cpu().numpy())
    assert abs(float(loss) - want[0]) <= 1e-5 * want[0]
    for got, w in zip((gWe, gbe, gWd, gbd), want[1:]):
        close(got, w, 1e-4)


@pytest.mark.parametrize("T,d_in,d_sae,k", [(300, 128, 1024, 32), (100, 64, 4096, 128)])
def test_backward_with_a_bf16_forward_pass(T, d_in, d_sae, k):
    """The tensor cores pick the active set from bf16 copies of the parameters; the gradient is taken in fp32 on the
    fp32 parameters with the code recomputed for that set, which is what the oracle does with the same ids."""
    d = _dev()
    params = [p.to(d) for p in _params(T + 7, d_in, d_sae)]
    x = torch.randn((T, d_in), generator=torch.Generator().manual_seed(T)).to(d)
    W16 = S.s3_cast_f32_to_bf16(params[0])
    assert torch.equal(W16, params[0].to(torch.bfloat16))                   # round to nearest even, like the library cast
    sae = S.Sae(W16, params[1], params[3])
    ids = torch.empty((T, k), dtype=torch.int32, device=d)
    vals = torch.empty((T, k), dtype=torch.float32, device=d)
    ws = S.new_workspace(sae.encode_workspace_bytes(T, k), d)
    S.s3_sae_encode_topk(sae, S.s3_cast_f32_to_bf16(x), k, ids, vals, ws)
    loss, gWe, gbe, gWd, gbd = S.s3_sae_backward(params[0], params[2], params[3], x, ids, None, b_enc=params[1])
    torch.cuda.synchronize()
    want = O.sae_loss_and_grads(x.cpu().numpy(), *[p.cpu().numpy() for p in params], ids.cpu().numpy())
    assert abs(float(loss) - want[0]) <= 1e-5 * want[0]
    for got, w in zip((gWe, gbe, gWd, gbd), want[1:]):
        close(got, w, 1e-4)
    with pytest.raises(S.S3Error):
        S.s3_sae_backward(params[0], params[2], params[3], x, ids, None)     # neither vals nor b_enc


def test_adam_matches_oracle_over_steps():
    d = _dev()
    rng = np.random.default_rng(0)
    n = 10007
    p = rng.standard_normal(n).astype(np.float32)
    m, v = np.zeros(n), np.zeros(n)
    pg, mg, vg = torch.from_numpy(p).to(d), torch.zeros(n, device=d), torch.zeros(n, device=d)
    po = p.astype(np.float64)
    g_abs = np.zeros(n)                                                    # what the moments' rounding errors scale with
    for step in range(1, 6):
        g = (rng.standard_normal(n) * 10.0 ** rng.integers(-4, 2, size=n)).astype(np.float32)
        g[::100] = 0.0
        g_abs += np.abs(g)
        S.s3_adam_update(pg, mg, vg, torch.from_numpy(g).to(d), LR, B1, B2, EPS, step)
        po, m, v = O.adam_update(po, m, v, g, LR, B1, B2, EPS, step)
    torch.cuda.synchronize()
    np.testing.assert_allclose(pg.cpu().numpy(), po, rtol=2e-6, atol=2e-7)
    assert (np.abs(mg.cpu().numpy() - m) <= 5e-7 * g_abs + 1e-30).all()     # m mixes gradients of both signs: absolute bound
    np.testing.assert_allclose(vg.cpu().numpy(), v, rtol=1e-5, atol=1e-30)
    with pytest.raises(S.S3Error):
        S.s3_adam_update(pg, mg, vg, pg.clone(), LR, B1, B2, EPS, 0)


def test_two_training_steps_follow_the_oracle_and_reduce_the_loss():
    d = _dev()
    T, d_in, d_sae, k = 512, 64, 512, 16
    params = [p.to(d) for p in _params(5, d_in, d_sae)]
    ref = [p.cpu().numpy().astype(np.float64) for p in params]
    moments = [(torch.zeros_like(p), torch.zeros_like(p)) for p in params]
    ref_m = [(np.zeros(p.shape), np.zeros(p.shape)) for p in ref]
    x = torch.randn((T, d_in), generator=torch.Generator().manual_seed(6)).to(d)
    lr = LR                                                               # the paper's learning rate
    losses = []
    for step in (1, 2, 3):
        ids, vals = gpu_encode(params, x, k)
        loss, gWe, gbe, gWd, gbd = S.s3_sae_backward(params[0], params[2], params[3], x, ids, vals)
        losses.append(float(loss))
        # the oracle steps from its own parameters on the active set the GPU selected
        o = O.sae_loss_and_grads(x.cpu().numpy(), *ref, ids.cpu().numpy())
        assert abs(losses[-1] - o[0]) <= 1e-4 * o[0]
        for i, g in enumerate((gWe, gbe, gWd, gbd)):
            S.s3_adam_update(params[i], moments[i][0], moments[i][1], g, lr, B1, B2, EPS, step)
            ref[i], m, v = O.adam_update(ref[i], ref_m[i][0], ref_m[i][1], o[1 + i], lr, B1, B2, EPS, step)
            ref_m[i] = (m, v)
    torch.cuda.synchronize()
    assert losses[2] < losses[1] < losses[0]
    for p, r in zip(params, ref):
        # Adam's step is lr * sign-like: parameters that received a gradient moved by about 3 * lr; agreement to a small
        # fraction of that (entries whose tiny gradients round differently may differ by a fraction of lr)
        assert np.abs(p.cpu().numpy() - r).max() < 0.5 * lr


def test_backward_error_paths():
    d = _dev()
    W = torch.zeros((8, 16), device=d)
    Wd = torch.zeros((16, 8), device=d)
    b = torch.zeros(8, device=d)
    x = torch.zeros((4, 8), device=d)
    ids = torch.zeros((4, 2), dtype=torch.int32, device=d)
    vals = torch.zeros((4, 2), device=d)
    with pytest.raises(S.S3Error):
        S.s3_sae_backward(W, Wd, b, x, ids, vals, ws=torch.zeros(64, dtype=torch.uint8, device=d))
