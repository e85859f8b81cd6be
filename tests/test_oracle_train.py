"""Pins of the oracle's SAE training step: the analytic gradients against central finite differences of an independently
written loss (active set fixed), special cases with known gradients, and Adam's closed forms."""
import numpy as np

import oracle as O


def _setup(seed=0, T=7, d=6, D=20, k=4):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d))
    W_enc = rng.standard_normal((d, D)) / d ** 0.5
    b_enc = rng.standard_normal(D) * 0.1 + 1.0            # keeps the selected pre-activations positive
    W_dec = rng.standard_normal((D, d)) / d ** 0.5
    b_dec = rng.standard_normal(d) * 0.1
    ids = np.stack([rng.permutation(D)[:k] for _ in range(T)]).astype(np.int32)
    ids[2, -1] = -1
    return x, W_enc, b_enc, W_dec, b_dec, ids


def _loss(x, W_enc, b_enc, W_dec, b_dec, ids):
    # written densely and separately from the oracle: a masked code matrix times the dictionary
    T, D = x.shape[0], W_enc.shape[1]
    pre = (x - b_dec) @ W_enc + b_enc
    mask = np.zeros((T, D))
    for t in range(T):
        mask[t, ids[t][ids[t] >= 0]] = 1.0
    x_hat = (pre * mask) @ W_dec + b_dec
    return ((x_hat - x) ** 2).sum() / T


def test_gradients_match_finite_differences():
    x, W_enc, b_enc, W_dec, b_dec, ids = _setup()
    loss, gWe, gbe, gWd, gbd = O.sae_loss_and_grads(x, W_enc, b_enc, W_dec, b_dec, ids)
    assert abs(loss - _loss(x, W_enc, b_enc, W_dec, b_dec, ids)) < 1e-12
    params = dict(W_enc=W_enc, b_enc=b_enc, W_dec=W_dec, b_dec=b_dec)
    grads = dict(W_enc=gWe, b_enc=gbe, W_dec=gWd, b_dec=gbd)
    rng = np.random.default_rng(1)
    h = 1e-6
    for name, p in params.items():
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in p.shape)
            plus, minus = {k: v.copy() for k, v in params.items()}, {k: v.copy() for k, v in params.items()}
            plus[name][idx] += h
            minus[name][idx] -= h
            fd = (_loss(x, plus["W_enc"], plus["b_enc"], plus["W_dec"], plus["b_dec"], ids) -
                  _loss(x, minus["W_enc"], minus["b_enc"], minus["W_dec"], minus["b_dec"], ids)) / (2 * h)
            assert abs(fd - grads[name][idx]) < 1e-6 * (1 + abs(fd)), (name, idx, fd, grads[name][idx])


def test_perfect_reconstruction_has_zero_gradients():
    # orthonormal dictionary with all of +-Q active where positive: x_hat = x, so loss and every gradient vanish
    rng = np.random.default_rng(2)
    d = 5
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    W_enc = np.concatenate([Q, -Q], axis=1)
    x = rng.standard_normal((4, d))
    pre = x @ W_enc
    ids = np.stack([np.nonzero(pre[t] > 0)[0][:d] for t in range(4)]).astype(np.int32)
    loss, *grads = O.sae_loss_and_grads(x, W_enc, np.zeros(2 * d), W_enc.T.copy(), np.zeros(d), ids)
    assert loss < 1e-25 and all(np.abs(g).max() < 1e-12 for g in grads)


def test_inactive_features_get_no_gradient_and_bias_only_case():
    x, W_enc, b_enc, W_dec, b_dec, ids = _setup(seed=3)
    _, gWe, gbe, gWd, _ = O.sae_loss_and_grads(x, W_enc, b_enc, W_dec, b_dec, ids)
    unused = np.setdiff1d(np.arange(W_enc.shape[1]), ids[ids >= 0])
    assert unused.size and (gWe[:, unused] == 0).all() and (gbe[unused] == 0).all() and (gWd[unused] == 0).all()
    # no active feature at all: x_hat = b_dec, loss = mean ||b_dec - x||^2, gb_dec = 2 mean (b_dec - x)
    none = np.full_like(ids, -1)
    loss, gWe, gbe, gWd, gbd = O.sae_loss_and_grads(x, W_enc, b_enc, W_dec, b_dec, none)
    np.testing.assert_allclose(loss, ((b_dec - x) ** 2).sum() / len(x), rtol=1e-14)
    np.testing.assert_allclose(gbd, 2 * (b_dec - x).mean(axis=0), rtol=1e-13)
    assert not gWe.any() and not gbe.any() and not gWd.any()


def test_adam_closed_forms():
    g = np.array([0.5, -2.0, 0.0, 1e-3])
    p0 = np.array([1.0, 1.0, 1.0, 1.0])
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    p, m, v = O.adam_update(p0, np.zeros(4), np.zeros(4), g, lr, b1, b2, eps, 1)
    np.testing.assert_allclose(p, p0 - lr * g / (np.abs(g) + eps), rtol=1e-12)      # first step: m_hat = g, v_hat = g^2
    np.testing.assert_allclose(m, 0.1 * g)
    np.testing.assert_allclose(v, 0.001 * g * g)
    for step in (2, 3, 4):                                                          # a constant gradient keeps m_hat = g
        p_prev = p
        p, m, v = O.adam_update(p, m, v, g, lr, b1, b2, eps, step)
        np.testing.assert_allclose(p, p_prev - lr * g / (np.abs(g) + eps), rtol=1e-9)
    assert p[2] == 1.0                                                              # zero gradient: untouched
