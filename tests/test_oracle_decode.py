"""Pins of the oracle's SAE decode (Sec. 3.3: x_hat = z_hat W_dec + b_dec): a hand example, the dense matrix
product of the scattered code (library routine), exact reconstruction through an orthonormal dictionary, padding,
and the error's closed forms."""
import numpy as np

import oracle as O


def test_hand_example():
    W_dec = np.array([[1, 0, 2], [0, 1, -1], [3, 3, 3], [0.5, 0, 0]], np.float32)        # 4 features, d_in 3
    b_dec = np.array([10, 20, 30], np.float32)
    ids = np.array([[2, 0], [1, -1]], np.int32)
    vals = np.array([[2.0, 0.5], [4.0, 0.0]], np.float32)
    # token 0: 2*(3,3,3) + 0.5*(1,0,2) + b = (16.5, 26, 37);  token 1: 4*(0,1,-1) + b = (10, 24, 26)
    x = np.array([[16.5, 26, 36], [10, 24, 26]], np.float32)
    xh, err = O.decode(ids, vals, W_dec, b_dec, x)
    assert xh.tolist() == [[16.5, 26.0, 37.0], [10.0, 24.0, 26.0]]
    assert err.tolist() == [1.0, 0.0]


def test_matches_dense_product_of_scattered_code():
    rng = np.random.default_rng(0)
    T, k, D, d = 37, 5, 64, 24
    ids = np.argsort(rng.random((T, D)), axis=1)[:, :k].astype(np.int32)
    vals = rng.random((T, k)).astype(np.float32)
    ids[3, 2:] = -1
    W_dec = rng.standard_normal((D, d)).astype(np.float32)
    b_dec = rng.standard_normal(d).astype(np.float32)
    z = np.zeros((T, D))
    for t in range(T):
        for j in range(k):
            if ids[t, j] >= 0:
                z[t, ids[t, j]] = vals[t, j]
    want = z @ W_dec.astype(np.float64) + b_dec
    x = rng.standard_normal((T, d)).astype(np.float32)
    xh, err = O.decode(ids, vals, W_dec, b_dec, x)
    np.testing.assert_allclose(xh, want, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(err, ((x - want) ** 2).sum(axis=1), rtol=1e-12)


def test_orthonormal_dictionary_reconstructs_through_the_encoder():
    # W_enc = [Q, -Q] with Q orthogonal, W_dec = W_enc^T, zero biases: the positive parts of +-Q^T x are at most d
    # non-zeros, and decoding all of them gives x back (x = Q Q^T x).
    rng = np.random.default_rng(1)
    d = 16
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    W_enc = np.concatenate([Q, -Q], axis=1).astype(np.float32)               # [d, 2d]
    x = rng.standard_normal((9, d)).astype(np.float32)
    zero_e, zero_d = np.zeros(2 * d, np.float32), np.zeros(d, np.float32)
    ids, vals = O.encode_topk(x, W_enc, zero_e, zero_d, d)
    xh, err = O.decode(ids, vals, np.ascontiguousarray(W_enc.T), zero_d, x)
    np.testing.assert_allclose(xh, x, atol=2e-6)
    assert err.max() < 1e-10
    # keeping fewer features loses exactly the dropped coefficients' energy (orthonormal directions)
    ids4, vals4 = O.encode_topk(x, W_enc, zero_e, zero_d, 4)
    _, err4 = O.decode(ids4, vals4, np.ascontiguousarray(W_enc.T), zero_d, x)
    dropped = (vals.astype(np.float64) ** 2).sum(axis=1) - (vals4.astype(np.float64) ** 2).sum(axis=1)
    np.testing.assert_allclose(err4, dropped, rtol=1e-4, atol=1e-6)


def test_padding_only_rows_give_the_bias():
    W_dec = np.ones((4, 3), np.float32)
    b = np.array([1, 2, 3], np.float32)
    xh = O.decode(np.full((2, 3), -1, np.int32), np.zeros((2, 3), np.float32), W_dec, b)
    assert xh.tolist() == [[1, 2, 3], [1, 2, 3]]
