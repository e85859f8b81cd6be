"""Comparison rules shared by the GPU parity tests (numpy only; no method arithmetic beyond sorting)."""
import numpy as np


def check_topk_against_preact(pre, ids, vals, k, tol):
    """pre: oracle fp64 pre-activations [T, D]; ids/vals: the implementation's [T, k] output.

    Values: |val - pre| / (|pre| + 1) <= tol for every reported id.
    Sets: with thr the oracle's k-th largest positive value (0 if fewer than k are positive) and
    band = tol * (|thr| + 1): every feature above thr + band must be reported, nothing at or below
    thr - band (or <= -band) may be, and when no other feature lies inside the band the reported
    set equals the oracle's exactly. Rows are value-descending with distinct ids, padded -1 / 0.
    Returns the number of rows that needed the band."""
    T, D = pre.shape
    banded = 0
    for t in range(T):
        z = pre[t]
        g = ids[t]
        n = int((g >= 0).sum())
        assert (g[:n] >= 0).all() and (g[n:] == -1).all(), f"row {t}: padding must trail"
        assert (vals[t, n:] == 0).all()
        G = g[:n]
        assert len(set(G.tolist())) == n, f"row {t}: duplicate ids"
        assert (G < D).all()
        v = vals[t, :n].astype(np.float64)
        assert (np.diff(v) <= 0).all(), f"row {t}: values not descending"
        assert (v > 0).all()
        err = np.abs(v - z[G]) / (np.abs(z[G]) + 1.0)
        assert err.max(initial=0.0) <= tol, f"row {t}: value error {err.max()}"
        pos = np.flatnonzero(z > 0)
        order = pos[np.lexsort((pos, -z[pos]))]
        oset = order[:k]
        thr = z[order[k - 1]] if len(order) >= k else 0.0
        band = tol * (abs(thr) + 1.0)
        must = np.flatnonzero(z > thr + band)
        maybe = np.flatnonzero((np.abs(z - thr) <= band) & (z > -band))
        Gs = set(G.tolist())
        assert set(must.tolist()) <= Gs, f"row {t}: a feature clearly above the threshold is missing"
        assert Gs <= set(must.tolist()) | set(maybe.tolist()), f"row {t}: a feature clearly below the threshold was reported"
        extra = set(maybe.tolist()) - set(oset.tolist())
        if not extra:
            assert Gs == set(oset.tolist()), f"row {t}: id set differs with no near-tie to excuse it"
            # equal values must come out in ascending id order
            assert G.tolist() == oset.tolist() or _only_value_ties_reordered(z, G, oset, tol)
        else:
            banded += 1
            assert len(must) <= n <= k
    return banded


def _only_value_ties_reordered(z, G, oset, tol):
    # the two orders may differ only where the oracle values are within the tolerance of each other
    for a, b in zip(G.tolist(), oset.tolist()):
        if a != b and abs(z[a] - z[b]) > tol * (abs(z[b]) + 1.0):
            return False
    return True


def csr_equal(row_ptr_a, pos_a, row_ptr_b, pos_b):
    ra = np.asarray(row_ptr_a).astype(np.int64)
    rb = np.asarray(row_ptr_b).astype(np.int64)
    np.testing.assert_array_equal(ra, rb)
    n = int(ra[-1])
    np.testing.assert_array_equal(np.asarray(pos_a)[:n], np.asarray(pos_b)[:n])
