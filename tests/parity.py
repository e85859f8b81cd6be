"""Comparison rules shared by the GPU parity tests (numpy only; no method arithmetic beyond sorting)."""
import numpy as np


def check_topk_against_preact(pre, ids, vals, k, tol, stats=None):
    """pre: oracle fp64 pre-activations [T, D]; ids/vals: the implementation's [T, k] output.

    Values: |val - pre| / (|pre| + 1) <= tol for every reported id.
    Sets: with thr the oracle's k-th largest positive value (0 if fewer than k are positive) and
    band = tol * (|thr| + 1): every feature above thr + band must be reported, nothing at or below
    thr - band (or <= -band) may be, and when no other feature lies inside the band the reported
    set equals the oracle's exactly. In a row that needs the band the count is still fixed (k ids when k
    pre-activations are clearly positive, never more than the possibly positive ones) and no unreported
    feature may beat the weakest reported one by more than the two values' error bounds.
    Rows are value-descending with distinct ids, padded -1 / 0.
    Returns the number of rows that needed the band; `stats` (a dict) accumulates rows, banded rows, rows whose
    id list equals the oracle's Top-k exactly, and the largest |val - pre| / (|pre| + 1) seen."""
    T, D = pre.shape
    banded = 0
    if stats is not None:
        for key in ("rows", "banded", "exact"):
            stats.setdefault(key, 0)
        stats.setdefault("max_rel_err", 0.0)
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
        exact = G.tolist() == oset.tolist()
        if not extra:
            assert Gs == set(oset.tolist()), f"row {t}: id set differs with no near-tie to excuse it"
            # equal values must come out in ascending id order
            assert exact or _only_value_ties_reordered(z, G, oset, tol)
        else:
            banded += 1
            lo = min(k, int((z > tol).sum()))
            hi = min(k, int((z > -tol).sum()))
            assert lo <= n <= hi, f"row {t}: {n} ids reported, between {lo} and {hi} expected"
            rest = np.ones(D, dtype=bool)
            rest[G] = False
            if rest.any():
                weakest = z[G].min() if n == k else 0.0
                slack = tol * (abs(weakest) + 1.0) + tol * (np.abs(z[rest]).max(initial=0.0) + 1.0) if n < k else 2.0 * band
                assert z[rest].max() <= weakest + slack, f"row {t}: an unreported feature beats the weakest reported one"
        if stats is not None:
            stats["rows"] += 1
            stats["banded"] += 1 if extra else 0
            stats["exact"] += 1 if exact else 0
            stats["max_rel_err"] = max(stats["max_rel_err"], float(err.max(initial=0.0)))
    return banded


def assert_tight(stats, min_exact=0.98, max_rel_err=2e-4):
    """The statistic that is much tighter than the acceptance band: nearly every row's id list is the oracle's
    Top-k in the oracle's order, and the values agree to fp32-accumulation accuracy."""
    assert stats["rows"] > 0
    assert stats["exact"] >= min_exact * stats["rows"], f"only {stats['exact']} of {stats['rows']} rows equal the oracle's Top-k"
    assert stats["max_rel_err"] <= max_rel_err, f"largest relative value error {stats['max_rel_err']}"


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


# --------------------------------------------------------------------------------------------- density, known case
# The per-position relevance takes every weight in 2^-24 fixed point, w = rint(aQ * IDF * 2^24) / 2^24, on both sides.
# The one way two correct implementations can differ: a product aQ * IDF that lies within one ulp of a rounding
# half-way point, where the two sides' `log` (last place) decide the unit differently. Such a feature's weight is one
# unit apart, every position that holds it moves by one unit, and nothing else changes. The helpers below recognise
# exactly that and re-derive density and peaks from the shifted integers; any other difference stays a failure.
UNIT = 16777216.0   # 2^24


def _box_density(s_fix, K):
    L = len(s_fix)
    c = np.concatenate([[0], np.cumsum(s_fix.astype(np.int64))])
    t = np.arange(L)
    lo = np.clip(t - K // 2, 0, L)
    hi = np.clip(t - K // 2 + K, 0, L)
    return c[hi] - c[lo]


def _nms_centres(d_fix, R, N):
    alive = np.ones(len(d_fix), bool)
    centres, dens = np.full(N, -1, np.int32), np.zeros(N, np.float32)
    for i in range(N):
        cand = np.where(alive & (d_fix > 0), d_fix, -1)
        if len(cand) == 0 or cand.max() < 0:
            break
        best = int(np.argmax(cand))                  # first of equals = lowest position
        centres[i], dens[i] = best, np.float32(d_fix[best] / UNIT)
        alive[max(0, best - R):best + R + 1] = False
    return centres, dens


def density_weight_shifts(ctx, q_ids, d_sae, stop_freq, oS_q, gS_q, qi, max_features=8):
    """For one query: the list of (layer, feature, +-1) weight shifts that turns the oracle's S into the GPU's, or
    None when no such list of at most `max_features` distinct features exists. [] when they are equal."""
    n_layers, L, _ = ctx.shape
    s_fix = np.rint(np.asarray(oS_q, np.float64) * UNIT).astype(np.int64)
    g32 = np.asarray(gS_q, np.float32)
    shifts = []
    for _ in range(max_features + 1):
        bad = np.nonzero((s_fix / UNIT).astype(np.float32) != g32)[0]
        if len(bad) == 0:
            return shifts
        if len(shifts) == max_features:
            return None
        p = int(bad[0])
        sign = 1 if float(g32[p]) > s_fix[p] / UNIT else -1
        best = None
        for l in range(n_layers):
            qf = np.unique(q_ids[l, qi][q_ids[l, qi] >= 0])
            for f in np.intersect1d(qf, ctx[l, p][ctx[l, p] >= 0]).tolist():
                if any(l == sl and f == sf for sl, sf, _ in shifts):
                    continue
                cnt = (ctx[l] == f).sum(axis=1).astype(np.int64)
                if stop_freq > 0 and int(cnt.sum()) > stop_freq:
                    continue
                left = int(((((s_fix + sign * cnt) / UNIT).astype(np.float32)) != g32).sum())
                if best is None or left < best[0]:
                    best = (left, l, f, cnt)
        if best is None or best[0] >= len(bad):
            return None
        s_fix = s_fix + sign * best[3]
        shifts.append((best[1], best[2], sign))
    return None


def check_density(ctx, q_ids, d_sae, K, R, N, stop_freq, oracle_out, gpu_out):
    """Exact agreement returns None. A difference that is fully explained by weights one fixed-point unit apart
    (S, the density and the peaks all re-derived from the shifted integers) returns a text naming the features: the
    known case. Anything else raises."""
    oS, oD, oc, odens = oracle_out
    gS, gD, gc, gdens = gpu_out
    same = (np.array_equal(gS, oS.astype(np.float32)) and np.array_equal(gD, oD.astype(np.float32))
            and np.array_equal(gc, oc) and np.array_equal(gdens, odens))
    if same:
        return None
    notes = []
    for qi in range(oS.shape[0]):
        shifts = density_weight_shifts(ctx, q_ids, d_sae, stop_freq, oS[qi], gS[qi], qi)
        assert shifts is not None, f"query {qi}: S differs from the oracle by more than single-unit weight shifts"
        s_fix = np.rint(oS[qi] * UNIT).astype(np.int64)
        for l, f, sg in shifts:
            s_fix += sg * (ctx[l] == f).sum(axis=1)
        d_fix = _box_density(s_fix, K)
        np.testing.assert_array_equal(gD[qi], (d_fix / UNIT).astype(np.float32))
        c, dn = _nms_centres(d_fix, R, N)
        np.testing.assert_array_equal(gc[qi], c)
        np.testing.assert_array_equal(gdens[qi], dn)
        notes += [f"query {qi} layer {l} feature {f}: {sg:+d} unit" for l, f, sg in shifts]
    assert notes, "outputs differ although S agrees"
    return "weights one 2^-24 unit apart (rounding half-way case): " + "; ".join(notes)
