"""The comparison rules of tests/parity.py, tried on the oracle's own output with planted mistakes (CPU only)."""
import numpy as np
import pytest

import oracle as O
from parity import assert_tight, check_topk_against_preact


def _case(seed=0, T=40, D=512, k=16):
    pre = np.random.default_rng(seed).standard_normal((T, D))
    ids, vals = O.topk(pre, k)
    return pre, ids, vals, k


def test_oracle_output_passes_and_is_tight():
    pre, ids, vals, k = _case()
    st = {}
    banded = check_topk_against_preact(pre, ids, vals, k, 2e-2, st)
    assert st["rows"] == 40 and st["banded"] == banded and st["exact"] == 40
    assert_tight(st)


def test_a_banded_row_that_returns_too_few_ids_fails():
    pre, ids, vals, k = _case()
    ids[:, -1] = -1
    vals[:, -1] = 0
    with pytest.raises(AssertionError, match="ids reported"):
        check_topk_against_preact(pre, ids, vals, k, 2e-2)


def test_a_far_weaker_feature_in_place_of_the_kth_fails():
    pre, ids, vals, k = _case()
    weak = int(np.argsort(-pre[0])[60])
    ids[0, -1], vals[0, -1] = weak, pre[0, weak]
    with pytest.raises(AssertionError):
        check_topk_against_preact(pre, ids, vals, k, 2e-2)


def test_a_swap_inside_the_band_passes_but_is_not_exact():
    pre, ids, vals, k = _case()
    z = pre[0]
    order = np.argsort(-z)
    z[order[k]] = z[order[k - 1]] - 1e-4            # the (k+1)-th value sits just under the k-th
    ids[0, -1], vals[0, -1] = order[k], z[order[k]]
    st = {}
    check_topk_against_preact(pre, ids, vals, k, 2e-2, st)
    assert st["exact"] == st["rows"] - 1
    with pytest.raises(AssertionError):
        assert_tight(st, min_exact=1.0)


def test_value_error_beyond_fp32_accumulation_fails_the_tight_bound():
    pre, ids, vals, k = _case()
    vals = vals * (1 + 1e-3)
    st = {}
    check_topk_against_preact(pre, ids, vals.astype(np.float32), k, 2e-2, st)
    with pytest.raises(AssertionError, match="relative value error"):
        assert_tight(st)


# ---- the density checker: what it lets through as the known case and what it does not
def _density_case():
    import oracle as O
    rng = np.random.default_rng(5)
    L, k, D, Q, nq, kq, K, R, N = 700, 4, 48, 2, 3, 4, 9, 5, 6
    ctx = np.argsort(rng.random((2, L, D)), axis=2)[:, :, :k].astype(np.int32)
    q = np.argsort(rng.random((2, Q * nq, D)), axis=2)[:, :, :kq].astype(np.int32).reshape(2, Q, nq, kq)
    qv = (rng.random(q.shape) * 3).astype(np.float32)
    out = O.position_density(ctx, q, qv, D, K, R, N, 0)
    return ctx, q, D, K, R, N, out


def _shifted(ctx, out, K, R, N, qi, layer, f, units):
    from parity import UNIT, _box_density, _nms_centres
    oS, oD, oc, odens = out
    gS, gD, gc, gdens = oS.astype(np.float32), oD.astype(np.float32), oc.copy(), odens.copy()
    s_fix = np.rint(oS[qi] * UNIT).astype(np.int64) + units * (ctx[layer] == f).sum(axis=1)
    d_fix = _box_density(s_fix, K)
    gS[qi], gD[qi] = (s_fix / UNIT).astype(np.float32), (d_fix / UNIT).astype(np.float32)
    gc[qi], gdens[qi] = _nms_centres(d_fix, R, N)
    return gS, gD, gc, gdens


def test_density_checker_rederives_the_oracles_density_and_peaks():
    from parity import check_density
    ctx, q, D, K, R, N, out = _density_case()
    same = _shifted(ctx, out, K, R, N, 0, 0, int(q[0, 0, 0, 0]), 0)          # no shift: the numpy re-derivation itself
    assert check_density(ctx, q, D, K, R, N, 0, out, same) is None


def test_density_checker_names_a_single_unit_weight_shift():
    from parity import check_density
    ctx, q, D, K, R, N, out = _density_case()
    f = int(q[1, 1, 2, 1])
    note = check_density(ctx, q, D, K, R, N, 0, out, _shifted(ctx, out, K, R, N, 1, 1, f, -1))
    assert note is not None and f"query 1 layer 1 feature {f}: -1 unit" in note


def test_density_checker_rejects_everything_else():
    from parity import check_density
    ctx, q, D, K, R, N, out = _density_case()
    f = int(q[0, 0, 0, 0])
    with pytest.raises(AssertionError):                                       # two units is not the rounding case
        check_density(ctx, q, D, K, R, N, 0, out, _shifted(ctx, out, K, R, N, 0, 0, f, 2))
    notq = next(x for x in range(D) if x not in set(q[0, 0].ravel().tolist()))
    with pytest.raises(AssertionError):                                       # a feature the query does not hold
        check_density(ctx, q, D, K, R, N, 0, out, _shifted(ctx, out, K, R, N, 0, 0, notq, 1))
    gS, gD, gc, gdens = _shifted(ctx, out, K, R, N, 0, 0, f, 0)
    gS[0, 17] += np.float32(1.0 / 65536)                                      # one position alone
    with pytest.raises(AssertionError):
        check_density(ctx, q, D, K, R, N, 0, out, (gS, gD, gc, gdens))
    gS, gD, gc, gdens = _shifted(ctx, out, K, R, N, 0, 0, f, 1)
    gc[0, 0] += 1                                                             # right shift, wrong peak
    with pytest.raises(AssertionError):
        check_density(ctx, q, D, K, R, N, 0, out, (gS, gD, gc, gdens))
