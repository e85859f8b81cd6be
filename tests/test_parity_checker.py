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
