"""Pins for the oracle's per-head top-k (Section 2.3: a KV index row holds the top-k entries of a head)."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from helpers import cu_of


def exhaustive(x, k):
    """Independent restatement: rank by (value descending, +0 before -0, position ascending), keep k, emit ascending."""
    order = sorted(range(len(x)), key=lambda t: (-float(x[t]) if x[t] != 0 else 0.0, bool(np.signbit(x[t])), t))
    return sorted(order[:k])


def run(x_rows, lens, ks):
    """x_rows: [L][Hkv][T] float32."""
    cu, ck = cu_of(lens), cu_of(ks)
    return oracle.select_topk(np.asarray(x_rows, dtype=np.float32), cu, ck), cu, ck


@pytest.mark.parametrize("seed", range(5))
def test_topk_matches_exhaustive_sort(seed):
    rng = np.random.default_rng(seed)
    lens, ks = (17, 1, 40, 8), (5, 1, 0, 8)
    L, Hkv = 2, 3
    x = rng.standard_normal((L, Hkv, sum(lens))).astype(np.float32)
    x[rng.random(x.shape) < 0.3] = 0.25            # many ties
    sel, cu, ck = run(x, lens, ks)
    for l in range(L):
        for g in range(Hkv):
            for b in range(len(lens)):
                got = sel[l, g, ck[b]:ck[b + 1]].tolist()
                assert got == exhaustive(x[l, g, cu[b]:cu[b + 1]], ks[b])


def test_topk_budget_count_unique_ascending_in_range():
    rng = np.random.default_rng(10)
    lens, ks = (100, 33), (10, 33)
    x = rng.random((1, 2, 133)).astype(np.float32)
    sel, cu, ck = run(x, lens, ks)
    for g in range(2):
        for b in range(2):
            row = sel[0, g, ck[b]:ck[b + 1]]
            assert len(row) == ks[b] and len(set(row.tolist())) == ks[b]
            assert np.all(np.diff(row) > 0) and row.min() >= 0 and row.max() < lens[b]
            seg = x[0, g, cu[b]:cu[b + 1]]
            rest = np.setdiff1d(np.arange(lens[b]), row)
            if len(rest):
                assert seg[row].min() >= seg[rest].max()


def test_topk_all_equal_takes_lowest_positions_and_full_budget_is_identity():
    x = np.full((1, 1, 50), 3.0, dtype=np.float32)
    sel, _, _ = run(x, (50,), (7,))
    assert sel[0, 0].tolist() == list(range(7))
    rng = np.random.default_rng(0)
    y = rng.standard_normal((1, 1, 50)).astype(np.float32)
    sel, _, _ = run(y, (50,), (50,))
    assert sel[0, 0].tolist() == list(range(50))


def test_topk_tie_at_threshold_prefers_lower_index():
    x = np.array([[[1, 5, 2, 5, 2, 2, 0, 2]]], dtype=np.float32)
    sel, _, _ = run(x, (8,), (4,))
    assert sel[0, 0].tolist() == [1, 2, 3, 4]        # both 5s, then the two lowest-index 2s


def test_topk_special_values():
    inf = np.inf
    den = np.float32(1e-42)                           # a subnormal
    x = np.array([[[0.0, -0.0, inf, -inf, den, -den, 1.0, -1.0]]], dtype=np.float32)
    # descending order: inf, 1, den, +0, -0, -den, -1, -inf
    want_order = [2, 6, 4, 0, 1, 5, 7, 3]
    for k in range(1, 9):
        sel, _, _ = run(x, (8,), (k,))
        assert sel[0, 0].tolist() == sorted(want_order[:k])


def test_topk_infinite_importance_is_always_kept():
    """Eq. 1 gives forced entries infinite importance; they must come before any finite value."""
    rng = np.random.default_rng(3)
    x = rng.random((1, 1, 64)).astype(np.float32) * 100
    forced = [5, 17, 40]
    x[0, 0, forced] = np.inf
    sel, _, _ = run(x, (64,), (3,))
    assert sel[0, 0].tolist() == forced


@settings(max_examples=60, deadline=None)
@given(st.lists(st.sampled_from([-2.0, -0.0, 0.0, 0.5, 0.5000001, 7.0]), min_size=1, max_size=40), st.data())
def test_topk_hypothesis_few_distinct_values(vals, data):
    k = data.draw(st.integers(min_value=0, max_value=len(vals)))
    x = np.asarray(vals, dtype=np.float32)
    sel, _, _ = run(x[None, None], (len(vals),), (k,))
    assert sel[0, 0].tolist() == exhaustive(x, k)


def test_topk_rejects_budget_above_length():
    with pytest.raises(RuntimeError):
        run(np.zeros((1, 1, 4), dtype=np.float32), (4,), (5,))


def _nan(sign, payload):
    """A float32 NaN with the given sign bit and mantissa payload (non-zero)."""
    return np.array([(sign << 31) | 0x7F800000 | payload], dtype=np.uint32).view(np.float32)[0]


def test_topk_nan_takes_the_place_of_its_bit_pattern():
    """The order of values is the total order of the fp32 bit patterns: a NaN with a clear sign bit ranks above
    +inf (larger payload first), one with a set sign bit below -inf.  Restated here with plain integers: the rank of a
    value is its sign-magnitude pattern read as a signed quantity."""
    vals = np.array([1.0, _nan(0, 1), np.inf, _nan(0, 0x400000), -np.inf, _nan(1, 1), 0.0, _nan(1, 0x400000), -2.0, 1.0],
                    dtype=np.float32)
    bits = vals.view(np.uint32).astype(np.int64)
    rank = np.where(bits >> 31 == 1, -(bits & 0x7FFFFFFF) - 1, bits & 0x7FFFFFFF)      # -0 just below +0
    order = sorted(range(len(vals)), key=lambda t: (-int(rank[t]), t))
    assert order[:3] == [3, 1, 2] and order[-2:] == [5, 7]                         # quiet NaN, NaN(1), +inf ... -NaNs last
    for k in range(len(vals) + 1):
        sel, _, _ = run(vals[None, None], (len(vals),), (k,))
        assert sel[0, 0].tolist() == sorted(order[:k])
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 2, 300)).astype(np.float32)
    xb = x.view(np.uint32)
    xb[0, :, ::7] = 0x7FC00000 | rng.integers(0, 1 << 22, size=xb[0, :, ::7].shape).astype(np.uint32)
    xb[0, :, 3::11] = 0xFFC00000 | rng.integers(0, 1 << 22, size=xb[0, :, 3::11].shape).astype(np.uint32)
    sel, cu, ck = run(x, (300,), (60,))
    for g in range(2):
        b_ = x[0, g].view(np.uint32).astype(np.int64)
        r_ = np.where(b_ >> 31 == 1, -(b_ & 0x7FFFFFFF) - 1, b_ & 0x7FFFFFFF)
        want = sorted(sorted(range(300), key=lambda t: (-int(r_[t]), t))[:60])
        assert sel[0, g].tolist() == want
