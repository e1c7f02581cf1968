"""Pins for the oracle's threshold (alpha) selection: brute force, hand example, limits of alpha, the cap, ties."""
import numpy as np
import pytest

import oracle
from helpers import cu_of


def brute(x, alpha, cap):
    """Independent statement of the rule with numpy on one row."""
    x = np.asarray(x, dtype=np.float32)
    thr = np.float32(x.max()) - np.float32(alpha)
    cand = [t for t in range(len(x)) if x[t] > thr]
    cand.sort(key=lambda t: (-float(x[t]), t))
    return sorted(cand[:cap])


def test_hand_example():
    """Scores 5, 1, 4.5, 3, 4.9, 0 with alpha = 1: the maximum is 5, the threshold 4, positions 0, 2, 4 exceed it.
    With a cap of two the two largest (5 and 4.9) stay; a score equal to the threshold is not selected."""
    x = np.array([[[5, 1, 4.5, 3, 4.9, 0]]], dtype=np.float32)
    cu = cu_of((6,))
    sel, cnt = oracle.select_threshold(x, cu, 1.0, cu_of((6,)))
    assert cnt[0, 0, 0] == 3 and sel[0, 0].tolist() == [0, 2, 4, -1, -1, -1]
    sel, cnt = oracle.select_threshold(x, cu, 1.0, cu_of((2,)))
    assert cnt[0, 0, 0] == 2 and sel[0, 0].tolist() == [0, 4]
    x[0, 0, 3] = 4.0                                             # exactly max - alpha: "exceeding" is strict
    sel, cnt = oracle.select_threshold(x, cu, 1.0, cu_of((6,)))
    assert cnt[0, 0, 0] == 3 and 3 not in sel[0, 0].tolist()


@pytest.mark.parametrize("seed", range(4))
def test_matches_brute_force_on_ragged_batches(seed):
    rng = np.random.default_rng(seed)
    lens = (37, 5, 64, 1)
    caps = (8, 5, 13, 1)
    L, Hkv = 2, 3
    cu, cc = cu_of(lens), cu_of(caps)
    x = rng.standard_normal((L, Hkv, int(cu[-1]))).astype(np.float32) * 2
    x[0, 0, 3] = x[0, 0, 7]                                      # a tie inside a row
    for alpha in (0.0, 0.5, 1.5, 100.0):
        sel, cnt = oracle.select_threshold(x, cu, alpha, cc)
        for l in range(L):
            for g in range(Hkv):
                for b, n in enumerate(lens):
                    want = brute(x[l, g, cu[b]:cu[b + 1]], alpha, caps[b])
                    row = sel[l, g, cc[b]:cc[b + 1]]
                    assert cnt[l, b, g] == len(want)
                    assert row[:len(want)].tolist() == want and np.all(row[len(want):] == -1)


def test_limits_of_alpha_and_relation_to_topk():
    rng = np.random.default_rng(9)
    lens, caps = (200, 50), (40, 10)
    cu, cc = cu_of(lens), cu_of(caps)
    x = rng.random((1, 2, 250)).astype(np.float32)
    sel0, cnt0 = oracle.select_threshold(x, cu, 0.0, cc)         # nothing exceeds the maximum itself
    assert np.all(cnt0 == 0) and np.all(sel0 == -1)
    selinf, cntinf = oracle.select_threshold(x, cu, 1e9, cc)     # everything exceeds: the cap binds -> plain top-k
    assert np.array_equal(selinf, oracle.select_topk(x, cu, cc))
    assert np.array_equal(cntinf[0], np.array([[40, 40], [10, 10]]))
    prev = None
    for alpha in (0.01, 0.05, 0.1, 0.3, 1.0):                    # the selection grows with alpha, nested
        sel, cnt = oracle.select_threshold(x, cu, alpha, cc)
        sets = [set(sel[0, g, cc[b]:cc[b] + cnt[0, b, g]].tolist()) for g in range(2) for b in range(2)]
        if prev is not None:
            assert all(p <= s for p, s in zip(prev, sets))
        prev = sets


def test_ties_at_the_cap_go_to_the_lower_index_and_nan_is_never_selected():
    x = np.array([[[2, 7, 7, 7, 1, 7, np.nan, 6.5]]], dtype=np.float32)
    cu = cu_of((8,))
    sel, cnt = oracle.select_threshold(x, cu, 1.0, cu_of((3,)))  # five scores exceed 6, the cap keeps three 7s
    assert cnt[0, 0, 0] == 3 and sel[0, 0].tolist() == [1, 2, 3]
    sel, cnt = oracle.select_threshold(x, cu, 1.0, cu_of((8,)))
    assert sel[0, 0, :cnt[0, 0, 0]].tolist() == [1, 2, 3, 5, 7]


def test_counted_pack_and_decode_equal_the_plain_path_on_the_trimmed_selection():
    """Ragged per-head counts: packing the first count entries of each row and attending only those packed rows is the
    same as the plain path run head by head with that head's own budget (the definition of the plain path)."""
    from helpers import rand_bf16
    rng = np.random.default_rng(5)
    lens, caps, Hq, Hkv, d = (60, 33), (12, 7), 4, 2, 16
    cu, cc = cu_of(lens), cu_of(caps)
    T = int(cu[-1])
    k, v = rand_bf16(rng, (1, T, Hkv, d)), rand_bf16(rng, (1, T, Hkv, d))
    q = rand_bf16(rng, (len(lens), Hq, d))
    x = rng.standard_normal((1, Hkv, T)).astype(np.float32)
    sel, cnt = oracle.select_threshold(x, cu, 0.8, cc)
    assert len(set(cnt.ravel().tolist())) > 1                      # counts really differ per head
    pk, pv = oracle.pack_kv(k, v, cu, sel, cc, sel_count=cnt, fill=0x7fc0)
    loc = np.zeros((Hkv, 0), dtype=np.int32)
    out, lse = oracle.sparse_decode_attn(q, pk[0], pv[0], cc, k[0], v[0], cu, loc, cu_of((0, 0)), packed_count=cnt[0])
    G = Hq // Hkv
    for g in range(Hkv):                                           # one KV head at a time, uniform budget = that head's count
        for b in range(len(lens)):
            n = int(cnt[0, b, g])
            rows = pk[0].reshape(-1, d)[cc[b] * Hkv + g * caps[b]: cc[b] * Hkv + g * caps[b] + n]
            want_rows = k[0, cu[b] + sel[0, g, cc[b]:cc[b] + n], g]
            assert np.array_equal(rows, want_rows)
            rest = pk[0].reshape(-1, d)[cc[b] * Hkv + g * caps[b] + n: cc[b] * Hkv + (g + 1) * caps[b]]
            assert np.all(rest == 0x7fc0)                          # rows beyond the count are not written
            if n == 0:
                assert np.all(out[b, g * G:(g + 1) * G] == 0) and np.all(np.isneginf(lse[b, g * G:(g + 1) * G]))
                continue
            # dense attention over exactly those tokens, in numpy
            from helpers import widen
            kk, vv = widen(k[0, cu[b] + sel[0, g, cc[b]:cc[b] + n], g]), widen(v[0, cu[b] + sel[0, g, cc[b]:cc[b] + n], g])
            for h in range(g * G, (g + 1) * G):
                s = kk @ widen(q[b, h]) / np.sqrt(d)
                p = np.exp(s - s.max()); p /= p.sum()
                assert np.allclose(out[b, h], p @ vv, atol=1e-6)
