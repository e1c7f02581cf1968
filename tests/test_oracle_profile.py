"""Pins for the oracle's profile-based proactive selection (Section 4.1: Eq. 1, Eq. 2, top-K_r blocks; Section 4.2 mask)."""
import numpy as np
import pytest

import oracle
from helpers import cu_of


def test_accumulate_counts_each_selection_once():
    cu, ck = cu_of((5, 3)), cu_of((2, 3))
    idx = np.array([[0, 4, 0, 1, 2], [1, 2, 0, 1, 2]], dtype=np.int32)
    c = np.zeros((2, 8), dtype=np.int32)
    oracle.profile_accumulate(c, idx, cu, ck)
    oracle.profile_accumulate(c, idx, cu, ck)
    want = np.zeros((2, 8), dtype=np.int32)
    want[0, [0, 4]] = 2; want[0, [5, 6, 7]] = 2
    want[1, [1, 2]] = 2; want[1, [5, 6, 7]] = 2
    assert np.array_equal(c, want)
    assert c.sum() == 2 * idx.size


def test_eq1_hand_example():
    """L = 3, one sequence of 6 tokens, 2 heads, M = 3 blocks of 2 tokens: layer 2's means by hand."""
    counts = np.zeros((3, 2, 6), dtype=np.int32)
    counts[2, 0] = [1, 2, 3, 4, 5, 6]
    counts[2, 1] = [0, 0, 1, 1, 10, 0]
    I = oracle.block_importance(counts, cu_of((6,)), 3)
    assert np.all(np.isposinf(I[:2]))                       # layers 0 and 1 are always selected
    np.testing.assert_allclose(I[2], [(1 + 2 + 0 + 0) / 4, (3 + 4 + 1 + 1) / 4, (5 + 6 + 10 + 0) / 4])


def test_eq1_mean_over_ragged_sequences_and_mass_invariant():
    rng = np.random.default_rng(0)
    lens, L, Hkv, M = (37, 10, 64), 4, 3, 8
    cu = cu_of(lens)
    counts = rng.integers(0, 50, size=(L, Hkv, int(cu[-1])), dtype=np.int32)
    I = oracle.block_importance(counts, cu, M).astype(np.float64)
    # independent restatement with numpy: block of token t is floor(t*M/N)
    blk = np.concatenate([np.arange(n) * M // n for n in lens])
    for l in range(2, L):
        for m in range(M):
            sel = counts[l][:, blk == m]
            assert abs(I[l, m] - sel.mean()) < 1e-5 * max(1.0, sel.mean())
        entries = np.array([(blk == m).sum() * Hkv for m in range(M)])
        assert abs((I[l] * entries).sum() - counts[l].sum()) < 1e-3 * counts[l].sum()
    # uniform counts -> every block has the same importance
    I = oracle.block_importance(np.full((3, Hkv, int(cu[-1])), 7, dtype=np.int32), cu, M)
    assert np.all(I[2] == 7.0)


def test_eq2_budget_and_clip():
    L, M = 32, 1024
    assert oracle.transfer_budget(L, M, 0.5, 1.0) == 1024 * 31 // 2          # M (L-1) T_p / T_t
    assert oracle.transfer_budget(L, M, 1.0, 6.5) == int(1024 * 31 / 6.5)    # transfer 6.5x the prefill time
    assert oracle.transfer_budget(L, M, 1e-6, 1.0) == 2 * M                  # clipped from below: two layers always go
    assert oracle.transfer_budget(L, M, 10.0, 1.0) == L * M                  # low network load: full transfer
    assert oracle.transfer_budget(L, M, 1.0, 1.0) == M * (L - 1)             # equal times: all but one layer's worth


def test_top_kr_always_contains_the_first_two_layers_and_full_budget_is_everything():
    rng = np.random.default_rng(1)
    L, M, Hkv = 6, 16, 2
    cu = cu_of((200,))
    counts = rng.integers(0, 9, size=(L, Hkv, 200), dtype=np.int32)
    I = oracle.block_importance(counts, cu, M)
    for tp in (1e-3, 0.3, 100.0):
        kr = oracle.transfer_budget(L, M, tp, 1.0)
        sel = oracle.select_topk(I.reshape(1, 1, L * M), cu_of((L * M,)), cu_of((kr,)))[0, 0]
        assert set(range(2 * M)) <= set(sel.tolist()) and len(sel) == kr
        if kr == L * M:
            assert sel.tolist() == list(range(L * M))
        rest = np.setdiff1d(np.arange(2 * M, L * M), sel)
        chosen = np.setdiff1d(sel, np.arange(2 * M))
        if len(rest) and len(chosen):
            assert I.ravel()[chosen].min() >= I.ravel()[rest].max()


def test_proactive_mask_marks_exactly_the_selected_blocks():
    lens, M, L = (50, 9), 8, 4
    cu = cu_of(lens)
    selected = np.array(sorted([2 * M + 1, 2 * M + 7, 3 * M + 0, 0, 5]), dtype=np.int32)
    blk = np.concatenate([np.arange(n) * M // n for n in lens])
    for layer in range(L):
        mask = oracle.proactive_mask(cu, M, layer, selected)
        want = np.where(np.isin(layer * M + blk, selected), 1, 2).astype(np.int8)
        assert np.array_equal(mask, want)
    assert set(np.unique(oracle.proactive_mask(cu, M, 1, selected)).tolist()) == {2}      # no block of layer 1 selected here
    full = np.arange(L * M, dtype=np.int32)
    assert np.all(oracle.proactive_mask(cu, M, 3, full) == 1)                             # full transfer: everything local


def test_speculative_schedule_matches_printed_iteration_counts():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "speculative_iterations.txt")
    L, M = 40, 1000
    kr = oracle.transfer_budget(L, M, 1e-9, 1.0)            # minimal proactive transfer: 2M blocks
    assert kr == 2 * M
    for line in open(path):
        if not line.strip() or line.startswith("#"):
            continue
        ratio, iters, tol = line.split()
        it = 0
        while oracle.speculative_delivered(L, M, kr, float(ratio), it) < L * M:
            it += 1
        assert abs(it - int(iters)) <= int(tol)
    # monotone, starts at K_r, saturates at L*M, at least one block per iteration
    seq = [oracle.speculative_delivered(L, M, kr, 0.1, i) for i in range(12)]
    assert seq[0] == kr and seq[-1] == L * M and all(b >= a for a, b in zip(seq, seq[1:]))
    assert oracle.speculative_delivered(4, 2, 4, 1e-6, 3) == 7


def _caches(seed, lens, Hkv, d):
    rng = np.random.default_rng(seed)
    T = int(sum(lens))
    mk = lambda: rng.integers(0, 1 << 16, size=(T, Hkv, d), dtype=np.uint16)
    return mk(), mk(), mk(), mk()


def test_push_blocks_hand_example():
    """Section 4.1, online transfer: 10 tokens in M = 4 blocks are {0,1,2} {3,4} {5,6,7} {8,9} (token t is in block
    floor(t M / N)); pushing blocks 1 and 3 of layer 2 moves rows 3, 4, 8, 9 and nothing else."""
    sk, sv, dk, dv = _caches(0, (10,), 2, 8)
    M, layer = 4, 2
    gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu_of((10,)), M, layer, np.array([0, 5, layer * M + 1, layer * M + 3, 13], dtype=np.int32))
    moved = np.array([3, 4, 8, 9])
    kept = np.array([0, 1, 2, 5, 6, 7])
    assert np.array_equal(gk[moved], sk[moved]) and np.array_equal(gv[moved], sv[moved])
    assert np.array_equal(gk[kept], dk[kept]) and np.array_equal(gv[kept], dv[kept])


def test_push_blocks_agrees_with_the_kv_mask_and_covers_all_heads():
    """The pushed rows are exactly the rows the proactive KV mask marks local (1); rows marked remote (2) keep the
    destination's old bytes; K and V, every head, every element of a pushed row."""
    lens = (37, 5, 64, 1)
    cu = cu_of(lens)
    M, L = 8, 5
    rng = np.random.default_rng(3)
    selected = np.sort(rng.choice(L * M, size=17, replace=False)).astype(np.int32)
    sk, sv, dk, dv = _caches(1, lens, 3, 16)
    for layer in range(L):
        gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu, M, layer, selected)
        local = oracle.proactive_mask(cu, M, layer, selected) == 1
        blk = np.concatenate([np.arange(n) * M // n for n in lens])         # independent block geometry
        assert np.array_equal(local, np.isin(layer * M + blk, selected))
        assert np.array_equal(gk, np.where(local[:, None, None], sk, dk))
        assert np.array_equal(gv, np.where(local[:, None, None], sv, dv))


def test_push_blocks_all_and_none():
    lens = (20, 33)
    cu = cu_of(lens)
    sk, sv, dk, dv = _caches(2, lens, 2, 8)
    M = 6
    gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu, M, 1, np.arange(M, 2 * M, dtype=np.int32))
    assert np.array_equal(gk, sk) and np.array_equal(gv, sv)
    gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu, M, 1, np.arange(0, M, dtype=np.int32))     # another layer's blocks
    assert np.array_equal(gk, dk) and np.array_equal(gv, dv)
    gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu, M, 0, np.zeros(0, dtype=np.int32))
    assert np.array_equal(gk, dk) and np.array_equal(gv, dv)


def test_push_blocks_more_blocks_than_tokens():
    """M > N: most blocks are empty, every token is alone in its block floor(t M / N)."""
    sk, sv, dk, dv = _caches(4, (3,), 1, 8)
    gk, gv = oracle.push_blocks(sk, sv, dk, dv, cu_of((3,)), 8, 0, np.array([2, 3], dtype=np.int32))   # token 1 -> block 2
    assert np.array_equal(gk[1], sk[1]) and np.array_equal(gk[[0, 2]], dk[[0, 2]])
    assert np.array_equal(gv[1], sv[1]) and np.array_equal(gv[[0, 2]], dv[[0, 2]])


def test_push_blocks_updates_the_kv_mask_of_the_pushed_tokens_only():
    """Section 4.2: pushing a block also sets the decode-side KV mask of its tokens to 1; a mask that starts all-remote (2,
    with 0 for padding) and receives the pushes of the selected blocks ends up as the proactive mask, padding untouched."""
    lens, M, L = (50, 9), 8, 4
    cu = cu_of(lens)
    T = int(cu[-1])
    sk, sv, dk, dv = _caches(5, lens, 2, 8)
    selected = np.array(sorted([2 * M + 1, 2 * M + 7, 3 * M + 0, 0, 5]), dtype=np.int32)
    for layer in range(L):
        start = np.full(T, 2, dtype=np.int8)
        start[[3, 55]] = 0                                       # padding entries
        _, _, km = oracle.push_blocks(sk, sv, dk, dv, cu, M, layer, selected, kv_mask=start)
        want = oracle.proactive_mask(cu, M, layer, selected)
        pushed = want == 1
        assert np.array_equal(km[pushed], np.ones(pushed.sum(), dtype=np.int8))
        assert np.array_equal(km[~pushed], start[~pushed])
    # speculative transfer: pushing the remaining blocks later turns the rest local, nothing is ever set back
    first = oracle.push_blocks(sk, sv, dk, dv, cu, M, 2, selected, kv_mask=np.full(T, 2, dtype=np.int8))[2]
    rest = np.setdiff1d(np.arange(L * M, dtype=np.int32), selected)
    second = oracle.push_blocks(sk, sv, dk, dv, cu, M, 2, rest, kv_mask=first)[2]
    assert np.all(second == 1)
