"""Pins for the oracle's importance score (Section 2.1 attention formula; Section 4.1 importance).

Each test compares `oracle.score` with something fixed independently of it: a library softmax over
a library matmul, a closed form, or an invariant of the definition.
"""
import numpy as np
import pytest
from scipy.special import softmax

import oracle
from helpers import cu_of, rand_bf16, widen


def brute_importance(q_win, k, cu):
    """Textbook form: per query row, softmax(q K^T / sqrt(d)) over the causally visible keys; sum rows."""
    L, B, W, Hq, d = q_win.shape
    _, T, Hkv, _ = k.shape
    G = Hq // Hkv
    qf, kf = widen(q_win), widen(k)
    imp = np.zeros((L, Hkv, T))
    for l in range(L):
        for b in range(B):
            n = cu[b + 1] - cu[b]
            weff = min(W, n)
            for h in range(Hq):
                g = h // G
                keys = kf[l, cu[b]:cu[b + 1], g]                    # [n][d]
                for i in range(weff):
                    pos = n - weff + i
                    s = keys[: pos + 1] @ qf[l, b, i, h] / np.sqrt(d)
                    imp[l, g, cu[b]: cu[b] + pos + 1] += softmax(s)
    return imp


@pytest.mark.parametrize("lens,W,Hq,Hkv,d", [((37,), 5, 4, 2, 16), ((9, 1, 20), 4, 6, 2, 8),
                                             ((3, 12), 8, 2, 2, 32), ((50,), 1, 1, 1, 64)])
def test_score_matches_library_softmax(lens, W, Hq, Hkv, d):
    rng = np.random.default_rng(1)
    cu = cu_of(lens)
    L, B, T = 2, len(lens), int(cu[-1])
    q = rand_bf16(rng, (L, B, W, Hq, d))
    k = rand_bf16(rng, (L, T, Hkv, d))
    got = oracle.score(q, k, cu)
    want = brute_importance(q, k, cu)
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-12)


def test_score_mass_is_rows():
    """Every softmax row sums to one, so the importance of a (layer, sequence, KV head) sums to G*W_eff."""
    rng = np.random.default_rng(2)
    lens = (40, 3, 17)
    cu = cu_of(lens)
    W, Hq, Hkv, d = 6, 8, 2, 16
    q = rand_bf16(rng, (1, 3, W, Hq, d), 2.0)
    k = rand_bf16(rng, (1, int(cu[-1]), Hkv, d), 2.0)
    imp = oracle.score(q, k, cu).astype(np.float64)
    for b, n in enumerate(lens):
        for g in range(Hkv):
            assert abs(imp[0, g, cu[b]:cu[b + 1]].sum() - (Hq // Hkv) * min(W, n)) < 1e-5
    assert (imp >= 0).all()


def test_score_identical_keys_closed_form():
    """All keys equal: each query spreads 1/(pos+1) on keys 0..pos, so importance[t] = G * sum_{pos_i >= t} 1/(pos_i+1)."""
    rng = np.random.default_rng(3)
    N, W, Hq, Hkv, d = 29, 7, 6, 3, 8
    G = Hq // Hkv
    krow = rand_bf16(rng, (1, 1, Hkv, d))
    k = np.repeat(krow, N, axis=1)
    q = rand_bf16(rng, (1, 1, W, Hq, d))
    imp = oracle.score(q, k, cu_of((N,)))
    pos = np.arange(N - W, N)
    want = np.array([G * np.sum(1.0 / (pos[pos >= t] + 1)) for t in range(N)])
    for g in range(Hkv):
        np.testing.assert_allclose(imp[0, g], want, rtol=1e-6)


def test_score_dominant_key_takes_all_mass():
    rng = np.random.default_rng(4)
    N, W, Hq, Hkv, d = 64, 4, 4, 2, 16
    q = np.abs(widen(rand_bf16(rng, (1, 1, W, Hq, d)))) + 0.5     # all-positive queries
    from paper_2607_28150_b200.workloads import f32_to_bf16_bits
    qb = f32_to_bf16_bits(q.astype(np.float32))
    k = rand_bf16(rng, (1, N, Hkv, d), 0.1)
    k[0, 10] = f32_to_bf16_bits(np.full((Hkv, d), 30.0, dtype=np.float32))   # aligned with every query
    imp = oracle.score(qb, k, cu_of((N,)))
    R = (Hq // Hkv) * W
    assert np.all(np.abs(imp[0, :, 10] - R) < 1e-3)
    assert np.all(np.delete(imp[0], 10, axis=1) < 1e-3)


def test_score_permutation_equivariance_outside_window():
    """Keys at positions before the window are all visible to all window queries: permuting them permutes importance."""
    rng = np.random.default_rng(5)
    N, W, Hq, Hkv, d = 48, 8, 4, 2, 16
    q = rand_bf16(rng, (1, 1, W, Hq, d))
    k = rand_bf16(rng, (1, N, Hkv, d))
    perm = np.concatenate([rng.permutation(N - W), np.arange(N - W, N)])
    a = oracle.score(q, k, cu_of((N,)))
    b = oracle.score(q, k[:, perm], cu_of((N,)))
    np.testing.assert_allclose(b, a[:, :, perm], rtol=1e-6, atol=1e-12)


def test_score_window_longer_than_prompt():
    """W > N: only the first N window rows are used, at positions 0..N-1 (query i sees keys 0..i)."""
    rng = np.random.default_rng(6)
    N, W, d = 3, 8, 8
    q = rand_bf16(rng, (1, 1, W, 1, d))
    k = rand_bf16(rng, (1, N, 1, d))
    imp = oracle.score(q, k, cu_of((N,)))[0, 0]
    qf, kf = widen(q)[0, 0, :, 0], widen(k)[0, :, 0]
    want = np.zeros(N)
    for i in range(N):
        want[: i + 1] += softmax(kf[: i + 1] @ qf[i] / np.sqrt(d))
    np.testing.assert_allclose(imp, want, rtol=1e-6)
    assert abs(imp.sum() - N) < 1e-5


def test_score_scale_is_inverse_sqrt_d():
    """A wrong scale (1/d, none) changes a two-key softmax whose value is known in closed form."""
    from paper_2607_28150_b200.workloads import f32_to_bf16_bits
    d = 16
    q = f32_to_bf16_bits(np.full((1, 1, 1, 1, d), 1.0, dtype=np.float32))
    k = np.zeros((1, 2, 1, d), dtype=np.float32)
    k[0, 1] = 0.5                                   # s0 = 0, s1 = 16*0.5/4 = 2
    imp = oracle.score(q, f32_to_bf16_bits(k), cu_of((2,)))[0, 0]
    np.testing.assert_allclose(imp, [1 / (1 + np.exp(2.0)), 1 / (1 + np.exp(-2.0))], rtol=1e-6)
