"""Pins for the oracle's two-source decode attention (Section 2.1 formula; Section 4.2 two-lane fetching
and the order-invariance of attention along the sequence axis)."""
import numpy as np
import pytest
import torch
from scipy.special import logsumexp

import oracle
from helpers import cu_of, rand_bf16, widen
from paper_2607_28150_b200.workloads import f32_to_bf16_bits


def make_case(seed, lens=(23, 9), Hq=4, Hkv=2, d=16, ks=(6, 9), nls=(5, 0)):
    rng = np.random.default_rng(seed)
    cu, ck, cl = cu_of(lens), cu_of(ks), cu_of(nls)
    T = int(cu[-1])
    k = rand_bf16(rng, (1, T, Hkv, d))
    v = rand_bf16(rng, (1, T, Hkv, d))
    q = rand_bf16(rng, (len(lens), Hq, d))
    sel = np.zeros((1, Hkv, int(ck[-1])), dtype=np.int32)
    loc = np.zeros((Hkv, int(cl[-1])), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            perm = rng.permutation(n).astype(np.int32)
            sel[0, g, ck[b]:ck[b + 1]] = np.sort(perm[: ks[b]])
            loc[g, cl[b]:cl[b + 1]] = perm[ks[b]: ks[b] + nls[b]]
    pk, pv = oracle.pack_kv(k, v, cu, sel, ck)
    return dict(q=q, k=k[0], v=v[0], pk=pk[0], pv=pv[0], sel=sel[0], loc=loc, cu=cu, ck=ck, cl=cl,
                lens=lens, Hq=Hq, Hkv=Hkv, d=d)


def run(c, **kw):
    return oracle.sparse_decode_attn(c["q"], c["pk"], c["pv"], c["ck"], c["k"], c["v"], c["cu"], c["loc"], c["cl"], **kw)


def dense_over_set(c, b, h):
    """Library softmax attention restricted to the union index list of (b, h)."""
    g = h // (c["Hq"] // c["Hkv"])
    idx = np.concatenate([c["sel"][g, c["ck"][b]:c["ck"][b + 1]], c["loc"][g, c["cl"][b]:c["cl"][b + 1]]])
    K = torch.from_numpy(widen(c["k"])[c["cu"][b] + idx, g])
    V = torch.from_numpy(widen(c["v"])[c["cu"][b] + idx, g])
    qv = torch.from_numpy(widen(c["q"])[b, h])
    s = K @ qv / np.sqrt(c["d"])
    return (torch.softmax(s, 0) @ V).numpy(), float(torch.logsumexp(s, 0))


@pytest.mark.parametrize("seed", range(3))
def test_decode_matches_dense_attention_on_the_index_set(seed):
    c = make_case(seed)
    out, lse = run(c)
    for b in range(len(c["lens"])):
        for h in range(c["Hq"]):
            o, l = dense_over_set(c, b, h)
            np.testing.assert_allclose(out[b, h], o, rtol=1e-5, atol=1e-6)
            assert abs(lse[b, h] - l) < 1e-5


@pytest.mark.parametrize("n_local_frac", [0.0, 0.3, 1.0])
def test_full_budget_equals_full_attention(n_local_frac):
    """Fallback to full transfer (Section 4.4): with every token required, the result is plain attention over
    the whole prompt, wherever the split between the packed source and the local source falls."""
    lens, Hq, Hkv, d = (31, 12), 6, 2, 32
    nls = tuple(int(round(n_local_frac * n)) for n in lens)
    ks = tuple(n - m for n, m in zip(lens, nls))
    c = make_case(7, lens, Hq, Hkv, d, ks, nls)
    out, _ = run(c)
    G = Hq // Hkv
    for b, n in enumerate(lens):
        K = torch.from_numpy(widen(c["k"])[c["cu"][b]:c["cu"][b + 1]]).permute(1, 0, 2)    # [Hkv][n][d]
        V = torch.from_numpy(widen(c["v"])[c["cu"][b]:c["cu"][b + 1]]).permute(1, 0, 2)
        Q = torch.from_numpy(widen(c["q"])[b]).reshape(Hkv, G, d)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V).reshape(Hq, d).numpy()
        np.testing.assert_allclose(out[b], ref, rtol=1e-5, atol=1e-6)


def test_order_invariance():
    """Permuting the packed rows of a head, or its local index list, leaves the output unchanged."""
    c = make_case(11)
    out0, lse0 = run(c)
    rng = np.random.default_rng(0)
    c2 = dict(c)
    pk, pv = c["pk"].copy(), c["pv"].copy()
    Hkv = c["Hkv"]
    for b in range(len(c["lens"])):
        kb = c["ck"][b + 1] - c["ck"][b]
        for g in range(Hkv):
            base = c["ck"][b] * Hkv + g * kb
            p = rng.permutation(kb)
            pk[base: base + kb] = c["pk"][base + p]
            pv[base: base + kb] = c["pv"][base + p]
    loc = c["loc"].copy()
    for g in range(Hkv):
        for b in range(len(c["lens"])):
            seg = slice(c["cl"][b], c["cl"][b + 1])
            loc[g, seg] = rng.permutation(loc[g, seg])
    c2.update(pk=pk, pv=pv, loc=loc)
    out1, lse1 = run(c2)
    np.testing.assert_allclose(out1, out0, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(lse1, lse0, atol=1e-5)


def test_split_invariance_between_sources():
    """Moving entries from the packed source to the local source does not change the result."""
    lens, Hq, Hkv, d = (40,), 4, 2, 16
    a = make_case(5, lens, Hq, Hkv, d, (20,), (0,))
    out_a, lse_a = run(a)
    # same 20 tokens per head: first 12 (ascending) stay packed, the other 8 become local indices
    sel = a["sel"]
    sel_b = sel[:, :12].copy()
    loc_b = sel[:, 12:].copy()
    ck, cl = cu_of((12,)), cu_of((8,))
    pk, pv = oracle.pack_kv(a["k"][None], a["v"][None], a["cu"], sel_b[None], ck)
    out_b, lse_b = oracle.sparse_decode_attn(a["q"], pk[0], pv[0], ck, a["k"], a["v"], a["cu"], loc_b, cl)
    np.testing.assert_allclose(out_b, out_a, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(lse_b, lse_a, atol=1e-5)


def test_lse_merge_identity():
    """Split-softmax combine: the results over two disjoint parts, merged with their log-sum-exps,
    reproduce the one-pass result (m = max m_j, l = sum l_j e^{m_j - m})."""
    c = make_case(21, (30,), 4, 2, 16, (10,), (7,))
    out, lse = run(c)
    # part 1: packed only; part 2: local only
    z = cu_of((0,))
    o1, l1 = oracle.sparse_decode_attn(c["q"], c["pk"], c["pv"], c["ck"], c["k"], c["v"], c["cu"],
                                       np.zeros((2, 0), np.int32), z)
    o2, l2 = oracle.sparse_decode_attn(c["q"], np.zeros((0, 16), np.uint16), np.zeros((0, 16), np.uint16), z,
                                       c["k"], c["v"], c["cu"], c["loc"], c["cl"])
    m = np.maximum(l1, l2)
    w1, w2 = np.exp(l1 - m), np.exp(l2 - m)
    merged = (o1 * w1[..., None] + o2 * w2[..., None]) / (w1 + w2)[..., None]
    np.testing.assert_allclose(merged, out, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(m + np.log(w1 + w2), lse, atol=1e-5)


def test_single_token_returns_its_value_and_identical_keys_average_values():
    rng = np.random.default_rng(2)
    N, Hq, Hkv, d = 10, 2, 1, 8
    k = rand_bf16(rng, (N, Hkv, d))
    v = rand_bf16(rng, (N, Hkv, d))
    q = rand_bf16(rng, (1, Hq, d))
    cu, z = cu_of((N,)), cu_of((0,))
    loc = np.array([[4]], dtype=np.int32)
    out, lse = oracle.sparse_decode_attn(q, np.zeros((0, d), np.uint16), np.zeros((0, d), np.uint16), z,
                                         k, v, cu, loc, cu_of((1,)))
    np.testing.assert_allclose(out[0, 0], widen(v)[4, 0], rtol=1e-6)
    np.testing.assert_allclose(lse[0], widen(k)[4, 0] @ widen(q)[0].T / np.sqrt(d), rtol=1e-5, atol=1e-6)
    k2 = np.repeat(k[:1], N, axis=0)
    loc = np.arange(N, dtype=np.int32)[None]
    out, _ = oracle.sparse_decode_attn(q, np.zeros((0, d), np.uint16), np.zeros((0, d), np.uint16), z,
                                       k2, v, cu, loc, cu_of((N,)))
    np.testing.assert_allclose(out[0, 1], widen(v)[:, 0].mean(0), rtol=1e-5, atol=1e-6)


def test_lse_is_logsumexp_of_scaled_scores_and_scale_override():
    c = make_case(33, (16,), 2, 1, 8, (16,), (0,))
    for scale in (0.0, 0.37):
        _, lse = run(c, softmax_scale=scale)
        sc = scale if scale > 0 else 1 / np.sqrt(8)
        for h in range(2):
            s = widen(c["k"])[:, 0] @ widen(c["q"])[0, h] * sc
            assert abs(lse[0, h] - logsumexp(s)) < 1e-5


def test_empty_sources_give_zero_and_minus_inf():
    c = make_case(1, (5, 7), 2, 1, 8, (0, 3), (0, 2))
    out, lse = run(c)
    assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0]))
    assert np.all(np.isfinite(lse[1]))


def test_duplicates_count_twice():
    """Multiset semantics: a token present in both sources is weighted twice."""
    rng = np.random.default_rng(9)
    d = 8
    k = rand_bf16(rng, (2, 1, d))
    v = rand_bf16(rng, (2, 1, d))
    q = rand_bf16(rng, (1, 1, d))
    cu = cu_of((2,))
    sel = np.array([[[0, 1]]], dtype=np.int32)
    pk, pv = oracle.pack_kv(k[None], v[None], cu, sel, cu_of((2,)))
    loc = np.array([[1]], dtype=np.int32)
    out, _ = oracle.sparse_decode_attn(q, pk[0], pv[0], cu_of((2,)), k, v, cu, loc, cu_of((1,)))
    s = widen(k)[:, 0] @ widen(q)[0, 0] / np.sqrt(d)
    w = np.exp(s) * np.array([1.0, 2.0])
    np.testing.assert_allclose(out[0, 0], (w[:, None] * widen(v)[:, 0]).sum(0) / w.sum(), rtol=1e-5, atol=1e-6)
