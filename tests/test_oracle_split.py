"""Pins for the oracle's Algorithm 1 (KV index splitting and reordering, Section 4.2)."""
import os

import numpy as np
import pytest

import oracle
from helpers import cu_of


def make(seed, lens=(30, 12), ks=(10, 12), Hkv=3, p=(0.1, 0.5, 0.4)):
    rng = np.random.default_rng(seed)
    cu, ck = cu_of(lens), cu_of(ks)
    mask = rng.choice(np.array([0, 1, 2], dtype=np.int8), size=int(cu[-1]), p=p)
    idx = np.zeros((Hkv, int(ck[-1])), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            idx[g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    return idx, mask, cu, ck


@pytest.mark.parametrize("seed", range(4))
def test_split_matches_numpy_indexing(seed):
    """Operators 1-5 written with numpy fancy indexing and a library stable sort."""
    idx, mask, cu, ck = make(seed)
    re, loc, rem, nl, nr = oracle.split_index(idx, mask, cu, ck, reorder=True)
    for g in range(idx.shape[0]):
        for b in range(len(cu) - 1):
            row = idx[g, ck[b]:ck[b + 1]]
            m = mask[cu[b] + row]                                   # (1)
            order = np.argsort(-m.astype(np.int32), kind="stable")  # (4)
            row2, m2 = row[order], m[order]                         # (5)
            assert re[g, ck[b]:ck[b + 1]].tolist() == row2.tolist()
            assert loc[g, ck[b]: ck[b] + nl[b, g]].tolist() == row2[m2 == 1].tolist()   # (2)
            assert rem[g, ck[b]: ck[b] + nr[b, g]].tolist() == row2[m2 == 2].tolist()   # (3)


def test_split_partition_and_remote_first():
    idx, mask, cu, ck = make(9, p=(0.0, 0.6, 0.4))
    re, loc, rem, nl, nr = oracle.split_index(idx, mask, cu, ck, reorder=True)
    for g in range(idx.shape[0]):
        for b in range(len(cu) - 1):
            row = set(idx[g, ck[b]:ck[b + 1]].tolist())
            l = loc[g, ck[b]: ck[b] + nl[b, g]].tolist()
            r = rem[g, ck[b]: ck[b] + nr[b, g]].tolist()
            assert set(l) | set(r) == row and not (set(l) & set(r))          # no padding here: a partition
            # descending mask order: the remote entries are the first n_remote entries of the reordered row
            assert re[g, ck[b]: ck[b] + nr[b, g]].tolist() == r
            assert re[g, ck[b] + nr[b, g]: ck[b + 1]].tolist() == l


def test_split_without_reordering_keeps_row_order_and_drops_padding():
    idx, mask, cu, ck = make(5)
    re, loc, rem, nl, nr = oracle.split_index(idx, mask, cu, ck, reorder=False)
    assert np.array_equal(re, idx)
    for g in range(idx.shape[0]):
        for b in range(len(cu) - 1):
            row = idx[g, ck[b]:ck[b + 1]]
            m = mask[cu[b] + row]
            assert nl[b, g] + nr[b, g] == int((m != 0).sum())
            assert loc[g, ck[b]: ck[b] + nl[b, g]].tolist() == row[m == 1].tolist()
            assert rem[g, ck[b]: ck[b] + nr[b, g]].tolist() == row[m == 2].tolist()


def test_kv_mask_of_the_printed_example_has_the_printed_footprint():
    """Section 4.2 prints the cost of the KV mask for 64K tokens on a 40-layer model: one int8 per token and layer,
    2.5 MB in all.  The masks the oracle builds (proactive transfer of the global top blocks, one mask per layer)
    must have exactly that footprint, hold only the classes 1 / 2, and be the structure Algorithm 1 indexes."""
    path = os.path.join(os.path.dirname(__file__), "golden", "kv_mask_footprint.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    tokens, layers, per_layer, total_mb = int(rows[0][0]), int(rows[0][1]), int(rows[0][2]), float(rows[0][3])
    cu = np.array([0, tokens], dtype=np.int32)
    M = 64
    selected = np.arange(0, layers * M, 3, dtype=np.int32)          # every third block, ascending flat ids
    masks = [oracle.proactive_mask(cu, M, l, selected) for l in range(layers)]
    assert all(m.dtype == np.int8 and m.shape == (tokens,) for m in masks)
    assert masks[0].nbytes == per_layer
    assert sum(m.nbytes for m in masks) / 2**20 == total_mb
    for l in (0, 1, layers - 1):
        blocks = (np.arange(tokens, dtype=np.int64) * M) // tokens
        want = np.where(np.isin(l * M + blocks, selected), 1, 2).astype(np.int8)
        assert np.array_equal(masks[l], want)
    # the same mask drives Algorithm 1 at that size: a row of indices splits into the two classes it marks
    idx = np.arange(0, tokens, 97, dtype=np.int32)[None, :]
    ck = np.array([0, idx.shape[1]], dtype=np.int32)
    _, loc, rem, nl, nr = oracle.split_index(idx, masks[2], cu, ck, reorder=False)
    assert nl[0, 0] + nr[0, 0] == idx.shape[1]
    assert loc[0, : nl[0, 0]].tolist() == idx[0][masks[2][idx[0]] == 1].tolist()
    assert rem[0, : nr[0, 0]].tolist() == idx[0][masks[2][idx[0]] == 2].tolist()


def test_two_lane_fetching_equals_attention_over_the_kv_index():
    """Section 4.2 end to end on the oracle: split and reorder the KV index by the KV mask (Algorithm 1), fetch the remote
    entries into a packed buffer, attend [packed remote rows] ++ [local rows by index]; the result is attention over the
    KV index set itself (order along the sequence axis does not matter)."""
    import oracle
    from helpers import cu_of, rand_bf16
    rng = np.random.default_rng(8)
    lens, ks, Hq, Hkv, d = (70, 41), (20, 9), 4, 2, 16
    cu, ck = cu_of(lens), cu_of(ks)
    T, Kt = int(cu[-1]), int(ck[-1])
    k, v = rand_bf16(rng, (1, T, Hkv, d)), rand_bf16(rng, (1, T, Hkv, d))
    q = rand_bf16(rng, (len(lens), Hq, d))
    kv_index = np.zeros((Hkv, Kt), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            kv_index[g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    kv_mask = rng.choice(np.array([1, 2], dtype=np.int8), size=T)
    reordered, loc, rem, nl, nr = oracle.split_index(kv_index, kv_mask, cu, ck, reorder=True)
    assert len(set(nr.ravel().tolist())) > 1
    # remote lane: the first nr[b][g] entries of every reordered row are fetched and packed (counts per head)
    pk, pv = oracle.pack_kv(k, v, cu, reordered[None], ck, sel_count=nr[None])
    # two-lane attention: packed remote rows, then the local rest of the reordered row read by index from the cache
    out, lse = oracle.sparse_decode_attn(q, pk[0], pv[0], ck, k[0], v[0], cu, reordered, ck, packed_count=nr, local_skip=nr)
    # reference: everything read by index (one lane)
    empty = np.zeros((0, d), dtype=np.uint16)
    want, want_lse = oracle.sparse_decode_attn(q, empty, empty, cu_of((0, 0)), k[0], v[0], cu, kv_index, ck)
    assert np.allclose(out, want, atol=1e-6) and np.allclose(lse, want_lse, atol=1e-6)
