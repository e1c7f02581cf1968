"""Pins for the oracle's gather-pack (Section 4.2: selected KV of shape BH x k x d)."""
import numpy as np

import oracle
from helpers import cu_of


def test_pack_rows_are_bytewise_copies():
    rng = np.random.default_rng(0)
    lens, ks = (11, 4, 30), (3, 4, 7)
    L, Hkv, d = 2, 3, 8
    cu, ck = cu_of(lens), cu_of(ks)
    k = rng.integers(0, 65536, size=(L, int(cu[-1]), Hkv, d), dtype=np.uint16)
    v = rng.integers(0, 65536, size=k.shape, dtype=np.uint16)
    sel = np.zeros((L, Hkv, int(ck[-1])), dtype=np.int32)
    for l in range(L):
        for g in range(Hkv):
            for b, n in enumerate(lens):
                sel[l, g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    pk, pv = oracle.pack_kv(k, v, cu, sel, ck)
    assert pk.shape == (L, int(ck[-1]) * Hkv, d)
    for l in range(L):
        for b in range(len(lens)):
            for g in range(Hkv):
                for j in range(ks[b]):
                    row = ck[b] * Hkv + g * ks[b] + j
                    t = cu[b] + sel[l, g, ck[b] + j]
                    assert np.array_equal(pk[l, row], k[l, t, g])
                    assert np.array_equal(pv[l, row], v[l, t, g])


def test_pack_full_budget_is_head_major_transpose():
    rng = np.random.default_rng(1)
    N, Hkv, d = 13, 4, 16
    k = rng.integers(0, 65536, size=(1, N, Hkv, d), dtype=np.uint16)
    v = rng.integers(0, 65536, size=k.shape, dtype=np.uint16)
    sel = np.tile(np.arange(N, dtype=np.int32), (1, Hkv, 1))
    pk, pv = oracle.pack_kv(k, v, cu_of((N,)), sel, cu_of((N,)))
    assert np.array_equal(pk[0].reshape(Hkv, N, d), k[0].transpose(1, 0, 2))
    assert np.array_equal(pv[0].reshape(Hkv, N, d), v[0].transpose(1, 0, 2))
