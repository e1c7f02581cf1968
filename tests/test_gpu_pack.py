"""GPU parity: sg_pack_kv against the oracle, bit-exact."""
import numpy as np
import pytest

import oracle
from helpers import cu_of
from paper_2607_28150_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def random_case(seed, lens, ks, L, Hkv, d):
    rng = np.random.default_rng(seed)
    cu, ck = cu_of(lens), cu_of(ks)
    k = rng.integers(0, 65536, size=(L, int(cu[-1]), Hkv, d), dtype=np.uint16)
    v = rng.integers(0, 65536, size=k.shape, dtype=np.uint16)
    sel = np.zeros((L, Hkv, int(ck[-1])), dtype=np.int32)
    for l in range(L):
        for g in range(Hkv):
            for b, n in enumerate(lens):
                sel[l, g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    return k, v, cu, sel, ck


@pytest.mark.parametrize("lens,ks,L,Hkv,d", [
    ((1024,), (128,), 1, 2, 64),                       # tiny config shape
    ((300, 1, 77, 513), (37, 1, 0, 513), 3, 8, 128),   # ragged, empty and full budgets, tail rows
    ((2048, 999), (205, 100), 2, 8, 128),
    ((50,), (7,), 1, 1, 64),
])
def test_pack_bit_exact(lens, ks, L, Hkv, d):
    import gpu_ops
    k, v, cu, sel, ck = random_case(0, lens, ks, L, Hkv, d)
    want_k, want_v = oracle.pack_kv(k, v, cu, sel, ck)
    got_k, got_v = gpu_ops.pack_kv(k, v, cu, sel, ck)
    assert np.array_equal(got_k, want_k) and np.array_equal(got_v, want_v)


def test_pack_out_of_range_index_is_flagged_and_zeroed():
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    k, v, cu, sel, ck = random_case(1, (64, 32), (8, 8), 1, 2, 128)
    sel[0, 1, 3] = 64          # one past the end of sequence 0
    sel[0, 0, 9] = -1
    got_k, got_v = gpu_ops.pack_kv(k, v, cu, sel, ck, expect_status=1 << sg.SG_ERR_INDEX)
    good = sel.copy()
    good[0, 1, 3] = 0
    good[0, 0, 9] = 0
    want_k, want_v = oracle.pack_kv(k, v, cu, good, ck)
    bad_rows = [0 * 2 + 1 * 8 + 3, 8 * 2 + 0 * 8 + 1]
    for r in bad_rows:
        assert not got_k[0, r].any() and not got_v[0, r].any()
    mask = np.ones(got_k.shape[1], dtype=bool)
    mask[bad_rows] = False
    assert np.array_equal(got_k[0, mask], want_k[0, mask]) and np.array_equal(got_v[0, mask], want_v[0, mask])


def test_pack_strided_cache_view():
    """A cache whose token stride is wider than H_kv*d (a slice of a larger allocation)."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    k, v, cu, sel, ck = random_case(2, (200,), (33,), 2, 4, 128)
    L, T, Hkv, d = k.shape
    pad = 2
    kbig = np.zeros((L, T, Hkv + pad, d), dtype=np.uint16); kbig[:, :, :Hkv] = k
    vbig = np.zeros_like(kbig); vbig[:, :, :Hkv] = v
    shp = gpu_ops.shape_of(L, Hkv, Hkv, d, 1, cu, layer_stride=T * (Hkv + pad) * d, token_stride=(Hkv + pad) * d)
    pk = torch.zeros((L, 33 * Hkv, d), dtype=torch.int16, device="cuda")
    pv = torch.zeros_like(pk)
    sg.sg_pack_kv(shp, gpu_ops.dev(kbig), gpu_ops.dev(vbig), gpu_ops.dev(sel), gpu_ops.dev(ck), 33, pk, pv)
    want_k, want_v = oracle.pack_kv(k, v, cu, sel, ck)
    assert np.array_equal(pk.cpu().numpy().view(np.uint16), want_k)
    assert np.array_equal(pv.cpu().numpy().view(np.uint16), want_v)


def test_pack_varlen_config_sampled_rows():
    """Full-size ragged batch (8 prompts of 2K-32K tokens, 10 % budget): every packed row checked bytewise
    against the cache row its index names (the oracle's definition applied row by row)."""
    import gpu_ops
    cfg = wl.varlen(0.10)
    data = wl.make_prefill(cfg)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    sel, _, _, _ = wl.make_index_split(cfg, 0, 0, cfg.budgets(), np.zeros(cfg.batch, dtype=np.int64))
    sel = sel[None]
    got_k, got_v = gpu_ops.pack_kv(data["k"], data["v"], cu, sel, ck)
    Hkv = cfg.num_kv_heads
    for b in range(cfg.batch):
        kb = ck[b + 1] - ck[b]
        for g in range(Hkv):
            rows = ck[b] * Hkv + g * kb + np.arange(kb)
            toks = cu[b] + sel[0, g, ck[b]:ck[b + 1]]
            assert np.array_equal(got_k[0, rows], data["k"][0, toks, g])
            assert np.array_equal(got_v[0, rows], data["v"][0, toks, g])
