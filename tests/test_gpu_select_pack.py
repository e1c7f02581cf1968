"""GPU parity: sg_select_pack_kv (selection and gather in one call) against the oracle's select_topk followed by
pack_kv, bit-exact, on shapes that take the fused kernel (each of its four row-length classes, both head
dimensions) and on shapes that take the two-kernel route."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def case(seed, lens, ks, L, Hkv, d, ties=True):
    rng = np.random.default_rng(seed)
    cu, ck = cu_of(lens), cu_of(ks)
    T = int(cu[-1])
    k = rng.integers(0, 65536, size=(L, T, Hkv, d), dtype=np.uint16)
    v = rng.integers(0, 65536, size=k.shape, dtype=np.uint16)
    imp = rng.random((L, Hkv, T), dtype=np.float32)
    if ties:                                   # many equal values around the threshold: lowest positions win
        imp = np.round(imp * 64).astype(np.float32) / 64
    imp[0, 0, : min(T, 5)] = np.float32(np.inf)
    return imp, k, v, cu, ck


def check(imp, k, v, cu, ck, expect_status=0):
    import gpu_ops
    want_sel = oracle.select_topk(imp, cu, ck)
    got_sel, got_k, got_v = gpu_ops.select_pack_kv(imp, k, v, cu, ck, expect_status=expect_status)
    assert np.array_equal(got_sel, want_sel)
    want_k, want_v = oracle.pack_kv(k, v, cu, want_sel, ck)
    assert np.array_equal(got_k, want_k) and np.array_equal(got_v, want_v)


@pytest.mark.parametrize("lens,ks,L,Hkv,d", [
    ((300, 1, 77, 513), (37, 1, 0, 513), 5, 8, 128),        # 160 rows, <= 4096 tokens; empty and full budgets
    ((4096, 1000, 17, 2049), (410, 100, 2, 205), 5, 8, 64),
    ((8192, 4097), (820, 410), 10, 8, 128),                 # <= 8192 tokens
    ((5000, 8191, 3), (1, 4095, 3), 7, 8, 64),
    ((16384, 9000), (1638, 33), 10, 8, 64),                 # <= 16384 tokens
    ((8193, 100), (819, 99), 19, 4, 128),
    ((17000, 300, 50, 1), (1700, 30, 5, 1), 5, 8, 64),      # <= 32768 tokens
    ((20000, 5, 3, 2), (2000, 5, 1, 0), 5, 8, 128),
])
def test_fused_route_bit_exact(lens, ks, L, Hkv, d):
    assert L * len(lens) * Hkv >= 148
    check(*case(3, lens, ks, L, Hkv, d))


@pytest.mark.parametrize("lens,ks,L,Hkv,d", [
    ((1024,), (128,), 1, 2, 64),                            # few rows: two kernels
    ((2048, 999), (205, 100), 2, 8, 128),
    ((40000,), (4000,), 1, 2, 64),                          # rows beyond the register-resident kernels
])
def test_two_kernel_route_bit_exact(lens, ks, L, Hkv, d):
    check(*case(4, lens, ks, L, Hkv, d))


def test_fused_matches_the_two_calls_on_continuous_scores():
    import gpu_ops
    imp, k, v, cu, ck = case(5, (3000, 777, 4000), (300, 77, 400), 7, 8, 128, ties=False)
    sel2 = gpu_ops.select_topk(imp, cu, ck)
    k2, v2 = gpu_ops.pack_kv(k, v, cu, sel2, ck)
    sel1, k1, v1 = gpu_ops.select_pack_kv(imp, k, v, cu, ck)
    assert np.array_equal(sel1, sel2) and np.array_equal(k1, k2) and np.array_equal(v1, v2)


def test_fused_oversized_budget_sets_both_bits_and_zero_rows():
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    lens, ks, L, Hkv, d = (100, 40), (10, 44), 10, 8, 64     # second sequence asks for more rows than it has tokens
    imp, k, v, cu, ck = case(6, lens, ks, L, Hkv, d)
    bits = (1 << sg.SG_ERR_INVALID) | (1 << sg.SG_ERR_INDEX)
    sel, pk, pv = gpu_ops.select_pack_kv(imp, k, v, cu, ck, expect_status=bits)
    assert np.array_equal(sel[:, :, 10:50], np.broadcast_to(np.arange(40, dtype=np.int32), (L, Hkv, 40)))
    assert (sel[:, :, 50:] == -1).all()
    for g in range(Hkv):
        base = 10 * Hkv + g * 44
        assert np.array_equal(pk[:, base:base + 40], k[:, 100:140, g]) and np.array_equal(pv[:, base:base + 40], v[:, 100:140, g])
        assert not pk[:, base + 40:base + 44].any() and not pv[:, base + 40:base + 44].any()
    # the first sequence is a normal selection
    want = oracle.select_topk(np.ascontiguousarray(imp[:, :, :100]), cu_of((100,)), cu_of((10,)))
    assert np.array_equal(sel[:, :, :10], want)


def test_fused_strided_cache_view():
    """The fused kernel gathers through the cache strides of the shape: a cache whose token stride is wider than
    H_kv * d (a slice of a larger allocation), 160 rows so that the one-kernel route is taken."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    lens, ks, L, Hkv, d = (200, 77), (33, 8), 10, 8, 128
    imp, k, v, cu, ck = case(8, lens, ks, L, Hkv, d)
    T, pad, Ktot = int(cu[-1]), 2, int(ck[-1])
    kbig = np.zeros((L, T, Hkv + pad, d), dtype=np.uint16); kbig[:, :, :Hkv] = k
    vbig = np.zeros_like(kbig); vbig[:, :, :Hkv] = v
    shp = gpu_ops.shape_of(L, Hkv, Hkv, d, 1, cu, layer_stride=T * (Hkv + pad) * d, token_stride=(Hkv + pad) * d)
    sel = torch.full((L, Hkv, Ktot), -99, dtype=torch.int32, device="cuda")
    pk = torch.zeros((L, Ktot * Hkv, d), dtype=torch.int16, device="cuda")
    pv = torch.zeros_like(pk)
    st = gpu_ops.status_word()
    sg.sg_select_pack_kv(shp, gpu_ops.dev(imp), gpu_ops.dev(ck), Ktot, gpu_ops.dev(kbig), gpu_ops.dev(vbig), sel, pk, pv, st)
    assert gpu_ops.read_status(st) == 0
    want_sel = oracle.select_topk(imp, cu, ck)
    want_k, want_v = oracle.pack_kv(k, v, cu, want_sel, ck)
    assert np.array_equal(sel.cpu().numpy(), want_sel)
    assert np.array_equal(pk.cpu().numpy().view(np.uint16), want_k)
    assert np.array_equal(pv.cpu().numpy().view(np.uint16), want_v)
