"""GPU parity: sg_select_topk against the oracle, bit-exact index sets in ascending order."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def check(x, lens, ks, expect_status=0):
    import gpu_ops
    cu, ck = cu_of(lens), cu_of(ks)
    want = oracle.select_topk(x, cu, ck)
    got = gpu_ops.select_topk(x, cu, ck, expect_status)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("lens,ks,L,Hkv", [
    ((1024,), (128,), 1, 2),
    ((8192,), (820,), 2, 8),
    ((33, 1, 700, 5000), (5, 1, 0, 4999), 2, 3),
    ((32768,), (2048,), 1, 2),
    ((12000, 9000), (1200, 1), 1, 2),     # 16 keys per thread in registers
    ((40000,), (4000,), 1, 1),            # shared-memory key buffer variant
    ((60000,), (3000,), 1, 1),            # longer than the shared-memory key buffer: global-memory path
])
def test_select_random_values(lens, ks, L, Hkv):
    rng = np.random.default_rng(0)
    x = rng.random((L, Hkv, sum(lens)), dtype=np.float32) ** 4
    check(x, lens, ks)


def test_select_heavy_ties_and_special_values():
    rng = np.random.default_rng(1)
    n = 4096
    x = rng.choice(np.array([0.0, -0.0, 1e-42, 0.5, 0.5, 0.5, 2.0, np.inf, -np.inf, -3.0], dtype=np.float32), size=(1, 4, n))
    for k in (1, 7, 400, 2048, 4095, 4096):
        check(x, (n,), (k,))


def test_select_all_equal_and_full_budget():
    x = np.full((1, 2, 1000), 0.125, dtype=np.float32)
    check(x, (1000,), (10,))
    check(x, (600, 400), (600, 1))


def test_select_softmax_like_rows():
    """Importance-like input: a few large masses, a long tail of tiny positive values with many exact ties."""
    rng = np.random.default_rng(2)
    n = 8192
    x = (rng.random((1, 8, n), dtype=np.float32) * 1e-4).astype(np.float32)
    x[:, :, rng.choice(n, 80, replace=False)] += 3.0
    x[:, :, 100:4000] = np.float32(2.5e-5)
    check(x, (n,), (820,))


def test_select_budget_above_length_is_flagged():
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    x = np.arange(8, dtype=np.float32)[None, None]
    got = gpu_ops.select_topk(x, cu_of((8,)), cu_of((10,)), expect_status=1 << sg.SG_ERR_INVALID)
    assert got[0, 0].tolist() == list(range(8)) + [-1, -1]


def test_select_narrow_clustered_and_wide_key_ranges():
    """Rows whose values span a few ulps, rows with half of the values inside a 4096-ulp cluster that holds the threshold
    (many keys stay in the interval after two narrowing passes), and rows spread over the whole float range."""
    rng = np.random.default_rng(7)
    n = 8192
    one = np.float32(1.0).view(np.uint32)
    narrow = (one + rng.integers(0, 40, size=(1, 4, n)).astype(np.uint32)).view(np.float32)
    check(narrow, (n,), (820,))
    bits = (np.uint32(0x10000000) + rng.integers(0, 1 << 29, size=(1, 4, n)).astype(np.uint32))
    cluster = rng.random((1, 4, n)) < 0.5
    bits[cluster] = one + rng.integers(0, 4096, size=int(cluster.sum())).astype(np.uint32)
    clustered = bits.view(np.float32)
    check(clustered, (n,), (820,))
    check(np.ascontiguousarray(clustered[:, :, :8190]), (5001, 3189), (4000, 7))     # unaligned second row
    wide = (rng.standard_normal((2, 4, n)) * 10.0 ** rng.uniform(-35, 35, size=(2, 4, n))).astype(np.float32)
    wide[:, :, ::97] = np.float32(np.inf)
    wide[:, :, 5::101] = -np.float32(np.inf)
    check(wide, (n,), (1000,))
    check(wide, (4096, 4096), (4000, 2))


def test_select_nan_ordered_by_bit_pattern():
    """NaNs rank where their bit patterns put them (clear sign bit: above +inf; set sign bit: below -inf), on every
    kernel variant: registers (8 / 16 / 32 keys per thread), keys in shared memory, keys re-read from global memory."""
    rng = np.random.default_rng(11)
    for n, k in ((3000, 100), (8192, 820), (30000, 2500), (40000, 3000), (60000, 500)):
        x = rng.standard_normal((1, 2, n)).astype(np.float32)
        xb = x.view(np.uint32)
        xb[0, :, ::13] = 0x7FC00000 | rng.integers(0, 1 << 22, size=xb[0, :, ::13].shape).astype(np.uint32)
        xb[0, :, 5::17] = 0xFFC00000 | rng.integers(0, 1 << 22, size=xb[0, :, 5::17].shape).astype(np.uint32)
        xb[0, :, 7::19] = 0x7F800001                      # signalling NaN with the smallest payload
        check(x, (n,), (k,))
        check(x, (n,), (n - 3,))                          # the negative NaNs are the ones left out


def test_select_row_longer_than_max_seqlen_is_flagged_not_read():
    """shape->max_seqlen sizes the kernels' key storage.  A sequence longer than it must set SG_ERR_INVALID and get
    an empty row (-1), with no access outside the buffers, in the selection, the fused selection + gather, and the
    shared-memory variant; the other sequences of the batch are selected as usual."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(12)
    for lens, ks, lie, L, Hkv in (((3000, 9000), (30, 90), 4096, 1, 2), ((1000, 9000), (10, 90), 4096, 10, 8),
                                  ((1000, 50000), (10, 100), 34000, 1, 1)):
        cu, ck = cu_of(lens), cu_of(ks)
        T, Kt, d = int(cu[-1]), int(ck[-1]), 64
        x = rng.random((L, Hkv, T), dtype=np.float32)
        shp = sg.make_shape(L, Hkv, Hkv, d, 1, gpu_ops.dev(cu), T, lie)
        want = oracle.select_topk(x, cu, ck)
        want[:, :, ck[1]:ck[2]] = -1
        sel = gpu_ops.Guarded((L, Hkv, Kt), torch.int32, -99)
        st = gpu_ops.status_word()
        sg.sg_select_topk(shp, gpu_ops.dev(x), gpu_ops.dev(ck), Kt, sel.view, None, st)
        assert np.array_equal(sel.numpy(), want)
        assert gpu_ops.read_status(st) == 1 << sg.SG_ERR_INVALID
        if lie > 32768:
            continue
        k = rng.integers(0, 1 << 16, size=(L, T, Hkv, d), dtype=np.uint16)
        v = rng.integers(0, 1 << 16, size=(L, T, Hkv, d), dtype=np.uint16)
        sel = gpu_ops.Guarded((L, Hkv, Kt), torch.int32, -99)
        pk = gpu_ops.Guarded((L, Kt * Hkv, d), torch.int16, 0x5555)
        pv = gpu_ops.Guarded((L, Kt * Hkv, d), torch.int16, 0x5555)
        st = gpu_ops.status_word()
        sg.sg_select_pack_kv(shp, gpu_ops.dev(x), gpu_ops.dev(ck), Kt, gpu_ops.dev(k), gpu_ops.dev(v), sel.view, pk.view,
                             pv.view, st)
        assert np.array_equal(sel.numpy(), want)
        assert gpu_ops.read_status(st) == (1 << sg.SG_ERR_INVALID) | (1 << sg.SG_ERR_INDEX)
        safe = np.where(want < 0, 0, want)
        pk_o, pv_o = oracle.pack_kv(k, v, cu, safe, ck)
        rows = slice(ck[1] * Hkv, ck[2] * Hkv)
        pk_o[:, rows] = 0
        pv_o[:, rows] = 0
        assert np.array_equal(pk.numpy(), pk_o) and np.array_equal(pv.numpy(), pv_o)
