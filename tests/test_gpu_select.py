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
