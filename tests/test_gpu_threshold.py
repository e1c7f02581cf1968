"""GPU parity: threshold (alpha) selection under a cap against the oracle, bit-exact indices and counts."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def run(x, lens, caps, alpha):
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    cu, cc = cu_of(lens), cu_of(caps)
    L, Hkv, T = x.shape
    shp = gpu_ops.shape_of(L, Hkv, Hkv, 128, 1, cu)
    sel = gpu_ops.Guarded((L, Hkv, int(cc[-1])), torch.int32, -7)
    cnt = gpu_ops.Guarded((L, len(lens), Hkv), torch.int32, -7)
    st = gpu_ops.status_word()
    sg.sg_select_threshold(shp, gpu_ops.dev(x), alpha, gpu_ops.dev(cc), int(cc[-1]), sel.view, cnt.view, st)
    got_sel, got_cnt = sel.numpy(), cnt.numpy()
    assert gpu_ops.read_status(st) == 0
    want_sel, want_cnt = oracle.select_threshold(x, cu, alpha, cc)
    assert np.array_equal(got_cnt, want_cnt)
    assert np.array_equal(got_sel, want_sel)
    return got_sel, got_cnt


@pytest.mark.parametrize("alpha", [0.0, 0.05, 0.5, 5.0, 1e9])
def test_threshold_matches_oracle_ragged(alpha):
    rng = np.random.default_rng(0)
    lens = (300, 64, 5000, 77, 1)
    caps = tuple(max(1, -(-n // 5)) for n in lens)               # the paper's maximum selection ratio, 20 %
    x = (rng.standard_normal((2, 4, sum(lens))) * 0.7).astype(np.float32)
    run(x, lens, caps, alpha)


def test_threshold_on_importance_like_rows_of_the_8b_shape():
    """Rows shaped like sg_score's output on the 8B-shaped cache (mostly small, 1 % heavy hitters), cap 20 %."""
    rng = np.random.default_rng(1)
    N, L, Hkv = 8192, 3, 8
    x = (rng.random((L, Hkv, N)) * 0.02).astype(np.float32)
    heavy = rng.choice(N, N // 100, replace=False)
    x[:, :, heavy] += rng.random((L, Hkv, len(heavy))).astype(np.float32) * 4
    for alpha in (0.5, 2.0, 3.99):
        sel, cnt = run(x, (N,), (1639,), alpha)
        assert cnt.max() <= 1639 and cnt.min() >= 1


def test_threshold_ties_zero_signs_and_subnormals():
    x = np.zeros((1, 2, 512), dtype=np.float32)
    x[0, 0, :] = 1.0                                             # all equal: nothing exceeds max - 0, everything exceeds max - 1
    x[0, 1, :] = np.float32(1e-42)                               # subnormal scores
    x[0, 1, 100:110] = 0.0
    x[0, 1, 110:120] = -0.0
    for alpha, cap in ((0.0, 100), (1.0, 100), (1.0, 512), (np.float32(1e-42), 300), (np.float32(5e-43), 300)):
        run(x, (512,), (cap,), float(alpha))


def test_threshold_long_rows_use_the_wide_select():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 1, 40000)).astype(np.float32)
    run(x, (40000,), (8000,), 1.0)
    run(x, (40000,), (8000,), 6.0)
