"""GPU parity: sg_score against the fp64 oracle, elementwise |d| <= 1e-4 |ref| + 1e-30."""
import numpy as np
import pytest

import oracle
from helpers import cu_of, rand_bf16
from paper_2607_28150_b200 import workloads as wl

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-30


def assert_close(got, want):
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = RTOL * np.abs(want.astype(np.float64)) + ATOL
    bad = err > bound
    assert not bad.any(), "max rel err %.3e at %s (got %r want %r)" % (
        (err / np.maximum(np.abs(want), 1e-300)).max(), np.argwhere(bad)[0], got[bad][0], want[bad][0])


def run_random(seed, lens, L, W, Hq, Hkv, d, kscale=1.0):
    import gpu_ops
    rng = np.random.default_rng(seed)
    cu = cu_of(lens)
    q = rand_bf16(rng, (L, len(lens), W, Hq, d))
    k = rand_bf16(rng, (L, int(cu[-1]), Hkv, d), kscale)
    want = oracle.score(q, k, cu)
    got = gpu_ops.score(q, k, cu)
    assert_close(got, want)
    return got


def test_score_tiny_config():
    import gpu_ops
    cfg = wl.tiny()
    data = wl.make_prefill(cfg)
    want = oracle.score(data["q_win"], data["k"], data["cu_seqlens"])
    got = gpu_ops.score(data["q_win"], data["k"], data["cu_seqlens"])
    assert_close(got, want)


def test_score_llama8b_shape_two_layers():
    import gpu_ops
    cfg = wl.llama8b(num_layers=2)
    data = wl.make_prefill(cfg)
    want = oracle.score(data["q_win"], data["k"], data["cu_seqlens"])
    got = gpu_ops.score(data["q_win"], data["k"], data["cu_seqlens"])
    assert_close(got, want)
    # every softmax row sums to one: the mass of a (layer, head) is G*W
    np.testing.assert_allclose(got.astype(np.float64).sum(-1), cfg.group * cfg.window, rtol=1e-4)


@pytest.mark.parametrize("lens,L,W,Hq,Hkv,d", [
    ((300, 1, 77, 5000, 129), 2, 32, 32, 8, 128),     # ragged: prompts shorter than the window, tile tails
    ((3000,), 1, 64, 16, 2, 128),                      # R = 512: four row blocks, two K stages
    ((1500, 40), 1, 16, 2, 2, 64),                     # R = 16, G = 1
    ((700,), 1, 5, 6, 2, 64),                          # R = 15: padded to 16 columns
    ((1000, 2000), 1, 24, 16, 2, 128),                 # R = 192: one full and one partial row block
    ((4096,), 1, 8, 32, 2, 64),                        # G = 16, R = 128
    ((2000, 300), 1, 64, 16, 1, 64),                   # R = 1024 at d = 64: the largest supported row count
])
def test_score_random_shapes(lens, L, W, Hq, Hkv, d):
    run_random(1, lens, L, W, Hq, Hkv, d)


def test_score_peaked_rows():
    """Keys with large norms: exponent ranges of ~100 between the largest and typical scores."""
    run_random(2, (2048,), 1, 32, 8, 2, 128, kscale=3.0)


def test_score_llama70b_shape_one_head_full_length():
    """R = 512, N = 32768 (the long-context shape) on one KV head, heavy hitters clustered in spans."""
    import gpu_ops
    cfg = wl.Config("c4_one_head", 4, 1, 8, 1, 128, 64, (32768,), 2048, heavy="spans")
    data = wl.make_prefill(cfg)
    want = oracle.score(data["q_win"], data["k"], data["cu_seqlens"])
    got = gpu_ops.score(data["q_win"], data["k"], data["cu_seqlens"])
    assert_close(got, want)


def test_score_strided_cache():
    """K cache given as a view into a wider allocation (token stride > H_kv*d)."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(3)
    lens, L, W, Hq, Hkv, d, pad = (900,), 2, 16, 8, 2, 128, 3
    cu = cu_of(lens)
    T = int(cu[-1])
    q = rand_bf16(rng, (L, 1, W, Hq, d))
    k = rand_bf16(rng, (L, T, Hkv, d))
    kbig = rand_bf16(rng, (L, T, Hkv + pad, d))
    kbig[:, :, :Hkv] = k
    shp = gpu_ops.shape_of(L, Hq, Hkv, d, W, cu, layer_stride=T * (Hkv + pad) * d, token_stride=(Hkv + pad) * d)
    imp = torch.zeros((L, Hkv, T), dtype=torch.float32, device="cuda")
    ws = sg.alloc_workspace(sg.SG_OP_SCORE, shp)
    sg.sg_score(shp, gpu_ops.dev(q), gpu_ops.dev(kbig), imp, ws)
    assert_close(imp.cpu().numpy(), oracle.score(q, k, cu))


def test_score_late_key_far_above_everything_before_it():
    """A key whose score lies more than 2^127 (in exp2 terms) above every earlier key of its row, met in the SECOND
    key tile a warpgroup sees within a work item: pass 1 sums each chunk against a running reference that is only
    refreshed when the sum leaves the safe range, so this is the case where it must be refreshed (the unguarded sum
    would be +inf).  The shape has enough (layer, head) units that work items span eight key tiles, two per
    warpgroup.  Also the mirror case, a dominant key first and tiny ones after it."""
    import gpu_ops
    from paper_2607_28150_b200.workloads import f32_to_bf16_bits
    rng = np.random.default_rng(9)
    L, N, W, Hq, Hkv, d = 32, 4096, 8, 8, 8, 64
    cu = cu_of((N,))
    for where in (5 * 128 + 20, 3):
        qv = rng.standard_normal((L, Hkv, d)).astype(np.float32)
        q = np.broadcast_to(qv[:, None, None], (L, 1, W, Hq, d)).copy()
        k = (0.01 * rng.standard_normal((L, N, Hkv, d))).astype(np.float32)
        k[:, where] = 20.0 * qv                     # score ~ 20 |q|^2 / sqrt(d) ~ 160 nats above the rest
        qb, kb = f32_to_bf16_bits(q), f32_to_bf16_bits(k)
        want = oracle.score(qb, kb, cu)
        got = gpu_ops.score(qb, kb, cu)
        assert_close(got, want)
        assert np.all(np.isfinite(got)) and np.abs(got[:, :, where] - W).max() < 1e-2
