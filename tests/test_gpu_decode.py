"""GPU parity: sg_sparse_decode_attn against the fp64 oracle (bf16 output within 2e-2 absolute, lse 1e-3)."""
import numpy as np
import pytest

import oracle
from helpers import cu_of, rand_bf16
from paper_2607_28150_b200 import workloads as wl

pytestmark = pytest.mark.gpu

OUT_ATOL = 2e-2     # bf16 attention outputs against the fp32-rounded fp64 oracle
LSE_ATOL = 1e-3


def build(seed, lens, ks, nls, Hq, Hkv, d, scale=1.0):
    rng = np.random.default_rng(seed)
    cu, ck, cl = cu_of(lens), cu_of(ks), cu_of(nls)
    T = int(cu[-1])
    k = rand_bf16(rng, (T, Hkv, d), scale)
    v = rand_bf16(rng, (T, Hkv, d))
    q = rand_bf16(rng, (len(lens), Hq, d))
    sel = np.zeros((1, Hkv, int(ck[-1])), dtype=np.int32)
    loc = np.zeros((Hkv, int(cl[-1])), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            perm = rng.permutation(n).astype(np.int32)
            sel[0, g, ck[b]:ck[b + 1]] = np.sort(perm[: ks[b]])
            loc[g, cl[b]:cl[b + 1]] = perm[ks[b]: ks[b] + nls[b]]
    pk, pv = oracle.pack_kv(k[None], v[None], cu, sel, ck)
    return q, pk[0], pv[0], ck, k, v, cu, loc, cl


def compare(args, **kw):
    import gpu_ops
    want_o, want_l = oracle.sparse_decode_attn(*args, **{k: v for k, v in kw.items() if k == "softmax_scale"})
    got_o, got_l = gpu_ops.sparse_decode_attn(*args, **kw)
    assert np.abs(got_o - want_o).max() <= OUT_ATOL
    fin = np.isfinite(want_l)
    assert np.array_equal(np.isneginf(got_l), np.isneginf(want_l))
    assert np.abs(got_l[fin] - want_l[fin]).max(initial=0.0) <= LSE_ATOL


@pytest.mark.parametrize("lens,ks,nls,Hq,Hkv,d", [
    ((1024,), (128,), (32,), 8, 2, 64),                       # tiny config
    ((8192,), (820,), (422,), 32, 8, 128),                    # one layer of the 8B-shaped config
    ((300, 64, 5000, 77), (37, 64, 1000, 0), (11, 0, 777, 70), 32, 8, 128),   # ragged; empty sources
    ((4096,) * 3, (100, 4096, 1), (3996, 0, 0), 8, 8, 128),   # G = 1, full budget, single token
    ((2000,), (333,), (100,), 32, 2, 128),                    # G = 16
    ((513,), (65,), (63,), 16, 2, 64),                        # G = 8, d = 64, ragged tiles
    ((3000,), (700,), (300,), 2, 2, 64),                      # G = 1, d = 64: clusters of 8, eight outputs per owner
    ((2500,), (350,), (150,), 4, 2, 64),                      # G = 2, d = 64, short list: 4-warp CTAs in clusters of 8
    ((4096,) * 2, (1000,) * 2, (229,) * 2, 32, 8, 128),       # two sequences: 8-warp CTAs in clusters of 4
    ((12000,), (5000,), (3333,), 8, 2, 128),                  # few heads, long lists: clusters of 8, many slices per warp
    ((9000, 100), (4100, 10), (4500, 90), 4, 1, 128),         # one head, ragged pair of sequences
    ((25000,) * 3, (12000,) * 3, (8000,) * 3, 8, 8, 128),     # clusters of 4, long CTA ranges
    (tuple(200 + 13 * i for i in range(40)), tuple(5 * i for i in range(40)), tuple(150 - 3 * i for i in range(40)), 32, 8, 128),   # more pairs than SMs: 4-warp CTAs, no clusters
    (tuple(90 + 7 * i for i in range(80)), (33,) * 80, tuple(i % 50 for i in range(80)), 32, 2, 64),   # same, G = 16, d = 64
])
def test_decode_matches_oracle(lens, ks, nls, Hq, Hkv, d):
    compare(build(0, lens, ks, nls, Hq, Hkv, d))


def test_decode_peaked_softmax_and_scale_override():
    args = build(1, (3000,), (500,), (300,), 32, 8, 128, scale=3.0)
    compare(args)
    compare(args, softmax_scale=0.02)


def test_decode_empty_sequence_gives_zero_and_minus_inf():
    compare(build(2, (100, 200), (0, 20), (0, 10), 8, 2, 128))


def test_decode_full_budget_equals_full_attention_any_split():
    """Selected fraction 100 %: every token attended once, wherever the packed/local split falls."""
    import gpu_ops
    import torch
    from helpers import widen
    n, Hq, Hkv, d = 4096, 32, 8, 128
    outs = []
    for rho in (0.0, 0.25, 0.5):
        nl = int(round(rho * n))
        args = build(3, (n,), (n - nl,), (nl,), Hq, Hkv, d)
        got_o, _ = gpu_ops.sparse_decode_attn(*args)
        q, _, _, _, k, v = args[:6]
        K = torch.from_numpy(widen(k)).permute(1, 0, 2)
        V = torch.from_numpy(widen(v)).permute(1, 0, 2)
        Q = torch.from_numpy(widen(q)[0]).reshape(Hkv, Hq // Hkv, d)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V).reshape(Hq, d).numpy()
        assert np.abs(got_o[0] - ref).max() <= OUT_ATOL
        outs.append(got_o)


def test_decode_bad_local_index_is_skipped_and_flagged():
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    q, pk, pv, ck, k, v, cu, loc, cl = build(4, (500,), (50,), (40,), 8, 2, 128)
    bad = loc.copy()
    bad[0, 5] = 500
    bad[1, 17] = -3
    got_o, got_l = gpu_ops.sparse_decode_attn(q, pk, pv, ck, k, v, cu, bad, cl, expect_status=1 << sg.SG_ERR_INDEX)
    # the oracle on the same lists with the two bad entries removed (39 good entries per head)
    clean = np.stack([np.delete(loc[0], 5), np.delete(loc[1], 17)])
    want_o, want_l = oracle.sparse_decode_attn(q, pk, pv, ck, k, v, cu, clean, cu_of((39,)))
    assert np.abs(got_o - want_o).max() <= OUT_ATOL
    assert np.abs(got_l - want_l).max() <= LSE_ATOL


def test_decode_batched_sweep_point():
    """A point of the decode-heavy sweep: 16 sequences of 4096 tokens, 20 % required, 25 % of it index-addressed."""
    cfg = wl.decode_sweep(16, 0.20, 0.25)
    ks, nls = cfg.budgets(), cfg.n_local()
    compare(build(5, cfg.seqlens, tuple(ks), tuple(nls), 32, 8, 128))
