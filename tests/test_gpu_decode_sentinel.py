"""GPU parity of sg_sparse_decode_attn on inputs built so that the 2e-2 output tolerance bites.

With i.i.d. N(0,1) keys and values, a single dropped, duplicated or misplaced V row moves a 1000-token attention
output by about 1e-3: far below the tolerance.  Here every (sequence, KV head) list has about 400 "live" tokens
spread at random over the whole list -- packed part and index-addressed part alike -- whose keys are one and the
same vector aligned with the group's query (score ~ 35), while all other keys are zero (weight e^-35).  The softmax is
therefore uniform over the live tokens whatever the list length, and the value rows are sentinels: row j of the list
holds a single non-zero of 48..80 in column (j mod d).  Dropping, duplicating or mispairing ONE live row moves one
output column by at least 48 / 400 = 0.12, six times the tolerance, while bf16 rounding of P and of the output stays
near 2e-3.  The shapes reach every launch plan of the kernel (clusters of 8 / 4 / 2, many slices per warp, more
(sequence, head) pairs than SMs with 4-warp CTAs, G = 16, d = 64) and the counted variant with local_skip.
"""
import numpy as np
import pytest

import oracle
from helpers import cu_of
from paper_2607_28150_b200.workloads import f32_to_bf16_bits

pytestmark = pytest.mark.gpu

OUT_ATOL, LSE_ATOL = 2e-2, 1e-3
LIVE = 400


def build_sentinel(seed, lens, ks, nls, Hq, Hkv, d):
    rng = np.random.default_rng(seed)
    cu, ck, cl = cu_of(lens), cu_of(ks), cu_of(nls)
    T, B, G = int(cu[-1]), len(lens), Hq // Hkv
    k = np.zeros((T, Hkv, d), dtype=np.float32)
    v = np.zeros((T, Hkv, d), dtype=np.float32)
    qg = rng.standard_normal((B, Hkv, d)).astype(np.float32)
    q = np.repeat(qg, G, axis=1)                               # every query head of a group holds the group's vector
    sel = np.zeros((1, Hkv, int(ck[-1])), dtype=np.int32)
    loc = np.zeros((Hkv, int(cl[-1])), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            perm = rng.permutation(n).astype(np.int32)
            s_ = np.sort(perm[: ks[b]])
            l_ = perm[ks[b]: ks[b] + nls[b]]
            sel[0, g, ck[b]:ck[b + 1]] = s_
            loc[g, cl[b]:cl[b + 1]] = l_
            order = np.concatenate([s_, l_])                    # the list of (b, g): packed rows, then local rows
            nlist = len(order)
            if nlist == 0:
                continue
            live = rng.choice(nlist, size=min(LIVE, nlist), replace=False)
            qq = qg[b, g]
            k[cu[b] + order[live], g] = 3.0 * qq
            j = np.arange(nlist)
            v[cu[b] + order, g, j % d] = 48.0 + 4.0 * (j % 9)
            # tokens of the sequence outside the list: loud values that must never show up
            rest = np.setdiff1d(np.arange(n), order)
            k[cu[b] + rest, g] = 3.0 * qq
            v[cu[b] + rest, g, :] = 1000.0
    kb, vb, qb = f32_to_bf16_bits(k), f32_to_bf16_bits(v), f32_to_bf16_bits(q)
    pk, pv = oracle.pack_kv(kb[None], vb[None], cu, sel, ck)
    return qb, pk[0], pv[0], ck, kb, vb, cu, loc, cl


def check(args):
    import gpu_ops
    want_o, want_l = oracle.sparse_decode_attn(*args)
    got_o, got_l = gpu_ops.sparse_decode_attn(*args)
    assert np.abs(got_o - want_o).max() <= OUT_ATOL
    fin = np.isfinite(want_l)
    assert np.array_equal(np.isneginf(got_l), np.isneginf(want_l))
    assert np.abs(got_l[fin] - want_l[fin]).max(initial=0.0) <= LSE_ATOL
    return want_o


@pytest.mark.parametrize("lens,ks,nls,Hq,Hkv,d", [
    ((8192,), (820,), (422,), 32, 8, 128),                    # the 8B-shaped call: clusters of 8
    ((4096,) * 2, (1000,) * 2, (229,) * 2, 32, 8, 128),       # two sequences: clusters of 4
    ((12000,), (5000,), (3333,), 8, 2, 128),                  # few heads, long lists: many slices per warp
    ((25000,) * 3, (12000,) * 3, (8000,) * 3, 8, 8, 128),     # clusters of 4, long CTA ranges
    ((3000,), (700,), (300,), 2, 2, 64),                      # G = 1, d = 64: clusters of 8
    ((2000,), (333,), (100,), 32, 2, 128),                    # G = 16
    ((4096,) * 16, (614,) * 16, (205,) * 16, 32, 8, 128),     # 128 pairs: the sweep's batch-16 point
    (tuple(600 + 13 * i for i in range(40)), tuple(300 + 5 * i for i in range(40)), tuple(150 - 3 * i for i in range(40)), 32, 8, 128),   # more pairs than SMs: 4-warp CTAs, no clusters
    (tuple(500 + 7 * i for i in range(80)), (233,) * 80, tuple(100 + i % 50 for i in range(80)), 32, 2, 64),   # same, G = 16, d = 64
    ((5000,), (0,), (1500,), 32, 8, 128),                     # index-addressed rows only
    ((5000,), (1500,), (0,), 32, 8, 128),                     # packed rows only
])
def test_decode_sentinel_values(lens, ks, nls, Hq, Hkv, d):
    want = check(build_sentinel(0, lens, ks, nls, Hq, Hkv, d))
    # the construction does what it says: dropping one live row would move the oracle's own output well beyond the tolerance
    assert want.max() >= 48.0 / LIVE * 0.9


def test_sentinel_inputs_make_one_dropped_row_visible():
    """The tolerance bites on these inputs: the oracle itself, given the list with ONE live local row removed, differs
    from the full answer by more than five times the tolerance."""
    q, pk, pv, ck, k, v, cu, loc, cl = build_sentinel(1, (8192,), (820,), (422,), 32, 8, 128)
    full, _ = oracle.sparse_decode_attn(q, pk, pv, ck, k, v, cu, loc, cl)
    live_rows = np.flatnonzero(k[loc[0], 0].any(axis=1))
    assert len(live_rows) > 10
    short = np.stack([np.delete(loc[g], live_rows[0] if g == 0 else 0) for g in range(loc.shape[0])])
    dropped, _ = oracle.sparse_decode_attn(q, pk, pv, ck, k, v, cu, short, cu_of((421,)))
    assert np.abs(dropped[0, :4] - full[0, :4]).max() > 5 * OUT_ATOL


def test_decode_sentinel_counted_with_local_skip():
    """The counted variant on sentinel inputs: per-head packed counts below the cap and a per-head number of skipped
    local entries; the rows left out are live ones as often as not, so attending one too many or too few shows."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    lens, ks, nls, Hq, Hkv, d = (6000, 3000), (900, 500), (700, 300), 32, 8, 128
    q, pk, pv, ck, k, v, cu, loc, cl = build_sentinel(2, lens, ks, nls, Hq, Hkv, d)
    rng = np.random.default_rng(3)
    B = len(lens)
    cnt = np.stack([rng.integers(ks[b] // 2, ks[b] + 1, size=Hkv) for b in range(B)]).astype(np.int32)
    skip = np.stack([rng.integers(0, nls[b] // 2, size=Hkv) for b in range(B)]).astype(np.int32)
    want_o, want_l = oracle.sparse_decode_attn(q, pk, pv, ck, k, v, cu, loc, cl, packed_count=cnt, local_skip=skip)
    shp = gpu_ops.shape_of(1, Hq, Hkv, d, 1, cu)
    out = gpu_ops.Guarded((B, Hq, d), torch.int16, 0x5555)
    lse = gpu_ops.Guarded((B, Hq), torch.float32, -7.0)
    st = gpu_ops.status_word()
    sg.sg_sparse_decode_attn_counted(shp, gpu_ops.dev(q), gpu_ops.dev(pk), gpu_ops.dev(pv), gpu_ops.dev(ck), int(ck[-1]),
                                     gpu_ops.dev(cnt), gpu_ops.dev(k), gpu_ops.dev(v), gpu_ops.dev(loc), gpu_ops.dev(cl),
                                     int(cl[-1]), out.view, lse.view, 0.0, st, None, gpu_ops.dev(skip))
    from paper_2607_28150_b200.workloads import bf16_bits_to_f32
    got_o, got_l = bf16_bits_to_f32(out.numpy()), lse.numpy()
    assert gpu_ops.read_status(st) == 0
    assert np.abs(got_o - want_o).max() <= OUT_ATOL
    assert np.abs(got_l - want_l).max() <= LSE_ATOL
