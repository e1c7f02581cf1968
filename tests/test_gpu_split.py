"""GPU parity: sg_split_index (Algorithm 1) against the oracle, bit-exact."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def run_gpu(idx, mask, cu, ck, reorder, expect_status=0):
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    Hkv, Ktot = idx.shape
    B = len(cu) - 1
    shp = gpu_ops.shape_of(1, Hkv, Hkv, 128, 1, cu)
    re_ = gpu_ops.Guarded((Hkv, Ktot), torch.int32, -99)
    loc = gpu_ops.Guarded((Hkv, Ktot), torch.int32, -1)
    rem = gpu_ops.Guarded((Hkv, Ktot), torch.int32, -1)
    nl = gpu_ops.Guarded((B, Hkv), torch.int32, -5)
    nr = gpu_ops.Guarded((B, Hkv), torch.int32, -5)
    st = gpu_ops.status_word()
    sg.sg_split_index(shp, gpu_ops.dev(idx), gpu_ops.dev(ck), Ktot, gpu_ops.dev(mask), reorder, re_.view, loc.view,
                      rem.view, nl.view, nr.view, st)
    out = re_.numpy(), loc.numpy(), rem.numpy(), nl.numpy(), nr.numpy()
    assert gpu_ops.read_status(st) == expect_status
    return out


def make(seed, lens, ks, Hkv, p):
    rng = np.random.default_rng(seed)
    cu, ck = cu_of(lens), cu_of(ks)
    mask = rng.choice(np.array([0, 1, 2], dtype=np.int8), size=int(cu[-1]), p=p)
    idx = np.zeros((Hkv, int(ck[-1])), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            idx[g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    return idx, mask, cu, ck


@pytest.mark.parametrize("lens,ks,Hkv,p", [
    ((1024,), (128,), 2, (0.0, 0.7, 0.3)),
    ((8192,), (820,), 8, (0.0, 0.5, 0.5)),
    ((300, 1, 5000, 77, 40), (37, 1, 1000, 0, 40), 3, (0.1, 0.5, 0.4)),     # padding, empty row, full row
    ((32768,), (6554,), 8, (0.0, 0.34, 0.66)),
])
@pytest.mark.parametrize("reorder", [True, False])
def test_split_matches_oracle(lens, ks, Hkv, p, reorder):
    idx, mask, cu, ck = make(0, lens, ks, Hkv, p)
    want = oracle.split_index(idx, mask, cu, ck, reorder=reorder)
    got = run_gpu(idx, mask, cu, ck, reorder)
    assert np.array_equal(got[3], want[3]) and np.array_equal(got[4], want[4])
    assert np.array_equal(got[0], want[0])
    # the lists are defined up to their counts; the oracle pads with -1 and the kernel leaves the rest untouched (-1 here)
    assert np.array_equal(got[1], want[1]) and np.array_equal(got[2], want[2])


def test_split_all_local_and_all_remote():
    idx, mask, cu, ck = make(1, (500,), (100,), 2, (0.0, 1.0, 0.0))
    got = run_gpu(idx, mask, cu, ck, True)
    assert np.array_equal(got[1], idx) and (got[4] == 0).all() and (got[3] == 100).all()
    mask[:] = 2
    got = run_gpu(idx, mask, cu, ck, True)
    assert np.array_equal(got[2], idx) and np.array_equal(got[0], idx) and (got[3] == 0).all()


def test_split_out_of_range_index_is_padding_and_flagged():
    import paper_2607_28150_b200.binding as sg
    idx, mask, cu, ck = make(2, (64,), (16,), 1, (0.0, 0.5, 0.5))
    idx[0, 3] = 64
    got = run_gpu(idx, mask, cu, ck, True, expect_status=1 << sg.SG_ERR_INDEX)
    good = np.delete(idx[0], 3)
    m = mask[good]
    assert got[2][0, : got[4][0, 0]].tolist() == good[m == 2].tolist()
    assert got[1][0, : got[3][0, 0]].tolist() == good[m == 1].tolist()
    assert got[0][0, -1] == 64                       # the bad entry sorts last, with the padding class


def test_split_feeds_two_lane_decode():
    """Chain: KV index -> Algorithm 1 -> remote rows packed, local rows by index -> attention equals attention
    over the whole KV index (order and lane do not matter)."""
    import gpu_ops
    from helpers import rand_bf16
    rng = np.random.default_rng(3)
    lens, ks, Hq, Hkv, d = (3000, 700), (600, 140), 8, 2, 128
    idx, mask, cu, ck = make(4, lens, ks, Hkv, (0.0, 0.4, 0.6))
    k = rand_bf16(rng, (int(cu[-1]), Hkv, d)); v = rand_bf16(rng, (int(cu[-1]), Hkv, d)); q = rand_bf16(rng, (2, Hq, d))
    _, loc, rem, nl, nr = run_gpu(idx, mask, cu, ck, True)
    # the mask is per token, so every head of a sequence has its own counts; build per-head ragged lists by padding
    # is not possible with one cu per call, so check head by head
    pk_all, pv_all = oracle.pack_kv(k[None], v[None], cu, idx[None], ck)
    want_o, want_l = oracle.sparse_decode_attn(q, pk_all[0], pv_all[0], ck, k, v, cu, np.zeros((Hkv, 0), np.int32), cu_of((0, 0)))
    G = Hq // Hkv
    for g in range(Hkv):
        cr, cl = cu_of(nr[:, g]), cu_of(nl[:, g])
        rem_g = np.concatenate([rem[g, ck[b]: ck[b] + nr[b, g]] for b in range(2)])[None]
        loc_g = np.concatenate([loc[g, ck[b]: ck[b] + nl[b, g]] for b in range(2)])[None]
        pk, pv = gpu_ops.pack_kv(k[None, :, g:g + 1], v[None, :, g:g + 1], cu, rem_g[None], cr)
        got_o, got_l = gpu_ops.sparse_decode_attn(q[:, g * G:(g + 1) * G], pk[0], pv[0], cr, k[:, g:g + 1], v[:, g:g + 1], cu, loc_g, cl)
        assert np.abs(got_o - want_o[:, g * G:(g + 1) * G]).max() <= 2e-2
        assert np.abs(got_l - want_l[:, g * G:(g + 1) * G]).max() <= 1e-3
