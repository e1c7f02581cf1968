"""GPU parity of the per-head-count path: threshold selection -> counted gather-pack -> counted decode attention."""
import numpy as np
import pytest

import oracle
from helpers import cu_of, rand_bf16
from paper_2607_28150_b200.workloads import bf16_bits_to_f32

pytestmark = pytest.mark.gpu


def run_chain(seed, lens, ratio, alpha, Hq, Hkv, d, nls, L=1):
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(seed)
    B = len(lens)
    caps = tuple(min(n, max(1, int(np.ceil(ratio * n)))) for n in lens)
    cu, cc, cl = cu_of(lens), cu_of(caps), cu_of(nls)
    T, cap_tot, NL = int(cu[-1]), int(cc[-1]), int(cl[-1])
    k, v = rand_bf16(rng, (L, T, Hkv, d)), rand_bf16(rng, (L, T, Hkv, d))
    q = rand_bf16(rng, (B, Hq, d))
    x = (rng.standard_normal((L, Hkv, T)) * 0.8).astype(np.float32)
    shpL = gpu_ops.shape_of(L, Hq, Hkv, d, 1, cu)
    shp1 = gpu_ops.shape_of(1, Hq, Hkv, d, 1, cu)
    st = gpu_ops.status_word()
    # selection (already checked bit-exact elsewhere; here it feeds the chain)
    d_sel = torch.empty((L, Hkv, cap_tot), dtype=torch.int32, device="cuda")
    d_cnt = torch.empty((L, B, Hkv), dtype=torch.int32, device="cuda")
    sg.sg_select_threshold(shpL, gpu_ops.dev(x), alpha, gpu_ops.dev(cc), cap_tot, d_sel, d_cnt, st)
    sel_o, cnt_o = oracle.select_threshold(x, cu, alpha, cc)
    assert np.array_equal(d_sel.cpu().numpy(), sel_o) and np.array_equal(d_cnt.cpu().numpy(), cnt_o)
    # counted pack: rows beyond a head's count keep the sentinel
    pk = gpu_ops.Guarded((L, cap_tot * Hkv, d), torch.int16, 0x7fc0)
    pv = gpu_ops.Guarded((L, cap_tot * Hkv, d), torch.int16, 0x7fc0)
    sg.sg_pack_kv_counted(shpL, gpu_ops.dev(k), gpu_ops.dev(v), d_sel, gpu_ops.dev(cc), cap_tot, d_cnt, pk.view, pv.view, st)
    got_pk, got_pv = pk.numpy(), pv.numpy()
    want_pk, want_pv = oracle.pack_kv(k, v, cu, sel_o, cc, sel_count=cnt_o, fill=0x7fc0)
    assert np.array_equal(got_pk, want_pk) and np.array_equal(got_pv, want_pv)
    # counted decode on every layer: packed rows of the head's count, plus index-addressed local rows
    loc = np.zeros((Hkv, NL), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            loc[g, cl[b]:cl[b + 1]] = rng.choice(n, nls[b], replace=False)
    for l in range(L):
        out = gpu_ops.Guarded((B, Hq, d), torch.int16, 0x5555)
        lse = gpu_ops.Guarded((B, Hq), torch.float32, -7.0)
        sg.sg_sparse_decode_attn_counted(shp1, gpu_ops.dev(q), pk.view[l], pv.view[l], gpu_ops.dev(cc), cap_tot, d_cnt[l].contiguous(),
                                         gpu_ops.dev(k[l]), gpu_ops.dev(v[l]), gpu_ops.dev(loc) if NL else None, gpu_ops.dev(cl), NL,
                                         out.view, lse.view, 0.0, st)
        got_o, got_l = bf16_bits_to_f32(out.numpy()), lse.numpy()
        want_o, want_l = oracle.sparse_decode_attn(q, want_pk[l], want_pv[l], cc, k[l], v[l], cu, loc, cl, packed_count=cnt_o[l])
        assert np.abs(got_o - want_o).max() <= 2e-2
        fin = np.isfinite(want_l)
        assert np.array_equal(np.isneginf(got_l), np.isneginf(want_l))
        assert np.abs(got_l[fin] - want_l[fin]).max(initial=0.0) <= 1e-3
    assert gpu_ops.read_status(st) == 0
    return cnt_o


def test_counted_chain_ragged_batch():
    cnt = run_chain(0, (300, 64, 5000, 77), 0.2, 0.8, 32, 8, 128, (11, 0, 400, 20), L=2)
    assert len(set(cnt.ravel().tolist())) > 4


def test_counted_chain_single_long_sequence_uses_clusters():
    run_chain(1, (8192,), 0.2, 1.5, 32, 8, 128, (422,))


def test_counted_chain_many_pairs_and_d64():
    run_chain(2, tuple(100 + 9 * i for i in range(40)), 0.25, 0.6, 16, 8, 64, tuple(i % 7 for i in range(40)))


def test_counts_equal_to_the_caps_reproduce_the_plain_calls():
    """alpha so large that every cap binds: counted pack/decode equal sg_pack_kv / sg_sparse_decode_attn bit for bit."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(3)
    lens, caps, Hq, Hkv, d = (700, 1300), (70, 130), 32, 8, 128
    cu, cc = cu_of(lens), cu_of(caps)
    T, cap_tot = int(cu[-1]), int(cc[-1])
    k, v = rand_bf16(rng, (1, T, Hkv, d)), rand_bf16(rng, (1, T, Hkv, d))
    q = rand_bf16(rng, (2, Hq, d))
    x = rng.standard_normal((1, Hkv, T)).astype(np.float32)
    sel, cnt = oracle.select_threshold(x, cu, 1e9, cc)
    assert np.array_equal(cnt[0], np.array([[70] * 8, [130] * 8]))
    pk_a, pv_a = gpu_ops.pack_kv(k, v, cu, sel, cc)
    shp = gpu_ops.shape_of(1, Hq, Hkv, d, 1, cu)
    pk_b = torch.zeros((1, cap_tot * Hkv, d), dtype=torch.int16, device="cuda"); pv_b = torch.zeros_like(pk_b)
    sg.sg_pack_kv_counted(shp, gpu_ops.dev(k), gpu_ops.dev(v), gpu_ops.dev(sel), gpu_ops.dev(cc), cap_tot, gpu_ops.dev(cnt), pk_b, pv_b)
    assert np.array_equal(pk_b.cpu().numpy().view(np.uint16), pk_a) and np.array_equal(pv_b.cpu().numpy().view(np.uint16), pv_a)
    loc, cl = np.zeros((Hkv, 0), dtype=np.int32), cu_of((0, 0))
    out_a, lse_a = gpu_ops.sparse_decode_attn(q, pk_a[0], pv_a[0], cc, k[0], v[0], cu, loc, cl)
    out_b = torch.empty((2, Hq, d), dtype=torch.int16, device="cuda"); lse_b = torch.empty((2, Hq), dtype=torch.float32, device="cuda")
    sg.sg_sparse_decode_attn_counted(shp, gpu_ops.dev(q), pk_b[0], pv_b[0], gpu_ops.dev(cc), cap_tot, gpu_ops.dev(cnt[0]),
                                     gpu_ops.dev(k[0]), gpu_ops.dev(v[0]), None, gpu_ops.dev(cl), 0, out_b, lse_b)
    assert np.array_equal(bf16_bits_to_f32(out_b.cpu().numpy().view(np.uint16)), out_a)
    assert np.array_equal(lse_b.cpu().numpy(), lse_a)


@pytest.mark.parametrize("lens,ks,Hq,Hkv,d,remote_share", [
    ((8192,), (820,), 32, 8, 128, 0.34),                      # 8B-shaped layer, the paper's on-demand ratio
    ((300, 64, 5000, 77), (37, 64, 1000, 5), 32, 8, 128, 0.5),
    (tuple(120 + 11 * i for i in range(40)), tuple(10 + i for i in range(40)), 16, 8, 64, 0.2),
    ((2000,), (333,), 32, 2, 128, 1.0),                       # everything remote
    ((2000,), (333,), 32, 2, 128, 0.0),                       # everything local
])
def test_two_lane_fetching_on_the_gpu(lens, ks, Hq, Hkv, d, remote_share):
    """Section 4.2 end to end through the C ABI: Algorithm 1 (split + reorder) -> fetch the remote lane into a packed
    buffer with per-head counts -> attend [packed remote rows] ++ [local rest of the row, by index].  Equals the oracle's
    attention over the KV index set read in one lane."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(4)
    B = len(lens)
    cu, ck = cu_of(lens), cu_of(ks)
    T, Kt = int(cu[-1]), int(ck[-1])
    k, v = rand_bf16(rng, (1, T, Hkv, d)), rand_bf16(rng, (1, T, Hkv, d))
    q = rand_bf16(rng, (B, Hq, d))
    kv_index = np.zeros((Hkv, Kt), dtype=np.int32)
    for g in range(Hkv):
        for b, n in enumerate(lens):
            kv_index[g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, ks[b], replace=False))
    kv_mask = np.where(rng.random(T) < remote_share, 2, 1).astype(np.int8)
    shp = gpu_ops.shape_of(1, Hq, Hkv, d, 1, cu)
    st = gpu_ops.status_word()
    d_idx, d_ck = gpu_ops.dev(kv_index), gpu_ops.dev(ck)
    reo = torch.empty_like(d_idx); loc = torch.empty_like(d_idx); rem = torch.empty_like(d_idx)
    nl = torch.empty((B, Hkv), dtype=torch.int32, device="cuda"); nr = torch.empty_like(nl)
    sg.sg_split_index(shp, d_idx, d_ck, Kt, gpu_ops.dev(kv_mask), True, reo, loc, rem, nl, nr, st)
    # remote lane: fetch the first n_remote entries of every reordered row from the prefill-side cache
    pk = torch.zeros((1, Kt * Hkv, d), dtype=torch.int16, device="cuda"); pv = torch.zeros_like(pk)
    d_k, d_v = gpu_ops.dev(k), gpu_ops.dev(v)
    sg.sg_pack_kv_counted(shp, d_k, d_v, reo.unsqueeze(0).contiguous(), d_ck, Kt, nr.unsqueeze(0).contiguous(), pk, pv, st)
    # both lanes
    out = gpu_ops.Guarded((B, Hq, d), torch.int16, 0x5555)
    lse = gpu_ops.Guarded((B, Hq), torch.float32, -7.0)
    sg.sg_sparse_decode_attn_counted(shp, gpu_ops.dev(q), pk[0], pv[0], d_ck, Kt, nr, d_k[0], d_v[0], reo, d_ck, Kt,
                                     out.view, lse.view, 0.0, st, local_skip=nr)
    got_o, got_l = bf16_bits_to_f32(out.numpy()), lse.numpy()
    assert gpu_ops.read_status(st) == 0
    empty = np.zeros((0, d), dtype=np.uint16)
    want_o, want_l = oracle.sparse_decode_attn(q, empty, empty, cu_of((0,) * B), k[0], v[0], cu, kv_index, ck)
    assert np.abs(got_o - want_o).max() <= 2e-2 and np.abs(got_l - want_l).max() <= 1e-3
    n_remote = nr.cpu().numpy()
    assert n_remote.sum() == int((kv_mask[np.concatenate([cu[b] + kv_index[:, ck[b]:ck[b + 1]].ravel() for b in range(B)])] == 2).sum())
