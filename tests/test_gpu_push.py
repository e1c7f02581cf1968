"""GPU parity: block-granular online transfer of one layer (Section 4.1) against the oracle, bytes exact."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def run_case(seed, lens, Hkv, d, M, L, n_sel, head_major=False):
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(seed)
    cu = cu_of(lens)
    T = int(cu[-1])
    selected = np.sort(rng.choice(L * M, size=n_sel, replace=False)).astype(np.int32)
    mk = lambda: rng.integers(0, 1 << 16, size=(T, Hkv, d), dtype=np.uint16)
    sk, sv, dk, dv = mk(), mk(), mk(), mk()
    strides = {}
    to_dev = lambda a: gpu_ops.dev(a.view(np.int16))
    if head_major:                                           # cache stored [H_kv][T][d], addressed through the strides
        strides = dict(token_stride=d, head_stride=T * d)
        to_dev = lambda a: gpu_ops.dev(np.ascontiguousarray(a.transpose(1, 0, 2)).view(np.int16))
    shp = gpu_ops.shape_of(1, Hkv, Hkv, d, 1, cu, **strides)
    d_sel = gpu_ops.dev(selected) if n_sel else None
    for layer in sorted(set((0, 1, L // 2, L - 1))):
        want_k, want_v = oracle.push_blocks(sk, sv, dk, dv, cu, M, layer, selected)
        gk, gv = gpu_ops.Guarded((T * Hkv * d,), torch.int16, 0x5a5a), gpu_ops.Guarded((T * Hkv * d,), torch.int16, 0x5a5a)
        gk.view.copy_(to_dev(dk).view(-1)); gv.view.copy_(to_dev(dv).view(-1))
        sg.sg_push_blocks(shp, M, layer, d_sel, to_dev(sk), to_dev(sv), gk.view, gv.view)
        got_k, got_v = gk.numpy(), gv.numpy()
        if head_major:
            got_k = got_k.reshape(Hkv, T, d).transpose(1, 0, 2); got_v = got_v.reshape(Hkv, T, d).transpose(1, 0, 2)
        assert np.array_equal(got_k.reshape(T, Hkv, d), want_k) and np.array_equal(got_v.reshape(T, Hkv, d), want_v)


@pytest.mark.parametrize("lens,Hkv,d,M,L,n_sel", [
    ((1024,), 2, 64, 16, 4, 20),                              # tiny config
    ((8192,), 8, 128, 1024, 32, 13000),                       # 8B-shaped layer, M = 1K as in the paper, ~40 % of blocks
    ((300, 64, 5000, 77, 1), 8, 128, 64, 6, 150),             # ragged batch, a one-token sequence, M > N for some
    ((4096,) * 3, 1, 128, 7, 3, 21),                          # every block selected: dst becomes src
    ((2000,), 4, 64, 50, 5, 0),                               # nothing selected: dst untouched
])
def test_push_blocks_matches_oracle(lens, Hkv, d, M, L, n_sel):
    run_case(0, lens, Hkv, d, M, L, n_sel)


def test_push_blocks_strided_cache():
    run_case(1, (700, 1300), 4, 128, 32, 4, 50, head_major=True)


def test_push_blocks_follows_the_profile_chain():
    """Blocks chosen by Eq. 1 + Eq. 2 + global top-K_r: the pushed rows are the rows whose KV mask is 1."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(2)
    lens, L, Hkv, d, M = (3000, 500), 6, 2, 64, 32
    cu = cu_of(lens); T = int(cu[-1])
    I = rng.random((L, M)).astype(np.float32); I[:2] = np.inf
    kr = sg.sg_transfer_budget(L, M, 0.5, 1.0)
    sel = gpu_ops.select_topk(I.reshape(1, 1, L * M), cu_of((L * M,)), cu_of((kr,)))[0, 0]
    shp = gpu_ops.shape_of(1, Hkv, Hkv, d, 1, cu)
    src = torch.randn(T, Hkv, d, device="cuda").to(torch.bfloat16)
    for layer in range(L):
        dst_k = torch.zeros_like(src); dst_v = torch.zeros_like(src)
        mask = torch.zeros(T, dtype=torch.int8, device="cuda")
        sg.sg_proactive_mask(shp, M, layer, gpu_ops.dev(sel), mask)
        sg.sg_push_blocks(shp, M, layer, gpu_ops.dev(sel), src, src * 2, dst_k, dst_v)
        local = (mask == 1)[:, None, None]
        assert torch.equal(dst_k, torch.where(local, src, torch.zeros_like(src)))
        assert torch.equal(dst_v, torch.where(local, src * 2, torch.zeros_like(src)))
        if layer < 2:                                        # Eq. 1: the first two layers are always pushed whole
            assert torch.equal(dst_k, src)


def test_push_blocks_several_layers_in_one_call():
    """One call over layers 1..3 of a 5-layer cache equals the oracle's three single-layer pushes."""
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(7)
    lens, Hkv, d, M, L = (900, 333), 2, 128, 24, 5
    cu = cu_of(lens); T = int(cu[-1])
    selected = np.sort(rng.choice(L * M, size=60, replace=False)).astype(np.int32)
    mk = lambda: rng.integers(0, 1 << 16, size=(L, T, Hkv, d), dtype=np.uint16)
    sk, sv, dk, dv = mk(), mk(), mk(), mk()
    shp3 = gpu_ops.shape_of(3, Hkv, Hkv, d, 1, cu)
    gk, gv = gpu_ops.dev(dk), gpu_ops.dev(dv)
    sg.sg_push_blocks(shp3, M, 1, gpu_ops.dev(selected), gpu_ops.dev(sk)[1:], gpu_ops.dev(sv)[1:], gk[1:], gv[1:])
    got_k, got_v = gk.cpu().numpy().view(np.uint16), gv.cpu().numpy().view(np.uint16)
    for layer in range(L):
        if 1 <= layer <= 3:
            want_k, want_v = oracle.push_blocks(sk[layer], sv[layer], dk[layer], dv[layer], cu, M, layer, selected)
        else:
            want_k, want_v = dk[layer], dv[layer]
        assert np.array_equal(got_k[layer], want_k) and np.array_equal(got_v[layer], want_v)


def test_push_blocks_updates_the_kv_mask():
    """The pushed tokens become local (1) in the decode-side KV mask, every other entry (remote 2, padding 0) keeps its
    value; several layers in one call; pushing the remaining blocks afterwards completes the mask."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(11)
    lens, Hkv, d, M, L = (900, 333, 5), 2, 64, 24, 4
    cu = cu_of(lens); T = int(cu[-1])
    selected = np.sort(rng.choice(L * M, size=40, replace=False)).astype(np.int32)
    mk = lambda: rng.integers(0, 1 << 16, size=(L, T, Hkv, d), dtype=np.uint16)
    sk, sv, dk, dv = mk(), mk(), mk(), mk()
    start = np.full((L, T), 2, dtype=np.int8)
    start[:, [7, 901, T - 1]] = 0
    shpL = gpu_ops.shape_of(L, Hkv, Hkv, d, 1, cu)
    gk, gv = gpu_ops.dev(dk), gpu_ops.dev(dv)
    mask = gpu_ops.Guarded((L, T), torch.int8, 9)
    mask.view.copy_(torch.from_numpy(start).cuda())
    sg.sg_push_blocks(shpL, M, 0, gpu_ops.dev(selected), gpu_ops.dev(sk), gpu_ops.dev(sv), gk, gv, kv_mask=mask.view)
    got_mask = mask.numpy()
    for layer in range(L):
        want_k, want_v, want_m = oracle.push_blocks(sk[layer], sv[layer], dk[layer], dv[layer], cu, M, layer, selected, kv_mask=start[layer])
        assert np.array_equal(got_mask[layer], want_m)
        assert np.array_equal(gk[layer].cpu().numpy().view(np.uint16), want_k)
        assert np.array_equal(gv[layer].cpu().numpy().view(np.uint16), want_v)
    # the speculative transfer delivers the rest: afterwards every token (a pushed padding entry included) is local
    rest = np.setdiff1d(np.arange(L * M, dtype=np.int32), selected).astype(np.int32)
    sg.sg_push_blocks(shpL, M, 0, gpu_ops.dev(rest), gpu_ops.dev(sk), gpu_ops.dev(sv), gk, gv, kv_mask=mask.view)
    final = mask.numpy()
    assert np.array_equal(final, np.ones_like(start))
    assert np.array_equal(gk.cpu().numpy().view(np.uint16), sk)
