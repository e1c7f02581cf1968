"""Run the C-ABI calls on numpy inputs (through the Python binding) and return numpy outputs.

Every output buffer is allocated with guard bands filled with a sentinel on both sides; the helpers
assert that the guards are untouched after the call, and that the device status word is as expected.
"""
import numpy as np
import torch

import paper_2607_28150_b200.binding as sg

GUARD = 64  # elements on each side


def dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


class Guarded:
    def __init__(self, shape, dtype, sentinel):
        n = int(np.prod(shape))
        self.n, self.shape, self.sentinel = n, tuple(shape), sentinel
        self.buf = torch.full((n + 2 * GUARD,), sentinel, dtype=dtype, device="cuda")
        self.view = self.buf[GUARD:GUARD + n].view(*shape) if n else self.buf[GUARD:GUARD].view(*shape)

    def numpy(self):
        torch.cuda.synchronize()
        b = self.buf.cpu()
        assert bool((b[:GUARD] == self.sentinel).all()) and bool((b[GUARD + self.n:] == self.sentinel).all()), \
            "guard band overwritten"
        out = b[GUARD:GUARD + self.n].view(*self.shape).numpy()
        return out.view(np.uint16) if out.dtype == np.int16 else out


def shape_of(L, Hq, Hkv, d, W, cu, **strides):
    cu = np.asarray(cu, dtype=np.int32)
    lens = np.diff(cu)
    return sg.make_shape(L, Hq, Hkv, d, W, dev(cu), int(cu[-1]), int(lens.max()) if len(lens) else 0, **strides)


def status_word():
    return torch.zeros(4, dtype=torch.int32, device="cuda")


def read_status(st):
    torch.cuda.synchronize()
    return int(st[0].item())


def score(q_win, k_cache, cu, expect_status=0):
    L, B, W, Hq, d = q_win.shape
    _, T, Hkv, _ = k_cache.shape
    shp = shape_of(L, Hq, Hkv, d, W, cu)
    imp = Guarded((L, Hkv, T), torch.float32, -7.0)
    ws = sg.alloc_workspace(sg.SG_OP_SCORE, shp)
    st = status_word()
    sg.sg_score(shp, dev(q_win), dev(k_cache), imp.view, ws, st)
    out = imp.numpy()
    assert read_status(st) == expect_status
    return out


def select_topk(importance, cu, cu_k, expect_status=0):
    L, Hkv, T = importance.shape
    shp = shape_of(L, Hkv, Hkv, 128, 1, cu)
    cu_k = np.asarray(cu_k, dtype=np.int32)
    sel = Guarded((L, Hkv, int(cu_k[-1])), torch.int32, -99)
    st = status_word()
    sg.sg_select_topk(shp, dev(np.asarray(importance, np.float32)), dev(cu_k), int(cu_k[-1]), sel.view, None, st)
    out = sel.numpy()
    assert read_status(st) == expect_status
    return out


def pack_kv(k_cache, v_cache, cu, sel_idx, cu_k, expect_status=0):
    L, T, Hkv, d = k_cache.shape
    shp = shape_of(L, Hkv, Hkv, d, 1, cu)
    cu_k = np.asarray(cu_k, dtype=np.int32)
    Ktot = int(cu_k[-1])
    pk = Guarded((L, Ktot * Hkv, d), torch.int16, 0x5555)
    pv = Guarded((L, Ktot * Hkv, d), torch.int16, 0x5555)
    st = status_word()
    sg.sg_pack_kv(shp, dev(k_cache), dev(v_cache), dev(sel_idx), dev(cu_k), Ktot, pk.view, pv.view, st)
    a, b = pk.numpy(), pv.numpy()
    assert read_status(st) == expect_status
    return a, b


def select_pack_kv(importance, k_cache, v_cache, cu, cu_k, expect_status=0):
    L, T, Hkv, d = k_cache.shape
    shp = shape_of(L, Hkv, Hkv, d, 1, cu)
    cu_k = np.asarray(cu_k, dtype=np.int32)
    Ktot = int(cu_k[-1])
    sel = Guarded((L, Hkv, Ktot), torch.int32, -99)
    pk = Guarded((L, Ktot * Hkv, d), torch.int16, 0x5555)
    pv = Guarded((L, Ktot * Hkv, d), torch.int16, 0x5555)
    st = status_word()
    sg.sg_select_pack_kv(shp, dev(np.asarray(importance, np.float32)), dev(cu_k), Ktot, dev(k_cache), dev(v_cache),
                         sel.view, pk.view, pv.view, st)
    s_, a, b = sel.numpy(), pk.numpy(), pv.numpy()
    assert read_status(st) == expect_status
    return s_, a, b


def sparse_decode_attn(q, packed_k, packed_v, cu_k, local_k, local_v, cu, local_idx, cu_nloc, softmax_scale=0.0,
                       expect_status=0):
    B, Hq, d = q.shape
    T, Hkv, _ = local_k.shape
    shp = shape_of(1, Hq, Hkv, d, 1, cu)
    cu_k = np.asarray(cu_k, dtype=np.int32)
    cu_nloc = np.asarray(cu_nloc, dtype=np.int32)
    Ktot, NLtot = int(cu_k[-1]), int(cu_nloc[-1])
    out = Guarded((B, Hq, d), torch.int16, 0x5555)
    lse = Guarded((B, Hq), torch.float32, -7.0)
    ws = sg.alloc_workspace(sg.SG_OP_SPARSE_DECODE_ATTN, shp, Ktot, NLtot)
    st = status_word()
    sg.sg_sparse_decode_attn(shp, dev(q), dev(packed_k) if Ktot else None, dev(packed_v) if Ktot else None, dev(cu_k),
                             Ktot, dev(local_k), dev(local_v), dev(local_idx) if NLtot else None, dev(cu_nloc), NLtot,
                             out.view, lse.view, softmax_scale, ws, st)
    o, l = out.numpy(), lse.numpy()
    assert read_status(st) == expect_status
    from paper_2607_28150_b200.workloads import bf16_bits_to_f32
    return bf16_bits_to_f32(o), l
