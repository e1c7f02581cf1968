"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only the tests, the smoke check and the benchmark's cpu-baseline leg may import this package.
It compiles ``sgo.c`` with gcc on first use and marshals numpy arrays; all arithmetic is in the C
file.  bf16 tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sgo.c")
_LIB = os.path.join(_HERE, "libsgo.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp) next to its source; returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.sgo_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(_load().sgo_max_threads())


def set_threads(n: int) -> None:
    _load().sgo_set_threads(ctypes.c_int(int(n)))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype != dtype:
        raise TypeError("expected %s, got %s" % (np.dtype(dtype), a.dtype))
    return np.ascontiguousarray(a)


def _i64(x):
    return ctypes.c_int64(int(x))


def score(q_win: np.ndarray, k_cache: np.ndarray, cu_seqlens: np.ndarray, window: Optional[int] = None) -> np.ndarray:
    """importance float32 [L][H_kv][T] from q_win uint16 [L][B][W][H_q][d] and k_cache uint16 [L][T][H_kv][d]."""
    q_win, k_cache, cu = _c(q_win, np.uint16), _c(k_cache, np.uint16), _c(cu_seqlens, np.int32)
    L, B, W, Hq, d = q_win.shape
    L2, T, Hkv, d2 = k_cache.shape
    assert L == L2 and d == d2 and cu.shape == (B + 1,) and cu[-1] == T
    assert window is None or window == W
    imp = np.zeros((L, Hkv, T), dtype=np.float32)
    rc = _load().sgo_score(L, B, Hq, Hkv, d, W, _p(cu), _p(q_win), _p(k_cache),
                           _i64(T * Hkv * d), _i64(Hkv * d), _i64(d), _p(imp))
    if rc:
        raise RuntimeError("sgo_score failed: %d" % rc)
    return imp


def select_topk(importance: np.ndarray, cu_seqlens: np.ndarray, cu_k: np.ndarray) -> np.ndarray:
    """sel_idx int32 [L][H_kv][K_tot] (ascending, sequence-local) from importance float32 [L][H_kv][T]."""
    imp, cu, ck = _c(importance, np.float32), _c(cu_seqlens, np.int32), _c(cu_k, np.int32)
    L, Hkv, T = imp.shape
    B = cu.shape[0] - 1
    assert cu[-1] == T and ck.shape == (B + 1,)
    sel = np.zeros((L, Hkv, int(ck[-1])), dtype=np.int32)
    rc = _load().sgo_select_topk(L, B, Hkv, _p(cu), _p(imp), _p(ck), _p(sel))
    if rc:
        raise RuntimeError("sgo_select_topk failed: %d" % rc)
    return sel


def select_threshold(scores: np.ndarray, cu_seqlens: np.ndarray, alpha: float, cu_cap: np.ndarray):
    """Threshold selection: per (layer, sequence, KV head) the tokens with score > row max - alpha, at most
    cap_b of them (the largest, ties to the lower index).  Returns sel_idx int32 [L][H_kv][cap_tot] (ascending,
    then -1) and sel_count int32 [L][B][H_kv]."""
    x, cu, cc = _c(scores, np.float32), _c(cu_seqlens, np.int32), _c(cu_cap, np.int32)
    L, Hkv, T = x.shape
    B = cu.shape[0] - 1
    assert cu[-1] == T and cc.shape == (B + 1,)
    sel = np.zeros((L, Hkv, int(cc[-1])), dtype=np.int32)
    cnt = np.zeros((L, B, Hkv), dtype=np.int32)
    rc = _load().sgo_select_threshold(L, B, Hkv, _p(cu), _p(x), ctypes.c_float(alpha), _p(cc), _p(sel), _p(cnt))
    if rc:
        raise RuntimeError("sgo_select_threshold failed: %d" % rc)
    return sel, cnt


def pack_kv(k_cache: np.ndarray, v_cache: np.ndarray, cu_seqlens: np.ndarray, sel_idx: np.ndarray, cu_k: np.ndarray,
            sel_count: Optional[np.ndarray] = None, fill: int = 0):
    """packed_k, packed_v uint16 [L][K_tot*H_kv][d]; row of (b, g, j) is cu_k[b]*H_kv + g*k_b + j.
    With sel_count (int32 [L][B][H_kv]) only the first sel_count[l][b][g] entries of each row are packed; the other
    rows keep `fill`."""
    k, v = _c(k_cache, np.uint16), _c(v_cache, np.uint16)
    cu, ck, sel = _c(cu_seqlens, np.int32), _c(cu_k, np.int32), _c(sel_idx, np.int32)
    L, T, Hkv, d = k.shape
    B = cu.shape[0] - 1
    Ktot = int(ck[-1])
    assert v.shape == k.shape and sel.shape == (L, Hkv, Ktot)
    pk = np.full((L, Ktot * Hkv, d), fill, dtype=np.uint16)
    pv = np.full_like(pk, fill)
    sc = None if sel_count is None else _c(sel_count, np.int32)
    assert sc is None or sc.shape == (L, B, Hkv)
    rc = _load().sgo_pack_kv(L, B, Hkv, d, _p(cu), _p(k), _p(v), _i64(T * Hkv * d), _i64(Hkv * d), _i64(d),
                             _p(sel), _p(ck), _p(pk), _p(pv), None if sc is None else _p(sc))
    if rc:
        raise RuntimeError("sgo_pack_kv failed: %d" % rc)
    return pk, pv


def sparse_decode_attn(q, packed_k, packed_v, cu_k, local_k, local_v, cu_seqlens, local_idx, cu_nloc,
                       softmax_scale: float = 0.0, packed_count: Optional[np.ndarray] = None,
                       local_skip: Optional[np.ndarray] = None):
    """(out float32 [B][H_q][d], lse float32 [B][H_q]) of attention over packed rows ++ indexed local rows.

    q uint16 [B][H_q][d]; packed_k/v uint16 [K_tot*H_kv][d]; local_k/v uint16 [T][H_kv][d];
    local_idx int32 [H_kv][NL_tot].  With packed_count (int32 [B][H_kv]) only the first packed_count[b][g] packed rows
    of each (sequence, KV head) are attended; with local_skip (int32 [B][H_kv]) the first local_skip[b][g] entries of
    each local-index row are left out.
    """
    q, pk, pv = _c(q, np.uint16), _c(packed_k, np.uint16), _c(packed_v, np.uint16)
    lk, lv = _c(local_k, np.uint16), _c(local_v, np.uint16)
    cu, ck, cl, li = _c(cu_seqlens, np.int32), _c(cu_k, np.int32), _c(cu_nloc, np.int32), _c(local_idx, np.int32)
    B, Hq, d = q.shape
    T, Hkv, d2 = lk.shape
    assert d == d2 and li.shape == (Hkv, int(cl[-1])) and pk.shape == (int(ck[-1]) * Hkv, d)
    out = np.zeros((B, Hq, d), dtype=np.float32)
    lse = np.zeros((B, Hq), dtype=np.float32)
    rc = _load().sgo_sparse_decode_attn(B, Hq, Hkv, d, _p(cu), _p(q), _p(pk), _p(pv), _p(ck), _p(lk), _p(lv),
                                        _i64(Hkv * d), _i64(d), _p(li), _p(cl), ctypes.c_double(softmax_scale),
                                        _p(out), _p(lse), None if packed_count is None else _p(_c(packed_count, np.int32)),
                                        None if local_skip is None else _p(_c(local_skip, np.int32)))
    if rc:
        raise RuntimeError("sgo_sparse_decode_attn failed: %d" % rc)
    return out, lse


def split_index(kv_index, kv_mask, cu_seqlens, cu_k, reorder: bool = True):
    """Algorithm 1.  Returns (reordered, local_index, remote_index, n_local [B][H_kv], n_remote [B][H_kv])."""
    idx, mask = _c(kv_index, np.int32), _c(kv_mask, np.int8)
    cu, ck = _c(cu_seqlens, np.int32), _c(cu_k, np.int32)
    Hkv, Ktot = idx.shape
    B = cu.shape[0] - 1
    assert Ktot == ck[-1] and mask.shape == (int(cu[-1]),)
    reordered = np.zeros_like(idx)
    loc = np.full_like(idx, -1)
    rem = np.full_like(idx, -1)
    nl = np.zeros((B, Hkv), dtype=np.int32)
    nr = np.zeros((B, Hkv), dtype=np.int32)
    rc = _load().sgo_split_index(B, Hkv, _p(cu), _p(ck), _p(idx), _p(mask), int(bool(reorder)),
                                 _p(reordered), _p(loc), _p(rem), _p(nl), _p(nr))
    if rc:
        raise RuntimeError("sgo_split_index failed: %d" % rc)
    return reordered, loc, rem, nl, nr


def profile_accumulate(counts, kv_index, cu_seqlens, cu_k):
    """counts int32 [H_kv][T] += 1 at every entry of kv_index int32 [H_kv][K_tot] (in place; returns counts)."""
    c, idx, cu, ck = _c(counts, np.int32), _c(kv_index, np.int32), _c(cu_seqlens, np.int32), _c(cu_k, np.int32)
    assert c is counts or np.shares_memory(c, counts)
    Hkv, T = c.shape
    rc = _load().sgo_profile_accumulate(cu.shape[0] - 1, Hkv, _p(cu), _p(ck), _p(idx), _p(c))
    if rc:
        raise RuntimeError("sgo_profile_accumulate failed: %d" % rc)
    return counts


def block_importance(counts, cu_seqlens, num_blocks: int) -> np.ndarray:
    """Eq. 1: float32 [L][M] from selection counts int32 [L][H_kv][T]."""
    c, cu = _c(counts, np.int32), _c(cu_seqlens, np.int32)
    L, Hkv, T = c.shape
    out = np.zeros((L, num_blocks), dtype=np.float32)
    _load().sgo_block_importance(L, cu.shape[0] - 1, Hkv, num_blocks, _p(cu), _p(c), _p(out))
    return out


def transfer_budget(num_layers: int, num_blocks: int, t_prefill: float, t_transfer: float) -> int:
    """Eq. 2 with its clip to [2M, LM]."""
    lib = _load()
    lib.sgo_transfer_budget.restype = ctypes.c_int64
    return int(lib.sgo_transfer_budget(num_layers, num_blocks, ctypes.c_double(t_prefill), ctypes.c_double(t_transfer)))


def proactive_mask(cu_seqlens, num_blocks: int, layer: int, selected) -> np.ndarray:
    """int8 [T]: 1 for tokens of layer `layer` whose block is in `selected` (flat ids l*M+m, ascending), else 2."""
    cu, sel = _c(cu_seqlens, np.int32), _c(selected, np.int32)
    mask = np.zeros(int(cu[-1]), dtype=np.int8)
    _load().sgo_proactive_mask(cu.shape[0] - 1, num_blocks, _p(cu), layer, _p(sel), sel.shape[0], _p(mask))
    return mask


def push_blocks(src_k, src_v, dst_k, dst_v, cu_seqlens, num_blocks: int, layer: int, selected, kv_mask=None):
    """Online proactive transfer of one layer (Section 4.1): returns copies of dst_k, dst_v ([T][Hkv][d] uint16)
    with the rows of every selected block of `layer` overwritten by the source cache's rows; with kv_mask (int8 [T])
    also a copy of it with the pushed tokens set to 1."""
    cu, sel = _c(cu_seqlens, np.int32), _c(selected, np.int32)
    sk, sv = _c(src_k, np.uint16), _c(src_v, np.uint16)
    dk, dv = _c(dst_k, np.uint16).copy(), _c(dst_v, np.uint16).copy()
    T, Hkv, d = sk.shape
    assert int(cu[-1]) == T and sv.shape == sk.shape == dk.shape == dv.shape
    km = None if kv_mask is None else _c(kv_mask, np.int8).copy()
    _load().sgo_push_blocks(cu.shape[0] - 1, Hkv, d, num_blocks, _p(cu), layer, _p(sel), sel.shape[0],
                            _p(sk), _p(sv), _p(dk), _p(dv), None if km is None else _p(km))
    return (dk, dv) if km is None else (dk, dv, km)


def speculative_delivered(num_layers: int, num_blocks: int, k_r: int, ratio: float, iteration: int) -> int:
    """Blocks on the decode node after `iteration` speculative transfers (Section 4.3)."""
    lib = _load()
    lib.sgo_speculative_delivered.restype = ctypes.c_int64
    return int(lib.sgo_speculative_delivered(num_layers, num_blocks, ctypes.c_int64(k_r), ctypes.c_double(ratio), iteration))
