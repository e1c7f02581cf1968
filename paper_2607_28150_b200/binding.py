"""ctypes binding of libsmartgen.so: same names as the C ABI, argument marshalling only.

Every function takes torch CUDA tensors (PyTorch is used for device memory and streams, nothing
else), checks dtypes/contiguity, passes raw pointers to the library and raises `SmartGenError` on a
non-zero status.  All computation happens in the library's CUDA kernels; there is no fallback --
importing this module without the built library raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsmartgen.so")

SG_OK, SG_ERR_INVALID, SG_ERR_UNSUPPORTED, SG_ERR_WORKSPACE, SG_ERR_CUDA, SG_ERR_INDEX, SG_ERR_TIMEOUT = range(7)
SG_OP_SCORE, SG_OP_SELECT_TOPK, SG_OP_PACK_KV, SG_OP_SPARSE_DECODE_ATTN, SG_OP_SPLIT_INDEX = range(5)

# every symbol include/smartgen.h declares
EXPORTED = ("sg_workspace_bytes", "sg_score", "sg_select_topk", "sg_pack_kv", "sg_sparse_decode_attn",
            "sg_score_static", "sg_select_pack_kv", "sg_select_threshold", "sg_pack_kv_counted", "sg_sparse_decode_attn_counted", "sg_split_index", "sg_profile_accumulate", "sg_block_importance",
            "sg_transfer_budget", "sg_proactive_mask", "sg_push_blocks", "sg_speculative_delivered", "sg_strerror", "sg_last_cuda_error",
            "sg_testing_score_fault", "sg_testing_score_clock", "sg_testing_score_grid", "sg_testing_decode_overlap")
SG_SCORE_STATIC_SCRATCH_BYTES = 8 << 20

if not os.path.exists(LIB_PATH):
    raise ImportError("libsmartgen.so is not built (%s): run `python __graft_entry__.py` or "
                      "`python -m paper_2607_28150_b200.build`; there is no CPU fallback" % LIB_PATH)
_lib = ctypes.CDLL(LIB_PATH)


class SmartGenError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.sg_strerror(status).decode()
        if status == SG_ERR_CUDA:
            msg += " [cuda error %d]" % _lib.sg_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


class Shape(ctypes.Structure):
    """Mirror of `sg_shape`."""
    _fields_ = [("num_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("window", ctypes.c_int32),
                ("total_tokens", ctypes.c_int32), ("max_seqlen", ctypes.c_int32),
                ("cu_seqlens", ctypes.c_void_p), ("cache_layer_stride", ctypes.c_int64),
                ("cache_token_stride", ctypes.c_int64), ("cache_head_stride", ctypes.c_int64)]


_vp, _i32, _sz, _f = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
_sp = ctypes.POINTER(Shape)
_lib.sg_strerror.restype = ctypes.c_char_p
_lib.sg_strerror.argtypes = [ctypes.c_int]
_lib.sg_last_cuda_error.restype = ctypes.c_int
_lib.sg_workspace_bytes.restype = _sz
_lib.sg_workspace_bytes.argtypes = [ctypes.c_int, _sp, _i32, _i32]
_lib.sg_score.restype = ctypes.c_int
_lib.sg_score.argtypes = [_sp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.sg_score_static.restype = ctypes.c_int
_lib.sg_score_static.argtypes = [_sp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_select_topk.restype = ctypes.c_int
_lib.sg_select_topk.argtypes = [_sp, _vp, _vp, _i32, _vp, _vp, _sz, _vp, _vp]
_lib.sg_pack_kv.restype = ctypes.c_int
_lib.sg_pack_kv.argtypes = [_sp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp]
_lib.sg_profile_accumulate.restype = ctypes.c_int
_lib.sg_profile_accumulate.argtypes = [_sp, _vp, _vp, _i32, _vp, _vp, _vp]
_lib.sg_block_importance.restype = ctypes.c_int
_lib.sg_block_importance.argtypes = [_sp, _vp, _i32, _vp, _vp]
_lib.sg_transfer_budget.restype = ctypes.c_int64
_lib.sg_transfer_budget.argtypes = [_i32, _i32, ctypes.c_double, ctypes.c_double]
_lib.sg_speculative_delivered.restype = ctypes.c_int64
_lib.sg_speculative_delivered.argtypes = [_i32, _i32, ctypes.c_int64, ctypes.c_double, _i32]
_lib.sg_proactive_mask.restype = ctypes.c_int
_lib.sg_proactive_mask.argtypes = [_sp, _i32, _i32, _vp, _i32, _vp, _vp]
_lib.sg_select_pack_kv.restype = ctypes.c_int
_lib.sg_select_pack_kv.argtypes = [_sp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_pack_kv_counted.restype = ctypes.c_int
_lib.sg_pack_kv_counted.argtypes = [_sp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.sg_sparse_decode_attn_counted.restype = ctypes.c_int
_lib.sg_sparse_decode_attn_counted.argtypes = [_sp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _f, _vp, _vp, _vp, _vp]
_lib.sg_select_threshold.restype = ctypes.c_int
_lib.sg_select_threshold.argtypes = [_sp, _vp, _f, _vp, _i32, _vp, _vp, _vp, _vp]
_lib.sg_push_blocks.restype = ctypes.c_int
_lib.sg_push_blocks.argtypes = [_sp, _i32, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_split_index.restype = ctypes.c_int
_lib.sg_split_index.argtypes = [_sp, _vp, _vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_sparse_decode_attn.restype = ctypes.c_int
_lib.sg_sparse_decode_attn.argtypes = [_sp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _i32, _f, _vp, _vp, _vp,
                                       _sz, _vp, _vp]


_lib.sg_testing_score_fault.restype = None
_lib.sg_testing_score_fault.argtypes = [_i32, _i32]
_lib.sg_testing_score_clock.restype = None
_lib.sg_testing_score_clock.argtypes = [_vp]
_lib.sg_testing_decode_overlap.restype = None
_lib.sg_testing_decode_overlap.argtypes = [_i32]
_lib.sg_testing_score_grid.restype = _i32
_lib.sg_testing_score_grid.argtypes = [_sp]


def sg_testing_score_fault(withhold_unit: int = -1, wait_limit_ms: int = 0) -> None:
    """Test hook: withhold the done-count of one scoring unit and/or shorten every bounded wait (0 / -1 = off)."""
    _lib.sg_testing_score_fault(withhold_unit, wait_limit_ms)


def sg_testing_score_clock(buffer: Optional[torch.Tensor]) -> None:
    """Measurement hook: the next scoring kernels record their start/end clock64 and globaltimer per CTA into
    `buffer` (int64, at least 32 words per CTA); None switches it off."""
    _lib.sg_testing_score_clock(None if buffer is None else buffer.data_ptr())


def sg_testing_decode_overlap(allowed: bool) -> None:
    """Measurement hook: False launches sg_sparse_decode_attn fully ordered behind earlier work (no overlap of calls)."""
    _lib.sg_testing_decode_overlap(1 if allowed else 0)


def sg_testing_score_grid(shape: "Shape") -> int:
    return int(_lib.sg_testing_score_grid(ctypes.byref(shape)))


def make_shape(num_layers: int, num_q_heads: int, num_kv_heads: int, head_dim: int, window: int,
               cu_seqlens: torch.Tensor, total_tokens: int, max_seqlen: int,
               layer_stride: Optional[int] = None, token_stride: Optional[int] = None,
               head_stride: Optional[int] = None) -> Shape:
    """Build an `sg_shape`.  `cu_seqlens` is a device int32 tensor of B+1 prefix sums; the caller passes the
    host-side totals (no device read happens here).  Strides default to a dense [L][T][H_kv][d] cache."""
    _check(cu_seqlens, torch.int32, "cu_seqlens")
    ts = num_kv_heads * head_dim if token_stride is None else token_stride
    hs = head_dim if head_stride is None else head_stride
    ls = total_tokens * ts if layer_stride is None else layer_stride
    s = Shape(num_layers, cu_seqlens.numel() - 1, num_q_heads, num_kv_heads, head_dim, window, total_tokens,
              max_seqlen, cu_seqlens.data_ptr(), ls, ts, hs)
    s._keep = cu_seqlens          # keep the device array alive as long as the struct
    return s


def _check(t: Optional[torch.Tensor], dtype, name: str, allow_none: bool = False):
    if t is None:
        if allow_none:
            return
        raise TypeError("%s is required" % name)
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    dtypes = dtype if isinstance(dtype, (tuple, list)) else (dtype,)
    if t.dtype not in dtypes:
        raise TypeError("%s: expected dtype %s, got %s" % (name, dtypes, t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous (strided caches go through the sg_shape strides)" % name)


_BF16 = (torch.bfloat16, torch.int16, torch.uint16)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None or t.numel() == 0 else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def _ws(workspace: Optional[torch.Tensor]):
    if workspace is None:
        return None, 0
    return workspace.data_ptr(), workspace.numel() * workspace.element_size()


def sg_strerror(status: int) -> str:
    return _lib.sg_strerror(status).decode()


def sg_last_cuda_error() -> int:
    return int(_lib.sg_last_cuda_error())


def sg_workspace_bytes(op: int, shape: Shape, total_sel: int = 0, total_loc: int = 0) -> int:
    return int(_lib.sg_workspace_bytes(op, ctypes.byref(shape), total_sel, total_loc))


def alloc_workspace(op: int, shape: Shape, total_sel: int = 0, total_loc: int = 0, device="cuda") -> Optional[torch.Tensor]:
    """Device scratch of the size the library asks for (None when the operation needs none)."""
    n = sg_workspace_bytes(op, shape, total_sel, total_loc)
    return torch.empty(n, dtype=torch.uint8, device=device) if n else None


def sg_score(shape: Shape, q_win: torch.Tensor, k_cache: torch.Tensor, importance: torch.Tensor,
             workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(q_win, _BF16, "q_win"); _check(k_cache, _BF16, "k_cache"); _check(importance, torch.float32, "importance")
    _check(dev_status, torch.int32, "dev_status", True)
    w, wb = _ws(workspace)
    rc = _lib.sg_score(ctypes.byref(shape), _ptr(q_win), k_cache.data_ptr(), _ptr(importance), w, wb,
                       _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_score")


def sg_score_static(shape: Shape, q_win: torch.Tensor, k_cache: torch.Tensor, importance: torch.Tensor,
                    dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """`sg_score` for callers that cannot allocate device memory: the scratch between the two scoring
    passes is a fixed array inside the library (SG_SCORE_STATIC_SCRATCH_BYTES), shared by all calls on a
    device, so calls must not overlap on the GPU.  Shapes that need more scratch raise SG_ERR_WORKSPACE."""
    _check(q_win, _BF16, "q_win"); _check(k_cache, _BF16, "k_cache"); _check(importance, torch.float32, "importance")
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_score_static(ctypes.byref(shape), _ptr(q_win), k_cache.data_ptr(), _ptr(importance),
                              _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_score_static")


def sg_select_topk(shape: Shape, importance: torch.Tensor, cu_k: torch.Tensor, total_sel: int,
                   sel_idx: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                   dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(importance, torch.float32, "importance"); _check(cu_k, torch.int32, "cu_k")
    _check(sel_idx, torch.int32, "sel_idx"); _check(dev_status, torch.int32, "dev_status", True)
    w, wb = _ws(workspace)
    rc = _lib.sg_select_topk(ctypes.byref(shape), _ptr(importance), cu_k.data_ptr(), total_sel, _ptr(sel_idx), w, wb,
                             _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_select_topk")


def sg_pack_kv(shape: Shape, k_cache: torch.Tensor, v_cache: torch.Tensor, sel_idx: torch.Tensor,
               cu_k: torch.Tensor, total_sel: int, packed_k: torch.Tensor, packed_v: torch.Tensor,
               dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(k_cache, _BF16, "k_cache"); _check(v_cache, _BF16, "v_cache"); _check(sel_idx, torch.int32, "sel_idx")
    _check(cu_k, torch.int32, "cu_k"); _check(packed_k, _BF16, "packed_k"); _check(packed_v, _BF16, "packed_v")
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_pack_kv(ctypes.byref(shape), k_cache.data_ptr(), v_cache.data_ptr(), _ptr(sel_idx), cu_k.data_ptr(),
                         total_sel, _ptr(packed_k), _ptr(packed_v), _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_pack_kv")


def sg_sparse_decode_attn(shape: Shape, q: torch.Tensor, packed_k: Optional[torch.Tensor],
                          packed_v: Optional[torch.Tensor], cu_k: torch.Tensor, total_sel: int,
                          local_k: Optional[torch.Tensor], local_v: Optional[torch.Tensor],
                          local_idx: Optional[torch.Tensor], cu_nloc: torch.Tensor, total_loc: int,
                          out: torch.Tensor, lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                          workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                          stream=None) -> None:
    _check(q, _BF16, "q"); _check(out, _BF16, "out"); _check(cu_k, torch.int32, "cu_k")
    _check(cu_nloc, torch.int32, "cu_nloc"); _check(packed_k, _BF16, "packed_k", True)
    _check(packed_v, _BF16, "packed_v", True); _check(local_k, _BF16, "local_k", True)
    _check(local_v, _BF16, "local_v", True); _check(local_idx, torch.int32, "local_idx", True)
    _check(lse, torch.float32, "lse", True); _check(dev_status, torch.int32, "dev_status", True)
    w, wb = _ws(workspace)
    rc = _lib.sg_sparse_decode_attn(ctypes.byref(shape), q.data_ptr(), _ptr(packed_k), _ptr(packed_v), cu_k.data_ptr(),
                                    total_sel, _ptr(local_k), _ptr(local_v), _ptr(local_idx), cu_nloc.data_ptr(),
                                    total_loc, softmax_scale, out.data_ptr(), _ptr(lse), w, wb, _ptr(dev_status),
                                    _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_sparse_decode_attn")


def sg_split_index(shape: Shape, kv_index: torch.Tensor, cu_k: torch.Tensor, total_sel: int, kv_mask: torch.Tensor,
                   reorder: bool, reordered: Optional[torch.Tensor], local_index: torch.Tensor,
                   remote_index: torch.Tensor, n_local: torch.Tensor, n_remote: torch.Tensor,
                   dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Algorithm 1: split each KV index row into local (mask 1) and remote (mask 2) lists, optionally reordering
    the row so that remote entries come first."""
    _check(kv_index, torch.int32, "kv_index"); _check(cu_k, torch.int32, "cu_k"); _check(kv_mask, torch.int8, "kv_mask")
    _check(reordered, torch.int32, "reordered", True); _check(local_index, torch.int32, "local_index")
    _check(remote_index, torch.int32, "remote_index"); _check(n_local, torch.int32, "n_local")
    _check(n_remote, torch.int32, "n_remote"); _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_split_index(ctypes.byref(shape), _ptr(kv_index), cu_k.data_ptr(), total_sel, _ptr(kv_mask),
                             1 if reorder else 0, _ptr(reordered), _ptr(local_index), _ptr(remote_index),
                             n_local.data_ptr(), n_remote.data_ptr(), _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_split_index")


def sg_profile_accumulate(shape: Shape, kv_index: torch.Tensor, cu_k: torch.Tensor, total_sel: int, counts: torch.Tensor,
                          dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """S(e) += 1 for every entry of one layer's KV index (counts int32 [H_kv][T], caller-zeroed)."""
    _check(kv_index, torch.int32, "kv_index"); _check(cu_k, torch.int32, "cu_k"); _check(counts, torch.int32, "counts")
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_profile_accumulate(ctypes.byref(shape), _ptr(kv_index), cu_k.data_ptr(), total_sel, _ptr(counts),
                                    _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_profile_accumulate")


def sg_block_importance(shape: Shape, counts: torch.Tensor, num_blocks: int, importance: torch.Tensor, stream=None) -> None:
    """Eq. 1: importance fp32 [L][M] from counts int32 [L][H_kv][T]."""
    _check(counts, torch.int32, "counts"); _check(importance, torch.float32, "importance")
    rc = _lib.sg_block_importance(ctypes.byref(shape), _ptr(counts), num_blocks, _ptr(importance), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_block_importance")


def sg_transfer_budget(num_layers: int, num_blocks: int, t_prefill: float, t_transfer: float) -> int:
    """Eq. 2: K_r = M (L-1) T_p / T_t, rounded down and clipped to [2M, LM] (host arithmetic)."""
    return int(_lib.sg_transfer_budget(num_layers, num_blocks, t_prefill, t_transfer))


def sg_proactive_mask(shape: Shape, num_blocks: int, layer: int, selected: Optional[torch.Tensor], kv_mask: torch.Tensor,
                      stream=None) -> None:
    """KV mask (int8 [T]) of one layer after the proactive transfer: 1 inside the selected blocks, 2 elsewhere."""
    _check(selected, torch.int32, "selected", True); _check(kv_mask, torch.int8, "kv_mask")
    n = 0 if selected is None else selected.numel()
    rc = _lib.sg_proactive_mask(ctypes.byref(shape), num_blocks, layer, _ptr(selected), n, _ptr(kv_mask), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_proactive_mask")


def sg_select_threshold(shape: Shape, scores: torch.Tensor, alpha: float, cu_cap: torch.Tensor, total_cap: int,
                        sel_idx: torch.Tensor, sel_count: torch.Tensor, dev_status: Optional[torch.Tensor] = None,
                        stream=None) -> None:
    """Threshold selection under a cap: per row the positions with score > row max - alpha (at most cap_b, the
    largest first, ties to the lower index), ascending then -1, plus the count per (layer, sequence, KV head)."""
    _check(scores, torch.float32, "scores"); _check(cu_cap, torch.int32, "cu_cap")
    _check(sel_idx, torch.int32, "sel_idx", total_cap == 0); _check(sel_count, torch.int32, "sel_count")
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_select_threshold(ctypes.byref(shape), _ptr(scores), alpha, _ptr(cu_cap), total_cap, _ptr(sel_idx),
                                  _ptr(sel_count), _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_select_threshold")


def sg_select_pack_kv(shape: Shape, importance: torch.Tensor, cu_k: torch.Tensor, total_sel: int, k_cache: torch.Tensor,
                      v_cache: torch.Tensor, sel_idx: torch.Tensor, packed_k: torch.Tensor, packed_v: torch.Tensor,
                      dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """sg_select_topk then sg_pack_kv in one call (one fused kernel where that pays); same outputs as the two calls."""
    _check(importance, torch.float32, "importance"); _check(cu_k, torch.int32, "cu_k")
    _check(k_cache, _BF16, "k_cache"); _check(v_cache, _BF16, "v_cache"); _check(sel_idx, torch.int32, "sel_idx", total_sel == 0)
    _check(packed_k, _BF16, "packed_k", total_sel == 0); _check(packed_v, _BF16, "packed_v", total_sel == 0)
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_select_pack_kv(ctypes.byref(shape), _ptr(importance), _ptr(cu_k), total_sel, _ptr(k_cache), _ptr(v_cache),
                                _ptr(sel_idx), _ptr(packed_k), _ptr(packed_v), _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_select_pack_kv")


def sg_pack_kv_counted(shape: Shape, k_cache: torch.Tensor, v_cache: torch.Tensor, sel_idx: torch.Tensor,
                       cu_cap: torch.Tensor, total_cap: int, sel_count: torch.Tensor, packed_k: torch.Tensor,
                       packed_v: torch.Tensor, dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """sg_pack_kv for per-head counts: only the first sel_count[l][b][g] entries of each row of sel_idx are packed."""
    _check(k_cache, _BF16, "k_cache"); _check(v_cache, _BF16, "v_cache"); _check(sel_idx, torch.int32, "sel_idx", total_cap == 0)
    _check(cu_cap, torch.int32, "cu_cap"); _check(sel_count, torch.int32, "sel_count")
    _check(packed_k, _BF16, "packed_k", total_cap == 0); _check(packed_v, _BF16, "packed_v", total_cap == 0)
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_pack_kv_counted(ctypes.byref(shape), _ptr(k_cache), _ptr(v_cache), _ptr(sel_idx), _ptr(cu_cap), total_cap,
                                 _ptr(sel_count), _ptr(packed_k), _ptr(packed_v), _ptr(dev_status), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_pack_kv_counted")


def sg_sparse_decode_attn_counted(shape: Shape, q: torch.Tensor, packed_k: Optional[torch.Tensor], packed_v: Optional[torch.Tensor],
                                  cu_cap: torch.Tensor, total_cap: int, packed_count: Optional[torch.Tensor],
                                  local_k: Optional[torch.Tensor], local_v: Optional[torch.Tensor],
                                  local_idx: Optional[torch.Tensor], cu_nloc: torch.Tensor, total_loc: int, out: torch.Tensor,
                                  lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                                  dev_status: Optional[torch.Tensor] = None, stream=None,
                                  local_skip: Optional[torch.Tensor] = None) -> None:
    """sg_sparse_decode_attn for per-head counts: of the cap_b packed rows of (b, g) only the first packed_count[b][g]
    are attended, and the first local_skip[b][g] entries of its local-index row are left out."""
    _check(q, _BF16, "q"); _check(out, _BF16, "out"); _check(cu_cap, torch.int32, "cu_cap"); _check(cu_nloc, torch.int32, "cu_nloc")
    _check(packed_count, torch.int32, "packed_count", True); _check(local_skip, torch.int32, "local_skip", True)
    _check(packed_k, _BF16, "packed_k", True); _check(packed_v, _BF16, "packed_v", True)
    _check(local_k, _BF16, "local_k", True); _check(local_v, _BF16, "local_v", True)
    _check(local_idx, torch.int32, "local_idx", True); _check(lse, torch.float32, "lse", True)
    _check(dev_status, torch.int32, "dev_status", True)
    rc = _lib.sg_sparse_decode_attn_counted(ctypes.byref(shape), _ptr(q), _ptr(packed_k), _ptr(packed_v), _ptr(cu_cap), total_cap,
                                            _ptr(packed_count), _ptr(local_k), _ptr(local_v), _ptr(local_idx), _ptr(cu_nloc),
                                            total_loc, _ptr(local_skip), softmax_scale, _ptr(out), _ptr(lse), _ptr(dev_status),
                                            _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_sparse_decode_attn_counted")


def sg_push_blocks(shape: Shape, num_blocks: int, layer: int, selected: Optional[torch.Tensor], src_k: torch.Tensor,
                   src_v: torch.Tensor, dst_k: torch.Tensor, dst_v: torch.Tensor, kv_mask: Optional[torch.Tensor] = None,
                   stream=None) -> None:
    """Online proactive transfer: copy the rows (all KV heads, K and V) of every selected block of the layers
    `layer` .. `layer + shape.num_layers - 1` from the source cache to the same positions of the destination
    cache (the tensors start at `layer`); other rows are untouched.  With `kv_mask` (int8 [layers][T]) the pushed
    tokens are also marked local (1) in the decode-side KV mask."""
    _check(selected, torch.int32, "selected", True)
    for name, t in (("src_k", src_k), ("src_v", src_v), ("dst_k", dst_k), ("dst_v", dst_v)):
        _check(t, _BF16, name)
    _check(kv_mask, torch.int8, "kv_mask", True)
    n = 0 if selected is None else selected.numel()
    rc = _lib.sg_push_blocks(ctypes.byref(shape), num_blocks, layer, _ptr(selected), n, _ptr(src_k), _ptr(src_v),
                             _ptr(dst_k), _ptr(dst_v), _ptr(kv_mask), _stream(stream))
    if rc:
        raise SmartGenError(rc, "sg_push_blocks")


def sg_speculative_delivered(num_layers: int, num_blocks: int, k_r: int, ratio: float, iteration: int) -> int:
    """Blocks on the decode node after `iteration` speculative transfers of at most `ratio` of all blocks each."""
    return int(_lib.sg_speculative_delivered(num_layers, num_blocks, k_r, ratio, iteration))
