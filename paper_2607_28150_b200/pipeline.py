"""Buffer management around the four C-ABI calls (allocation and argument marshalling only).

`HotPath` owns the device buffers of one batch of prompts -- importance, KV index, packed K/V,
workspaces, status word -- and issues the library calls in the order of the path:

    prefill side:  sg_score -> sg_select_topk -> sg_pack_kv      (all layers in one call each, or layer by
                                                                   layer with select+pack on a second stream)
    decode side :  sg_sparse_decode_attn                          (one call per layer per step)

No arithmetic of the method happens here; every step runs in the library's CUDA kernels.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as sg


def as_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    """Upload a numpy array; uint16 (bf16 bit patterns) becomes an int16 tensor with the same bits."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).to(device)


class HotPath:
    def __init__(self, num_layers: int, num_q_heads: int, num_kv_heads: int, head_dim: int, window: int,
                 seqlens: Sequence[int], budgets: Sequence[int], device="cuda"):
        self.L, self.Hq, self.Hkv, self.d, self.W = num_layers, num_q_heads, num_kv_heads, head_dim, window
        self.device = torch.device(device)
        lens = np.asarray(seqlens, dtype=np.int64)
        ks = np.asarray(budgets, dtype=np.int64)
        self.B = len(lens)
        self.T = int(lens.sum())
        self.max_seqlen = int(lens.max())
        self.K_tot = int(ks.sum())
        self.cu_host = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        self.cu_k_host = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
        self.cu = as_device(self.cu_host, device)
        self.cu_k = as_device(self.cu_k_host, device)
        self.shape = sg.make_shape(self.L, self.Hq, self.Hkv, self.d, self.W, self.cu, self.T, self.max_seqlen)
        self.shape1 = sg.make_shape(1, self.Hq, self.Hkv, self.d, self.W, self.cu, self.T, self.max_seqlen)
        self.importance = torch.empty((self.L, self.Hkv, self.T), dtype=torch.float32, device=device)
        self.sel_idx = torch.empty((self.L, self.Hkv, self.K_tot), dtype=torch.int32, device=device)
        self.packed_k = torch.empty((self.L, self.K_tot * self.Hkv, self.d), dtype=torch.int16, device=device)
        self.packed_v = torch.empty_like(self.packed_k)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        self.ws_score = sg.alloc_workspace(sg.SG_OP_SCORE, self.shape, device=device)
        self._ws_decode = None
        self._ws_decode_for = -1

    # ---- prefill side -------------------------------------------------------------------------
    def score(self, q_win: torch.Tensor, k_cache: torch.Tensor, stream=None) -> torch.Tensor:
        sg.sg_score(self.shape, q_win, k_cache, self.importance, self.ws_score, self.status, stream)
        return self.importance

    def select(self, stream=None) -> torch.Tensor:
        sg.sg_select_topk(self.shape, self.importance, self.cu_k, self.K_tot, self.sel_idx, None, self.status, stream)
        return self.sel_idx

    def pack(self, k_cache: torch.Tensor, v_cache: torch.Tensor, stream=None):
        sg.sg_pack_kv(self.shape, k_cache, v_cache, self.sel_idx, self.cu_k, self.K_tot, self.packed_k, self.packed_v,
                      self.status, stream)
        return self.packed_k, self.packed_v

    def select_pack(self, k_cache: torch.Tensor, v_cache: torch.Tensor, stream=None):
        """select() then pack() as one library call (one fused kernel where the library finds that it pays)."""
        sg.sg_select_pack_kv(self.shape, self.importance, self.cu_k, self.K_tot, k_cache, v_cache, self.sel_idx,
                             self.packed_k, self.packed_v, self.status, stream)
        return self.packed_k, self.packed_v

    def prefill(self, q_win, k_cache, v_cache, stream=None):
        self.score(q_win, k_cache, stream)
        return self.select_pack(k_cache, v_cache, stream)

    def prefill_layer(self, layer: int, q_win: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                      stream=None, aux_stream=None):
        """score -> select -> pack of ONE layer, as a prefill engine calls them when that layer's KV is ready
        (the paper transfers layer by layer, overlapped with the prefill of the following layers).
        `q_win`, `k_cache`, `v_cache` are the full [L][...] tensors.  With `aux_stream`, select and pack run
        there behind an event, so the next layer's scoring on `stream` does not wait for them; the caller joins
        with `join_aux` before reading the results on `stream`."""
        main = stream if stream is not None else torch.cuda.current_stream(self.device)
        sg.sg_score(self.shape1, q_win[layer], k_cache[layer], self.importance[layer], self.ws_score, self.status, main)
        side = main
        if aux_stream is not None:
            ev = torch.cuda.Event()
            ev.record(main)
            aux_stream.wait_event(ev)
            side = aux_stream
        sg.sg_select_topk(self.shape1, self.importance[layer], self.cu_k, self.K_tot, self.sel_idx[layer], None,
                          self.status, side)
        sg.sg_pack_kv(self.shape1, k_cache[layer], v_cache[layer], self.sel_idx[layer], self.cu_k, self.K_tot,
                      self.packed_k[layer], self.packed_v[layer], self.status, side)

    def join_aux(self, aux_stream, stream=None) -> None:
        """Make `stream` wait for everything queued on `aux_stream` so far."""
        main = stream if stream is not None else torch.cuda.current_stream(self.device)
        ev = torch.cuda.Event()
        ev.record(aux_stream)
        main.wait_event(ev)

    def prefill_layerwise(self, q_win, k_cache, v_cache, stream=None, aux_stream=None):
        for layer in range(self.L):
            self.prefill_layer(layer, q_win, k_cache, v_cache, stream, aux_stream)
        if aux_stream is not None:
            self.join_aux(aux_stream, stream)
        return self.packed_k, self.packed_v

    # ---- decode side --------------------------------------------------------------------------
    def decode_workspace(self, total_loc: int) -> torch.Tensor:
        if self._ws_decode is None or self._ws_decode_for < total_loc:
            self._ws_decode = sg.alloc_workspace(sg.SG_OP_SPARSE_DECODE_ATTN, self.shape1, self.K_tot, total_loc,
                                                 device=self.device)
            self._ws_decode_for = total_loc
        return self._ws_decode

    def decode(self, layer: int, q: torch.Tensor, local_k: torch.Tensor, local_v: torch.Tensor,
               local_idx: Optional[torch.Tensor], cu_nloc: torch.Tensor, total_loc: int, out: torch.Tensor,
               lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0, stream=None) -> torch.Tensor:
        """One layer of one decode step: packed rows of `layer` plus `local_idx`-addressed rows of local_k/v."""
        ws = self.decode_workspace(total_loc)
        sg.sg_sparse_decode_attn(self.shape1, q, self.packed_k[layer], self.packed_v[layer], self.cu_k, self.K_tot,
                                 local_k, local_v, local_idx, cu_nloc, total_loc, out, lse, softmax_scale, ws,
                                 self.status, stream)
        return out

    def read_status(self) -> int:
        """Device status word (bit i set = sg_status i was raised by a kernel); synchronises."""
        return int(self.status[0].item())
