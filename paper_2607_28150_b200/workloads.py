"""Seeded synthetic workloads: GQA-shaped KV caches, window queries, index splits.

This module only *shapes inputs*.  It holds none of the method's arithmetic (no
scoring, no selection, no attention) and imports neither the CUDA binding nor
any CPU checker, so the same arrays can be fed to both sides of a parity test.

Everything is numpy with a counter-based generator (``Philox``), keyed by
``(config id, layer, tensor id)``, so any layer of any configuration can be
regenerated independently and identically on any machine.

The caches stand in for real model caches on long-document prompts: i.i.d.
N(0,1) keys/values in bf16 plus the structure that makes selective KV transfer
meaningful -- a few "sink" tokens at the start of each prompt and a sparse set
of heavy-hitter keys (norm x4, aligned with the mean window query of their KV
head), either scattered (1 % of tokens) or clustered in contiguous spans.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence

import numpy as np
from numpy.random import Generator, Philox

# tensor ids used in seeds
_TID_Q, _TID_K, _TID_V, _TID_HH, _TID_QDEC, _TID_IDX, _TID_LEN = 1, 2, 3, 4, 5, 6, 7


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(config_id: int, layer: int, tensor_id: int) -> Generator:
    return Generator(Philox(key=1000 * config_id + 10 * layer + tensor_id))


@dataclasses.dataclass(frozen=True)
class Config:
    """One workload configuration (shapes follow the benchmark's config list)."""
    name: str
    config_id: int
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    window: int
    seqlens: tuple                 # prompt length of every sequence in the batch
    budget: object                 # int (tokens per KV head) or float (fraction of the prompt)
    heavy: str = "scatter"         # "scatter": 1 % of tokens; "count16": 16 tokens; "spans": 4 spans of 256
    local_ratio: float = 0.34      # on-demand share of the required entries in a decode step
    n_local_fixed: Optional[int] = None
    decode_steps: int = 1

    @property
    def batch(self) -> int:
        return len(self.seqlens)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seqlens)]).astype(np.int32)

    def budgets(self, fraction: Optional[float] = None) -> np.ndarray:
        """Selected tokens per KV head for every sequence: k_b = min(N_b, max(1, ceil(f N_b)))."""
        b = self.budget if fraction is None else fraction
        out = []
        for n in self.seqlens:
            k = int(b) if isinstance(b, (int, np.integer)) else int(math.ceil(float(b) * n - 1e-9))
            out.append(min(n, max(1, k)))
        return np.asarray(out, dtype=np.int32)

    def cu_k(self, fraction: Optional[float] = None) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.budgets(fraction))]).astype(np.int32)

    def n_local(self, fraction: Optional[float] = None) -> np.ndarray:
        """Index-addressed entries per KV head in a decode step, per sequence."""
        k = self.budgets(fraction)
        if self.n_local_fixed is not None:
            n = np.full_like(k, self.n_local_fixed)
        else:
            rho = self.local_ratio
            n = np.rint(k * rho / (1.0 - rho)).astype(np.int32)
        return np.minimum(n, np.asarray(self.seqlens, dtype=np.int32) - k).astype(np.int32)


def variable_lengths(config_id: int = 3, batch: int = 8, lo: int = 2048, hi: int = 32768) -> tuple:
    return tuple(int(x) for x in _rng(config_id, 0, _TID_LEN).integers(lo, hi, endpoint=True, size=batch))


def tiny() -> Config:
    return Config("c1_tiny", 1, 1, 8, 2, 64, 16, (1024,), 128, heavy="count16", n_local_fixed=32)


def llama8b(num_layers: int = 32, seqlen: int = 8192) -> Config:
    return Config("c2_llama3_8b", 2, num_layers, 32, 8, 128, 32, (seqlen,), 0.10, decode_steps=64)


def varlen(fraction: float = 0.10, num_layers: int = 1, seqlens: Optional[Sequence[int]] = None) -> Config:
    lens = tuple(seqlens) if seqlens is not None else variable_lengths()
    return Config("c3_varlen", 3, num_layers, 32, 8, 128, 32, lens, float(fraction))


def llama70b(num_layers: int = 8, seqlen: int = 32768, budget: int = 2048) -> Config:
    return Config("c4_llama3_70b", 4, num_layers, 64, 8, 128, 64, (seqlen,), budget, heavy="spans")


def decode_sweep(batch: int, sel: float, rho: float, seqlen: int = 4096) -> Config:
    """Decode-only point: `sel` = required fraction of the prompt, `rho` = index-addressed share of it."""
    n_req = min(seqlen, max(1, int(math.ceil(sel * seqlen - 1e-9))))
    n_loc = int(round(rho * n_req))
    return Config("c5_decode", 5, 1, 32, 8, 128, 32, (seqlen,) * batch, n_req - n_loc,
                  local_ratio=rho, n_local_fixed=n_loc)


def _unit(x: np.ndarray) -> np.ndarray:
    return x / np.maximum(np.linalg.norm(x, axis=-1, keepdims=True), 1e-30)


def heavy_positions(cfg: Config, layer: int, b: int) -> np.ndarray:
    """Token positions (sequence-local, sinks 0-3 included) of the heavy-hitter keys of sequence b."""
    n = cfg.seqlens[b]
    rng = Generator(Philox(key=1000 * cfg.config_id + 10 * layer + _TID_HH + 100000 * (b + 1)))
    lo, hi = 4, max(5, n - cfg.window)
    if cfg.heavy == "count16":
        pos = rng.choice(np.arange(lo, hi), size=min(16, hi - lo), replace=False)
    elif cfg.heavy == "spans":
        span, nspan = 256, 4
        slots = (hi - lo) // span
        if slots >= nspan:
            starts = lo + span * rng.choice(slots, size=nspan, replace=False)
            pos = (starts[:, None] + np.arange(span)[None, :]).ravel()
        else:
            pos = np.arange(lo, hi)
    else:
        cnt = max(1, (n + 50) // 100) if hi - lo > 1 else 0
        pos = rng.choice(np.arange(lo, hi), size=min(cnt, hi - lo), replace=False)
    sinks = np.arange(0, min(4, n))
    return np.unique(np.concatenate([sinks, pos])).astype(np.int64)


def make_layer(cfg: Config, layer: int, identical_heavy: bool = False) -> Dict[str, np.ndarray]:
    """One layer of prefill-side inputs as bf16 bit patterns (uint16).

    q_win [B][W][H_q][d]  -- the last W prompt queries of every sequence (row i is position N-W_eff+i)
    k, v  [T][H_kv][d]    -- ragged, token-major caches, sequences packed back to back
    """
    B, W, Hq, Hkv, d, G = cfg.batch, cfg.window, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.group
    T = cfg.total_tokens
    cu = cfg.cu_seqlens()
    q = _rng(cfg.config_id, layer, _TID_Q).standard_normal((B, W, Hq, d), dtype=np.float32)
    k = _rng(cfg.config_id, layer, _TID_K).standard_normal((T, Hkv, d), dtype=np.float32)
    v = _rng(cfg.config_id, layer, _TID_V).standard_normal((T, Hkv, d), dtype=np.float32)
    for b in range(B):
        u = _unit(q[b].reshape(W, Hkv, G, d).mean(axis=(0, 2)))          # [H_kv][d] mean window query direction
        pos = heavy_positions(cfg, layer, b)
        if pos.size == 0:
            continue
        eps = _unit(k[cu[b] + pos])                                       # [n][H_kv][d]
        if identical_heavy:
            eps = np.zeros_like(eps)
            mix = np.broadcast_to(u[None], eps.shape)
        else:
            mix = 0.9 * u[None] + 0.436 * eps
        k[cu[b] + pos] = (4.0 * math.sqrt(d)) * _unit(mix)
    return {"q_win": f32_to_bf16_bits(q), "k": f32_to_bf16_bits(k), "v": f32_to_bf16_bits(v)}


def make_prefill(cfg: Config, layers: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
    """Stack `make_layer` over layers: q_win [L][B][W][H_q][d], k/v [L][T][H_kv][d] (uint16 bf16 bits)."""
    layers = list(range(cfg.num_layers)) if layers is None else list(layers)
    per = [make_layer(cfg, l) for l in layers]
    out = {name: np.stack([p[name] for p in per]) for name in ("q_win", "k", "v")}
    out["cu_seqlens"] = cfg.cu_seqlens()
    return out


def make_decode_queries(cfg: Config, layer: int, step: int, q_win_layer: Optional[np.ndarray] = None) -> np.ndarray:
    """Decode-step queries [B][H_q][d] (bf16 bits): N(0,1) plus the mean window query of the same head."""
    B, Hq, d = cfg.batch, cfg.num_q_heads, cfg.head_dim
    rng = Generator(Philox(key=1000 * cfg.config_id + 10 * layer + _TID_QDEC + 100000 * (step + 1)))
    q = rng.standard_normal((B, Hq, d), dtype=np.float32)
    if q_win_layer is not None:
        q = q + bf16_bits_to_f32(q_win_layer).mean(axis=1)
    return f32_to_bf16_bits(q)


def make_index_split(cfg: Config, layer: int, step: int, n_sel: Sequence[int], n_loc: Sequence[int],
                     exclude: Optional[np.ndarray] = None, cu_excl: Optional[np.ndarray] = None):
    """Seeded uniform index sets per (sequence, KV head).

    Returns (sel_idx [H_kv][sum n_sel] ascending per row segment, cu_k,
             local_idx [H_kv][sum n_loc] in drawn (unsorted) order, cu_nloc).
    `sel` and `local` of one (sequence, head) are disjoint.  If `exclude` ([H_kv][K_tot] with prefix
    sums `cu_excl`) is given, no selected set is drawn (n_sel is ignored) and the local indices are
    drawn from the complement of `exclude`.
    """
    Hkv = cfg.num_kv_heads
    n_sel = np.asarray(n_sel, dtype=np.int64)
    n_loc = np.asarray(n_loc, dtype=np.int64)
    cu_k = np.concatenate([[0], np.cumsum(n_sel)]).astype(np.int32)
    cu_l = np.concatenate([[0], np.cumsum(n_loc)]).astype(np.int32)
    sel = np.zeros((Hkv, int(cu_k[-1])), dtype=np.int32)
    loc = np.zeros((Hkv, int(cu_l[-1])), dtype=np.int32)
    for b, n in enumerate(cfg.seqlens):
        for g in range(Hkv):
            rng = Generator(Philox(key=1000 * cfg.config_id + 10 * layer + _TID_IDX
                                   + 100000 * (step + 1) + 10000000 * (b * Hkv + g + 1)))
            if exclude is not None:
                taken = exclude[g, cu_excl[b]:cu_excl[b + 1]]
                rest = np.setdiff1d(np.arange(n, dtype=np.int32), taken, assume_unique=False)
                loc[g, cu_l[b]:cu_l[b + 1]] = rng.permutation(rest)[: n_loc[b]]
            else:
                perm = rng.permutation(n).astype(np.int32)
                sel[g, cu_k[b]:cu_k[b + 1]] = np.sort(perm[: n_sel[b]])
                loc[g, cu_l[b]:cu_l[b + 1]] = perm[n_sel[b]: n_sel[b] + n_loc[b]]
    return sel, cu_k, loc, cu_l
