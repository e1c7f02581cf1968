"""One small pass of the hot path on cuda:0, checked against the CPU oracle (used by the driver's smoke step)."""
from __future__ import annotations

import numpy as np
import torch


def run(verbose: bool = True) -> None:
    if not torch.cuda.is_available():
        raise RuntimeError("smoke() needs a CUDA device: the hot path has no CPU fallback")
    import oracle                                   # test infrastructure: only used to check the result
    from . import workloads as wl
    from .pipeline import HotPath, as_device

    torch.cuda.set_device(0)
    cfg = wl.tiny()
    data = wl.make_prefill(cfg)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    hp = HotPath(cfg.num_layers, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window, cfg.seqlens, cfg.budgets())
    q_win, k, v = as_device(data["q_win"]), as_device(data["k"]), as_device(data["v"])
    hp.prefill(q_win, k, v)
    torch.cuda.synchronize()
    imp = hp.importance.cpu().numpy()
    sel = hp.sel_idx.cpu().numpy()
    pk = hp.packed_k.cpu().numpy().view(np.uint16)
    pv = hp.packed_v.cpu().numpy().view(np.uint16)

    imp_o = oracle.score(data["q_win"], data["k"], cu)
    assert np.all(np.abs(imp - imp_o) <= 1e-4 * np.abs(imp_o) + 1e-30), "score mismatch"
    assert np.array_equal(sel, oracle.select_topk(imp, cu, ck)), "top-k mismatch (given identical scores)"
    pk_o, pv_o = oracle.pack_kv(data["k"], data["v"], cu, sel, ck)
    assert np.array_equal(pk, pk_o) and np.array_equal(pv, pv_o), "pack mismatch"

    qd = wl.make_decode_queries(cfg, 0, 0, data["q_win"][0])
    _, _, loc, cl = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local(), exclude=sel[0], cu_excl=ck)
    out = torch.empty((cfg.batch, cfg.num_q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((cfg.batch, cfg.num_q_heads), dtype=torch.float32, device="cuda")
    hp.decode(0, as_device(qd), k[0], v[0], as_device(loc), as_device(cl), int(cl[-1]), out, lse)
    torch.cuda.synchronize()
    out_o, lse_o = oracle.sparse_decode_attn(qd, pk[0], pv[0], ck, data["k"][0], data["v"][0], cu, loc, cl)
    assert np.abs(out.float().cpu().numpy() - out_o).max() <= 2e-2, "decode attention mismatch"
    assert np.abs(lse.cpu().numpy() - lse_o).max() <= 1e-3, "lse mismatch"
    assert hp.read_status() == 0, "device status word set"
    if verbose:
        print("smoke ok: score/select/pack/decode match the oracle on the tiny config")
