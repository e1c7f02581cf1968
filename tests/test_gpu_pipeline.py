"""GPU parity of the chained path: score -> select -> pack -> two-source decode, each stage through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2607_28150_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def chain(cfg):
    import gpu_ops
    data = wl.make_prefill(cfg)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    imp_o = oracle.score(data["q_win"], data["k"], cu)
    sel_o = oracle.select_topk(imp_o, cu, ck)
    imp_g = gpu_ops.score(data["q_win"], data["k"], cu)
    sel_g = gpu_ops.select_topk(imp_g, cu, ck)
    return data, cu, ck, imp_o, sel_o, imp_g, sel_g


@pytest.mark.parametrize("cfg", [wl.tiny(), wl.llama8b(num_layers=2, seqlen=4096),
                                 wl.varlen(0.1, seqlens=(700, 2048, 130))], ids=lambda c: c.name)
def test_selection_differs_only_at_near_ties(cfg):
    """Each side selecting from its own scores: index sets may differ only where the oracle's importance is
    within 2e-4 relative of its k-th value."""
    data, cu, ck, imp_o, sel_o, imp_g, sel_g = chain(cfg)
    L, Hkv = imp_o.shape[:2]
    total, same = 0, 0
    for l in range(L):
        for g in range(Hkv):
            for b in range(cfg.batch):
                so = set(sel_o[l, g, ck[b]:ck[b + 1]].tolist())
                sg_ = set(sel_g[l, g, ck[b]:ck[b + 1]].tolist())
                seg = imp_o[l, g, cu[b]:cu[b + 1]].astype(np.float64)
                kth = np.sort(seg)[::-1][len(so) - 1]
                for t in so ^ sg_:
                    assert abs(seg[t] - kth) <= 2e-4 * abs(kth) + 1e-30
                total += len(so | sg_)
                same += len(so & sg_)
    assert same / total > 0.99          # Jaccard index over all heads


def test_identical_scores_give_identical_sets_and_packed_bytes():
    import gpu_ops
    cfg = wl.llama8b(num_layers=2, seqlen=4096)
    data, cu, ck, imp_o, sel_o, _, _ = chain(cfg)
    sel_g = gpu_ops.select_topk(imp_o, cu, ck)                 # the GPU selects from the oracle's fp32 scores
    assert np.array_equal(sel_g, sel_o)
    pk_g, pv_g = gpu_ops.pack_kv(data["k"], data["v"], cu, sel_g, ck)
    pk_o, pv_o = oracle.pack_kv(data["k"], data["v"], cu, sel_o, ck)
    assert np.array_equal(pk_g, pk_o) and np.array_equal(pv_g, pv_o)


def test_tiny_config_end_to_end_decode():
    """Tiny config: 128 selected tokens per KV head plus 32 local indices, one decode step."""
    import gpu_ops
    cfg = wl.tiny()
    data, cu, ck, imp_o, sel_o, imp_g, sel_g = chain(cfg)
    pk, pv = gpu_ops.pack_kv(data["k"], data["v"], cu, sel_g, ck)
    q = wl.make_decode_queries(cfg, 0, 0, data["q_win"][0])
    _, _, loc, cl = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local(), exclude=sel_g[0], cu_excl=ck)
    got_o, got_l = gpu_ops.sparse_decode_attn(q, pk[0], pv[0], ck, data["k"][0], data["v"][0], cu, loc, cl)
    want_o, want_l = oracle.sparse_decode_attn(q, pk[0], pv[0], ck, data["k"][0], data["v"][0], cu, loc, cl)
    assert np.abs(got_o - want_o).max() <= 2e-2 and np.abs(got_l - want_l).max() <= 1e-3


@pytest.mark.parametrize("two_streams", [False, True])
def test_layer_by_layer_prefill_matches_the_oracle_chain(two_streams):
    """score -> select -> pack issued layer by layer (optionally with select+pack on a second stream): scores within
    tolerance of the oracle, and index sets / packed bytes bit-exact against the oracle run on those same scores."""
    import torch
    from paper_2607_28150_b200.pipeline import HotPath, as_device
    cfg = wl.varlen(0.1, seqlens=(1500, 4096, 130), num_layers=5)
    data = wl.make_prefill(cfg)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    hp = HotPath(cfg.num_layers, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window, cfg.seqlens, cfg.budgets())
    q, k, v = as_device(data["q_win"]), as_device(data["k"]), as_device(data["v"])
    aux = torch.cuda.Stream() if two_streams else None
    hp.prefill_layerwise(q, k, v, aux_stream=aux)
    torch.cuda.synchronize()
    assert hp.read_status() == 0
    imp_g = hp.importance.cpu().numpy()
    imp_o = oracle.score(data["q_win"], data["k"], cu)
    assert np.all(np.abs(imp_g - imp_o) <= 1e-4 * np.abs(imp_o) + 1e-30)
    sel_o = oracle.select_topk(imp_g, cu, ck)
    assert np.array_equal(hp.sel_idx.cpu().numpy(), sel_o)
    pk_o, pv_o = oracle.pack_kv(data["k"], data["v"], cu, sel_o, ck)
    assert np.array_equal(hp.packed_k.cpu().numpy().view(np.uint16), pk_o)
    assert np.array_equal(hp.packed_v.cpu().numpy().view(np.uint16), pv_o)
