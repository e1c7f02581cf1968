"""GPU parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(all layers per prefill call, one decode call per layer).  Outputs the oracle can afford are compared
element by element on sampled layers / heads; the rest is checked through properties that hold at any size."""
import numpy as np
import pytest

import oracle
from paper_2607_28150_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def close(got, want, rtol=1e-4, atol=1e-30):
    return bool(np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= rtol * np.abs(want.astype(np.float64)) + atol))


def run_prefill(cfg):
    import torch
    from paper_2607_28150_b200.pipeline import HotPath, as_device
    data = wl.make_prefill(cfg)
    hp = HotPath(cfg.num_layers, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window, cfg.seqlens, cfg.budgets())
    q, k, v = as_device(data["q_win"]), as_device(data["k"]), as_device(data["v"])
    hp.prefill(q, k, v)
    torch.cuda.synchronize()
    assert hp.read_status() == 0
    out = dict(imp=hp.importance.cpu().numpy(), sel=hp.sel_idx.cpu().numpy(),
               pk=hp.packed_k.cpu().numpy().view(np.uint16), pv=hp.packed_v.cpu().numpy().view(np.uint16))
    return data, hp, (q, k, v), out


def check_select_and_pack(cfg, data, out, layers):
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    Hkv = cfg.num_kv_heads
    # top-k from the GPU's own fp32 scores: bit-exact against the oracle on the sampled layers
    sel_o = oracle.select_topk(out["imp"][layers], cu, ck)
    assert np.array_equal(out["sel"][layers], sel_o)
    # every layer: budget count, ascending, in range
    for b in range(cfg.batch):
        seg = out["sel"][:, :, ck[b]:ck[b + 1]]
        assert seg.min() >= 0 and seg.max() < cfg.seqlens[b] and np.all(np.diff(seg, axis=-1) > 0)
    # pack: every row of every layer equals the cache row its index names
    for l in range(cfg.num_layers):
        for b in range(cfg.batch):
            kb = ck[b + 1] - ck[b]
            for g in range(Hkv):
                rows = ck[b] * Hkv + g * kb + np.arange(kb)
                toks = cu[b] + out["sel"][l, g, ck[b]:ck[b + 1]]
                assert np.array_equal(out["pk"][l, rows], data["k"][l, toks, g])
                assert np.array_equal(out["pv"][l, rows], data["v"][l, toks, g])


def test_llama8b_config_all_layers():
    """32 layers, 8192-token prompt, W = 32, 10 % budget; then decode calls with 422 local indices."""
    import torch
    from paper_2607_28150_b200.pipeline import as_device
    cfg = wl.llama8b()
    data, hp, (q, k, v), out = run_prefill(cfg)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    # scores: row-mass invariant on every (layer, head); full comparison on sampled layers
    np.testing.assert_allclose(out["imp"].astype(np.float64).sum(-1), cfg.group * cfg.window, rtol=1e-4)
    layers = [0, 13, 31]
    imp_o = oracle.score(data["q_win"][layers], data["k"][layers], cu)
    assert close(out["imp"][layers], imp_o)
    check_select_and_pack(cfg, data, out, layers)
    # heavy hitters and sinks are found in every layer and head
    pos = set(wl.heavy_positions(cfg, 5, 0).tolist())
    assert all(pos <= set(out["sel"][5, g].tolist()) for g in range(cfg.num_kv_heads))
    # decode: sampled (layer, step) calls against the oracle
    nloc = cfg.n_local()
    for l, step in [(0, 0), (31, 63)]:
        qd = wl.make_decode_queries(cfg, l, step, data["q_win"][l])
        _, _, loc, cl = wl.make_index_split(cfg, l, step, cfg.budgets(), nloc, exclude=out["sel"][l], cu_excl=ck)
        o = torch.empty((cfg.batch, cfg.num_q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((cfg.batch, cfg.num_q_heads), dtype=torch.float32, device="cuda")
        hp.decode(l, as_device(qd), k[l], v[l], as_device(loc), as_device(cl), int(cl[-1]), o, lse)
        torch.cuda.synchronize()
        want_o, want_l = oracle.sparse_decode_attn(qd, out["pk"][l], out["pv"][l], ck, data["k"][l], data["v"][l], cu, loc, cl)
        assert np.abs(o.float().cpu().numpy() - want_o).max() <= 2e-2
        assert np.abs(lse.cpu().numpy() - want_l).max() <= 1e-3
    assert hp.read_status() == 0


def test_varlen_config_budget_sweep():
    """8 prompts of 2K-32K tokens, budgets 5 / 10 / 20 %: scores on two sampled KV heads, select and pack everywhere."""
    for frac in (0.05, 0.10, 0.20):
        cfg = wl.varlen(frac)
        data, hp, _, out = run_prefill(cfg)
        cu = data["cu_seqlens"]
        mass = np.add.reduceat(out["imp"].astype(np.float64), cu[:-1], axis=-1)
        np.testing.assert_allclose(mass, cfg.group * cfg.window, rtol=1e-4)
        if frac == 0.10:
            G = cfg.group
            for g in (0, 5):
                imp_o = oracle.score(data["q_win"][:, :, :, g * G:(g + 1) * G], data["k"][:, :, g:g + 1], cu)
                assert close(out["imp"][:, g:g + 1], imp_o)
        check_select_and_pack(cfg, data, out, [0])


def test_llama70b_config_long_context():
    """8 layers, 64/8 heads, 32768-token prompt, W = 64 (512 score rows per KV head), budget 2048."""
    cfg = wl.llama70b()
    data, hp, _, out = run_prefill(cfg)
    cu = data["cu_seqlens"]
    np.testing.assert_allclose(out["imp"].astype(np.float64).sum(-1), cfg.group * cfg.window, rtol=1e-4)
    G = cfg.group
    for l, g in [(0, 0), (7, 6)]:
        imp_o = oracle.score(data["q_win"][l:l + 1, :, :, g * G:(g + 1) * G], data["k"][l:l + 1, :, g:g + 1], cu)
        assert close(out["imp"][l:l + 1, g:g + 1], imp_o)
    check_select_and_pack(cfg, data, out, [0, 7])
    # the clustered spans carry the mass: every span token is selected
    pos = set(wl.heavy_positions(cfg, 3, 0).tolist())
    assert all(pos <= set(out["sel"][3, g].tolist()) for g in range(cfg.num_kv_heads))


@pytest.mark.parametrize("batch,sel,rho", [(128, 0.20, 0.25), (32, 1.0, 0.5), (1, 0.05, 0.0), (8, 0.5, 0.1)])
def test_decode_sweep_points(batch, sel, rho):
    """Decode-heavy sweep: B sequences of 4096 tokens, `sel` of the prompt required, `rho` of that index-addressed."""
    import gpu_ops
    cfg = wl.decode_sweep(batch, sel, rho)
    rng = np.random.default_rng(batch)
    from helpers import rand_bf16
    T = cfg.total_tokens
    k = rand_bf16(rng, (T, 8, 128)); v = rand_bf16(rng, (T, 8, 128)); q = rand_bf16(rng, (batch, 32, 128))
    sel_idx, ck, loc, cl = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local())
    cu = cfg.cu_seqlens()
    pk, pv = oracle.pack_kv(k[None], v[None], cu, sel_idx[None], ck)
    want_o, want_l = oracle.sparse_decode_attn(q, pk[0], pv[0], ck, k, v, cu, loc, cl)
    got_o, got_l = gpu_ops.sparse_decode_attn(q, pk[0], pv[0], ck, k, v, cu, loc, cl)
    assert np.abs(got_o - want_o).max() <= 2e-2 and np.abs(got_l - want_l).max() <= 1e-3
