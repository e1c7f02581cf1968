"""The synthetic workloads have the stated shapes and structure, and are reproducible."""
import numpy as np

import oracle
from paper_2607_28150_b200 import workloads as wl


def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.0e38], dtype=np.float32)
    b = wl.f32_to_bf16_bits(x)
    y = wl.bf16_bits_to_f32(b)
    assert y[0] == 1.0 and y[3] == -2.5 and y[4] == 0.0
    assert y[1] == 1.0            # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: goes to the even mantissa
    assert y[2] == 1.015625       # 1 + 3*2^-8 is a tie between 1+2^-7 and 1+2^-6: even is 1+2^-6
    assert np.array_equal(wl.f32_to_bf16_bits(y), b)


def test_tiny_config_shapes_and_determinism():
    cfg = wl.tiny()
    a, b = wl.make_prefill(cfg), wl.make_prefill(cfg)
    assert a["q_win"].shape == (1, 1, 16, 8, 64) and a["k"].shape == (1, 1024, 2, 64)
    for name in ("q_win", "k", "v"):
        assert np.array_equal(a[name], b[name])
    assert cfg.budgets().tolist() == [128] and cfg.n_local().tolist() == [32]
    pos = wl.heavy_positions(cfg, 0, 0)
    assert len(pos) == 20 and pos[:4].tolist() == [0, 1, 2, 3]
    norms = np.linalg.norm(wl.bf16_bits_to_f32(a["k"])[0, pos], axis=-1)
    assert np.allclose(norms, 4 * 8.0, rtol=0.02)


def test_heavy_hitters_and_sinks_are_selected_by_the_oracle():
    """Structure check: the seeded heavy hitters carry the attention mass the selection is meant to find."""
    cfg = wl.tiny()
    data = wl.make_prefill(cfg)
    imp = oracle.score(data["q_win"], data["k"], data["cu_seqlens"])
    sel = oracle.select_topk(imp, data["cu_seqlens"], cfg.cu_k())
    pos = set(wl.heavy_positions(cfg, 0, 0).tolist())
    for g in range(cfg.num_kv_heads):
        assert pos <= set(sel[0, g].tolist())


def test_config_shapes():
    c2 = wl.llama8b()
    assert (c2.num_layers, c2.group, c2.budgets().tolist()) == (32, 4, [820])
    c3 = wl.varlen(0.05)
    assert c3.batch == 8 and all(2048 <= n <= 32768 for n in c3.seqlens)
    assert c3.seqlens == wl.varlen(0.2).seqlens
    c4 = wl.llama70b()
    assert c4.group * c4.window == 512 and c4.budgets().tolist() == [2048]
    assert len(wl.heavy_positions(c4, 0, 0)) == 4 + 4 * 256
    c5 = wl.decode_sweep(4, 1.0, 0.25)
    assert c5.budgets()[0] + c5.n_local()[0] == 4096


def test_index_split_is_disjoint_and_seeded():
    cfg = wl.decode_sweep(2, 0.2, 0.5, seqlen=256)
    sel, ck, loc, cl = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local())
    sel2, _, loc2, _ = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local())
    assert np.array_equal(sel, sel2) and np.array_equal(loc, loc2)
    for g in range(cfg.num_kv_heads):
        for b in range(cfg.batch):
            s = set(sel[g, ck[b]:ck[b + 1]].tolist())
            l = set(loc[g, cl[b]:cl[b + 1]].tolist())
            assert len(s) == ck[b + 1] - ck[b] and len(l) == cl[b + 1] - cl[b] and not (s & l)
