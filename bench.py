#!/usr/bin/env python
"""Benchmark of the selective-KV hot path on B200: score -> select -> pack -> sparse decode.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c2|c4|c3|c5]

One "step" is one pass of the whole path over one batch of synthetic prompts: sg_score,
sg_select_topk and sg_pack_kv over all layers (one call each), then the workload's decode steps
(one sg_sparse_decode_attn call per layer per step, replayed from a CUDA graph).  The default
workload is the Llama-3-8B-shaped cache (32 layers, 8192-token prompt, 10 % budget, 64 decode
steps).  Rank 0 prints ONE JSON line:
  value                 (select + pack algorithmic bytes) / device time of the sg_select_pack_kv call (selection and gather in
                        one kernel on this workload), inputs resident in HBM; stage_ms.select / .pack: the two separate calls
  decode_tokens_per_s   batch * decode steps / decode-stage device time;  stage_ms: every stage of a step
  e2e                   the same step with host buffers (pinned H2D of caches and queries, D2H of the payload and outputs)
  roofline / rooflines  per-kernel achieved bytes/s (or flop/s) against the measured copy / bf16 peaks
  decode_sweep          the decode kernel alone on large-batch points; next_rows: timings of the widened rows
  cpu_baseline          the CPU oracle timed on a bounded sample of the same workload; clocks: sampled under load

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "prefill select+pack GB/s (sparse-decode tokens/s in decode_tokens_per_s)"
UNIT = "GB/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu --set full captures (bytes; None where no
# capture exists).  Keyed by workload then kernel.
NCU_TRAFFIC = {
    # captured on 8 of the 32 layers: per-launch bytes scaled x4 where a launch
    # covers all layers; the decode call is per layer.  (pack: its stores were still in L2 when the capture ended.)
    "c2": {"score": 4 * (142.152e6 + 6.255e6), "select": 4 * 2.125e6, "pack": 4 * (27.097e6 + 0.131e6),
           "select_pack": (32 / 24) * (86.950e6 + 27.208e6), "decode": 5.146e6},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def workload_config(name: str, args):
    from paper_2607_28150_b200 import workloads as wl
    if name == "c2":
        return wl.llama8b() if args.layers is None else wl.llama8b(num_layers=args.layers)
    if name == "c4":
        return wl.llama70b() if args.layers is None else wl.llama70b(num_layers=args.layers)
    if name == "c3":
        return wl.varlen(args.fraction)
    if name == "c5":
        return wl.decode_sweep(args.batch, args.sel, args.rho)
    if name == "c1":
        return wl.tiny()
    raise SystemExit("unknown workload %s" % name)


def algorithmic_work(cfg, n_loc):
    """Algorithmic bytes / flops of one step, per stage (what the method must move or compute, counted once)."""
    L, Hkv, d, G, W = cfg.num_layers, cfg.num_kv_heads, cfg.head_dim, cfg.group, cfg.window
    lens = np.asarray(cfg.seqlens, dtype=np.int64)
    ks = cfg.budgets().astype(np.int64)
    T, Ktot, NL = int(lens.sum()), int(ks.sum()), int(np.sum(n_loc))
    R = G * W
    work = {
        "score": {"flops": float(2 * R * d * T * Hkv * L),
                  "bytes": float(L * Hkv * (T * d * 2 + T * 4) + L * cfg.batch * W * cfg.num_q_heads * d * 2)},
        "select": {"bytes": float(L * Hkv * (T * 4 + Ktot * 4))},
        "pack": {"bytes": float(L * Hkv * Ktot * (2 * 2 * d * 2 + 4))},
        "decode_call": {"bytes": float(Hkv * (2 * (Ktot + NL) * d * 2 + NL * 4) + 2 * cfg.batch * cfg.num_q_heads * d * 2),
                        "flops": float(4 * G * d * (Ktot + NL) * Hkv)},
    }
    return work


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.strip().split(", ") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
            except ValueError:
                continue
            for nm, val in zip(names, r[4:8]):
                if val.strip().lower().startswith("active"):
                    reasons.add(nm)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# --------------------------------------------------------------------------------------------- oracle arm
def oracle_sample(cfg, layers, n_decode_layers=None):
    """Time the CPU oracle, as it stands, on `layers` of the workload: score, select, pack, one decode step."""
    import oracle
    from paper_2607_28150_b200 import workloads as wl
    data = wl.make_prefill(cfg, layers)
    cu, ck = data["cu_seqlens"], cfg.cu_k()
    t = {}
    t0 = time.perf_counter(); imp = oracle.score(data["q_win"], data["k"], cu); t["score"] = time.perf_counter() - t0
    t0 = time.perf_counter(); sel = oracle.select_topk(imp, cu, ck); t["select"] = time.perf_counter() - t0
    t0 = time.perf_counter(); pk, pv = oracle.pack_kv(data["k"], data["v"], cu, sel, ck); t["pack"] = time.perf_counter() - t0
    nloc = cfg.n_local()
    td = 0.0
    for i, l in enumerate(layers):
        q = wl.make_decode_queries(cfg, l, 0, data["q_win"][i])
        _, _, loc, cl = wl.make_index_split(cfg, l, 0, cfg.budgets(), nloc, exclude=sel[i], cu_excl=ck)
        t0 = time.perf_counter()
        oracle.sparse_decode_attn(q, pk[i], pv[i], ck, data["k"][i], data["v"][i], cu, loc, cl)
        td += time.perf_counter() - t0
    t["decode"] = td
    return t


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle
    cfg = workload_config(args.workload, args)
    layers = list(range(min(2, cfg.num_layers)))
    work = algorithmic_work(cfg, cfg.n_local())
    frac = len(layers) / cfg.num_layers
    for _ in range(args.warmup):
        oracle_sample(cfg, layers)
    t_all, t_sp, t_dec = 0.0, 0.0, 0.0
    for _ in range(args.steps):
        t0 = time.perf_counter()
        t = oracle_sample(cfg, layers)
        t_all += time.perf_counter() - t0
        t_sp += t["select"] + t["pack"]
        t_dec += t["decode"]
    value = (work["select"]["bytes"] + work["pack"]["bytes"]) * frac * args.steps / t_sp / 1e9
    dec_tok = cfg.batch * len(layers) / cfg.num_layers * args.steps / t_dec
    cores = oracle.max_threads()
    sample = "layers 0-%d of %s per step: oracle score+select+pack and one decode step over those layers" % (
        layers[-1], cfg.name)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "sample": sample},
            "decode_tokens_per_s": dec_tok,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------- CUDA arm

def next_rows_timing(dev, cfg, hp, k_cache, v_cache, layer=0, reps=20):
    """Device time of the "next" rows on the workload's shapes: Algorithm 1 (sg_split_index) on one layer's KV
    index, and the profile chain (sg_profile_accumulate per layer, sg_block_importance, sg_proactive_mask)."""
    import torch
    from paper_2607_28150_b200 import binding as sg
    B, Hkv, T, Ktot, L, M = hp.B, hp.Hkv, hp.T, hp.K_tot, hp.L, 1024
    gen = torch.Generator(device=dev); gen.manual_seed(77)
    mask = (torch.randint(0, 100, (T,), generator=gen, device=dev) < 34).to(torch.int8) + 1      # 34 % remote
    idx = hp.sel_idx[layer].contiguous()
    re_ = torch.empty_like(idx); loc = torch.empty_like(idx); rem = torch.empty_like(idx)
    nl = torch.empty((B, Hkv), dtype=torch.int32, device=dev); nr = torch.empty_like(nl)
    counts = torch.zeros((L, Hkv, T), dtype=torch.int32, device=dev)
    imp = torch.empty((L, M), dtype=torch.float32, device=dev)
    pmask = torch.empty(T, dtype=torch.int8, device=dev)
    selblk = torch.arange(0, 2 * M, dtype=torch.int32, device=dev)
    # block push: every block of one layer (Eq. 1 always selects layers 0 and 1), rotating over the layers so the
    # source is not L2-resident; one layer of K+V read and written per call
    dst_k = torch.empty_like(k_cache[0]); dst_v = torch.empty_like(v_cache[0])
    push_sel = [torch.arange(l * M, (l + 1) * M, dtype=torch.int32, device=dev) for l in range(L)]

    def push_all_layers():                                   # L calls, one per layer, replayed from a CUDA graph
        for l in range(L):
            sg.sg_push_blocks(hp.shape1, M, l, push_sel[l], k_cache[l], v_cache[l], dst_k, dst_v)
    push_bytes = 2 * 2 * T * Hkv * hp.d * 2
    # threshold selection on the step's importance: alpha = 2 of the R = G*W attention mass, cap 20 % of each prompt
    caps = [max(1, -(-int(n) // 5)) for n in np.diff(hp.cu_host)]
    cu_cap = torch.tensor(np.concatenate([[0], np.cumsum(caps)]).astype(np.int32), device=dev)
    cap_tot = int(sum(caps))
    thr_idx = torch.empty((L, Hkv, cap_tot), dtype=torch.int32, device=dev)
    thr_cnt = torch.empty((L, B, Hkv), dtype=torch.int32, device=dev)
    dst_all_k = torch.empty_like(k_cache); dst_all_v = torch.empty_like(v_cache)
    sel_all = torch.arange(0, L * M, dtype=torch.int32, device=dev)
    sel_40 = torch.arange(0, L * M, dtype=torch.int32, device=dev)[torch.randperm(L * M, generator=gen, device=dev)[: (2 * L * M) // 5]].sort().values.contiguous()

    def timeit(fn):
        fn(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record(); torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / reps

    def timeit_graph(fn):
        fn(); torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        g.replay(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            g.replay()
        e1.record(); torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / 5

    return {
        "split_index_us": timeit(lambda: sg.sg_split_index(hp.shape1, idx, hp.cu_k, Ktot, mask, True, re_, loc, rem, nl, nr)),
        "profile_accumulate_us_per_layer": timeit(lambda: sg.sg_profile_accumulate(hp.shape1, idx, hp.cu_k, Ktot, counts[layer])),
        "block_importance_us": timeit(lambda: sg.sg_block_importance(hp.shape, counts, M, imp)),
        "proactive_mask_us_per_layer": timeit(lambda: sg.sg_proactive_mask(hp.shape1, M, layer, selblk, pmask)),
        "select_threshold_all_layers_us": timeit(lambda: sg.sg_select_threshold(hp.shape, hp.importance, 2.0, cu_cap, cap_tot, thr_idx, thr_cnt)),
        "push_blocks_us_per_layer": (push_us := timeit_graph(push_all_layers) / L),
        "push_blocks_gbs": push_bytes / push_us / 1e3,
        "push_blocks_frac_of_copy_peak": push_bytes / push_us / 1e3 / load_peaks()["hbm_gbs"],
        "push_blocks_all_layers_one_call_us": (push_all_us := timeit(lambda: sg.sg_push_blocks(hp.shape, M, 0, sel_all, k_cache, v_cache, dst_all_k, dst_all_v))),
        "push_blocks_all_layers_frac_of_copy_peak": L * push_bytes / push_all_us / 1e3 / load_peaks()["hbm_gbs"],
        "push_blocks_40pct_one_call_us": (push_40_us := timeit(lambda: sg.sg_push_blocks(hp.shape, M, 0, sel_40, k_cache, v_cache, dst_all_k, dst_all_v))),
        "push_blocks_40pct_frac_of_copy_peak": 0.4 * L * push_bytes / push_40_us / 1e3 / load_peaks()["hbm_gbs"],
        "note": "push_blocks moves one whole layer per call (all M = 1024 blocks selected), 32 calls replayed from a CUDA graph; the others are launch-latency-bound integer kernels (a few KB to a few MB each); eager launches, CUDA events",
    }


def layerwise_prefill_timing(dev, hp, d_q, d_k, d_v, reps=5):
    """The prefill side issued layer by layer (one score/select/pack call per layer, as a prefill engine would
    when each layer's KV becomes ready), replayed from a CUDA graph: on one stream, and with select+pack on a
    second stream so that they overlap the next layer's scoring.  Device ms for all layers."""
    import torch

    def graph_ms(aux):
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            hp.prefill_layerwise(d_q, d_k, d_v, aux_stream=aux)            # warm-up outside the capture
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                hp.prefill_layerwise(d_q, d_k, d_v, aux_stream=aux)
            g.replay(); side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(reps):
                g.replay()
            e1.record(side); side.synchronize()
        return e0.elapsed_time(e1) / reps

    one = graph_ms(None)
    two = graph_ms(torch.cuda.Stream(device=dev))
    return {"one_stream_ms": one, "two_stream_ms": two, "layers": hp.L,
            "note": "3 kernels + 1 counter memset per layer; compare with score+select+pack of the all-layer calls in stage_ms"}


def full_first_two_timing(dev, cfg, d_q, d_k, d_v, reps=5):
    """The prefill side under the budget policy of Eq. 1 / Eq. 2's clip: layers 0 and 1 are transferred whole
    (k_b = N_b, the selection degenerates to the identity list), the other layers get the workload's budget.
    Two call groups replayed from one CUDA graph; device ms and the payload it produces."""
    import torch
    from paper_2607_28150_b200.pipeline import HotPath
    L = cfg.num_layers
    if L <= 2:
        return None
    args = (cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window, cfg.seqlens)
    first = HotPath(2, *args, list(cfg.seqlens), device=dev)
    rest = HotPath(L - 2, *args, cfg.budgets(), device=dev)

    def run():
        first.select_pack(d_k[:2], d_v[:2])
        rest.prefill(d_q[2:], d_k[2:], d_v[2:])

    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        run(); side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            run()
        g.replay(); side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(reps):
            g.replay()
        e1.record(side); side.synchronize()
    status = first.read_status() | rest.read_status()
    payload = 2 * (first.packed_k.numel() + rest.packed_k.numel()) * 2 + (first.sel_idx.numel() + rest.sel_idx.numel()) * 4
    return {"ms_prefill": e0.elapsed_time(e1) / reps, "payload_mb": payload / 1e6, "dev_status": status,
            "note": "layers 0-1 with k_b = N_b (whole layers), layers 2..%d with the workload's budget; score + select + pack" % (L - 1)}


def decode_sweep_points(dev, peaks, points=((64, 0.20, 0.25), (128, 1.0, 0.0), (128, 1.0, 0.5)), calls=16):
    """sg_sparse_decode_attn alone on points of the decode-heavy sweep (B sequences of 4096 tokens, `sel` of the
    prompt required, `rho` of that index-addressed): the sizes at which the kernel can reach the HBM roofline.
    K/V are seeded N(0,1) bf16 generated on the device; the packed buffer is built by sg_pack_kv; every call of a
    timed graph reads more than L2 holds.  Returns one dict per point."""
    import torch
    from paper_2607_28150_b200 import binding as sg, workloads as wl
    from paper_2607_28150_b200.pipeline import as_device
    out = []
    gen = torch.Generator(device=dev)
    for (B, sel, rho) in points:
        cfg = wl.decode_sweep(B, sel, rho)
        Hq, Hkv, d, N = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.seqlens[0]
        T = B * N
        gen.manual_seed(5000 + B)
        k = torch.randn((T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        v = torch.randn((T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        q = torch.randn((B, Hq, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        sel_idx, ck, loc, cl = wl.make_index_split(cfg, 0, 0, cfg.budgets(), cfg.n_local())
        Ktot, NL = int(ck[-1]), int(cl[-1])
        cu = as_device(cfg.cu_seqlens(), dev)
        d_ck, d_cl = as_device(ck, dev), as_device(cl, dev)
        shp = sg.make_shape(1, Hq, Hkv, d, 1, cu, T, N)
        pk = torch.empty((max(Ktot, 1) * Hkv, d), dtype=torch.bfloat16, device=dev)
        pv = torch.empty_like(pk)
        if Ktot:
            sg.sg_pack_kv(shp, k, v, as_device(sel_idx, dev), d_ck, Ktot, pk, pv)
        d_loc = as_device(loc, dev) if NL else None
        o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=dev)
        call = lambda: sg.sg_sparse_decode_attn(shp, q, pk if Ktot else None, pv if Ktot else None, d_ck, Ktot, k, v,
                                                d_loc, d_cl, NL, o)
        call()
        torch.cuda.synchronize()
        def graph_us_per_call():
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for _ in range(calls):
                    call()
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            best = float("inf")
            for _ in range(3):
                e0.record(); g.replay(); e1.record()
                torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            return best * 1e3 / calls
        us = graph_us_per_call()
        try:
            sg.sg_testing_decode_overlap(False)          # every call fully ordered behind the one before it
            us_serial = graph_us_per_call()
        finally:
            sg.sg_testing_decode_overlap(True)
        nbytes = Hkv * (2 * (Ktot + NL) * d * 2 + NL * 4) + 2 * B * Hq * d * 2
        gbs = nbytes / us / 1e3
        out.append({"batch": B, "sel": sel, "rho": rho, "n_sel": Ktot // B, "n_loc": NL // B, "us_per_call": us, "us_per_call_serialized": us_serial,
                    "bytes_per_call": nbytes, "l2": "larger than L2" if nbytes > 126e6 else "warm L2 (same buffers every call)",
                    "achieved_gbs": gbs, "frac_of_copy_peak": gbs / peaks["hbm_gbs"],
                    "tokens_per_s": B / (us * 1e-6)})
        del k, v, pk, pv
        torch.cuda.empty_cache()
    return out

def _graph_us(fn, dev, reps=7):
    """Median device time (us) of `fn` replayed from a CUDA graph on a side stream (CUDA events on that stream)."""
    import torch
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        fn(); side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
        g.replay(); side.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side); g.replay(); e1.record(side); side.synchronize()
            ts.append(e0.elapsed_time(e1))
    return 1e3 * float(np.median(ts))


def handover_timing(dev, hp, d_q, d_k, d_v):
    """What the kernel boundary between scoring and selection costs: device time of sg_score and sg_select_pack_kv each
    replayed alone, and of the two back to back in one graph.  `gap_us` = both - (score + select_pack) is everything a
    score -> select fusion could remove (launch hand-over, drained SMs, and the importance array's trip through L2/HBM:
    `importance_bytes` written once and read once)."""
    a = _graph_us(lambda: hp.score(d_q, d_k), dev)
    b = _graph_us(lambda: hp.select_pack(d_k, d_v), dev)

    def both():
        hp.score(d_q, d_k)
        hp.select_pack(d_k, d_v)
    c = _graph_us(both, dev)
    imp_bytes = hp.importance.numel() * 4
    return {"score_us": a, "select_pack_us": b, "back_to_back_us": c, "gap_us": c - a - b, "gap_frac_of_prefill": (c - a - b) / c,
            "importance_bytes": imp_bytes, "importance_round_trip_us_at_copy_peak": 2 * imp_bytes / load_peaks()["hbm_gbs"] / 1e3}

def score_clock(dev, hp, d_q, d_k):
    """SM clock (MHz) the scoring kernel really runs at: every CTA records clock64 and globaltimer at its start and end
    (testing hook of the library); a 200 ms nvidia-smi sample cannot see a kernel of a fraction of a millisecond."""
    import torch
    from paper_2607_28150_b200 import binding as sg
    grid = max(1, sg.sg_testing_score_grid(hp.shape))
    buf = torch.zeros(32 * grid, dtype=torch.int64, device=dev)
    for _ in range(2):
        hp.score(d_q, d_k)                       # same thermal / power state as the timed calls
    torch.cuda.synchronize()
    try:
        sg.sg_testing_score_clock(buf)
        hp.score(d_q, d_k)
        torch.cuda.synchronize()
    finally:
        sg.sg_testing_score_clock(None)
    rec = buf.cpu().numpy()[: 4 * grid].reshape(grid, 4).astype(np.float64)
    cyc, ns = rec[:, 1] - rec[:, 0], rec[:, 3] - rec[:, 2]
    ok = (cyc > 0) & (ns > 0)
    return float(1e3 * np.median(cyc[ok] / ns[ok])) if ok.any() else None


def measure_config(dev, peaks, cfg, fractions=None, decode=True):
    """Every stage of the path on one benchmark configuration, each timed alone (CUDA graph replay, CUDA events, median
    of 7): sg_score, sg_select_topk, sg_pack_kv, sg_select_pack_kv over all the configuration's layers in one call each,
    and one sg_sparse_decode_attn call (layer 0).  Inputs are the seeded synthetic caches of the workload recipe,
    resident in HBM.  Returns per stage: time, algorithmic bytes / flops, achieved rate, the roof that binds, frac."""
    import torch
    from paper_2607_28150_b200 import binding as sg, workloads as wl
    from paper_2607_28150_b200.pipeline import HotPath, as_device
    L, B, Hq, Hkv, d, W = cfg.num_layers, cfg.batch, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window
    T = cfg.total_tokens
    d_q = torch.empty((L, B, W, Hq, d), dtype=torch.int16, device=dev)
    d_k = torch.empty((L, T, Hkv, d), dtype=torch.int16, device=dev)
    d_v = torch.empty((L, T, Hkv, d), dtype=torch.int16, device=dev)
    for l in range(L):
        lay = wl.make_layer(cfg, l)
        d_q[l] = as_device(lay["q_win"], dev); d_k[l] = as_device(lay["k"], dev); d_v[l] = as_device(lay["v"], dev)
    tc_peak, hbm_peak = peaks["bf16_tflops_sustained"], peaks["hbm_gbs"]
    out = {"workload": "%s: L=%d B=%d Hq=%d Hkv=%d d=%d W=%d T=%d" % (cfg.name, L, B, Hq, Hkv, d, W, T), "stages": {}}

    def hbm(nbytes, us):
        a = nbytes / us / 1e3
        return {"us": us, "bytes": nbytes, "achieved": a, "unit": "GB/s", "bound": "hbm", "peak": hbm_peak, "frac": a / hbm_peak}

    first = True
    for frac in (fractions or [None]):
        budgets = cfg.budgets(frac) if frac is not None else cfg.budgets()
        hp = HotPath(L, Hq, Hkv, d, W, cfg.seqlens, budgets, device=dev)
        nloc = cfg.n_local(frac) if frac is not None else cfg.n_local()
        work = algorithmic_work(cfg if frac is None else wl.varlen(frac, L, cfg.seqlens), nloc)
        tag = "" if frac is None else "@%g%%" % (100 * frac)
        if first:
            us = _graph_us(lambda: hp.score(d_q, d_k), dev)
            r = hbm(work["score"]["bytes"], us)
            tf = work["score"]["flops"] / us / 1e6
            exps = 2.0 * work["score"]["flops"] / (2.0 * d)
            mhz = score_clock(dev, hp, d_q, d_k)
            r.update(tensor_tflops=tf, tensor_frac_of_sustained=tf / tc_peak, sfu_exp_per_s=exps / (us * 1e-6), sm_mhz_in_kernel=mhz,
                     sfu_frac_at_kernel_clock=(exps / (us * 1e-6)) / (16.0 * 148 * mhz * 1e6) if mhz else None)
            if cfg.group * W > tc_peak * 1e3 / hbm_peak:                  # above the ridge: tensor cores bind
                r.update(bound="tensor", achieved=tf, unit="TFLOP/s", peak=tc_peak, frac=tf / tc_peak)
            out["stages"]["score"] = r
        else:
            hp.score(d_q, d_k)
        torch.cuda.synchronize()
        out["stages"]["select" + tag] = hbm(work["select"]["bytes"], _graph_us(lambda: hp.select(), dev))
        out["stages"]["pack" + tag] = hbm(work["pack"]["bytes"], _graph_us(lambda: hp.pack(d_k, d_v), dev))
        out["stages"]["select_pack" + tag] = hbm(work["select"]["bytes"] + work["pack"]["bytes"],
                                                  _graph_us(lambda: hp.select_pack(d_k, d_v), dev))
        if decode and first:
            sel_host = hp.sel_idx[0].cpu().numpy()
            _, _, loc, cl = wl.make_index_split(cfg, 0, 0, budgets, nloc, exclude=sel_host, cu_excl=hp.cu_k_host)
            NL = int(cl[-1])
            qd = as_device(wl.make_decode_queries(cfg, 0, 0), dev)
            d_loc, d_cl = (as_device(loc, dev) if NL else None), as_device(cl, dev)
            o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=dev)
            hp.decode_workspace(NL)
            calls = 8

            def dec():
                for _ in range(calls):
                    hp.decode(0, qd, d_k[0], d_v[0], d_loc, d_cl, NL, o)
            us = _graph_us(dec, dev) / calls
            r = hbm(work["decode_call"]["bytes"], us)
            r["note"] = "one call (layer 0), %d back-to-back calls per graph, same buffers: warm L2 below 126 MB" % calls
            r["tokens_per_s"] = B / (us * 1e-6)
            out["stages"]["decode_call"] = r
        if first:
            out["score_select_handover"] = handover_timing(dev, hp, d_q, d_k, d_v)
        out["dev_status" + tag] = hp.read_status()
        first = False
        del hp
    del d_q, d_k, d_v
    torch.cuda.empty_cache()
    return out


def measure_configs(dev, peaks):
    """c1 (tiny), c3 (ragged batch, one layer: budgets 10 % with every stage, 5 % and 20 % for selection and gather) and
    c4 (long context, 8 layers) measured in the same run as the timed c2 step."""
    from paper_2607_28150_b200 import workloads as wl
    return {
        "c1": measure_config(dev, peaks, wl.tiny()),
        "c3": measure_config(dev, peaks, wl.varlen(0.10), fractions=[0.10, 0.05, 0.20]),
        "c4": measure_config(dev, peaks, wl.llama70b()),
    }

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_28150_b200 import build as _build
    if not os.path.exists(_build.LIB):
        _build.build()                                   # in-tree nvcc build; there is no fallback path
    from paper_2607_28150_b200 import binding as sg, workloads as wl
    from paper_2607_28150_b200.pipeline import HotPath

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    cfg = workload_config(args.workload, args)
    L, B, Hq, Hkv, d, W = cfg.num_layers, cfg.batch, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window
    T = cfg.total_tokens
    nsteps_dec = args.decode_steps if args.decode_steps is not None else cfg.decode_steps
    if args.decode_steps is None and args.workload == "c5":
        nsteps_dec = 16        # a single call per graph would measure the graph launch, not the kernel
    nloc = cfg.n_local()
    cu_nloc_h = np.concatenate([[0], np.cumsum(nloc)]).astype(np.int32)
    NL = int(cu_nloc_h[-1])
    work = algorithmic_work(cfg, nloc)

    # ---- synthetic inputs: generated on the host (seeded), kept in pinned memory for the end-to-end arm
    t_gen = time.perf_counter()
    h_q = torch.empty((L, B, W, Hq, d), dtype=torch.int16).pin_memory()
    h_k = torch.empty((L, T, Hkv, d), dtype=torch.int16).pin_memory()
    h_v = torch.empty((L, T, Hkv, d), dtype=torch.int16).pin_memory()
    for l in range(L):
        lay = wl.make_layer(cfg, l)
        h_q[l] = torch.from_numpy(lay["q_win"].view(np.int16))
        h_k[l] = torch.from_numpy(lay["k"].view(np.int16))
        h_v[l] = torch.from_numpy(lay["v"].view(np.int16))
    d_q, d_k, d_v = h_q.to(dev), h_k.to(dev), h_v.to(dev)
    hp = HotPath(L, Hq, Hkv, d, W, cfg.seqlens, cfg.budgets(), device=dev)
    Ktot = hp.K_tot

    # one untimed pass to obtain the selected sets, from which the local (on-demand) indices are drawn
    hp.prefill(d_q, d_k, d_v)
    torch.cuda.synchronize()
    sel_host = hp.sel_idx.cpu().numpy()
    h_qdec = torch.empty((nsteps_dec, L, B, Hq, d), dtype=torch.int16).pin_memory()
    h_idx = torch.empty((nsteps_dec, L, Hkv, max(NL, 1)), dtype=torch.int32).pin_memory()
    qwin_f = [wl.bf16_bits_to_f32(h_q[l].numpy().view(np.uint16)).mean(axis=1) for l in range(L)]
    for s in range(nsteps_dec):
        rng = np.random.Generator(np.random.Philox(key=1000 * cfg.config_id + 7 + 100000 * (s + 1)))
        qd = rng.standard_normal((L, B, Hq, d), dtype=np.float32) + np.stack(qwin_f)
        h_qdec[s] = torch.from_numpy(wl.f32_to_bf16_bits(qd).view(np.int16))
    if NL:
        ck = hp.cu_k_host
        for l in range(L):
            rng = np.random.Generator(np.random.Philox(key=1000 * cfg.config_id + 10 * l + 6))
            for b, n in enumerate(cfg.seqlens):
                if nloc[b] == 0:
                    continue
                for g in range(Hkv):
                    rest = np.setdiff1d(np.arange(n, dtype=np.int32), sel_host[l, g, ck[b]:ck[b + 1]])
                    draws = rng.permuted(np.tile(rest, (nsteps_dec, 1)), axis=1)[:, : nloc[b]]
                    h_idx[:, l, g, cu_nloc_h[b]:cu_nloc_h[b + 1]] = torch.from_numpy(draws)
    d_qdec, d_idx = h_qdec.to(dev), h_idx.to(dev)
    d_cu_nloc = torch.from_numpy(cu_nloc_h).to(dev)
    d_out = torch.empty((nsteps_dec, L, B, Hq, d), dtype=torch.bfloat16, device=dev)
    h_out = torch.empty((nsteps_dec, L, B, Hq, d), dtype=torch.bfloat16).pin_memory()
    h_pk = torch.empty(hp.packed_k.shape, dtype=torch.int16).pin_memory()
    h_pv = torch.empty(hp.packed_v.shape, dtype=torch.int16).pin_memory()
    h_sel = torch.empty(hp.sel_idx.shape, dtype=torch.int32).pin_memory()
    hp.decode_workspace(NL)
    gen_s = time.perf_counter() - t_gen

    # End-to-end arm: a step's queries and local indices travel as ONE host->device copy (a staging record per step,
    # queries first, then the index lists), as a serving loop stages the inputs of a step; the kernels read views of it.
    q_bytes, idx_bytes = L * B * Hq * d * 2, (L * Hkv * NL * 4 if NL else 0)
    rec = (q_bytes + idx_bytes + 255) // 256 * 256
    h_in = torch.empty((max(nsteps_dec, 1), rec), dtype=torch.uint8).pin_memory()
    d_in = torch.empty((max(nsteps_dec, 1), rec), dtype=torch.uint8, device=dev)
    for s in range(nsteps_dec):
        h_in[s, :q_bytes] = h_qdec[s].reshape(-1).view(torch.uint8)
        if NL:
            h_in[s, q_bytes:q_bytes + idx_bytes] = h_idx[s].reshape(-1).view(torch.uint8)
    e_q = [d_in[s, :q_bytes].view(torch.int16).view(L, B, Hq, d) for s in range(nsteps_dec)]
    e_idx = [d_in[s, q_bytes:q_bytes + idx_bytes].view(torch.int32).view(L, Hkv, NL) if NL else None for s in range(nsteps_dec)]

    def decode_all(with_copies: bool):
        for s in range(nsteps_dec):
            if with_copies:
                d_in[s].copy_(h_in[s], non_blocking=True)
            qs, ids = (e_q[s], e_idx[s]) if with_copies else (d_qdec[s], d_idx[s] if NL else None)
            for l in range(L):
                hp.decode(l, qs[l], d_k[l], d_v[l], ids[l] if NL else None, d_cu_nloc, NL, d_out[s, l])
            if with_copies:
                h_out[s].copy_(d_out[s], non_blocking=True)

    # eager once (sets kernel attributes), then capture both decode graphs
    if nsteps_dec:
        hp.decode(0, d_qdec[0, 0], d_k[0], d_v[0], d_idx[0, 0] if NL else None, d_cu_nloc, NL, d_out[0, 0])
    torch.cuda.synchronize()
    g_res, g_e2e = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    if nsteps_dec:
        with torch.cuda.graph(g_res):
            decode_all(False)
        with torch.cuda.graph(g_e2e):
            decode_all(True)
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream()

    def step(e2e: bool, ev, split: bool = False):
        """One pass of the path.  `ev` is a list of 7 events bracketing: h2d | score | select + pack | d2h | decode.
        Selection and packing are one library call (sg_select_pack_kv: one fused kernel on this workload); a `split`
        pass makes the two separate calls with an event between them (ev[3]) and gives the per-kernel times."""
        ev[0].record(stream)
        if e2e:
            d_q.copy_(h_q, non_blocking=True); d_k.copy_(h_k, non_blocking=True); d_v.copy_(h_v, non_blocking=True)
        ev[1].record(stream)
        hp.score(d_q, d_k)
        ev[2].record(stream)
        if split:
            hp.select()
            ev[3].record(stream)
            hp.pack(d_k, d_v)
        else:
            hp.select_pack(d_k, d_v)
        ev[4].record(stream)
        if e2e:
            h_pk.copy_(hp.packed_k, non_blocking=True); h_pv.copy_(hp.packed_v, non_blocking=True)
            h_sel.copy_(hp.sel_idx, non_blocking=True)
        ev[5].record(stream)
        if nsteps_dec:
            (g_e2e if e2e else g_res).replay()
        ev[6].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(e2e: bool, steps: int, warmup: int):
        mk = lambda: [torch.cuda.Event(enable_timing=True) for _ in range(7)]
        for _ in range(warmup):
            step(e2e, mk())
        evs = [mk() for _ in range(steps)]
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for i in range(steps):
            step(e2e, evs[i])
        t1.record(stream)
        barrier()
        total_ms = t0.elapsed_time(t1)
        spans = {"h2d": (0, 1), "score": (1, 2), "select_pack": (2, 4), "d2h": (4, 5), "decode": (5, 6)}
        stage = {n: sum(e[a].elapsed_time(e[b]) for e in evs) / steps for n, (a, b) in spans.items()}
        # per-kernel times of the two kernels inside the span, from passes with an event between them (not part of total_ms)
        sevs = [mk() for _ in range(steps)]
        for _ in range(min(warmup, 2)):
            step(e2e, mk(), split=True)
        for i in range(steps):
            step(e2e, sevs[i], split=True)
        torch.cuda.synchronize()
        stage["select"] = sum(e[2].elapsed_time(e[3]) for e in sevs) / steps
        stage["pack"] = sum(e[3].elapsed_time(e[4]) for e in sevs) / steps
        if world > 1:
            tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            total_ms = float(tt.item())
        return total_ms / steps, stage

    def e2e_pipelined_ms(reps: int = 3):
        """Prefill side with host buffers, layer by layer on three streams: while layer l is scored, selected and packed,
        layer l+1 is copied in and the packed rows of layer l-1 are copied out.  Returns device ms for all layers."""
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

        def run():
            start = torch.cuda.Event(); start.record(stream)
            s_in.wait_event(start); s_out.wait_event(start)
            for l in range(L):
                with torch.cuda.stream(s_in):
                    d_q[l].copy_(h_q[l], non_blocking=True); d_k[l].copy_(h_k[l], non_blocking=True); d_v[l].copy_(h_v[l], non_blocking=True)
                    e_in = torch.cuda.Event(); e_in.record(s_in)
                stream.wait_event(e_in)
                hp.prefill_layer(l, d_q, d_k, d_v)
                e_cmp = torch.cuda.Event(); e_cmp.record(stream)
                s_out.wait_event(e_cmp)
                with torch.cuda.stream(s_out):
                    h_pk[l].copy_(hp.packed_k[l], non_blocking=True); h_pv[l].copy_(hp.packed_v[l], non_blocking=True)
                    h_sel[l].copy_(hp.sel_idx[l], non_blocking=True)
            e_out = torch.cuda.Event(); e_out.record(s_out)
            stream.wait_event(e_out)

        run(); torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(reps):
            run()
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / reps

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_step, st = timed(False, args.steps, max(3, args.warmup))
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    ms_e2e, st_e = timed(True, e2e_steps, 1)
    ms_pipe = e2e_pipelined_ms() if world == 1 and not args.no_extras else None
    clocks = sampler.stop() if rank == 0 else {}       # sampled over both timed regions
    status = hp.read_status()

    from paper_2607_28150_b200 import replicas
    st, st_e = replicas.max_over_ranks(st), replicas.max_over_ranks(st_e)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    sp_bytes = work["select"]["bytes"] + work["pack"]["bytes"]
    value = world * sp_bytes / (st["select_pack"] * 1e-3) / 1e9
    dec_tok = world * B * nsteps_dec / (st["decode"] * 1e-3) if nsteps_dec else None
    e2e_value = world * sp_bytes / ((st_e["h2d"] + st_e["score"] + st_e["select_pack"] + st_e["d2h"]) * 1e-3) / 1e9
    e2e_dec_tok = world * B * nsteps_dec / (st_e["decode"] * 1e-3) if nsteps_dec else None
    h2d = (h_q.numel() + h_k.numel() + h_v.numel()) * 2 + (h_qdec.numel() * 2 + (h_idx.numel() * 4 if NL else 0))
    d2h = (h_pk.numel() + h_pv.numel()) * 2 + h_sel.numel() * 4 + h_out.numel() * 2

    # ---- rooflines, per kernel class, from the stage times of the device-resident arm
    ncalls_dec = nsteps_dec * L
    tc_peak = peaks["bf16_tflops_sustained"]
    ncu = NCU_TRAFFIC.get(args.workload, {})
    def hbm(name, nbytes, ms, launches):
        a = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
        return {"kernel": name, "bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": a / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy)", "ms_per_step": ms,
                "launches_per_step": launches, "traffic": ncu.get(name)}
    roofs = {
        "score": hbm("score", work["score"]["bytes"], st["score"], 1),
        "select": hbm("select", work["select"]["bytes"], st["select"], 1),
        "pack": hbm("pack", work["pack"]["bytes"], st["pack"], 1),
        "select_pack": hbm("select_pack", work["select"]["bytes"] + work["pack"]["bytes"], st["select_pack"], 1),
    }
    for n in ("select", "pack"):
        roofs[n]["launches_per_step"] = 0       # timed in the split passes; the step itself runs the fused kernel
    roofs["score"]["tensor_tflops"] = work["score"]["flops"] / (st["score"] * 1e-3) / 1e12
    roofs["score"]["tensor_frac_of_sustained"] = roofs["score"]["tensor_tflops"] / tc_peak
    roofs["select"]["rows"] = L * B * Hkv
    roofs["select"]["us_per_row_amortised"] = 1e3 * st["select"] / max(1, L * B * Hkv)
    # third ceiling of the scoring kernel: one exp2 per score element and pass on the SFU (16 per clock and SM)
    exps = 2.0 * work["score"]["flops"] / (2.0 * cfg.head_dim)
    sfu_peak = 16.0 * 148 * 1.965e9
    roofs["score"]["sfu_exp_per_s"] = exps / (st["score"] * 1e-3)
    roofs["score"]["sfu_frac_at_max_clock"] = roofs["score"]["sfu_exp_per_s"] / sfu_peak
    mhz = score_clock(dev, hp, d_q, d_k)
    roofs["score"]["sm_mhz_in_kernel"] = mhz
    roofs["score"]["sfu_frac_at_kernel_clock"] = roofs["score"]["sfu_exp_per_s"] / (16.0 * 148 * mhz * 1e6) if mhz else None
    R = cfg.group * W
    if R > peaks["bf16_tflops_sustained"] * 1e3 / peaks["hbm_gbs"]:       # above the ridge: tensor cores bind
        roofs["score"].update(bound="tensor", achieved=roofs["score"]["tensor_tflops"], peak=tc_peak, unit="TFLOP/s",
                              frac=roofs["score"]["tensor_frac_of_sustained"], peak_source=peaks["source"] + " (sustained bf16)")
    if ncalls_dec:
        roofs["decode"] = hbm("decode", work["decode_call"]["bytes"] * ncalls_dec, st["decode"], ncalls_dec)
        roofs["decode"]["us_per_call"] = 1e3 * st["decode"] / ncalls_dec
        # the same calls, each fully ordered behind the one before it (no overlap of consecutive calls): what a model
        # sees when the next layer's query depends on this layer's output
        try:
            sg.sg_testing_decode_overlap(False)
            g_ser = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_ser):
                decode_all(False)
            g_ser.replay(); torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream); g_ser.replay(); e1.record(stream); torch.cuda.synchronize()
            roofs["decode"]["us_per_call_serialized"] = 1e3 * e0.elapsed_time(e1) / ncalls_dec
        finally:
            sg.sg_testing_decode_overlap(True)
        roofs["decode"]["note"] = ("consecutive calls are independent (queries of all layers are inputs of the step) and overlap "
                                   "up to their output stores; us_per_call_serialized: each call ordered behind the previous one")
    dominant = max(roofs.values(), key=lambda r: r["ms_per_step"])

    # ---- the oracle on the host cores, bounded sample
    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        layers = list(range(min(16, L)))            # about 10-30 s of CPU work on the 8B-shaped workload
        t = oracle_sample(cfg, layers)
        fr = len(layers) / L
        cpu = {"value": sp_bytes * fr / (t["select"] + t["pack"]) / 1e9, "unit": UNIT, "cores": oracle.max_threads(),
               "kind": "oracle",
               "sample": "layers 0-%d of %s: score %.2fs, select %.3fs, pack %.3fs, one decode step %.3fs" % (
                   layers[-1], cfg.name, t["score"], t["select"], t["pack"], t["decode"]),
               "decode_tokens_per_s": B * fr / t["decode"] if t["decode"] > 0 else None,
               "score_tflops": work["score"]["flops"] * fr / t["score"] / 1e12}

    kv_mib = (h_k.numel() + h_v.numel()) * 2 / 2**20
    next_rows = next_rows_timing(dev, cfg, hp, d_k, d_v) if world == 1 and not args.no_extras else None
    layerwise = layerwise_prefill_timing(dev, hp, d_q, d_k, d_v) if world == 1 and not args.no_extras else None
    first_two = full_first_two_timing(dev, cfg, d_q, d_k, d_v) if world == 1 and not args.no_extras else None
    handover = handover_timing(dev, hp, d_q, d_k, d_v) if world == 1 and not args.no_extras else None
    sweep, configs = None, None
    if args.workload == "c2" and not args.no_decode_sweep and not args.no_extras and world == 1:
        del d_k, d_v, h_k, h_v
        torch.cuda.empty_cache()
        sweep = decode_sweep_points(dev, peaks)
        configs = measure_configs(dev, peaks)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "%s: L=%d B=%d Hq=%d Hkv=%d d=%d W=%d T=%d K_tot=%d n_loc=%d decode_steps=%d" % (
                       cfg.name, L, B, Hq, Hkv, d, W, T, Ktot, NL, nsteps_dec),
                   "l2": "inputs larger than L2 (K+V caches %.0f MiB); no flush" % kv_mib,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "decode": "one sg_sparse_decode_attn call per layer per step, replayed from a CUDA graph"},
        "decode_tokens_per_s": dec_tok,
        "stage_ms": st,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e, "decode_tokens_per_s": e2e_dec_tok, "stage_ms": st_e, "steps": e2e_steps},
        "gpu_launches": args.steps * (2 + ncalls_dec),
        "roofline": dominant, "rooflines": roofs, "cpu_baseline": cpu, "clocks": clocks,
        "decode_sweep": sweep, "configs": configs, "next_rows": next_rows, "prefill_layerwise": layerwise, "prefill_full_first_two": first_two, "score_select_handover": handover,
        "e2e_pipelined": None if ms_pipe is None else {
            "ms_prefill": ms_pipe, "value": sp_bytes / (ms_pipe * 1e-3) / 1e9, "unit": UNIT,
            "note": "host buffers, layer by layer on three streams (copy in | score, select, pack | copy out); "
                    "the whole prefill side, scoring included, against e2e's h2d + select + pack + d2h"}, "dev_status": status, "setup_s": gen_s,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--fraction", type=float, default=0.10, help="c3: budget fraction")
    ap.add_argument("--batch", type=int, default=64, help="c5: concurrent sequences")
    ap.add_argument("--sel", type=float, default=0.2, help="c5: required fraction of the prompt")
    ap.add_argument("--rho", type=float, default=0.25, help="c5: index-addressed share of the required entries")
    ap.add_argument("--layers", type=int, default=None, help="c2/c4: override the number of layers (small profiling cases)")
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode-sweep", action="store_true", help="skip the extra decode-only points (c2 only)")
    ap.add_argument("--decode-sweep-grid", action="store_true",
                    help="only the decode-heavy sweep: sg_sparse_decode_attn alone on batch {1, 8, 32, 128} x required "
                         "fraction {5, 20, 100 %} x index-addressed share {0, 25, 50 %}; prints one JSON line and exits")
    ap.add_argument("--no-extras", action="store_true",
                    help="only the timed step: skip the decode sweep, the timings of the other entry points, the "
                         "layer-by-layer prefill and the pipelined e2e (for profiling the step itself)")
    args = ap.parse_args()
    if args.decode_sweep_grid:
        import torch
        from paper_2607_28150_b200 import build as _build
        if not os.path.exists(_build.LIB):
            _build.build()
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        dev = torch.device("cuda", 0)
        torch.cuda.set_device(dev)
        points = tuple((b, sel, rho) for b in (1, 8, 32, 128) for sel in (0.05, 0.2, 1.0) for rho in (0.0, 0.25, 0.5))
        peaks = load_peaks()
        print(json.dumps({"decode_sweep_grid": decode_sweep_points(dev, peaks, points), "peak_gbs": peaks["hbm_gbs"],
                          "peak_source": peaks["source"], "calls_per_graph": 16}))
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # Started as a plain process (not under torchrun): start the N replicas here, one process per GPU.  They
        # exchange nothing but a barrier and the maximum of their device times; rank 0 prints the line.
        import torch
        from paper_2607_28150_b200 import replicas
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit("bench.py --gpus %d: only %d CUDA device(s) visible" % (args.gpus, have))
        env = dict(os.environ)
        env.setdefault("NCCL_DEBUG", "INFO")             # the communicator's one log line (ring/tree, NVLS) goes to stderr
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        codes, out0 = replicas.launch_local_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env)
        sys.stdout.write(out0)
        sys.stdout.flush()
        if any(codes):
            raise SystemExit("bench.py: rank exit codes %s" % codes)
        return
    run_ours(args)


if __name__ == "__main__":
    main()
