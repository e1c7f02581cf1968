"""GPU: a bounded device-side wait of the scoring kernel is made to run out, on purpose and harmlessly.

The test withholds the done-count of one (layer, KV head) unit through the library's testing hook and shortens every
wait to 10 ms.  The pass-2 work items of that unit then wait for a count that never comes; the wait gives up, the CTA
sets SG_ERR_TIMEOUT in the status word, waits (bounded) for its own copies and MMAs, frees its tensor memory and
returns.  Nothing traps, nothing spins without a limit, and the context stays usable: an ordinary sg_score call right
afterwards matches the oracle.
"""
import time

import numpy as np
import pytest

import oracle
from helpers import cu_of, rand_bf16

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_cleanly_and_the_next_call_is_correct():
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(5)
    L, Hq, Hkv, d, W = 6, 8, 2, 128, 16
    lens = (5000, 700)
    cu = cu_of(lens)
    T = int(cu[-1])
    q_h, k_h = rand_bf16(rng, (L, len(lens), W, Hq, d)), rand_bf16(rng, (L, T, Hkv, d))
    q, k = gpu_ops.dev(q_h), gpu_ops.dev(k_h)
    shp = gpu_ops.shape_of(L, Hq, Hkv, d, W, cu)
    ws = sg.alloc_workspace(sg.SG_OP_SCORE, shp)
    imp = torch.zeros((L, Hkv, T), dtype=torch.float32, device="cuda")
    st = gpu_ops.status_word()
    try:
        sg.sg_testing_score_fault(withhold_unit=3, wait_limit_ms=10)
        t0 = time.perf_counter()
        sg.sg_score(shp, q, k, imp, ws, st)
        torch.cuda.synchronize()                      # returns: every wait in the kernel is bounded
        elapsed = time.perf_counter() - t0
    finally:
        sg.sg_testing_score_fault(-1, 0)
    assert gpu_ops.read_status(st) & (1 << sg.SG_ERR_TIMEOUT)
    assert elapsed < 5.0, "a 10 ms limit must end the call within a few waits, took %.2f s" % elapsed
    # the context is intact: the same call without the hook is correct and raises nothing
    st2 = gpu_ops.status_word()
    imp.fill_(-1.0)
    sg.sg_score(shp, q, k, imp, ws, st2)
    torch.cuda.synchronize()
    assert gpu_ops.read_status(st2) == 0
    want = oracle.score(q_h, k_h, cu)
    got = imp.cpu().numpy()
    assert np.all(np.abs(got - want) <= 1e-4 * np.abs(want) + 1e-30)


def test_in_kernel_clock_record_is_plausible():
    """The measurement hook: every CTA of the scoring kernel records its start/end clock64 and globaltimer; the ratio
    is the SM clock the kernel ran at, which must lie between a few hundred MHz and the part's maximum."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(6)
    L, Hq, Hkv, d, W = 8, 32, 8, 128, 32
    cu = cu_of((8192,))
    q = gpu_ops.dev(rand_bf16(rng, (L, 1, W, Hq, d)))
    k = gpu_ops.dev(rand_bf16(rng, (L, 8192, Hkv, d)))
    shp = gpu_ops.shape_of(L, Hq, Hkv, d, W, cu)
    ws = sg.alloc_workspace(sg.SG_OP_SCORE, shp)
    imp = torch.empty((L, Hkv, 8192), dtype=torch.float32, device="cuda")
    grid = sg.sg_testing_score_grid(shp)
    assert 1 <= grid <= 148
    buf = torch.zeros(32 * grid, dtype=torch.int64, device="cuda")
    try:
        sg.sg_testing_score_clock(buf)
        sg.sg_score(shp, q, k, imp, ws, None)
        torch.cuda.synchronize()
    finally:
        sg.sg_testing_score_clock(None)
    rec = buf.cpu().numpy()[: 4 * grid].reshape(grid, 4).astype(np.float64)
    cycles, ns = rec[:, 1] - rec[:, 0], rec[:, 3] - rec[:, 2]
    assert np.all(cycles > 0) and np.all(ns > 0)
    mhz = 1e3 * np.median(cycles / ns)
    assert 300.0 < mhz < 2200.0, mhz
