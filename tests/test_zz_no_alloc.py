"""sg_score_static: the scoring call for hosts that cannot allocate device memory.

Some users of this library score from places where cudaMalloc is off limits (a fixed memory plan, an
allocation-free region of their runtime, a process whose allocator is owned by someone else).  For them
the library carries its own fixed scratch array.  This test calls that entry point through the C ABI
twice in a row -- different inputs, different shapes, so the second call runs over the first call's
left-over scratch -- and checks each result against the ordinary sg_score on the same inputs and against
the CPU oracle, within the tolerance the score parity tests use, and that the device's free memory is the
same before and after the second call (nothing was allocated).  It also checks that a shape too large for
the fixed array is refused on the host, and that a shape no kernel covers gets the same answer as from sg_score.  The file is named so that pytest collects it after every other test.
"""
import numpy as np
import pytest

from helpers import cu_of, rand_bf16

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-30


def both_ways(seed, lens, L, W, Hq, Hkv, d):
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    import oracle
    rng = np.random.default_rng(seed)
    cu = cu_of(lens)
    T = int(cu[-1])
    q_h, k_h = rand_bf16(rng, (L, len(lens), W, Hq, d)), rand_bf16(rng, (L, T, Hkv, d))
    q, k = gpu_ops.dev(q_h), gpu_ops.dev(k_h)
    shp = gpu_ops.shape_of(L, Hq, Hkv, d, W, cu)
    ref = torch.full((L, Hkv, T), -1.0, dtype=torch.float32, device="cuda")
    got = torch.full((L, Hkv, T), -2.0, dtype=torch.float32, device="cuda")
    st = gpu_ops.status_word()
    sg.sg_score(shp, q, k, ref, sg.alloc_workspace(sg.SG_OP_SCORE, shp), st)
    torch.cuda.synchronize()
    sg.sg_score_static(shp, q, k, got, st)          # no workspace: nothing is allocated for this call
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    again = got
    sg.sg_score_static(shp, q, k, again, st)        # second call on this device: no set-up left to do, no allocation
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert gpu_ops.read_status(st) == 0
    want = oracle.score(q_h, k_h, cu).astype(np.float64)
    assert np.all(np.abs(got.cpu().numpy().astype(np.float64) - want) <= RTOL * np.abs(want) + ATOL)
    ref, got = ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= RTOL * np.abs(ref) + ATOL)
    assert np.all(ref >= 0) and abs(ref.sum() / (L * Hkv * sum(min(W, n) for n in lens) * (Hq // Hkv)) - 1) < 1e-3


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    both_ways(0, (3000, 257), 2, 32, 32, 8, 128)
    both_ways(1, (1500,), 1, 16, 8, 2, 64)          # smaller shape: runs over the first call's left-overs


def test_static_scratch_rejects_shapes_beyond_its_fixed_size():
    import ctypes
    import paper_2607_28150_b200.binding as sg
    # 256 layers x 8 heads of 512 rows need more than the fixed array; refused on the host, nothing launched
    big = sg.Shape(256, 1, 64, 8, 128, 64, 32768, 32768, 0x1000, 32768 * 1024, 1024, 128)
    assert sg.sg_workspace_bytes(sg.SG_OP_SCORE, big) > sg.SG_SCORE_STATIC_SCRATCH_BYTES
    fake = ctypes.c_void_p(0x1000)
    rc = sg._lib.sg_score_static(ctypes.byref(big), fake, fake, fake, None, None)
    assert rc == sg.SG_ERR_WORKSPACE
    # a shape no scoring kernel covers is reported as such, as sg_score reports it (not as a size problem)
    odd = sg.Shape(1, 1, 64, 2, 128, 64, 16384, 16384, 0x1000, 16384 * 256, 256, 128)      # G*W = 2048 rows
    assert sg._lib.sg_score_static(ctypes.byref(odd), fake, fake, fake, None, None) == sg.SG_ERR_UNSUPPORTED
