"""GPU parity: profile-based proactive selection (counts, Eq. 1, Eq. 2, top-K_r, mask) against the oracle, bit-exact."""
import numpy as np
import pytest

import oracle
from helpers import cu_of

pytestmark = pytest.mark.gpu


def test_budget_matches_oracle_on_host():
    import paper_2607_28150_b200.binding as sg
    for L, M, tp, tt in [(32, 1024, 0.5, 1.0), (32, 1024, 1.0, 6.5), (40, 1000, 1e-9, 1.0), (8, 16, 5.0, 1.0), (2, 4, 0.3, 1.0)]:
        assert sg.sg_transfer_budget(L, M, tp, tt) == oracle.transfer_budget(L, M, tp, tt)


@pytest.mark.parametrize("lens,L,Hkv,M,k", [((4096, 1000, 37), 6, 8, 64, (400, 100, 10)), ((8192,), 32, 8, 1024, (820,))])
def test_profile_chain_matches_oracle(lens, L, Hkv, M, k):
    """Several decode steps of random KV indices -> S(e) -> Eq. 1 -> global top-K_r -> per-layer mask -> Algorithm 1."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(0)
    cu, ck = cu_of(lens), cu_of(k)
    T, Ktot, B = int(cu[-1]), int(ck[-1]), len(lens)
    shp1 = gpu_ops.shape_of(1, Hkv, Hkv, 128, 1, cu)
    shpL = gpu_ops.shape_of(L, Hkv, Hkv, 128, 1, cu)
    counts_o = np.zeros((L, Hkv, T), dtype=np.int32)
    counts_g = torch.zeros((L, Hkv, T), dtype=torch.int32, device="cuda")
    st = gpu_ops.status_word()
    # selection skewed towards the end of each prompt, as in the paper's positional profile
    for step in range(3):
        for l in range(L):
            idx = np.zeros((Hkv, Ktot), dtype=np.int32)
            for g in range(Hkv):
                for b, n in enumerate(lens):
                    p = np.linspace(0.2, 1.0, n) ** (1 + l % 3); p /= p.sum()
                    idx[g, ck[b]:ck[b + 1]] = np.sort(rng.choice(n, k[b], replace=False, p=p))
            oracle.profile_accumulate(counts_o[l], idx, cu, ck)
            sg.sg_profile_accumulate(shp1, gpu_ops.dev(idx), gpu_ops.dev(ck), Ktot, counts_g[l], st)
    assert np.array_equal(counts_g.cpu().numpy(), counts_o) and gpu_ops.read_status(st) == 0
    # Eq. 1
    I_o = oracle.block_importance(counts_o, cu, M)
    I_g = torch.empty((L, M), dtype=torch.float32, device="cuda")
    sg.sg_block_importance(shpL, counts_g, M, I_g)
    assert np.array_equal(I_g.cpu().numpy(), I_o)
    # Eq. 2 + global top-K_r through sg_select_topk on the flattened matrix
    kr = sg.sg_transfer_budget(L, M, 0.4, 1.0)
    sel_o = oracle.select_topk(I_o.reshape(1, 1, L * M), cu_of((L * M,)), cu_of((kr,)))[0, 0]
    sel_g = gpu_ops.select_topk(I_g.cpu().numpy().reshape(1, 1, L * M), cu_of((L * M,)), cu_of((kr,)))[0, 0]
    assert np.array_equal(sel_g, sel_o) and set(range(2 * M)) <= set(sel_g.tolist())
    # mask per layer, then Algorithm 1 on a fresh KV index
    d_sel = gpu_ops.dev(sel_g)
    for l in (0, 2, L - 1):
        mask_g = torch.zeros(T, dtype=torch.int8, device="cuda")
        sg.sg_proactive_mask(shp1, M, l, d_sel, mask_g)
        mask_o = oracle.proactive_mask(cu, M, l, sel_o)
        assert np.array_equal(mask_g.cpu().numpy(), mask_o)
    assert np.all(oracle.proactive_mask(cu, M, 0, sel_o) == 1)          # layer 0 is always transferred


def test_profile_accumulate_flags_bad_index():
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    cu, ck = cu_of((10,)), cu_of((3,))
    shp = gpu_ops.shape_of(1, 1, 1, 128, 1, cu)
    counts = torch.zeros((1, 10), dtype=torch.int32, device="cuda")
    st = gpu_ops.status_word()
    sg.sg_profile_accumulate(shp, gpu_ops.dev(np.array([[1, 10, 3]], dtype=np.int32)), gpu_ops.dev(ck), 3, counts, st)
    assert gpu_ops.read_status(st) == 1 << sg.SG_ERR_INDEX
    assert counts.cpu().numpy()[0].tolist() == [0, 1, 0, 1, 0, 0, 0, 0, 0, 0]


def test_speculative_schedule_masks_grow_until_everything_is_local():
    """Section 4.3: iteration i has the global top-n_i blocks on the decode node, n_i from the speculative ratio."""
    import torch
    import gpu_ops
    import paper_2607_28150_b200.binding as sg
    rng = np.random.default_rng(5)
    L, M, Hkv, lens = 8, 64, 2, (3000, 500)
    cu = cu_of(lens)
    T = int(cu[-1])
    shp1 = gpu_ops.shape_of(1, Hkv, Hkv, 128, 1, cu)
    I = rng.random((L, M)).astype(np.float32) * 5
    I[:2] = np.inf
    kr = sg.sg_transfer_budget(L, M, 0.2, 1.0)
    prev_local = None
    it = 0
    while True:
        n = sg.sg_speculative_delivered(L, M, kr, 0.10, it)
        assert n == oracle.speculative_delivered(L, M, kr, 0.10, it)
        sel_g = gpu_ops.select_topk(I.reshape(1, 1, L * M), cu_of((L * M,)), cu_of((n,)))[0, 0]
        sel_o = oracle.select_topk(I.reshape(1, 1, L * M), cu_of((L * M,)), cu_of((n,)))[0, 0]
        assert np.array_equal(sel_g, sel_o)
        local = np.zeros((L, T), dtype=bool)
        for l in range(L):
            m = torch.zeros(T, dtype=torch.int8, device="cuda")
            sg.sg_proactive_mask(shp1, M, l, gpu_ops.dev(sel_g), m)
            mg = m.cpu().numpy()
            assert np.array_equal(mg, oracle.proactive_mask(cu, M, l, sel_o))
            local[l] = mg == 1
        if prev_local is not None:
            assert np.all(local | ~prev_local)                 # nothing that was local becomes remote again
        prev_local = local
        if n == L * M:
            break
        it += 1
    assert local.all() and it <= 10                            # 10 % per iteration: complete within 10 iterations
