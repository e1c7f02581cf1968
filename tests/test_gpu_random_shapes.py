"""GPU parity on seeded random shapes: decode attention and the fused selection + gather against the oracle.
The hand-picked cases of the other files cover the code paths by construction; these catch what nobody thought of
(ragged batches, odd head counts, budgets from nothing to everything).  A longer run of the same generator
(a thousand shapes of each kind) passed during development."""
import numpy as np
import pytest

import test_gpu_decode as dec
import test_gpu_select_pack as sp

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(4))
def test_random_decode_shapes(seed):
    rng = np.random.default_rng(100 + seed)
    for _ in range(12):
        Hkv, G, d = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 8, 16])), int(rng.choice([64, 128]))
        B = int(rng.choice([1, 1, 2, 3, 4, 7, 16, 40]))
        lens = tuple(int(x) for x in rng.integers(1, 3000 if B <= 4 else 600, size=B))
        ks = tuple(int(rng.integers(0, n + 1)) for n in lens)
        nls = tuple(int(rng.integers(0, n - k + 1)) for n, k in zip(lens, ks))
        dec.compare(dec.build(int(rng.integers(1 << 30)), lens, ks, nls, G * Hkv, Hkv, d))


@pytest.mark.parametrize("seed", range(4))
def test_random_select_pack_shapes(seed):
    rng = np.random.default_rng(200 + seed)
    for _ in range(10):
        L, Hkv, d = int(rng.choice([1, 3, 20, 40])), int(rng.choice([2, 4, 8])), int(rng.choice([64, 128]))
        B = int(rng.choice([1, 2, 5]))
        lens = tuple(int(x) for x in rng.integers(1, int(rng.choice([300, 4096, 8192, 12000])) + 1, size=B))
        ks = tuple(int(rng.integers(0, n + 1)) for n in lens)
        L = max(1, min(L, int(3e8 / (sum(lens) * Hkv * d * 4))))      # keep the host-side cache under ~300 MB
        sp.check(*sp.case(int(rng.integers(1 << 30)), lens, ks, L, Hkv, d, ties=bool(rng.integers(2))))


@pytest.mark.parametrize("seed", range(3))
def test_random_score_shapes(seed):
    import test_gpu_score as sc
    rng = np.random.default_rng(300 + seed)
    done = 0
    while done < 25:
        Hkv, G, d = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 8, 16])), int(rng.choice([64, 128]))
        W = int(rng.choice([1, 3, 8, 16, 32, 64]))
        while G * W > (1024 if d == 64 else 512):          # row counts beyond the built tile shapes are refused by the call
            W //= 2
        B, L = int(rng.choice([1, 1, 2, 4])), int(rng.choice([1, 1, 2, 3, 9]))
        lens = tuple(int(x) for x in rng.integers(1, int(rng.choice([200, 900, 2500])) + 1, size=B))
        if L * sum(lens) * G * W * Hkv * d > 2e9:            # keep the oracle's share of the test short
            continue
        sc.run_random(int(rng.integers(1 << 30)), lens, L, W, G * Hkv, Hkv, d, kscale=float(rng.choice([1.0, 1.0, 3.0])))
        done += 1
