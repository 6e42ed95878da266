"""Seeded random sweeps of the entry points around the pass (hidden-state eviction, decode-time update, wide entropy),
each case checked against the oracle by the helpers of the fixed-shape tests."""
import random

import numpy as np
import pytest

import test_gpu_decode as td
import test_gpu_evict as te
import test_gpu_wide as tw

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [3, 11])
def test_random_entry_points(seed):
    from paper_2410_03090_b200 import binding as ub
    rng = random.Random(seed)
    for it in range(10):
        H, G = rng.choice([1, 2, 4, 8]), rng.choice([1, 2, 4, 8, 16])
        B, L = rng.choice([1, 2, 3]), rng.choice([1, 2])
        dt = rng.choice(["bf16", "bf16", "fp32"])
        N = rng.choice([2, 3, 31, 32, 33, 255, 1024, 1025, 2047, 5000, 9000])
        te._case(B, L, H, H * G, N, 8 * rng.randint(1, 64), dt, rng.randint(1, N), layer=L - 1, seed=it)

        units = B * L * H
        mc = rng.choice([1, 7, 40, 1023, 1024, 1500, 3000])
        caps = np.array([rng.randint(1, mc) for _ in range(units)])
        caps[0] = mc
        lens = np.array([rng.choice([c, c, max(0, c - rng.randint(0, 3))]) for c in caps])
        ctx = ub.Context(ub.make_shape(B, L, H, H * G, 16384, 128, 32, dt))
        st = td.State(B, L, H, H * G, dt, caps, lens, seed=it, start_pos=6000)
        protect = rng.choice([1, 1, 2, 50])
        for _ in range(3):
            td._step_and_check(ub, ctx, st, mc, protect=protect)

        Nw, Dw = rng.choice([2, 5, 63, 64, 65, 130, 300, 777, 1500, 3000]), 64 * rng.randint(2, 24)
        X = tw._matrix(1, Nw, Dw, rng.randint(1, 40), rng.choice([0.05, 0.3]), seed=it)
        tw._check(ub, X, rng.choice([1, 8, 32, 64]), rng.choice([0, 1]), rng.choice([0, 1]))
