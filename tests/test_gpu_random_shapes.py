"""Seeded sweep of the whole pass over random shapes (heads, grouped query heads, window, sequence length with ragged
tiles, layers, batch, budget, number of groups): every stage against the oracle, as in the fixed-shape parity tests."""
import random
from dataclasses import replace

import pytest
import torch

import parity
from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _shape(rng, it, dtype="bf16"):
    H = rng.choice([1, 2, 4, 8])
    w = rng.choice([8, 16, 32, 64])
    G = min(rng.choice([1, 2, 4, 8]), 512 // w)
    lengths = [w + 9, 129, 257, 1000, 1537, 4097, 6000, 9001] if dtype == "bf16" else [w + 9, 129, 257, 700, 1537]
    N = max(rng.choice(lengths), w + 9)
    L, B = rng.choice([1, 2, 3]), rng.choice([1, 2])
    P = N - w
    avg = rng.randint(w + 1, max(w + 1, min(N - 1, w + P // 2)))
    M = rng.choice([m for m in (1, 2, 4, 8) if m <= H])
    n_max = min(N, max(avg, min(2 * avg - w, int(round(5 * avg / 3)))))
    return replace(synth.WORKLOADS["c2"], name=f"rnd{it}", B=B, L=L, H=H, Hq=H * G, N=N, w=w, avg_budget=avg, M=M,
                   n_max=n_max, seed=1000 + it, dtype=dtype)


@pytest.mark.parametrize("seed,dtype,count", [(1, "bf16", 12), (7, "bf16", 12), (3, "fp32", 8)])
def test_random_shapes(seed, dtype, count):
    from paper_2410_03090_b200.compress import CompressionPass
    rng = random.Random(seed)
    for it in range(count):
        wl = _shape(rng, it, dtype)
        K, V, Qw = synth.generate(wl, "cuda")
        cp = CompressionPass(wl, "cuda")
        out = cp.run(K, V, Qw)
        torch.cuda.synchronize()
        assert cp.status() == 0, wl
        units = sorted({0, wl.units // 2, wl.units - 1})
        parity.check_entropy(wl, K, out.entropy, out.erank, units)
        parity.check_budgets(wl, out.erank, out.budgets, out.offsets, out.layer_group, out.layer_ctx)
        parity.check_scores(wl, K, Qw, out.scores, units[:2])
        parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, range(wl.units))
        parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, units)
        del cp, out, K, V, Qw
        torch.cuda.empty_cache()
