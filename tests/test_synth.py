"""The workload generator: determinism, shapes and the structure the recipe promises."""
import numpy as np
import torch

from paper_2410_03090_b200 import synth


def test_workload_table_matches_configs():
    w = synth.WORKLOADS
    assert (w["c1"].N, w["c1"].H, w["c1"].w, w["c1"].dtype, w["c1"].avg_budget) == (512, 8, 32, "fp32", 128)
    assert (w["c2"].L, w["c2"].Hq, w["c2"].N, w["c2"].avg_budget, w["c2"].n_max) == (32, 32, 8192, 410, 683)
    assert (w["c3"].N, w["c3"].w, w["c3"].avg_budget, w["c3"].n_max) == (32768, 64, 1540, 2567)
    assert (w["c4"].B, w["c4"].avg_budget, w["c4"].n_max) == (4, 3080, 5133)
    assert (w["c5"].L, w["c5"].Hq, w["c5"].N, w["c5"].avg_budget, w["c5"].n_max) == (80, 64, 131072, 2621, 4368)
    for wl in w.values():
        assert 2 * wl.avg_budget - wl.n_max >= wl.w      # smallest group target stays above the window


def test_units_are_reproducible_and_independent():
    wl = synth.scaled(synth.WORKLOADS["c2"], N=256, L=2)
    K, V, Q = synth.generate(wl)
    assert K.shape == (1, 2, 8, 256, 128) and Q.shape == (1, 2, 32, 32, 128) and K.dtype == torch.bfloat16
    k, v, q = synth.generate_unit(wl, 0, 1, 3)
    assert torch.equal(K[0, 1, 3], k) and torch.equal(V[0, 1, 3], v) and torch.equal(Q[0, 1, 12:16], q)
    assert not torch.equal(K[0, 0, 0], K[0, 0, 1])


def test_low_rank_structure_and_spikes():
    wl = synth.WORKLOADS["c1"]
    for h in (0, 2):
        k, _, _ = synth.generate_unit(wl, 0, 0, h)
        s = torch.linalg.svdvals(k.double())
        r = 1 << h
        assert s[r - 1] / s[0] > 1e-2 and s[r] / s[0] < 1e-3          # rank 2**h plus 1e-3 noise
    c4 = synth.scaled(synth.WORKLOADS["c4"], N=2048, L=1, B=2)
    m0, m1 = synth.spike_positions(c4, 0), synth.spike_positions(c4, 1)
    assert 5 <= int(m0.sum()) <= 50 and not torch.equal(m0, m1)
    k, _, _ = synth.generate_unit(c4, 0, 0, 0, spikes=m0)
    norms = k.float().norm(dim=1)
    assert norms[m0].mean() > 5 * norms[~m0].mean()
    c3 = synth.scaled(synth.WORKLOADS["c3"], N=1024, L=2)
    assert synth.unit_alpha(c3, 1, 1) == 0.0 and synth.unit_alpha(c3, 1, 2) == 2.0
