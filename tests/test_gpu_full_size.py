"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.

The oracle cannot run a whole workload, so float stages are checked on sampled units, the discrete stages
(budgets everywhere; selection and compaction on sampled or all units) under the stage protocol, and
size-independent properties are checked on every unit with plain tensor operations."""
import numpy as np
import pytest
import torch

import parity
from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _properties(wl, K, V, out):
    """Hold at any size: offsets are the prefix sum of budgets and end at the global budget; every unit's
    indices are strictly ascending, in range, and end with the window; compacted rows are the source rows."""
    bud = out.budgets.reshape(-1).long()
    off = out.offsets
    assert int(off[0]) == 0 and int(off[-1]) == wl.total_rows
    assert torch.equal(off[1:] - off[:-1], bud)
    assert int(bud.min()) >= wl.w and int(bud.max()) <= wl.N
    per_layer = bud.view(wl.B * wl.L, wl.H).sum(dim=1)
    assert bool((per_layer == wl.H * wl.avg_budget).all())
    idx = out.indices.long()
    assert int(idx.min()) >= 0 and int(idx.max()) == wl.N - 1
    unit_of_row = torch.repeat_interleave(torch.arange(wl.units, device=idx.device), bud)
    same_unit = unit_of_row[1:] == unit_of_row[:-1]
    assert bool(((idx[1:] > idx[:-1]) | ~same_unit).all())
    last = off[1:] - 1
    win = torch.arange(wl.w, device=idx.device)
    got = idx[(last[:, None] - (wl.w - 1 - win)[None, :])]
    assert torch.equal(got, (wl.N - wl.w + win)[None, :].expand(wl.units, -1))
    Kf, Vf = K.reshape(wl.units * wl.N, wl.d), V.reshape(wl.units * wl.N, wl.d)
    src = unit_of_row * wl.N + idx
    step = 1 << 20
    for a in range(0, src.numel(), step):
        assert torch.equal(out.Kc[a:a + step], Kf[src[a:a + step]])
        assert torch.equal(out.Vc[a:a + step], Vf[src[a:a + step]])
    # entropy bounds of the appendix: 0 <= H_k <= ln k
    assert float(out.entropy.min()) >= -1e-6 and float(out.entropy.max()) <= np.log(wl.k_trunc) + 1e-5


@pytest.mark.parametrize("name,n_float,n_select", [("c2", 6, 256), ("c3", 4, 256), ("c4", 3, 48), ("c5", 2, 24)])
def test_full_size_workload(name, n_float, n_select):
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.WORKLOADS[name]
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    assert cp.status() == 0
    _properties(wl, K, V, out)
    rng = np.random.default_rng(wl.seed)
    fl = sorted(rng.choice(wl.units, size=n_float, replace=False).tolist())
    if name == "c3":
        fl[0] = 0            # layer 0, head 0 is the near-isotropic unit of its layer
    sel = list(range(wl.units)) if n_select >= wl.units else sorted(rng.choice(wl.units, size=n_select, replace=False).tolist())
    parity.check_entropy(wl, K, out.entropy, out.erank, fl)
    parity.check_budgets(wl, out.erank, out.budgets, out.offsets, out.layer_group, out.layer_ctx)
    parity.check_scores(wl, K, Qw, out.scores, fl[:2])
    parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, sel)
    parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, fl)
    # the near-isotropic heads of c3 must have been given the largest budgets of their layer
    if name == "c3":
        b = out.budgets.cpu().numpy()[0]
        for l in range(wl.L):
            assert b[l, l % 8] == b[l].max()
    del K, V, Qw, cp, out
    torch.cuda.empty_cache()


def test_full_size_wide_entropy_hidden_states():
    """Hidden-state shape of the 8B models (D = 4096) at 8192 tokens, the size `bench.py --path wide` times: the
    entropy and the 32 largest eigenvalues against the oracle, plus properties that hold at any size."""
    import oracle
    from paper_2410_03090_b200 import binding as ub
    N, D, k = 8192, 4096, 32
    g = torch.Generator(device="cuda").manual_seed(11)
    W = torch.randn(256, D, generator=g, device="cuda") * (torch.arange(1, 257, device="cuda") ** -0.7)[:, None]
    X = (torch.randn(N, 256, generator=g, device="cuda") @ W + 0.05 * torch.randn(N, D, generator=g, device="cuda") + 0.3
         ).to(torch.bfloat16)[None]
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "bf16"))
    ent, er, spec = ub.uncomp_entropy_wide(ctx, X, k, spectrum=True)
    ent1, _, spec1 = ub.uncomp_entropy_wide(ctx, X, k, norm=1, spectrum=True)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    H, E, lam = oracle.entropy_wide(X[0].double().cpu().numpy(), k, return_spectrum=True)
    got = spec[0].cpu().numpy()
    assert np.abs(got - lam[:k]).max() <= 1e-4 * lam[0]
    assert abs(float(ent[0]) - H) <= parity.ENTROPY_RTOL * max(abs(H), 1.0)
    assert abs(float(er[0]) - E) <= 2e-4 * E
    # descending, non-negative, H_k <= ln k, same bits on a second run, whole-trace normalisation gives less entropy mass
    assert (np.diff(got) <= 0).all() and got[-1] > 0 and 0.0 <= float(ent[0]) <= np.log(k) + 1e-6
    assert torch.equal(spec, spec1) and float(ent1[0]) != float(ent[0])
    H1 = oracle.truncated_entropy(lam, k, 1)[0]
    assert abs(float(ent1[0]) - H1) <= parity.ENTROPY_RTOL * max(abs(H1), 1.0)
