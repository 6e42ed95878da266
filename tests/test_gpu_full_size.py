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


@pytest.mark.parametrize("name,n_float,n_select", [("c2", 8, 256), ("c3", 8, 256), ("c4", 8, 64), ("c5", 8, 32)])
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
    parity.check_scores(wl, K, Qw, out.scores, fl)          # the oracle runs these units on a thread pool
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


def test_full_size_hidden_state_eviction():
    """The configuration `bench.py --path hidden` times (B4, 32 query / 8 KV heads, N 32768, D 4096, keep half):
    scores of one sequence against the oracle, selection and gathered rows of every sequence."""
    import oracle
    from paper_2410_03090_b200 import binding as ub
    wl = synth.scaled(synth.WORKLOADS["c3"], L=1, B=4)
    D, n_keep = 4096, wl.N // 2
    K, _, Qw = synth.generate(wl, "cuda")
    Kl, q = K[:, 0], Qw[:, 0, :, -1, :].contiguous()
    X = synth.hidden_states(wl, D, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, 1, wl.H, wl.Hq, wl.N, wl.d, 1, wl.dtype))
    scores = torch.empty(wl.B, wl.N - 1, device="cuda")
    idx, Xout = ub.uncomp_evict_hidden(ctx, q, Kl, X, n_keep, scores=scores)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    ref = oracle.last_token_scores(q[1].double().cpu().numpy(), Kl[1].double().cpu().numpy())
    got = scores[1].double().cpu().numpy()
    assert (np.abs(got - ref[:-1]) <= parity.SCORE_RTOL * np.abs(ref[:-1]) + 1e-12 * ref.max()).all()
    assert abs(ref.sum() - wl.Hq) < 1e-9                         # every head's attention sums to one
    for b in range(wl.B):
        want = oracle.select(scores[b].double().cpu().numpy(), 1, n_keep)
        np.testing.assert_array_equal(idx[b].cpu().numpy(), want)
        assert torch.equal(Xout[b], X[b][idx[b].long()])


def test_full_size_decode_update_after_prefill():
    """The state `bench.py --path decode` starts from (the compressed cache of workload c3 after its prefill pass):
    three decode steps, sampled units against the oracle, invariants on all units."""
    import oracle
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.WORKLOADS["c3"]
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    o = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    offs = o.offsets.cpu().numpy()
    g = torch.Generator(device="cuda").manual_seed(3)
    cum = torch.rand(wl.total_rows, generator=g, device="cuda")
    pos, lens = o.indices.clone(), o.budgets.reshape(-1).clone()
    Kc, Vc = o.Kc.clone(), o.Vc.clone()
    max_cap = int(lens.max())
    sample = [0, 7, 100, 255]
    for step in range(3):
        qn = Qw[:, :, :, -1 - step, :].contiguous()
        kn, vn = K[:, :, :, -1 - step, :].contiguous(), V[:, :, :, -1 - step, :].contiguous()
        before = {u: (Kc[offs[u]:offs[u + 1]].double().cpu().numpy(), pos[offs[u]:offs[u + 1]].cpu().numpy(),
                      cum[offs[u]:offs[u + 1]].cpu().numpy()) for u in sample}
        pos_all = pos.clone()
        p = torch.empty(wl.total_rows + wl.units, device="cuda")
        ev = torch.empty(wl.units, dtype=torch.int32, device="cuda")
        npos = torch.full((wl.B,), wl.N + step, dtype=torch.int32, device="cuda")
        ub.uncomp_decode_update(cp.ctx, qn, kn, vn, npos, o.offsets, lens, max_cap, Kc, Vc, pos, cum, p=p, evicted=ev)
        torch.cuda.synchronize()
        assert cp.status() == 0
        for u in sample:
            Kb, pb, cb = before[u]
            n = len(pb)
            ref = oracle.decode_probs(qn.view(wl.units, wl.G, wl.d)[u].double().cpu().numpy(), Kb,
                                      kn.view(wl.units, wl.d)[u].double().cpu().numpy())
            got = p[offs[u] + u:offs[u] + u + n + 1].cpu().numpy()
            assert (np.abs(got - ref) <= parity.SCORE_RTOL * np.abs(ref) + 1e-12 * ref.max()).all()
            slot = oracle.decode_evict((cb + got[:n]).astype(np.float64), pb, wl.N + step, 1)
            assert int(ev[u]) == int(pb[slot]) and int(pos[offs[u] + slot]) == wl.N + step
            assert torch.equal(Kc[offs[u] + slot], kn.view(wl.units, wl.d)[u])
        # every unit: full caches stay full, exactly one position per unit changed, the evicted one is gone
        assert torch.equal(lens, o.budgets.reshape(-1))
        changed = (pos != pos_all).cpu().numpy()
        assert changed.sum() == wl.units and (np.add.reduceat(changed, offs[:-1]) == 1).all()
        assert (pos[torch.from_numpy(changed).cuda()] == wl.N + step).all()
