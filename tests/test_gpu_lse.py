"""The scorer with caller-supplied row normalisers (`d_lse` of uncomp_score_select): one sweep over K.

The log-sum-exp of a window row is what a prefill attention kernel keeps per row.  Here it comes from the oracle
(fp64, rounded to the fp32 the ABI takes); the scores must then hold the same 2e-3 tolerance against the oracle's
window scores as the two-sweep form, and the selection must follow from them bit for bit."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import parity
from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _ub():
    from paper_2410_03090_b200 import binding
    return binding


def _lse_tensor(wl, K, Qw, units=None, scale=None):
    """[B, L, Hq, w] float32: the oracle's log-sum-exp for `units` (all by default)."""
    units = range(wl.units) if units is None else units
    lse = torch.zeros(wl.B, wl.L, wl.Hq, wl.w, dtype=torch.float32)
    for u, v in parity.oracle_lse(wl, K, Qw, units, scale).items():
        b, l, h = synth.unit_index(wl, u)
        lse[b, l, h * wl.G:(h + 1) * wl.G] = torch.from_numpy(v.astype(np.float32))
    return lse.cuda()


def _device_lse(wl, K, Qw):
    """Stand-in for the prefill attention kernel's per-row log-sum-exp where the oracle would take too long: a plain
    fp32 matrix product and logsumexp on the device.  It is an INPUT of the call under test, never an expected value."""
    P = wl.N - wl.w
    out = torch.empty(wl.B, wl.L, wl.Hq, wl.w, dtype=torch.float32, device=K.device)
    pos = torch.arange(wl.N, device=K.device)[None, :]
    row_last = (P + torch.arange(wl.w, device=K.device))[:, None]
    for b in range(wl.B):
        for l in range(wl.L):
            for h in range(wl.H):
                q = Qw[b, l, h * wl.G:(h + 1) * wl.G].float()                       # [G, w, d]
                s = torch.einsum("gwd,nd->gwn", q, K[b, l, h].float()) / wl.d ** 0.5
                s = s.masked_fill((pos > row_last)[None], float("-inf"))
                out[b, l, h * wl.G:(h + 1) * wl.G] = torch.logsumexp(s, dim=-1)
    return out


@pytest.mark.parametrize("w,G,N,pool,mode", [(1, 1, 300, 1, 0), (8, 4, 515, 7, 0), (32, 2, 1027, 5, 1),
                                             (64, 8, 700, 7, 0), (17, 3, 401, 13, 1)])
@pytest.mark.parametrize("dtype,cuda_cores", [("bf16", False), ("bf16", True), ("fp32", False)])
def test_scorer_shapes_with_caller_lse(w, G, N, pool, mode, dtype, cuda_cores):
    ub = _ub()
    base = synth.scaled(synth.WORKLOADS["c2"], N=N, L=1)
    wl = replace(base, w=w, Hq=base.H * G, avg_budget=w + 40, n_max=w + 40, M=1, pool_kernel=pool, pool_mode=mode,
                 dtype=dtype)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    if cuda_cores:
        ub.uncomp_set_option(ctx, ub.UNCOMP_OPT_CUDA_CORES, 1)
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, 1, wl.n_max)
    lse = _lse_tensor(wl, K, Qw)
    scores = torch.empty(wl.B, wl.L, wl.H, N - w, device="cuda")
    idx = ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, pool, mode, 0.0, scores, lse=lse)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    parity.check_scores(wl, K, Qw, scores, range(wl.units))
    parity.check_select(wl, scores, b, o, idx, range(wl.units))
    # only the statistics sweep is gone: no score_stats launch, one column-sum launch
    ub.uncomp_profile_enable(ctx, True)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, pool, mode, 0.0, scores, lse=lse)
    prof = ub.uncomp_profile_read(ctx)
    ub.uncomp_profile_enable(ctx, False)
    assert prof["score_stats"][1] == 0 and prof["gram_score_stats"][1] == 0 and prof["score_colsum"][1] == 1


def test_custom_scale_with_lse_and_whole_pass_agrees_with_two_sweeps():
    from paper_2410_03090_b200.compress import CompressionPass
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c3"], N=2309, L=2)
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    two = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    two = [t.clone() for t in (two.entropy, two.budgets, two.scores, two.indices)]
    one = cp.run(K, V, Qw, lse=_lse_tensor(wl, K, Qw))
    torch.cuda.synchronize()
    assert cp.status() == 0
    units = range(0, wl.units, 3)
    parity.check_entropy(wl, K, one.entropy, one.erank, units)
    parity.check_budgets(wl, one.erank, one.budgets, one.offsets, one.layer_group, one.layer_ctx)
    parity.check_scores(wl, K, Qw, one.scores, units)
    parity.check_select(wl, one.scores, one.budgets, one.offsets, one.indices, range(wl.units))
    parity.check_compact(wl, K, V, one.indices, one.offsets, one.Kc, one.Vc, units)
    # same Gram summation order whether or not the statistics ride along? No: the fused sweep chunks differently,
    # so entropies agree to rounding only; scores of the two forms agree far inside the tolerance
    assert float((one.entropy - two[0]).abs().max()) < 1e-5
    rel = ((one.scores - two[2]).abs() / two[2].abs().clamp_min(1e-30)).max()
    assert float(rel) < 2e-4
    # a scale of the caller's own: the normalisers must be those of the same scaled logits
    ctx = cp.ctx
    scale = 0.05
    lse = _lse_tensor(wl, K, Qw, scale=scale)
    sc = torch.empty_like(one.scores)
    ub.uncomp_score_select(ctx, Qw, K, one.budgets, one.offsets, wl.total_rows, 7, 0, scale, sc, lse=lse)
    torch.cuda.synchronize()
    parity.check_scores(wl, K, Qw, sc, range(0, wl.units, 5), scale=scale)


def test_nonfinite_lse_is_reported_not_trapped():
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=640, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, 1, wl.avg_budget)
    lse = _lse_tensor(wl, K, Qw)
    good = torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, device="cuda")
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, 1, 0, 0.0, good, lse=lse)
    assert ub.uncomp_status(ctx) == 0
    for poison in (float("nan"), float("inf"), float("-inf")):
        bad = lse.clone()
        bad[0, 0, 5, 3] = poison                      # query head 5 belongs to KV head 1
        sc = torch.empty_like(good)
        idx = ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, 1, 0, 0.0, sc, lse=bad)
        assert ub.uncomp_status(ctx) == ub.UNCOMP_STATUS_NONFINITE
        assert torch.isfinite(sc).all() and int(idx.min()) >= 0 and int(idx.max()) == wl.N - 1
        # the poisoned row is left out of its unit, every other unit is untouched
        assert torch.equal(sc[0, 0, [0, 2, 3, 4, 5, 6, 7]], good[0, 0, [0, 2, 3, 4, 5, 6, 7]])
        assert bool((sc[0, 0, 1] <= good[0, 0, 1]).all()) and float((good[0, 0, 1] - sc[0, 0, 1]).sum()) > 0
    # the context stays usable
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, 1, 0, 0.0, good, lse=lse)
    assert ub.uncomp_status(ctx) == 0
    parity.check_scores(wl, K, Qw, good, [1], pool_kernel=1)


def test_reuse_flag_is_explicit_and_stale_statistics_are_not_picked_up_without_it():
    # statistics left by a fused entropy call are used only by a call that asks for them; a call that does not ask
    # recomputes, so keys rewritten in place in between are scored correctly
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=1500, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    ent, er = ub.uncomp_entropy(ctx, K, Qw=Qw)
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, wl.M, wl.n_max)
    K.mul_(0.5)                                                # same buffer, new contents
    sc = torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, device="cuda")
    ub.uncomp_profile_enable(ctx, True)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=sc)          # reuse_stats = 0
    prof = ub.uncomp_profile_read(ctx)
    assert prof["score_stats"][1] == 1
    parity.check_scores(wl, K, Qw, sc, [0, 5])
    # with the flag, after a fresh fused call, the sweep is skipped and the result is the same
    ub.uncomp_entropy(ctx, K, Qw=Qw)
    ub.uncomp_profile_read(ctx)
    sc2 = torch.empty_like(sc)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=sc2, reuse_stats=True)
    prof = ub.uncomp_profile_read(ctx)
    assert prof["score_stats"][1] == 0 and prof["score_colsum"][1] == 1
    parity.check_scores(wl, K, Qw, sc2, [0, 5])
    # the statistics are consumed: asking again without a new fused call recomputes
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=sc2, reuse_stats=True)
    assert ub.uncomp_profile_read(ctx)["score_stats"][1] == 1
    # switching kernel families in between drops them too
    ub.uncomp_entropy(ctx, K, Qw=Qw)
    ub.uncomp_set_option(ctx, ub.UNCOMP_OPT_CUDA_CORES, 1)
    ub.uncomp_set_option(ctx, ub.UNCOMP_OPT_CUDA_CORES, 0)
    ub.uncomp_profile_read(ctx)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=sc2, reuse_stats=True)
    assert ub.uncomp_profile_read(ctx)["score_stats"][1] == 1
    ub.uncomp_profile_enable(ctx, False)
    assert ub.uncomp_status(ctx) == 0
    parity.check_scores(wl, K, Qw, sc2, [3])


@pytest.mark.parametrize("name,n_units", [("c3", 6), ("c5", 4)])
def test_full_size_with_caller_lse(name, n_units):
    """Full-size workloads in the launch configuration the bench's `with_lse` record times: every unit gets a
    log-sum-exp (device-made for most, the oracle's for the sampled units), sampled units are compared."""
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.WORKLOADS[name]
    K, V, Qw = synth.generate(wl, "cuda")
    lse = _device_lse(wl, K, Qw)
    rng = np.random.default_rng(wl.seed + 17)
    units = sorted(rng.choice(wl.units, size=n_units, replace=False).tolist())
    for u, v in parity.oracle_lse(wl, K, Qw, units).items():
        b, l, h = synth.unit_index(wl, u)
        dev_v = lse[b, l, h * wl.G:(h + 1) * wl.G].double().cpu().numpy()
        assert np.abs(dev_v - v).max() < 1e-3          # the stand-in is a sane normaliser (not a parity claim)
        lse[b, l, h * wl.G:(h + 1) * wl.G] = torch.from_numpy(v.astype(np.float32)).cuda()
    cp = CompressionPass(wl, "cuda")
    for one_call in (False, True):          # the staged calls (two sweeps), then uncomp_compress (one sweep: the bench's form)
        out = cp.run_one_call(K, V, Qw, lse=lse) if one_call else cp.run(K, V, Qw, lse=lse)
        torch.cuda.synchronize()
        assert cp.status() == 0
        parity.check_scores(wl, K, Qw, out.scores, units)
        parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, units)
        parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, units[:2])
        assert int(out.offsets[-1]) == wl.total_rows
        if one_call:                         # its entropies come from Gram partials of the fused kernel
            parity.check_entropy(wl, K, out.entropy, out.erank, units)
            parity.check_budgets(wl, out.erank, out.budgets, out.offsets, out.layer_group, out.layer_ctx)
    del K, V, Qw, cp, out
    torch.cuda.empty_cache()
