"""`uncomp_compress`: the whole pass in one call.  With the caller's log-sum-exp the keys are swept ONCE: the
column-sum scorer and the Gram stage of the entropy run in the same kernel.  Every stage is checked against the
oracle exactly as for the staged calls (stage protocol), over shapes with one to four blocks of window rows, ragged
tiles, strided keys, fp32 keys (which take the staged path) and the call without normalisers."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import parity
from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _lse(wl, K, Qw):
    lse = torch.zeros(wl.B, wl.L, wl.Hq, wl.w, dtype=torch.float32)
    for u, v in parity.oracle_lse(wl, K, Qw, range(wl.units)).items():
        b, l, h = synth.unit_index(wl, u)
        lse[b, l, h * wl.G:(h + 1) * wl.G] = torch.from_numpy(v.astype(np.float32))
    return lse.cuda()


def _check(wl, K, V, Qw, out, units):
    parity.check_entropy(wl, K, out.entropy, out.erank, units)
    parity.check_budgets(wl, out.erank, out.budgets, out.offsets, out.layer_group, out.layer_ctx)
    parity.check_scores(wl, K, Qw, out.scores, units)
    parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, range(wl.units))
    parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, units)


@pytest.mark.parametrize("w,G,N,L", [(32, 4, 1000, 2), (64, 4, 2309, 2), (64, 6, 1111, 1), (64, 8, 1536, 1), (8, 1, 129, 3),
                                     (17, 3, 8200, 1)])
def test_one_sweep_with_caller_lse_matches_the_oracle(w, G, N, L):
    from paper_2410_03090_b200.compress import CompressionPass
    base = synth.scaled(synth.WORKLOADS["c3"], N=N, L=L)
    wl = replace(base, w=w, Hq=base.H * G, avg_budget=max(w + 16, base.avg_budget), n_max=max(w + 16, base.avg_budget),
                 M=1) if w != base.w or G != base.G else base
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    lse = _lse(wl, K, Qw)
    from paper_2410_03090_b200 import binding as ub
    ub.uncomp_profile_enable(cp.ctx, True)
    out = cp.run_one_call(K, V, Qw, lse=lse)
    torch.cuda.synchronize()
    prof = ub.uncomp_profile_read(cp.ctx)
    ub.uncomp_profile_enable(cp.ctx, False)
    assert cp.status() == 0
    # one sweep: the fused kernel ran once; neither the stand-alone Gram nor any statistics or column-sum kernel did
    assert prof["gram_score_colsum"][1] == 1
    assert all(prof[n][1] == 0 for n in ("gram", "score_stats", "gram_score_stats", "score_colsum"))
    _check(wl, K, V, Qw, out, range(0, wl.units, 3))
    # and a second time on the same context: nothing stale
    first = [t.clone() for t in (out.entropy, out.scores, out.indices, out.Kc)]
    out = cp.run_one_call(K, V, Qw, lse=lse)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(first, (out.entropy, out.scores, out.indices, out.Kc)))


def test_one_call_without_lse_equals_the_staged_calls_bit_for_bit():
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS["c3"], N=2309, L=3)
    K, V, Qw = synth.generate(wl, "cuda")
    a, b = CompressionPass(wl, "cuda"), CompressionPass(wl, "cuda")
    oa = a.run(K, V, Qw, eps=0.3, dn=256, n_last=512)
    ob = b.run_one_call(K, V, Qw, eps=0.3, dn=256, n_last=512)
    torch.cuda.synchronize()
    assert a.status() == 0 and b.status() == 0
    for name in ("entropy", "erank", "budgets", "offsets", "layer_group", "layer_ctx", "scores", "indices", "Kc", "Vc"):
        assert torch.equal(getattr(oa, name), getattr(ob, name)), name


def test_one_call_on_strided_keys_and_on_fp32_keys():
    from paper_2410_03090_b200.compress import CompressionPass
    # strided views: K and V are slices of wider buffers (token stride 160 elements)
    wl = synth.scaled(synth.WORKLOADS["c2"], N=900, L=1)
    K0, V0, Qw = synth.generate(wl, "cuda")
    wide = torch.zeros(wl.B, wl.L, wl.H, wl.N, 160, dtype=K0.dtype, device="cuda")
    wide[..., :128] = K0
    K = wide[..., :128]
    cp = CompressionPass(wl, "cuda")
    out = cp.run_one_call(K, V0, Qw, lse=_lse(wl, K0, Qw))
    torch.cuda.synchronize()
    assert cp.status() == 0
    _check(wl, K0, V0, Qw, out, range(wl.units))
    # fp32 keys have no tensor-core scorer: the call falls back to the staged schedule, normalisers still honoured
    wl32 = synth.WORKLOADS["c1"]
    K, V, Qw = synth.generate(wl32, "cuda")
    cp = CompressionPass(wl32, "cuda")
    out = cp.run_one_call(K, V, Qw, lse=_lse(wl32, K, Qw))
    torch.cuda.synchronize()
    assert cp.status() == 0
    _check(wl32, K, V, Qw, out, range(wl32.units))


def test_one_call_rejections():
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS["c2"], N=640, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    o = cp.out
    lse = torch.zeros(wl.B, wl.L, wl.Hq, wl.w, device="cuda")
    args = dict(entropy=o.entropy, erank=o.erank, budgets=o.budgets, offsets=o.offsets, layer_group=None,
                layer_ctx=None, scores=None, indices=o.indices, Kc=o.Kc, Vc=o.Vc, lse=lse)
    with pytest.raises(ub.UncompError) as ei:            # k_trunc < 1
        ub.uncomp_compress(cp.ctx, K, V, Qw, (0, 1, 0, 0), (wl.avg_budget, wl.M, wl.n_max, 0, 0.0, 0, 0), (7, 0, 0.0), **args)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:            # even pooling window
        ub.uncomp_compress(cp.ctx, K, V, Qw, (32, 1, 0, 0), (wl.avg_budget, wl.M, wl.n_max, 0, 0.0, 0, 0), (6, 0, 0.0), **args)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:            # budget below the window
        ub.uncomp_compress(cp.ctx, K, V, Qw, (32, 1, 0, 0), (wl.w - 1, wl.M, wl.n_max, 0, 0.0, 0, 0), (7, 0, 0.0), **args)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:            # one of the two layer outputs missing
        ub.uncomp_compress(cp.ctx, K, V, Qw, (32, 1, 0, 0), (wl.avg_budget, wl.M, wl.n_max, 0, 0.0, 0, 0), (7, 0, 0.0),
                           **dict(args, layer_group=o.layer_group))
    assert ei.value.code == ub.UNCOMP_E_NULL
    # scores may stay in the workspace
    ub.uncomp_compress(cp.ctx, K, V, Qw, (32, 1, 0, 0), (wl.avg_budget, wl.M, wl.n_max, 0, 0.0, 0, 0), (7, 0, 0.0),
                       **dict(args, lse=parity_lse(wl, K, Qw)))
    torch.cuda.synchronize()
    assert cp.status() == 0


def parity_lse(wl, K, Qw):
    return _lse(wl, K, Qw)
