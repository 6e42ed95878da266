"""Parity of the CUDA library against the CPU oracle, stage by stage, through the C ABI.

Tolerances (written out in tests/parity.py): entropies 1e-4 relative (floor |H| = 1), window scores 2e-3
relative; budgets, selected indices and compacted rows bit-exact under the stage protocol (the oracle's
rule applied to the GPU's own erank / pooled scores)."""
import numpy as np
import pytest
import torch

import parity
from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _ub():
    from paper_2410_03090_b200 import binding
    return binding


def _run(wl, **kw):
    from paper_2410_03090_b200.compress import CompressionPass
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw, **kw)
    torch.cuda.synchronize()
    assert cp.status() == 0
    return K, V, Qw, cp, out


def _check_all(wl, K, V, Qw, out, units, **bkw):
    parity.check_entropy(wl, K, out.entropy, out.erank, units)
    parity.check_budgets(wl, out.erank, out.budgets, out.offsets, out.layer_group, out.layer_ctx, **bkw)
    parity.check_scores(wl, K, Qw, out.scores, units)
    parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, range(wl.units))
    parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, units)
    assert int(out.offsets[-1]) == wl.total_rows


def test_config1_fp32_whole_pass():
    wl = synth.WORKLOADS["c1"]
    K, V, Qw, cp, out = _run(wl)
    _check_all(wl, K, V, Qw, out, range(wl.units))


@pytest.mark.parametrize("name,N,L", [("c2", 1000, 2), ("c3", 2309, 8), ("c5", 1536, 1)])
def test_bf16_small_whole_pass(name, N, L):
    # several token tiles and a ragged tail; c3 includes its near-isotropic head, c5 has G = 8, w = 64
    wl = synth.scaled(synth.WORKLOADS[name], N=N, L=L)
    K, V, Qw, cp, out = _run(wl, eps=0.3, dn=256, n_last=512)
    _check_all(wl, K, V, Qw, out, range(0, wl.units, 3), eps=0.3, dn=256, n_last=512)


def test_c4_batch_with_norm_spikes():
    wl = synth.scaled(synth.WORKLOADS["c4"], N=1280, L=1, B=2)
    K, V, Qw, cp, out = _run(wl)
    _check_all(wl, K, V, Qw, out, range(0, wl.units, 2))


def test_spectrum_matches_oracle_eigenvalues():
    import oracle
    ub = _ub()
    wl = synth.WORKLOADS["c1"]
    K, _, _ = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    spec = torch.empty(wl.B, wl.L, wl.H, 128, dtype=torch.float64, device="cuda")
    ent, er = ub.uncomp_entropy(ctx, K, k_trunc=128, norm=1, spectrum=spec)
    torch.cuda.synchronize()
    for u in range(wl.units):
        H, E, lam = oracle.entropy(parity.unit_np(K, wl, u), k_trunc=128, norm=1, return_spectrum=True)
        got = spec.reshape(-1, 128)[u].cpu().numpy()
        np.testing.assert_allclose(got, lam, rtol=0, atol=1e-11 * lam[0])
        assert abs(float(ent.reshape(-1)[u]) - H) <= 1e-4 * max(abs(H), 1.0)


@pytest.mark.parametrize("k_trunc,center,norm", [(16, 1, 0), (64, 0, 0), (32, 1, 1), (200, 0, 1)])
def test_entropy_variants(k_trunc, center, norm):
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=777, L=1)
    K, _, _ = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    ent, er = ub.uncomp_entropy(ctx, K, k_trunc=k_trunc, center=center, norm=norm)
    torch.cuda.synchronize()
    parity.check_entropy(wl, K, ent, er, range(wl.units), k_trunc=k_trunc, center=center, norm=norm)


def test_entropy_closed_forms_on_device():
    # rank-1 keys -> H = 0; +-a e_i rows -> H = ln m   (Appendix, proof of the entropy bounds)
    ub = _ub()
    N, H = 256, 2
    K = torch.zeros(1, 1, H, N, 128, device="cuda", dtype=torch.float32)
    g = torch.Generator(device="cuda").manual_seed(5)
    u = torch.randn(N, 1, generator=g, device="cuda")
    v = torch.randn(1, 128, generator=g, device="cuda")
    K[0, 0, 0] = u @ v
    m = 8
    for i in range(m):
        K[0, 0, 1, 2 * i, i] = 1.5
        K[0, 0, 1, 2 * i + 1, i] = -1.5
    ctx = ub.Context(ub.make_shape(1, 1, H, H, N, 128, 8, "fp32"))
    ent, er = ub.uncomp_entropy(ctx, K, k_trunc=32)
    torch.cuda.synchronize()
    assert abs(float(ent[0, 0, 0])) < 1e-6 and abs(float(er[0, 0, 0]) - 1.0) < 1e-6
    assert abs(float(ent[0, 0, 1]) - np.log(m)) < 1e-6 and abs(float(er[0, 0, 1]) - m) < 1e-5


@pytest.mark.parametrize("scope,M,avg,n_max", [(0, 8, 100, 160), (1, 8, 100, 160), (0, 3, 77, 120), (1, 5, 64, 96),
                                               (0, 1, 50, 50), (1, 24, 200, 360)])
def test_budget_variants_bit_exact(scope, M, avg, n_max):
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=3, B=2)
    g = torch.Generator(device="cuda").manual_seed(3)
    er = torch.rand(wl.B, wl.L, wl.H, generator=g, device="cuda") * 30 + 1
    er[0, 1, 2] = er[0, 1, 5]
    er[1, 0, 0] = er[1, 2, 7]
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    b, o, lg, lc = ub.uncomp_assign_budgets(ctx, er, avg, M, n_max, scope, eps=0.25, dn=64, n_last=128)
    torch.cuda.synchronize()
    parity.check_budgets(wl, er, b, o, lg, lc, M=M, avg=avg, n_max=n_max, scope=scope, eps=0.25, dn=64, n_last=128)
    assert int(b.sum()) == wl.units * avg


def test_budget_prefix_sum_beyond_one_block():
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=40, B=5)      # 1600 units > 1024 threads
    g = torch.Generator(device="cuda").manual_seed(4)
    er = torch.rand(wl.B, wl.L, wl.H, generator=g, device="cuda") * 30 + 1
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    b, o, lg, lc = ub.uncomp_assign_budgets(ctx, er, 100, 8, 160, 1)
    torch.cuda.synchronize()
    parity.check_budgets(wl, er, b, o, lg, lc, M=8, avg=100, n_max=160, scope=1)


@pytest.mark.parametrize("w,G,N,pool,mode", [(1, 1, 300, 1, 0), (8, 4, 515, 7, 0), (32, 2, 1027, 5, 1),
                                             (64, 8, 700, 7, 0), (17, 3, 401, 13, 1)])
def test_scorer_shapes(w, G, N, pool, mode):
    ub = _ub()
    base = synth.scaled(synth.WORKLOADS["c2"], N=N, L=1)
    from dataclasses import replace
    wl = replace(base, w=w, Hq=base.H * G, avg_budget=w + 40, n_max=w + 40, M=1, pool_kernel=pool, pool_mode=mode)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, 1, wl.n_max)
    scores = torch.empty(wl.B, wl.L, wl.H, N - w, device="cuda")
    idx = ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, pool, mode, 0.0, scores)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    parity.check_scores(wl, K, Qw, scores, range(wl.units))
    parity.check_select(wl, scores, b, o, idx, range(wl.units))
    # mass conservation: probabilities of a row sum to one, so the prefix mass is at most G * w
    if pool == 1:
        assert float(scores.sum(-1).max()) <= G * w * (1 + 1e-4)


@pytest.mark.parametrize("avg_kind", ["window_only", "one", "everything"])
def test_select_extreme_budgets(avg_kind):
    ub = _ub()
    from dataclasses import replace
    base = synth.scaled(synth.WORKLOADS["c2"], N=600, L=1)
    avg = {"window_only": base.w, "one": base.w + 1, "everything": base.N}[avg_kind]
    wl = replace(base, avg_budget=avg, n_max=avg, M=1)
    K, V, Qw, cp, out = _run(wl)
    parity.check_select(wl, out.scores, out.budgets, out.offsets, out.indices, range(wl.units))
    parity.check_compact(wl, K, V, out.indices, out.offsets, out.Kc, out.Vc, range(wl.units))
    if avg_kind == "everything":
        assert torch.equal(out.Kc.view(wl.units, wl.N, wl.d), K.view(wl.units, wl.N, wl.d))


def test_select_ties_take_lowest_positions():
    # all keys equal -> every prefix score is equal -> the first k positions are kept
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=400, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    K[:] = K[:, :, :, :1, :]
    from paper_2410_03090_b200.compress import CompressionPass
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    off = out.offsets.cpu().numpy()
    bud = out.budgets.reshape(-1).cpu().numpy()
    idx = out.indices.cpu().numpy()
    for u in range(wl.units):
        k = bud[u] - wl.w
        seg = idx[off[u]:off[u + 1]]
        assert seg.tolist() == list(range(k)) + list(range(wl.N - wl.w, wl.N))


def test_strided_inputs_and_determinism():
    # K / V as views of a larger [L, B, H, N, 2, d] buffer (interleaved K and V), two runs bit-identical
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS["c2"], N=640, L=2, B=2)
    K0, V0, Qw = synth.generate(wl, "cuda")
    big = torch.empty(wl.L, wl.B, wl.H, wl.N, 2, wl.d, dtype=K0.dtype, device="cuda")
    big[..., 0, :] = K0.permute(1, 0, 2, 3, 4)
    big[..., 1, :] = V0.permute(1, 0, 2, 3, 4)
    K = big[..., 0, :].permute(1, 0, 2, 3, 4)
    V = big[..., 1, :].permute(1, 0, 2, 3, 4)
    assert not K.is_contiguous()
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    first = [t.clone() for t in (out.entropy, out.budgets, out.scores, out.indices, out.Kc, out.Vc)]
    cp2 = CompressionPass(wl, "cuda")
    ref = cp2.run(K0, V0, Qw)
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    for a, b, c in zip(first, (out.entropy, out.budgets, out.scores, out.indices, out.Kc, out.Vc),
                       (ref.entropy, ref.budgets, ref.scores, ref.indices, ref.Kc, ref.Vc)):
        assert torch.equal(a, b) and torch.equal(a, c)
    _check_all(wl, K0, V0, Qw, out, range(0, wl.units, 5))


def test_host_side_rejections_and_status_word():
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    shape = ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype)
    ctx = ub.Context(shape)
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")

    def code(fn, *a, **k):
        with pytest.raises(ub.UncompError) as ei:
            fn(*a, **k)
        return ei.value.code

    assert code(ub.uncomp_entropy, ctx, K, k_trunc=0) == ub.UNCOMP_E_PARAM
    assert code(ub.uncomp_entropy, ctx, K.view(-1)[1:1 + 8 * 511 * 128].view(1, 1, 8, 511, 128)) == ub.UNCOMP_E_ALIGN
    assert code(ub.uncomp_assign_budgets, ctx, er, 100, 9, 160) == ub.UNCOMP_E_PARAM       # M > heads
    assert code(ub.uncomp_assign_budgets, ctx, er, 16, 8, 20) == ub.UNCOMP_E_PARAM         # avg < w
    assert code(ub.uncomp_assign_budgets, ctx, er, 100, 8, 190) == ub.UNCOMP_E_PARAM       # smallest target < w
    assert code(ub.uncomp_assign_budgets, ctx, er, 100, 8, 1000) == ub.UNCOMP_E_PARAM      # n_max > N
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, 100, 8, 160)
    assert code(ub.uncomp_score_select, ctx, Qw, K, b, o, wl.units * 100, pool_kernel=4) == ub.UNCOMP_E_PARAM
    # a workspace that is too small is refused at creation
    import ctypes as C
    h = C.c_void_p()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert ub.lib.uncomp_create(C.byref(h), C.byref(shape), C.c_void_p(small.data_ptr()), 1024) == ub.UNCOMP_E_WORKSPACE
    # device-side conditions arrive through the status word and leave the context usable
    ub.uncomp_entropy(ctx, K, max_iters=1)
    assert ub.uncomp_status(ctx) & ub.UNCOMP_STATUS_NOT_CONVERGED
    ent, _ = ub.uncomp_entropy(ctx, K)
    assert ub.uncomp_status(ctx) == 0
    parity.check_entropy(wl, K, ent, _, [0, 5])


@pytest.mark.parametrize("unit,value", [(3, "N+5"), (7, "N+5"), (7, "w-3"), (4, "0"), (2, "50"), (0, "-9")])
def test_bad_budget_stays_inside_its_slab(unit, value):
    # A budget that disagrees with its slab (too large, below the window, negative, or just different) is reported
    # and cut to the slab; the last unit is the one that would run off the end of d_indices.  The index buffer has
    # a guard region behind it that no case may touch, and it is sized so that even a unit writing N entries from
    # its offset would stay inside the allocation.
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, 100, 1, 100)
    total = wl.units * 100
    buf = torch.full((total + 2 * wl.N,), -7, dtype=torch.int32, device="cuda")
    scores = torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, device="cuda")
    bad = b.clone()
    bad.view(-1)[unit] = {"N+5": wl.N + 5, "w-3": wl.w - 3, "0": 0, "50": 50, "-9": -9}[value]
    ub.uncomp_score_select(ctx, Qw, K, bad, o, total, scores=scores, indices=buf[:total])
    assert ub.uncomp_status(ctx) == ub.UNCOMP_STATUS_BOUNDS
    assert bool((buf[total:] == -7).all())
    idx = buf[:total]
    parity.check_select(wl, scores, b, o, idx, [u for u in range(wl.units) if u != unit])
    slab = idx[unit * 100:(unit + 1) * 100].cpu().numpy()
    assert slab.min() >= 0 and slab.max() <= wl.N - 1          # every slot holds a valid position
    want = min(max(int(bad.view(-1)[unit]), 0), 100)
    if want >= wl.w:                                           # as much of the selection as budget and slab allow
        import oracle
        ref = oracle.select(scores.view(wl.units, -1)[unit].double().cpu().numpy(), wl.w, want)
        np.testing.assert_array_equal(slab[:want], ref)
    assert (slab[want:] == wl.N - 1).all()
    # the compaction of such a slab reads valid rows only
    Kc, Vc = ub.uncomp_compact(ctx, K, V, idx, o, total)
    assert ub.uncomp_status(ctx) == 0
    parity.check_compact(wl, K, V, idx, o, Kc, Vc, [unit])


def test_bad_offsets_write_nothing_outside_and_bad_indices_are_clamped():
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, 100, 1, 100)
    total = wl.units * 100
    scores = torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, device="cuda")
    for case in ("shifted", "negative", "beyond_end"):
        o2 = o.clone()
        if case == "shifted":
            o2[5] = 450                  # unit 4 gets 50 slots for a budget of 100, unit 5 gets 150
        elif case == "negative":
            o2[0] = -300
        else:
            o2[7] = total + 40           # unit 6 would end, and unit 7 start, beyond offsets[units]
        buf = torch.full((total + 2 * wl.N,), -7, dtype=torch.int32, device="cuda")
        ub.uncomp_score_select(ctx, Qw, K, b, o2, total, scores=scores, indices=buf[:total])
        assert ub.uncomp_status(ctx) == ub.UNCOMP_STATUS_BOUNDS, case
        assert bool((buf[total:] == -7).all()), case
        touched = {"shifted": (4, 5), "negative": (0,), "beyond_end": (6, 7)}[case]
        parity.check_select(wl, scores, b, o, buf[:total], [u for u in range(wl.units) if u not in touched])
        written = buf[:total][buf[:total] != -7]
        assert int(written.min()) >= 0 and int(written.max()) <= wl.N - 1, case
    # compaction: an index outside [0, N) is replaced by the nearest valid row and reported
    idx = ub.uncomp_score_select(ctx, Qw, K, b, o, total, scores=scores)
    assert ub.uncomp_status(ctx) == 0
    Kc0, Vc0 = ub.uncomp_compact(ctx, K, V, idx, o, total)
    hurt = idx.clone()
    hurt[250], hurt[251] = -1, wl.N                      # rows 50 and 51 of unit 2
    Kc, Vc = ub.uncomp_compact(ctx, K, V, hurt, o, total)
    assert ub.uncomp_status(ctx) == ub.UNCOMP_STATUS_BOUNDS
    keep = torch.ones(total, dtype=torch.bool, device="cuda")
    keep[250:252] = False
    assert torch.equal(Kc[keep], Kc0[keep]) and torch.equal(Vc[keep], Vc0[keep])
    assert torch.equal(Kc[250], K[0, 0, 2, 0]) and torch.equal(Kc[251], K[0, 0, 2, wl.N - 1])
    assert torch.equal(Vc[250], V[0, 0, 2, 0]) and torch.equal(Vc[251], V[0, 0, 2, wl.N - 1])


def _gram_oracle(K_unit_np):
    import oracle
    G = oracle.covariance(K_unit_np, center=False)
    return G, K_unit_np.sum(axis=0)


@pytest.mark.parametrize("N", [128, 200, 1000, 4096 + 77])
def test_gram_known_answer_integers(N):
    # integer-valued bf16 keys: every product and partial sum is exact in fp32, so the tensor-core Gram
    # must equal the oracle's X^T X and column sums exactly (this pins operand layout, swizzle and tiling)
    ub = _ub()
    H = 3
    g = torch.Generator(device="cuda").manual_seed(N)
    K = torch.randint(-3, 4, (1, 1, H, N, 128), generator=g, device="cuda").to(torch.bfloat16)
    K[0, 0, 1, :, 5] = 1.0          # a constant feature: its column sum is N
    K[0, 0, 2, N - 1, :] = 7.0      # the last token must be counted once
    ctx = ub.Context(ub.make_shape(1, 1, H, H, N, 128, 8, "bf16"))
    gram = ub.uncomp_gram(ctx, K)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    for u in range(H):
        G, s = _gram_oracle(K[0, 0, u].double().cpu().numpy())
        got = gram[u].cpu().numpy()
        np.testing.assert_array_equal(got[:128 * 128].reshape(128, 128), G)
        np.testing.assert_array_equal(got[128 * 128:], s)


def test_gram_tensor_core_vs_cuda_core_and_oracle():
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c3"], N=5000, L=2)
    K, _, _ = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    g_tc = ub.uncomp_gram(ctx, K).clone()
    ub.uncomp_set_option(ctx, ub.UNCOMP_OPT_CUDA_CORES, 1)
    g_cc = ub.uncomp_gram(ctx, K).clone()
    torch.cuda.synchronize()
    scale = g_cc[:, :128 * 128].abs().amax(dim=1, keepdim=True)
    assert float(((g_tc - g_cc).abs() / scale).max()) < 2e-6
    for u in (0, 9):
        G, s = _gram_oracle(parity.unit_np(K, wl, u))
        got = g_tc[u].cpu().numpy()
        assert np.abs(got[:128 * 128].reshape(128, 128) - G).max() <= 2e-6 * np.abs(G).max()
        assert np.abs(got[128 * 128:] - s).max() <= 2e-6 * np.abs(np.diag(G)).max() ** 0.5 * wl.N ** 0.5 + 1e-3


@pytest.mark.parametrize("name,N", [("c2", 3000), ("c3", 4500), ("c5", 2100)])
def test_scorer_tensor_core_vs_cuda_core(name, N):
    # the two implementations of the same definition must agree far inside the oracle tolerance
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS[name], N=N, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.ones(wl.B, wl.L, wl.H, device="cuda")
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, 1, wl.avg_budget)
    s_tc = torch.empty(wl.B, wl.L, wl.H, N - wl.w, device="cuda")
    s_cc = torch.empty_like(s_tc)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, 1, 0, 0.0, s_tc)
    ub.uncomp_set_option(ctx, ub.UNCOMP_OPT_CUDA_CORES, 1)
    ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, 1, 0, 0.0, s_cc)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    rel = ((s_tc - s_cc).abs() / (s_cc.abs() + 1e-12 * s_cc.amax(dim=-1, keepdim=True))).max()
    assert float(rel) < 5e-4, float(rel)


def test_bf16_spectrum_register_kernel_vs_oracle():
    # bf16 keys take the fp32 register-resident eigen kernel: its top-k spectrum against the oracle's
    # Jacobi eigenvalues (tolerance of an fp32 reduction: 2e-6 of the largest eigenvalue)
    import oracle
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c5"], N=3000, L=2)
    K, _, _ = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    spec = torch.empty(wl.B, wl.L, wl.H, 128, dtype=torch.float64, device="cuda")
    ent, er = ub.uncomp_entropy(ctx, K, k_trunc=128, norm=1, spectrum=spec)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    for u in range(0, wl.units, 3):
        H, E, lam = oracle.entropy(parity.unit_np(K, wl, u), k_trunc=128, norm=1, return_spectrum=True)
        got = spec.reshape(-1, 128)[u].cpu().numpy()
        np.testing.assert_allclose(got, lam, rtol=0, atol=2e-6 * lam[0])
        assert abs(float(ent.reshape(-1)[u]) - H) <= 1e-4 * max(abs(H), 1.0)


def test_fused_entropy_statistics_sweep_matches_separate_calls():
    # uncomp_entropy with the window queries forms the Gram matrices and the scorer's row statistics in one
    # sweep over K; everything downstream must agree with the two-sweep path
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS["c3"], N=9001, L=2)          # two scorer chunks, ragged tail
    K, V, Qw = synth.generate(wl, "cuda")
    outs = []
    for fused in (True, False):
        cp = CompressionPass(wl, "cuda", fused=fused)
        o = cp.run(K, V, Qw)
        torch.cuda.synchronize()
        assert cp.status() == 0
        outs.append({k: getattr(o, k).clone() for k in ("entropy", "budgets", "scores", "indices", "Kc", "Vc")})
    f, u = outs
    assert float((f["entropy"] - u["entropy"]).abs().max()) < 2e-6
    assert torch.equal(f["scores"], u["scores"])                   # same statistics, bit for bit
    if torch.equal(f["budgets"], u["budgets"]):
        assert torch.equal(f["indices"], u["indices"]) and torch.equal(f["Kc"], u["Kc"]) and torch.equal(f["Vc"], u["Vc"])
    _check_all(wl, K, V, Qw, CompressionPass(wl, "cuda", fused=True).run(K, V, Qw), range(0, wl.units, 5))


def test_fused_gram_is_exact_on_integer_keys():
    # integer-valued keys: every Gram partial is exact in fp32 whatever the chunking, so the fused sweep and the
    # stand-alone Gram kernel (itself pinned against the oracle exactly) must give identical spectra
    ub = _ub()
    N, H, G, w = 8192 + 300, 4, 2, 16
    g = torch.Generator(device="cuda").manual_seed(11)
    K = torch.randint(-3, 4, (1, 1, H, N, 128), generator=g, device="cuda").to(torch.bfloat16)
    Qw = torch.randn(1, 1, H * G, w, 128, generator=g, device="cuda").to(torch.bfloat16)
    ctx = ub.Context(ub.make_shape(1, 1, H, H * G, N, 128, w, "bf16"))
    spec_f = torch.empty(1, 1, H, 128, dtype=torch.float64, device="cuda")
    spec_u = torch.empty_like(spec_f)
    ent_f, _ = ub.uncomp_entropy(ctx, K, k_trunc=128, spectrum=spec_f, Qw=Qw)
    ent_f = ent_f.clone()
    ent_u, _ = ub.uncomp_entropy(ctx, K, k_trunc=128, spectrum=spec_u)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    assert torch.equal(spec_f, spec_u) and torch.equal(ent_f, ent_u)


@pytest.mark.parametrize("N,w,G", [(65, 64, 4), (33, 32, 1), (130, 2, 8), (129, 1, 2)])
def test_degenerate_lengths(N, w, G):
    # prefix of one token, sequences shorter than / just above one 128-token tile, single-row windows
    from dataclasses import replace
    from paper_2410_03090_b200.compress import CompressionPass
    base = synth.scaled(synth.WORKLOADS["c2"], N=max(N, 256), L=1)
    P = N - w
    avg = w + max(1, P // 2)
    wl = replace(base, N=N, w=w, Hq=base.H * G, avg_budget=avg, n_max=avg, M=1, name=f"tiny{N}")
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    assert cp.status() == 0
    _check_all(wl, K, V, Qw, out, range(wl.units))


def test_scores_may_stay_in_the_workspace():
    # d_scores = NULL: the pooled scores live in the workspace; selection must be unchanged
    ub = _ub()
    wl = synth.scaled(synth.WORKLOADS["c2"], N=900, L=1)
    K, V, Qw = synth.generate(wl, "cuda")
    ctx = ub.Context(ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype))
    er = torch.linspace(30, 2, wl.H, device="cuda").view(1, 1, wl.H).contiguous()
    b, o, _, _ = ub.uncomp_assign_budgets(ctx, er, wl.avg_budget, wl.M, wl.n_max)
    scores = torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, device="cuda")
    idx_a = ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=scores).clone()
    idx_b = ub.uncomp_score_select(ctx, Qw, K, b, o, wl.total_rows, scores=None)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0 and torch.equal(idx_a, idx_b)
    parity.check_select(wl, scores, b, o, idx_b, range(wl.units))


@pytest.mark.parametrize("units,N,w,budget", [(1, 9000, 32, 700), (4, 32768, 64, 5000), (8, 4200, 8, 4100), (3, 20001, 16, 16)])
def test_select_with_few_units_takes_the_cluster_kernel_and_matches_oracle(units, N, w, budget):
    """Few units and a long prefix: the selection runs as a cluster of CTAs per unit; same answer, bit for bit."""
    import oracle
    from paper_2410_03090_b200 import binding as ub
    g = torch.Generator(device="cuda").manual_seed(units * 7 + N)
    K = torch.randn(1, 1, units, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    Qw = torch.randn(1, 1, units, w, 128, generator=g, device="cuda").to(torch.bfloat16)
    dup = torch.arange(0, N - 1, 7, device="cuda")
    K[:, :, :, dup] = K[:, :, :, dup + 1]                      # duplicated keys: exact score ties
    ctx = ub.Context(ub.make_shape(1, 1, units, units, N, 128, w, "bf16"))
    budgets = torch.full((1, 1, units), budget, dtype=torch.int32, device="cuda")
    offsets = (torch.arange(units + 1, device="cuda") * budget).to(torch.int64)
    scores = torch.empty(1, 1, units, N - w, device="cuda")
    idx = torch.empty(units * budget, dtype=torch.int32, device="cuda")
    ub.uncomp_score_select(ctx, Qw, K, budgets, offsets, units * budget, 7, 0, 0.0, scores, idx)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    for u in range(units):
        want = oracle.select(scores[0, 0, u].double().cpu().numpy(), w, budget)
        np.testing.assert_array_equal(idx[u * budget:(u + 1) * budget].cpu().numpy(), want)
