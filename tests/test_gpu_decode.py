"""Decode-time cache update (paper Section 3.3.3, last sentence of "Dynamic KV Cache Eviction"; Algorithm 2,
decoding loop) through the C ABI against the oracle.  Attention mass p within 2e-3 relative; the cumulative
scores are the exact fp32 sum of the old score and the GPU's own p; the row that leaves is the oracle's choice on
those cumulative scores; every byte of the cache that should not change does not."""
import numpy as np
import pytest
import torch

import oracle
import parity

pytestmark = pytest.mark.gpu


class State:
    def __init__(self, B, L, H, Hq, dtype, caps, lens, seed, start_pos=5000):
        self.B, self.L, self.H, self.Hq, self.G = B, L, H, Hq, Hq // H
        self.units = B * L * H
        self.dt = torch.bfloat16 if dtype == "bf16" else torch.float32
        g = torch.Generator(device="cuda").manual_seed(seed)
        self.g = g
        caps = np.asarray(caps, dtype=np.int64)
        self.offsets = torch.tensor(np.concatenate([[0], np.cumsum(caps)]), dtype=torch.int64, device="cuda")
        self.lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
        total = int(caps.sum())
        self.W = torch.randn(4, 128, generator=g, device="cuda")
        self.Kc = self._rows(total)
        self.Vc = torch.randn(total, 128, generator=g, device="cuda").to(self.dt)
        rng = np.random.default_rng(seed)
        pos = np.full(total, -7, dtype=np.int32)
        o = 0
        for c, n in zip(caps, lens):
            pos[o:o + n] = rng.permutation(rng.choice(start_pos, size=n, replace=False)).astype(np.int32)
            o += c
        self.pos = torch.tensor(pos, device="cuda")
        # few distinct values: many ties in the cumulative scores
        self.cum = torch.tensor(rng.integers(0, 3, size=total).astype(np.float32) * 0.25, device="cuda")
        self.new_pos = start_pos
        self.caps = caps

    def _rows(self, n):
        g = self.g
        return (torch.randn(n, 4, generator=g, device="cuda") @ self.W * 0.9 +
                torch.randn(n, 128, generator=g, device="cuda") * 0.7).to(self.dt)

    def new_token(self):
        q = self._rows(self.units * self.G).view(self.B, self.L, self.Hq, 128)
        k = self._rows(self.units).view(self.B, self.L, self.H, 128)
        v = torch.randn(self.units, 128, generator=self.g, device="cuda").to(self.dt).view(self.B, self.L, self.H, 128)
        return q, k, v


def _bytes(t):
    return t.contiguous().view(torch.uint8).cpu().numpy().reshape(t.shape[0], -1)


def _step_and_check(ub, ctx, st, max_cap, protect):
    q, k, v = st.new_token()
    before = dict(K=_bytes(st.Kc), V=_bytes(st.Vc), pos=st.pos.cpu().numpy(), cum=st.cum.cpu().numpy(),
                  lens=st.lens.cpu().numpy())
    Kf = st.Kc.double().cpu().numpy()
    total = st.Kc.shape[0]
    p = torch.full((total + st.units,), -1.0, device="cuda")
    evicted = torch.full((st.units,), -99, dtype=torch.int32, device="cuda")
    new_pos = torch.full((st.B,), st.new_pos, dtype=torch.int32, device="cuda")
    ub.uncomp_decode_update(ctx, q, k, v, new_pos, st.offsets, st.lens, max_cap, st.Kc, st.Vc, st.pos, st.cum,
                            protect=protect, p=p, evicted=evicted)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    after = dict(K=_bytes(st.Kc), V=_bytes(st.Vc), pos=st.pos.cpu().numpy(), cum=st.cum.cpu().numpy(),
                 lens=st.lens.cpu().numpy())
    pg = p.cpu().numpy()
    qn = q.double().cpu().numpy().reshape(st.units, st.G, 128)
    kn, kb, vb = k.double().cpu().numpy().reshape(st.units, 128), _bytes(k.view(st.units, 128)), _bytes(v.view(st.units, 128))
    offs = st.offsets.cpu().numpy()
    ev = evicted.cpu().numpy()
    for u in range(st.units):
        o, cap, n = int(offs[u]), int(st.caps[u]), int(before["lens"][u])
        ref = oracle.decode_probs(qn[u], Kf[o:o + n], kn[u])
        got = pg[o + u:o + u + n + 1].astype(np.float64)
        assert (np.abs(got - ref) <= parity.SCORE_RTOL * np.abs(ref) + 1e-12 * ref.max()).all(), u
        cum_new = before["cum"][o:o + n] + pg[o + u:o + u + n]            # fp32 + fp32, as the kernel adds
        if n < cap:
            slot, gone = n, -1
            assert after["lens"][u] == n + 1
        else:
            slot = oracle.decode_evict(cum_new.astype(np.float64), before["pos"][o:o + n], st.new_pos, protect)
            gone = int(before["pos"][o + slot])
            assert after["lens"][u] == n
        assert ev[u] == gone, (u, ev[u], gone)
        want_cum = before["cum"][o:o + cap].copy()
        want_cum[:n] = cum_new
        want_cum[slot] = pg[o + u + n]
        want_pos = before["pos"][o:o + cap].copy()
        want_pos[slot] = st.new_pos
        wK, wV = before["K"][o:o + cap].copy(), before["V"][o:o + cap].copy()
        wK[slot], wV[slot] = kb[u], vb[u]
        np.testing.assert_array_equal(after["cum"][o:o + cap].view(np.uint32), want_cum.view(np.uint32))
        np.testing.assert_array_equal(after["pos"][o:o + cap], want_pos)
        assert (after["K"][o:o + cap] == wK).all() and (after["V"][o:o + cap] == wV).all()
    st.new_pos += 1


@pytest.mark.parametrize("B,L,H,Hq,dtype", [(1, 2, 4, 16, "bf16"), (2, 1, 2, 2, "bf16"), (1, 1, 2, 16, "bf16"),
                                            (1, 1, 1, 16, "bf16"), (1, 2, 2, 8, "fp32")])
def test_decode_steps_match_oracle(B, L, H, Hq, dtype):
    from paper_2410_03090_b200 import binding as ub
    units = B * L * H
    rng = np.random.default_rng(units * 31 + Hq)
    max_cap = 2300
    caps = rng.integers(1, max_cap + 1, size=units)
    caps[0] = max_cap                      # several chunks
    caps[-1] = 1023                        # with the new token exactly one chunk
    lens = caps.copy()
    lens[units // 2] = max(0, int(caps[units // 2]) - 2)    # fills up, then evicts
    ctx = ub.Context(ub.make_shape(B, L, H, Hq, 16384, 128, 32, dtype))
    st = State(B, L, H, Hq, dtype, caps, lens, seed=Hq)
    for _ in range(4):
        _step_and_check(ub, ctx, st, max_cap, protect=1)


def test_decode_degenerate_units():
    from paper_2410_03090_b200 import binding as ub
    # an empty cache, a cache of one row, a cache whose entries are all inside the protected span, 1024 / 1025 entries
    caps = [5, 1, 3, 1024, 1025, 40]
    lens = [0, 1, 3, 1024, 1025, 7]
    ctx = ub.Context(ub.make_shape(1, 1, 6, 24, 4096, 128, 32, "bf16"))
    st = State(1, 1, 6, 24, "bf16", caps, lens, seed=3, start_pos=3000)
    st.pos[6:9] = torch.tensor([2999, 2998, 2997], dtype=torch.int32, device="cuda")     # unit 2: all recent
    for _ in range(3):
        _step_and_check(ub, ctx, st, 1025, protect=8)


def test_decode_rejections_and_bad_unit():
    from paper_2410_03090_b200 import binding as ub
    ctx = ub.Context(ub.make_shape(1, 1, 2, 8, 512, 128, 32, "bf16"))
    st = State(1, 1, 2, 8, "bf16", [10, 300], [10, 300], seed=1)
    q, k, v = st.new_token()
    npos = torch.tensor([st.new_pos], dtype=torch.int32, device="cuda")
    args = (st.offsets, st.lens)
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_decode_update(ctx, q, k, v, npos, *args, 513, st.Kc, st.Vc, st.pos, st.cum)     # max_cap > N
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_decode_update(ctx, q, k, v, npos, *args, 300, st.Kc, st.Vc, st.pos, st.cum, protect=0)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    # a unit above max_cap is left alone and reported; the other unit is updated
    before = (_bytes(st.Kc), st.cum.cpu().numpy().copy(), st.pos.cpu().numpy().copy())
    ev = torch.zeros(2, dtype=torch.int32, device="cuda")
    ub.uncomp_decode_update(ctx, q, k, v, npos, *args, 100, st.Kc, st.Vc, st.pos, st.cum, evicted=ev)
    assert ub.uncomp_status(ctx) == ub.UNCOMP_STATUS_BOUNDS
    assert (_bytes(st.Kc)[10:] == before[0][10:]).all() and (st.cum.cpu().numpy()[10:] == before[1][10:]).all()
    assert (st.pos.cpu().numpy()[10:] == before[2][10:]).all() and int(ev[1]) == -1 and int(ev[0]) >= 0
    big = ub.Context(ub.make_shape(1, 1, 2, 32, 512, 128, 32, "bf16"))                           # logits do not fit
    st2 = State(1, 1, 2, 32, "bf16", [400, 400], [400, 400], seed=2)
    q2, k2, v2 = st2.new_token()
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_decode_update(big, q2, k2, v2, npos, st2.offsets, st2.lens, 400, st2.Kc, st2.Vc, st2.pos, st2.cum)
    assert ei.value.code == ub.UNCOMP_E_LIMIT


def test_decode_seed_matches_oracle():
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200 import synth
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS["c2"], N=2048, L=2)
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    o = cp.run(K, V, Qw)
    cum = ub.uncomp_decode_seed(cp.ctx, o.scores, o.indices, o.offsets)
    torch.cuda.synchronize()
    offs = o.offsets.cpu().numpy()
    sc = o.scores.reshape(wl.units, -1).double().cpu().numpy()
    idx = o.indices.cpu().numpy()
    got = cum.cpu().numpy()
    for u in range(wl.units):
        want = oracle.decode_seed(sc[u], idx[offs[u]:offs[u + 1]])
        np.testing.assert_array_equal(got[offs[u]:offs[u + 1]], want.astype(np.float32))
    # a unit that keeps only its window: every row starts at 0
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 64, 128, 8, "bf16"))
    scores = torch.rand(1, 1, 1, 56, device="cuda")
    idx1 = torch.arange(56, 64, dtype=torch.int32, device="cuda")
    off1 = torch.tensor([0, 8], dtype=torch.int64, device="cuda")
    assert float(ub.uncomp_decode_seed(ctx, scores, idx1, off1).abs().max()) == 0.0


def test_decode_update_same_bits_twice():
    from paper_2410_03090_b200 import binding as ub
    caps = [1500, 700, 2048, 33]
    results = []
    for _ in range(2):
        ctx = ub.Context(ub.make_shape(1, 1, 4, 16, 8192, 128, 32, "bf16"))
        st = State(1, 1, 4, 16, "bf16", caps, caps, seed=17)
        q, k, v = st.new_token()
        p = torch.zeros(sum(caps) + 4, device="cuda")
        npos = torch.tensor([st.new_pos], dtype=torch.int32, device="cuda")
        ub.uncomp_decode_update(ctx, q, k, v, npos, st.offsets, st.lens, 2048, st.Kc, st.Vc, st.pos, st.cum, p=p)
        torch.cuda.synchronize()
        results.append((p, st.cum.clone(), st.pos.clone(), st.Kc.clone()))
    assert all(torch.equal(a, b) for a, b in zip(*results))


def test_decode_cache_wrapper_runs_prefill_then_decode():
    from paper_2410_03090_b200 import synth
    from paper_2410_03090_b200.compress import CompressionPass, DecodeCache
    wl = synth.scaled(synth.WORKLOADS["c2"], N=2048, L=2)
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    cp.run(K, V, Qw)
    cache = DecodeCache(cp)
    offs = cache.offsets.cpu().numpy()
    for t in range(3):
        pos_before = cache.pos.clone()
        npos = torch.full((wl.B,), wl.N + t, dtype=torch.int32, device="cuda")
        ev = cache.step(Qw[:, :, :, -1 - t, :].contiguous(), K[:, :, :, -1 - t, :].contiguous(),
                        V[:, :, :, -1 - t, :].contiguous(), npos)
        torch.cuda.synchronize()
        assert cp.status() == 0
        changed = (cache.pos != pos_before).cpu().numpy()
        assert (np.add.reduceat(changed, offs[:-1]) == 1).all()            # one row per head took the new token
        assert (cache.pos[torch.from_numpy(changed).cuda()] == wl.N + t).all()
        gone = ev.cpu().numpy()
        for u in range(wl.units):
            assert gone[u] in pos_before[offs[u]:offs[u + 1]].cpu().numpy()
            assert gone[u] not in cache.pos[offs[u]:offs[u + 1]].cpu().numpy()


def test_decode_many_small_caches():
    """Many heads with tiny, uneven caches (1 to 40 rows), G = 2, fp32 and bf16: chunk and warp edges of every kernel."""
    from paper_2410_03090_b200 import binding as ub
    rng = np.random.default_rng(5)
    for dtype in ("bf16", "fp32"):
        B, L, H, Hq = 3, 4, 8, 16
        units = B * L * H
        caps = rng.integers(1, 41, size=units)
        lens = np.minimum(caps, rng.integers(0, 41, size=units))
        ctx = ub.Context(ub.make_shape(B, L, H, Hq, 512, 128, 8, dtype))
        st = State(B, L, H, Hq, dtype, caps, lens, seed=23, start_pos=400)
        for _ in range(3):
            _step_and_check(ub, ctx, st, 40, protect=2)
