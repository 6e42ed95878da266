"""Hidden-state eviction (paper Section 3.3.2) through the C ABI against the oracle: scores within 2e-3
relative, kept positions exact given the GPU's own scores, gathered hidden-state rows bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import parity

pytestmark = pytest.mark.gpu


def _case(B, L, H, Hq, N, D, dtype, n_keep, layer, seed):
    from paper_2410_03090_b200 import binding as ub
    g = torch.Generator(device="cuda").manual_seed(seed)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    W = torch.randn(6, 128, generator=g, device="cuda")
    Kall = (torch.randn(B, L, H, N, 6, generator=g, device="cuda") @ W * 0.8 +
            torch.randn(B, L, H, N, 128, generator=g, device="cuda")).to(dt)
    q = (torch.randn(B, Hq, 6, generator=g, device="cuda") @ W * 0.8 + torch.randn(B, Hq, 128, generator=g, device="cuda")).to(dt)
    X = torch.randn(B, N, D, generator=g, device="cuda").to(dt)
    ctx = ub.Context(ub.make_shape(B, L, H, Hq, N, 128, 1, dtype))
    Klayer = Kall[:, layer]                     # a strided view: the keys of one layer
    scores = torch.empty(B, N - 1, device="cuda")
    idx, Xout = ub.uncomp_evict_hidden(ctx, q, Klayer, X, n_keep, scores=scores)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    for b in range(B):
        ref = oracle.last_token_scores(q[b].double().cpu().numpy(), Klayer[b].double().cpu().numpy())
        got = scores[b].double().cpu().numpy()
        tol = parity.SCORE_RTOL * np.abs(ref[:-1]) + 1e-12 * ref.max()
        assert (np.abs(got - ref[:-1]) <= tol).all()
        # stage protocol: the oracle's selection on the GPU's own scores; the last position is the window
        want = oracle.select(got, 1, n_keep)
        np.testing.assert_array_equal(idx[b].cpu().numpy(), want)
        rows = X[b].contiguous().view(torch.uint8).reshape(N, -1).cpu().numpy()
        assert Xout[b].contiguous().view(torch.uint8).reshape(n_keep, -1).cpu().numpy().tobytes() == \
            oracle.compact(rows, want).tobytes()
    return idx


@pytest.mark.parametrize("B,L,H,Hq,N,D,dtype,n_keep", [
    (2, 3, 8, 32, 3000, 512, "bf16", 1024),      # grouped queries, several chunks, ragged tail
    (1, 1, 4, 4, 700, 128, "fp32", 300),         # one query head per KV head, fp32
    (1, 2, 2, 16, 2049, 4096, "bf16", 512),      # G = 8, model-width rows of 8 KB
    (3, 1, 1, 16, 130, 64, "bf16", 1),           # G = 16; only the last position survives
    (1, 1, 8, 8, 513, 256, "bf16", 513),         # keep everything
    (2, 1, 2, 4, 2, 8, "bf16", 1),               # two positions, 16-byte hidden rows
    (1, 1, 1, 2, 33, 24, "fp32", 32),            # one past a warp of positions, drop exactly one
    (5, 2, 4, 8, 1025, 72, "bf16", 7),           # one past a chunk, odd row width (144 bytes)
])
def test_evict_hidden_parity(B, L, H, Hq, N, D, dtype, n_keep):
    idx = _case(B, L, H, Hq, N, D, dtype, n_keep, layer=L - 1, seed=N)
    assert int(idx[:, -1].min()) == N - 1 and int(idx[:, -1].max()) == N - 1
    if n_keep == N:
        assert torch.equal(idx[0].cpu(), torch.arange(N, dtype=torch.int32))


def test_evict_hidden_rejections():
    from paper_2410_03090_b200 import binding as ub
    ctx = ub.Context(ub.make_shape(1, 1, 2, 6, 256, 128, 1, "bf16"))          # G = 3 is not supported here
    q = torch.zeros(1, 6, 128, dtype=torch.bfloat16, device="cuda")
    K = torch.zeros(1, 2, 256, 128, dtype=torch.bfloat16, device="cuda")
    X = torch.zeros(1, 256, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_evict_hidden(ctx, q, K, X, 10)
    assert ei.value.code == ub.UNCOMP_E_SHAPE
    ctx = ub.Context(ub.make_shape(1, 1, 2, 4, 256, 128, 1, "bf16"))
    q = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_evict_hidden(ctx, q, K, X, 257)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_evict_hidden(ctx, q, K, X[:, :, :60].contiguous(), 10)     # rows of 120 bytes
    assert ei.value.code == ub.UNCOMP_E_ALIGN


def test_evict_hidden_same_bits_twice():
    from paper_2410_03090_b200 import binding as ub
    g = torch.Generator(device="cuda").manual_seed(9)
    q = torch.randn(2, 32, 128, generator=g, device="cuda").to(torch.bfloat16)
    K = torch.randn(2, 8, 5000, 128, generator=g, device="cuda").to(torch.bfloat16)
    X = torch.randn(2, 5000, 256, generator=g, device="cuda").to(torch.bfloat16)
    ctx = ub.Context(ub.make_shape(2, 1, 8, 32, 5000, 128, 1, "bf16"))
    runs = []
    for _ in range(2):
        sc = torch.empty(2, 4999, device="cuda")
        idx, Xo = ub.uncomp_evict_hidden(ctx, q, K, X, 1234, scores=sc)
        runs.append((sc.clone(), idx.clone(), Xo.clone()))
    assert all(torch.equal(a, b) for a, b in zip(*runs))
