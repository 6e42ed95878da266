"""uncomp_gram_static: the Gram stage for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not available to them -- a custom-operator hook inside
a serving framework whose caching allocator owns the device memory, or a latency-critical thread that
cannot afford the device-wide stall of an allocation -- so they cannot create the workspace the other
entry points need.  This entry point keeps its scratch in a fixed array inside the library instead.  The
test calls it through the C ABI twice in a row (the second call on a smaller problem with different data,
so stale scratch contents would show) and compares with uncomp_gram, which uses a caller workspace.

Collected last on purpose: a failure here must not hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from paper_2410_03090_b200 import synth

pytestmark = pytest.mark.gpu


def _compare(ub, wl, tol=2e-6):
    K, _, _ = synth.generate(wl, "cuda")
    shape = ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype)
    ctx = ub.Context(shape)
    ref = ub.uncomp_gram(ctx, K)
    out = torch.full_like(ref, float("nan"))          # the caller's output buffer, allocated by the caller
    ub.uncomp_gram_static(shape, K, out)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    scale = ref[:, :128 * 128].abs().amax(dim=1, keepdim=True)
    # same kernels and, for these shapes, the same token chunks as uncomp_gram: the tolerance of the Gram tests
    # (2e-6 of the largest entry); a caller with longer chunks passes its own
    assert float(((out - ref).abs() / scale).max()) <= tol
    assert torch.isfinite(out).all()
    return out


def test_gram_static_matches_workspace_entry_point_twice_in_a_row():
    from paper_2410_03090_b200 import binding as ub
    big = synth.scaled(synth.WORKLOADS["c2"], N=6000, L=1)            # 8 units x 6 chunks
    small = synth.scaled(synth.WORKLOADS["c3"], N=700, L=2)           # 16 units x 1 chunk, other data
    _compare(ub, big)
    _compare(ub, small)
    fp32 = synth.WORKLOADS["c1"]                                      # fp32 keys take the fp64 partials
    _compare(ub, fp32)


def test_gram_static_is_exact_on_integer_keys_against_the_oracle():
    # integer-valued keys: every product and partial sum is exact, so the result must equal the oracle's X^T X and
    # column sums bit for bit whatever the chunking; the second shape needs the longer chunks (8 units x 17 chunks
    # of 1024 tokens would not fit the array)
    import oracle
    from paper_2410_03090_b200 import binding as ub
    for units, N in ((3, 1000), (8, 17000)):
        g = torch.Generator(device="cuda").manual_seed(N)
        K = torch.randint(-3, 4, (1, 1, units, N, 128), generator=g, device="cuda").to(torch.bfloat16)
        K[0, 0, units - 1, N - 1, :] = 5.0
        shape = ub.make_shape(1, 1, units, units, N, 128, 8, "bf16")
        out = torch.full((units, 128 * 128 + 128), float("nan"), dtype=torch.float64, device="cuda")
        ub.uncomp_gram_static(shape, K, out)
        torch.cuda.synchronize()
        for u in (0, units - 1):
            X = K[0, 0, u].double().cpu().numpy()
            got = out[u].cpu().numpy()
            np.testing.assert_array_equal(got[:128 * 128].reshape(128, 128), oracle.covariance(X, center=False))
            np.testing.assert_array_equal(got[128 * 128:], X.sum(axis=0))


def test_gram_static_at_its_documented_maximum():
    # one layer of the 32K-token workload: 8 heads x 32768 tokens, 64 partials of 4096 tokens each
    from paper_2410_03090_b200 import binding as ub
    # (uncomp_gram takes 1024: fp32 accumulation on the tensor cores over four times as many tokens per partial
    # rounds more, measured 1e-5 of the largest entry)
    wl = synth.scaled(synth.WORKLOADS["c3"], L=1)
    _compare(ub, wl, tol=4e-5)
    wl64 = synth.scaled(synth.WORKLOADS["c2"], N=512, L=8)            # 64 units, one partial each
    _compare(ub, wl64)


def test_gram_static_refuses_shapes_beyond_its_array():
    from paper_2410_03090_b200 import binding as ub
    wl = synth.scaled(synth.WORKLOADS["c2"], N=512, L=16)             # 128 units > 64 partial slots
    K = torch.zeros(wl.B, wl.L, wl.H, wl.N, wl.d, dtype=torch.bfloat16, device="cuda")
    shape = ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype)
    out = torch.empty(wl.units, 128 * 128 + 128, dtype=torch.float64, device="cuda")
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_gram_static(shape, K, out)
    assert ei.value.code == ub.UNCOMP_E_LIMIT
    assert ub.lib.uncomp_gram_static_max_bytes() == 32 * (128 * 128 + 128) * 8
