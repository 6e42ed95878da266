"""Truncated entropy of wide token matrices (paper Section 3.1 Eq. 1 with D beyond one head, Section 3.2) through
the C ABI against the oracle: |dH| <= 1e-4 max(|H|, 1), the k largest eigenvalues within 1e-4 of the largest."""
import numpy as np
import pytest
import torch

import oracle
import parity

pytestmark = pytest.mark.gpu


def _matrix(count, N, D, rank, noise, seed, offset=0.0, pad=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    W = torch.randn(rank, D, generator=g, device="cuda") * torch.linspace(2.0, 0.3, rank, device="cuda")[:, None]
    X = torch.randn(count, N, rank, generator=g, device="cuda") @ W + noise * torch.randn(count, N, D, generator=g, device="cuda")
    X = (X + offset).to(torch.bfloat16)
    if pad:
        buf = torch.zeros(count, N, D + pad, dtype=torch.bfloat16, device="cuda")
        buf[:, :, :D] = X
        X = buf[:, :, :D]
    return X


def _check(ub, X, k, center, norm):
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "bf16"))
    ent, er, spec = ub.uncomp_entropy_wide(ctx, X, k, center, norm, spectrum=True)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    for i in range(X.shape[0]):
        H, E, lam = oracle.entropy_wide(X[i].double().cpu().numpy(), k, bool(center), norm, return_spectrum=True)
        kk = min(k, X.shape[2])
        got = spec[i].cpu().numpy()
        assert np.abs(got - lam[:kk]).max() <= 1e-4 * lam[0], (i, np.abs(got - lam[:kk]).max() / lam[0])
        assert abs(float(ent[i]) - H) <= parity.ENTROPY_RTOL * max(abs(H), 1.0), (i, float(ent[i]), H)
        assert abs(float(er[i]) - E) <= 2e-4 * max(E, 1.0)


@pytest.mark.parametrize("N,D,rank,k,center,norm", [
    (700, 256, 12, 32, 1, 0),       # one block, ragged tokens
    (1000, 384, 40, 32, 1, 0),      # second block half empty
    (333, 512, 6, 16, 0, 0),        # N < D, uncentred
    (2500, 1024, 64, 64, 1, 1),     # ten block pairs, several token chunks, whole-trace normalisation
    (700, 1024, 30, 32, 1, 0),      # fewer tokens than features: token-space path, ragged token count, centred
    (100, 256, 8, 32, 1, 1),        # token-space matrix padded from 100 to 128, whole-trace normalisation
    (1000, 4096, 50, 64, 1, 0),     # hidden-state width, short prompt
    (60, 512, 5, 64, 1, 0),         # k_trunc beyond the number of tokens: the missing eigenvalues are zero
    (2, 128, 1, 8, 1, 0),           # two tokens: one non-zero eigenvalue after centring
    (128, 128, 9, 32, 1, 0),        # square: the feature-space path at its smallest size
    (129, 192, 9, 32, 0, 1),        # one token past a 64-token stage, token-space, uncentred, whole trace
    (64, 4096, 4, 16, 1, 0),        # a single stage of tokens against the widest matrix
])
def test_entropy_wide_parity(N, D, rank, k, center, norm):
    from paper_2410_03090_b200 import binding as ub
    _check(ub, _matrix(1, N, D, rank, 0.2, seed=N + D), k, center, norm)


def test_entropy_wide_batch_strided_rows_and_offset():
    from paper_2410_03090_b200 import binding as ub
    # two matrices, rows 64 elements wider than D, a common offset that centring must remove
    _check(ub, _matrix(2, 900, 640, 20, 0.1, seed=5, offset=3.0, pad=64), 32, 1, 0)


def test_entropy_wide_closed_forms():
    from paper_2410_03090_b200 import binding as ub
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "bf16"))
    # one direction: H = 0;  k orthogonal directions of equal weight: H = ln k
    N, D = 512, 256
    X = torch.zeros(1, N, D, dtype=torch.bfloat16, device="cuda")
    X[0, :, 3] = torch.where(torch.arange(N, device="cuda") % 2 == 0, 1.0, -1.0).to(torch.bfloat16)
    ent, _ = ub.uncomp_entropy_wide(ctx, X, 32)
    assert abs(float(ent[0])) < 1e-5
    X.zero_()
    # square waves of 8 different power-of-two periods are orthogonal and have zero mean; each is written to
    # four feature columns, so the scatter matrix has 8 equal non-zero eigenvalues
    for c in range(32):
        X[0, :, 5 * c] = torch.where((torch.arange(N, device="cuda") // (1 << (c % 8))) % 2 == 0, 1.0, -1.0).to(torch.bfloat16)
    ent, er, spec = ub.uncomp_entropy_wide(ctx, X, 8, spectrum=True)
    torch.cuda.synchronize()
    H, E, lam = oracle.entropy_wide(X[0].double().cpu().numpy(), 8, return_spectrum=True)
    assert abs(float(ent[0]) - H) < 1e-4 and abs(H - np.log(8)) < 1e-9


def test_entropy_wide_rejections():
    from paper_2410_03090_b200 import binding as ub
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "bf16"))
    X = torch.zeros(1, 64, 200, dtype=torch.bfloat16, device="cuda")           # D not a multiple of 64
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_entropy_wide(ctx, X, 8)
    assert ei.value.code == ub.UNCOMP_E_SHAPE
    X = torch.zeros(1, 64, 256, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_entropy_wide(ctx, X, 8, scratch=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == ub.UNCOMP_E_WORKSPACE
    assert ub.lib.uncomp_entropy_wide_scratch_bytes(64, 8192) == 0
    f32 = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "fp32"))
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_entropy_wide(f32, X, 8)
    assert ei.value.code == ub.UNCOMP_E_SHAPE


def test_l2_sweep_measurement_kernel_touches_every_element_once_per_pass():
    """`uncomp_measure_l2_sweep` defines the denominator of the tridiagonalisation's roofline: one fused multiply-add
    per element and pass, rows and ragged widths included, nothing outside the matrix."""
    from paper_2410_03090_b200 import binding as ub
    rows, cols, passes = 301, 4 * 131, 3
    buf = torch.full((rows + 2, cols), 7.0, device="cuda")
    A = buf[1:rows + 1]
    A.copy_(torch.arange(rows * cols, device="cuda", dtype=torch.float32).reshape(rows, cols) / (rows * cols))
    ref = A.clone().double()
    ub.uncomp_measure_l2_sweep(A, passes)
    torch.cuda.synchronize()
    for _ in range(passes):
        ref = ref * float(np.float32(0.999)) + float(np.float32(1e-6))
    assert float((A.double() - ref).abs().max()) < 1e-6
    assert float(buf[0].min()) == 7.0 and float(buf[-1].max()) == 7.0
    with pytest.raises(ub.UncompError):
        ub.uncomp_measure_l2_sweep(torch.zeros(4, 6, device="cuda"), 1)          # cols not a multiple of 4
