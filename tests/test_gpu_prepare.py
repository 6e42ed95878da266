"""Preparation stage (paper Section 3.3.1; Algorithm 1) through the C ABI against the oracle: the mean within fp32
rounding, every integer output bit-exact (labels of the mean on the GPU's own mean)."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("S,L,H,M,scope", [(500, 32, 8, 8, 0), (500, 32, 8, 2, 0), (500, 32, 8, 8, 1), (37, 5, 11, 4, 0),
                                           (1, 1, 3, 3, 0), (64, 80, 8, 5, 1), (9, 2, 4, 1, 1)])
def test_prepare_groups_parity(S, L, H, M, scope):
    from paper_2410_03090_b200 import binding as ub
    g = torch.Generator(device="cuda").manual_seed(S * 7 + M)
    base = torch.rand(L, H, generator=g, device="cuda") * 30 + 1
    erank = base[None] + torch.randn(S, L, H, generator=g, device="cuda") * 2.0
    erank[:, 0, :2] = 7.0                                    # exact ties inside a set
    erank = erank.round(decimals=1).contiguous()             # and many accidental ones
    ctx = ub.Context(ub.make_shape(1, L, H, H, 256, 128, 8, "bf16"))
    mean, gm, votes, gv = ub.uncomp_prepare_groups(ctx, erank, M, scope)
    torch.cuda.synchronize()
    e = erank.double().cpu().numpy()
    ref_mean = oracle.prepare_mean(e)
    np.testing.assert_allclose(mean.cpu().numpy(), ref_mean, rtol=1e-6)
    np.testing.assert_array_equal(gm.cpu().numpy(), oracle.group_labels(mean.double().cpu().numpy(), M, scope))
    ref_votes, ref_lab = oracle.majority_vote(e, M, scope)
    np.testing.assert_array_equal(votes.cpu().numpy(), ref_votes)
    np.testing.assert_array_equal(gv.cpu().numpy(), ref_lab)
    # a second call on the same buffers gives the same votes (the call clears them)
    _, _, votes2, _ = ub.uncomp_prepare_groups(ctx, erank, M, scope)
    assert torch.equal(votes2, votes)


def test_prepare_groups_rejections():
    from paper_2410_03090_b200 import binding as ub
    ctx = ub.Context(ub.make_shape(1, 4, 8, 8, 256, 128, 8, "bf16"))
    e = torch.ones(3, 4, 8, device="cuda")
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_prepare_groups(ctx, e, 9, 0)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    with pytest.raises(ub.UncompError) as ei:
        ub.uncomp_prepare_groups(ctx, e, 2, 2)
    assert ei.value.code == ub.UNCOMP_E_PARAM
    mean, gm, votes, gv = ub.uncomp_prepare_groups(ctx, e, 32, 1)        # all equal: rank = index
    assert torch.equal(gm.cpu().ravel(), torch.arange(32, dtype=torch.int32))


@pytest.mark.parametrize("L,H", [(32, 8), (2, 1), (80, 8), (300, 3)])
def test_retrieval_layer_parity(L, H):
    from paper_2410_03090_b200 import binding as ub
    g = torch.Generator(device="cuda").manual_seed(L * 13 + H)
    v = (torch.randn(L, H, generator=g, device="cuda") * 2 + 10).round(decimals=1).contiguous()
    if L > 4:
        v[3] = v[1]
        v[4] = v[2]                      # the rise 1 -> 2 occurs twice: the earlier one must win if it is the largest
    ctx = ub.Context(ub.make_shape(1, L, H, H, 256, 128, 8, "bf16"))
    layer, inc = ub.uncomp_retrieval_layer(ctx, v)
    torch.cuda.synchronize()
    want, winc = oracle.retrieval_layer(v.double().cpu().numpy())
    assert int(layer[0]) == want
    np.testing.assert_allclose(inc.cpu().numpy(), winc, rtol=1e-6, atol=1e-7)
