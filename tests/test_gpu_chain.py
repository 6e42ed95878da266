"""Chain-mode parity: the whole oracle chain against the whole GPU chain on the same stored inputs.

The acceptance tests compare stage by stage (the oracle's budget rule on the GPU's own effective ranks, the
oracle's selection on the GPU's own scores), because ranking and selection are discontinuous in their float
inputs.  Here nothing is handed over: entropy -> effective rank -> budgets -> window scores -> pooling ->
selection run end to end on both sides, and every place where the two chains end up with a different integer
is counted and must be explained by a near-tie in the ORACLE's own numbers:

* a unit whose budget differs must have, in its ranking set, a unit that the oracle gave that budget and whose
  oracle effective rank lies within 2e-4 relative (the entropy tolerance 1e-4, twice) of its own;
* a kept position that differs must have an oracle pooled score within 2e-3 relative (the score tolerance) of
  the unit's k-th largest oracle score, k = budget - window.

The counts are printed (pytest -s) so that they can be quoted."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2410_03090_b200 import synth


ERANK_GAP = 2e-4
SCORE_GAP = 2e-3


def _kept_position_diffs(got, ref, pooled, budget, w, where):
    """Number of kept prefix positions in which `got` differs from the oracle's selection `ref`; raises unless every
    differing position has an oracle score within SCORE_GAP (relative) of the oracle's k-th largest score."""
    assert len(got) == len(ref) == budget, where
    assert np.array_equal(got[-w:], ref[-w:]), where          # the window itself never differs
    k = budget - w
    if k == 0 or np.array_equal(got, ref):
        return 0
    odd = np.setxor1d(got[:k], ref[:k])
    kth = np.sort(pooled)[::-1][k - 1]
    rel = np.abs(pooled[odd] - kth) / kth
    assert rel.max() < SCORE_GAP, f"{where}: position {odd[rel.argmax()]} differs, score gap {rel.max():.2e}"
    return len(odd) // 2


def _oracle_chain(wl, K, Qw):
    """fp64 chain on every unit: (erank [B, L, H], budgets, offsets, pooled scores per unit)."""
    units = list(range(wl.units))
    ent = parity._map(lambda X: oracle.entropy(X, k_trunc=wl.k_trunc), [(parity.unit_np(K, wl, u),) for u in units], None)
    erank = np.array([e for _, e in ent], dtype=np.float64).reshape(wl.B, wl.L, wl.H)
    bud, off, _, _ = oracle.budgets(erank, wl.N, wl.w, wl.avg_budget, wl.M, wl.n_max)
    pooled = parity._map(lambda Q, X: oracle.pool(oracle.window_scores(Q, X), wl.pool_kernel, wl.pool_mode),
                         [(parity.unit_q_np(Qw, wl, u), parity.unit_np(K, wl, u)) for u in units], None)
    return erank, bud, off, pooled


@pytest.mark.gpu
@pytest.mark.parametrize("name,N,L,B", [("c2", 2048, 4, 1), ("c3", 4096, 2, 1), ("c4", 2048, 2, 2),
                                        ("c2", 8192, 32, 1)])          # the last one is workload c2 at its full size
def test_whole_chain_differs_from_the_oracle_chain_only_at_near_ties(name, N, L, B):
    from paper_2410_03090_b200.compress import CompressionPass
    wl = synth.scaled(synth.WORKLOADS[name], N=N, L=L, B=B)
    K, V, Qw = synth.generate(wl, "cuda")
    cp = CompressionPass(wl, "cuda")
    out = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    assert cp.status() == 0
    erank_o, bud_o, off_o, pooled_o = _oracle_chain(wl, K, Qw)
    bud_g = out.budgets.cpu().numpy()
    off_g = out.offsets.cpu().numpy()
    idx_g = out.indices.cpu().numpy()

    # ---- budgets: per ranking set (a layer) the GPU's budgets are a permutation of the oracle's
    budget_swaps = 0
    for b in range(wl.B):
        for l in range(wl.L):
            go, oo, eo = bud_g[b, l], bud_o[b, l], erank_o[b, l]
            assert sorted(go.tolist()) == sorted(oo.tolist())
            for h in np.nonzero(go != oo)[0]:
                budget_swaps += 1
                holders = np.nonzero(oo == go[h])[0]            # units the oracle gave this budget
                gap = np.min(np.abs(eo[holders] - eo[h])) / eo[h]
                assert gap < ERANK_GAP, f"unit ({b},{l},{h}): budget {go[h]} vs oracle {oo[h]}, erank gap {gap:.2e}"

    # ---- kept positions, at the GPU's budget of each unit
    index_diffs, units_with_diffs = 0, 0
    for u in range(wl.units):
        b, l, h = synth.unit_index(wl, u)
        budget = int(bud_g[b, l, h])
        ref = oracle.select(pooled_o[u], wl.w, budget)
        n = _kept_position_diffs(idx_g[off_g[u]:off_g[u + 1]], ref, pooled_o[u], budget, wl.w, f"unit {u}")
        index_diffs += n
        units_with_diffs += n > 0
    print(f"\nchain mode {wl.name} ({wl.units} units, {int(off_g[-1])} kept rows): {budget_swaps} units with a swapped "
          f"budget, {index_diffs} differing kept positions in {units_with_diffs} units; all at near-ties")


def test_the_position_check_itself_counts_near_ties_and_rejects_real_differences():
    # CPU only: the checker above on hand-made selections.  Scores 10, 9, ..., with two near-equal ones at the cut.
    pooled = np.array([10.0, 9.0, 8.0, 7.0, 6.0, 5.0 * (1 + 1e-4), 5.0, 4.0, 3.0, 2.0])
    w, budget = 2, 8                                  # k = 6 kept prefix positions, then the window 10, 11
    ref = oracle.select(pooled, w, budget)
    assert ref.tolist() == [0, 1, 2, 3, 4, 5, 10, 11]
    assert _kept_position_diffs(ref.copy(), ref, pooled, budget, w, "same") == 0
    near = np.array([0, 1, 2, 3, 4, 6, 10, 11])       # takes position 6 instead of 5: scores 1e-4 apart
    assert _kept_position_diffs(near, ref, pooled, budget, w, "near tie") == 1
    far = np.array([0, 1, 2, 3, 4, 8, 10, 11])        # takes position 8 (score 3) instead of 5
    with pytest.raises(AssertionError):
        _kept_position_diffs(far, ref, pooled, budget, w, "real difference")
    with pytest.raises(AssertionError):
        _kept_position_diffs(np.array([0, 1, 2, 3, 4, 5, 9, 11]), ref, pooled, budget, w, "window touched")
