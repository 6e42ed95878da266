"""Helpers shared by the GPU parity tests: run the CPU oracle on the stored inputs of single units and
compare with what the CUDA library produced.  The oracle never sees anything the CUDA path computed
except where the stage protocol says so (budgets from the GPU's erank, selection from the GPU's scores)."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import oracle
from paper_2410_03090_b200 import synth

ENTROPY_RTOL = 1e-4     # |dH| <= 1e-4 * max(|H_ref|, 1)
SCORE_RTOL = 2e-3       # |d| <= 2e-3 * |ref| + 1e-12 * max_j ref


def _map(fn, items, threads):
    """The oracle's C functions release the interpreter lock, so units can run side by side.  Inputs are fetched
    from the device on the calling thread."""
    items = list(items)
    if threads is None:
        threads = min(len(items), os.cpu_count() or 1, 16)
    if threads <= 1 or len(items) <= 1:
        return [fn(*it) for it in items]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(lambda it: fn(*it), items))


def unit_np(t: torch.Tensor, wl: synth.Workload, u: int) -> np.ndarray:
    b, l, h = synth.unit_index(wl, u)
    return t[b, l, h].double().cpu().numpy()


def unit_q_np(Qw: torch.Tensor, wl: synth.Workload, u: int) -> np.ndarray:
    b, l, h = synth.unit_index(wl, u)
    return Qw[b, l, h * wl.G:(h + 1) * wl.G].double().cpu().numpy()


def check_entropy(wl, K, entropy, erank, units, k_trunc=None, center=1, norm=0, threads=None):
    k = wl.k_trunc if k_trunc is None else k_trunc
    ent = entropy.reshape(-1).double().cpu().numpy()
    er = erank.reshape(-1).double().cpu().numpy()
    worst = 0.0
    units = list(units)
    refs = _map(lambda X: oracle.entropy(X, k_trunc=k, center=bool(center), norm=norm),
                [(unit_np(K, wl, u),) for u in units], threads)
    for u, (H, E) in zip(units, refs):
        tol = ENTROPY_RTOL * max(abs(H), 1.0)
        worst = max(worst, abs(ent[u] - H) / tol)
        assert abs(ent[u] - H) <= tol, f"unit {u}: entropy {ent[u]} vs oracle {H}"
        assert abs(er[u] - E) <= 2 * ENTROPY_RTOL * max(E, 1.0) * max(abs(H), 1.0), f"unit {u}: erank {er[u]} vs {E}"
    return worst


def oracle_lse(wl, K, Qw, units, scale=None, threads=None) -> dict:
    """{unit: [G, w] fp64 log-sum-exp of its window rows} from the oracle."""
    units = list(units)
    refs = _map(lambda Q, X: oracle.window_lse(Q, X, scale), [(unit_q_np(Qw, wl, u), unit_np(K, wl, u)) for u in units],
                threads)
    return dict(zip(units, refs))


def check_scores(wl, K, Qw, scores, units, pool_kernel=None, pool_mode=None, scale=None, threads=None):
    pk = wl.pool_kernel if pool_kernel is None else pool_kernel
    pm = wl.pool_mode if pool_mode is None else pool_mode
    P = wl.N - wl.w
    sc = scores.reshape(-1, P)
    worst = 0.0
    units = list(units)
    refs = _map(lambda Q, X: oracle.pool(oracle.window_scores(Q, X, scale), pk, pm),
                [(unit_q_np(Qw, wl, u), unit_np(K, wl, u)) for u in units], threads)
    for u, ref in zip(units, refs):
        got = sc[u].double().cpu().numpy()
        tol = SCORE_RTOL * np.abs(ref) + 1e-12 * ref.max()
        err = np.abs(got - ref) / tol
        worst = max(worst, float(err.max()))
        j = int(err.argmax())
        assert err.max() <= 1.0, f"unit {u}: score[{j}] {got[j]} vs oracle {ref[j]}"
    return worst


def check_budgets(wl, erank, budgets, offsets, layer_group=None, layer_ctx=None, M=None, avg=None, n_max=None,
                  scope=0, eps=0.0, dn=0, n_last=0):
    """Stage protocol: the oracle's budget rule applied to the GPU's own erank must agree bit for bit."""
    e = erank.cpu().numpy().astype(np.float64)
    rb, ro, rg, rc = oracle.budgets(e, wl.N, wl.w, wl.avg_budget if avg is None else avg, wl.M if M is None else M,
                                    wl.n_max if n_max is None else n_max, scope, float(np.float32(eps)), dn, n_last)
    np.testing.assert_array_equal(budgets.cpu().numpy(), rb)
    np.testing.assert_array_equal(offsets.cpu().numpy(), ro)
    if layer_group is not None:
        np.testing.assert_array_equal(layer_group.cpu().numpy(), rg)
        np.testing.assert_array_equal(layer_ctx.cpu().numpy(), rc)


def check_select(wl, scores, budgets, offsets, indices, units):
    """Stage protocol: the oracle's selection applied to the GPU's pooled scores and budgets."""
    P = wl.N - wl.w
    sc = scores.reshape(-1, P)
    bud = budgets.reshape(-1).cpu().numpy()
    off = offsets.cpu().numpy()
    idx = indices.cpu().numpy()
    for u in units:
        ref = oracle.select(sc[u].double().cpu().numpy(), wl.w, int(bud[u]))
        got = idx[off[u]:off[u + 1]]
        np.testing.assert_array_equal(got, ref, err_msg=f"unit {u}")


def check_compact(wl, K, V, indices, offsets, Kc, Vc, units):
    off = offsets.cpu().numpy()
    idx = indices.cpu().numpy()
    rb = wl.d * wl.elem_bytes
    for u in units:
        b, l, h = synth.unit_index(wl, u)
        seg = idx[off[u]:off[u + 1]]
        for src, dst in ((K, Kc), (V, Vc)):
            rows = src[b, l, h].contiguous().view(torch.uint8).reshape(wl.N, rb).cpu().numpy()
            ref = oracle.compact(rows, seg)
            got = dst[off[u]:off[u + 1]].contiguous().view(torch.uint8).reshape(-1, rb).cpu().numpy()
            assert got.tobytes() == ref.tobytes(), f"unit {u}: compacted rows differ"
