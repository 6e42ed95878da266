"""TEST INFRASTRUCTURE: Python face of the plain fp64 CPU oracle (oracle/uncomp_oracle.c).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the product
package never does.  All arrays are numpy; floating-point inputs are fp64 (stored bf16/fp32 values
widen to fp64 exactly).  Each function cites the paper passage it follows in the C source.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build as _build

_lib = C.CDLL(_build())

_dp = C.POINTER(C.c_double)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_u8p = C.POINTER(C.c_ubyte)

_lib.oracle_covariance.argtypes = [_dp, C.c_int, C.c_int, C.c_int, _dp]
_lib.oracle_covariance.restype = None
_lib.oracle_jacobi_eigenvalues.argtypes = [_dp, C.c_int, _dp]
_lib.oracle_jacobi_eigenvalues.restype = C.c_int
_lib.oracle_truncated_entropy.argtypes = [_dp, C.c_int, C.c_int, C.c_int, _dp, _dp]
_lib.oracle_truncated_entropy.restype = None
_lib.oracle_entropy.argtypes = [_dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, _dp, _dp, _dp]
_lib.oracle_entropy.restype = C.c_int
_lib.oracle_budgets.argtypes = [_dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                C.c_int, C.c_int, C.c_double, C.c_int, C.c_int,
                                _i32p, _i64p, _i32p, _i32p]
_lib.oracle_budgets.restype = C.c_int
_lib.oracle_window_scores.argtypes = [_dp, _dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _dp]
_lib.oracle_window_scores.restype = None
_lib.oracle_window_lse.argtypes = [_dp, _dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _dp]
_lib.oracle_window_lse.restype = None
_lib.oracle_last_token_scores.argtypes = [_dp, _dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _dp]
_lib.oracle_last_token_scores.restype = None
_lib.oracle_decode_probs.argtypes = [_dp, _dp, _dp, C.c_int, C.c_int, C.c_int, C.c_double, _dp]
_lib.oracle_decode_probs.restype = None
_lib.oracle_decode_evict.argtypes = [_dp, _i32p, C.c_int, C.c_int, C.c_int]
_lib.oracle_decode_evict.restype = C.c_int
_lib.oracle_prepare_mean.argtypes = [_dp, C.c_int, C.c_int, C.c_int, _dp]
_lib.oracle_prepare_mean.restype = None
_lib.oracle_group_labels.argtypes = [_dp, C.c_int, C.c_int, C.c_int, C.c_int, _i32p]
_lib.oracle_group_labels.restype = C.c_int
_lib.oracle_majority_vote.argtypes = [_dp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, _i32p, _i32p]
_lib.oracle_majority_vote.restype = C.c_int
_lib.oracle_decode_seed.argtypes = [_dp, C.c_int, _i32p, C.c_int, _dp]
_lib.oracle_decode_seed.restype = None
_lib.oracle_retrieval_layer.argtypes = [_dp, C.c_int, C.c_int, _dp]
_lib.oracle_retrieval_layer.restype = C.c_int
_lib.oracle_pool.argtypes = [_dp, C.c_int, C.c_int, C.c_int, _dp]
_lib.oracle_pool.restype = None
_lib.oracle_select.argtypes = [_dp, C.c_int, C.c_int, C.c_int, _i32p]
_lib.oracle_select.restype = None
_lib.oracle_compact.argtypes = [_u8p, C.c_size_t, _i32p, C.c_int, _u8p]
_lib.oracle_compact.restype = None


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(t)


def covariance(X, center: bool = True) -> np.ndarray:
    """Eq. 1 without the 1/(N-1) factor; X is [N, d]."""
    X = _f64(X)
    N, d = X.shape
    Cm = np.empty((d, d), dtype=np.float64)
    _lib.oracle_covariance(_p(X, _dp), N, d, int(center), _p(Cm, _dp))
    return Cm


def eigenvalues(A) -> np.ndarray:
    """Eigenvalues (descending) of a symmetric matrix by cyclic Jacobi."""
    A = _f64(A).copy()
    d = A.shape[0]
    lam = np.empty(d, dtype=np.float64)
    sweeps = _lib.oracle_jacobi_eigenvalues(_p(A, _dp), d, _p(lam, _dp))
    if sweeps < 0:
        raise RuntimeError("oracle Jacobi did not converge")
    return lam


def truncated_entropy(lam, k: int, norm: int = 0):
    """(H_k, erank_k) of a descending spectrum (Section 3.2)."""
    lam = _f64(lam)
    H, E = C.c_double(), C.c_double()
    _lib.oracle_truncated_entropy(_p(lam, _dp), lam.shape[0], int(k), int(norm), C.byref(H), C.byref(E))
    return H.value, E.value


def entropy(X, k_trunc: int = 32, center: bool = True, norm: int = 0, return_spectrum: bool = False):
    """(H_k, erank_k[, spectrum]) of one token matrix X [N, d]."""
    X = _f64(X)
    N, d = X.shape
    lam = np.empty(d, dtype=np.float64)
    H, E = C.c_double(), C.c_double()
    sweeps = _lib.oracle_entropy(_p(X, _dp), N, d, int(k_trunc), int(center), int(norm),
                                 C.byref(H), C.byref(E), _p(lam, _dp))
    if sweeps < 0:
        raise RuntimeError("oracle Jacobi did not converge")
    if return_spectrum:
        return H.value, E.value, lam
    return H.value, E.value


def budgets(erank, N: int, w: int, avg_budget: int, M: int, n_max: int, scope: int = 0,
            eps: float = 0.0, dn: int = 0, n_last: int = 0):
    """erank [B, L, H] -> (budgets [B,L,H] int32, offsets [units+1] int64,
    layer_group [B,L] int32, layer_ctx [B,L] int32).  Section 3.3.3 and 3.3.2."""
    e = _f64(erank)
    B, L, H = e.shape
    bud = np.zeros((B, L, H), dtype=np.int32)
    off = np.zeros(B * L * H + 1, dtype=np.int64)
    lg = np.zeros((B, L), dtype=np.int32)
    lc = np.zeros((B, L), dtype=np.int32)
    rc = _lib.oracle_budgets(_p(e, _dp), B, L, H, int(N), int(w), int(avg_budget), int(M), int(n_max),
                             int(scope), float(eps), int(dn), int(n_last),
                             _p(bud, _i32p), _p(off, _i64p), _p(lg, _i32p), _p(lc, _i32p))
    if rc != 0:
        raise ValueError("oracle_budgets: precondition violated")
    return bud, off, lg, lc


def window_scores(Q, K, scale: float | None = None) -> np.ndarray:
    """Raw window scores [N - w] of one unit; Q [G, w, d], K [N, d]."""
    Q, K = _f64(Q), _f64(K)
    G, w, d = Q.shape
    N = K.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    raw = np.empty(N - w, dtype=np.float64)
    _lib.oracle_window_scores(_p(Q, _dp), _p(K, _dp), N, d, w, G, float(scale), _p(raw, _dp))
    return raw


def window_lse(Q, K, scale: float | None = None) -> np.ndarray:
    """Natural-log sum of exponentials of every window row's scaled, causally visible logits: [G, w]."""
    Q, K = _f64(Q), _f64(K)
    G, w, d = Q.shape
    N = K.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    lse = np.empty((G, w), dtype=np.float64)
    _lib.oracle_window_lse(_p(Q, _dp), _p(K, _dp), N, d, w, G, float(scale), _p(lse, _dp))
    return lse


def pool(raw, pool_kernel: int = 7, pool_mode: int = 0) -> np.ndarray:
    raw = _f64(raw)
    out = np.empty_like(raw)
    _lib.oracle_pool(_p(raw, _dp), raw.shape[0], int(pool_kernel), int(pool_mode), _p(out, _dp))
    return out


def select(score, w: int, budget: int) -> np.ndarray:
    """Kept positions of one unit: top (budget - w) prefix positions ascending, then the window."""
    score = _f64(score)
    Pn = score.shape[0]
    idx = np.empty(int(budget), dtype=np.int32)
    _lib.oracle_select(_p(score, _dp), Pn, int(w), int(budget), _p(idx, _i32p))
    return idx


def compact(src_rows: np.ndarray, idx) -> np.ndarray:
    """Rows idx of src_rows ([N, row_bytes] uint8 view of one unit's K or V), bit for bit."""
    src = np.ascontiguousarray(src_rows, dtype=np.uint8)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.empty((idx.shape[0], src.shape[1]), dtype=np.uint8)
    _lib.oracle_compact(_p(src, _u8p), src.shape[1], _p(idx, _i32p), idx.shape[0], _p(out, _u8p))
    return out


def last_token_scores(q, K, scale: float | None = None) -> np.ndarray:
    """Hidden-state eviction scores [N] of one sequence and layer: q [Hq, d] (last position), K [H, N, d]."""
    q, K = _f64(q), _f64(K)
    Hq, d = q.shape
    H, N, _ = K.shape
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    out = np.empty(N, dtype=np.float64)
    _lib.oracle_last_token_scores(_p(q, _dp), _p(K, _dp), H, Hq, N, d, float(scale), _p(out, _dp))
    return out


def decode_probs(q, Kc, knew, scale: float | None = None) -> np.ndarray:
    """Attention of a new token over one head's cache plus itself, summed over the G query heads:
    q [G, d], Kc [len, d], knew [d] -> p [len + 1]."""
    q, Kc, knew = _f64(q), _f64(Kc), _f64(knew)
    G, d = q.shape
    n = Kc.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    p = np.empty(n + 1, dtype=np.float64)
    _lib.oracle_decode_probs(_p(q, _dp), _p(Kc, _dp), _p(knew, _dp), G, n, d, float(scale), _p(p, _dp))
    return p


def decode_evict(cum, pos, new_pos: int, protect: int = 1) -> int:
    """Entry of a full cache that leaves: lowest cumulative score among the entries older than the
    newest `protect` positions, equal scores to the lower position."""
    cum = _f64(cum)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    return int(_lib.oracle_decode_evict(_p(cum, _dp), _p(pos, _i32p), len(cum), int(new_pos), int(protect)))


def decode_update(q, Kc, Vc, pos, cum, knew, vnew, new_pos: int, cap: int, protect: int = 1,
                  scale: float | None = None):
    """One decode step of one head.  Returns (Kc', Vc', pos', cum', p, evicted position or -1); the cache
    stays ordered by position (the evicted row is removed, the new token goes to the end)."""
    Kc, Vc = np.asarray(Kc), np.asarray(Vc)
    pos = np.asarray(pos, dtype=np.int32)
    p = decode_probs(q, Kc, knew, scale)
    n = len(pos)
    cum2 = _f64(cum) + p[:n]
    evicted = -1
    keep = np.ones(n, dtype=bool)
    if n >= cap:
        e = decode_evict(cum2, pos, new_pos, protect)
        evicted = int(pos[e])
        keep[e] = False
    K2 = np.concatenate([Kc[keep], np.asarray(knew)[None]], axis=0)
    V2 = np.concatenate([Vc[keep], np.asarray(vnew)[None]], axis=0)
    pos2 = np.concatenate([pos[keep], np.array([new_pos], dtype=np.int32)])
    cum3 = np.concatenate([cum2[keep], p[n:]])
    return K2, V2, pos2, cum3, p, evicted


def prepare_mean(erank) -> np.ndarray:
    """Averaged effective rank over the samples: erank [S, L, H] -> [L, H]."""
    erank = _f64(erank)
    S, L, H = erank.shape
    out = np.empty((L, H), dtype=np.float64)
    _lib.oracle_prepare_mean(_p(erank, _dp), S, L, H, _p(out, _dp))
    return out


def group_labels(values, M: int, scope: int = 0) -> np.ndarray:
    """Rank-based group of every head: values [L, H] -> int32 [L, H], group 0 the highest values."""
    values = _f64(values)
    L, H = values.shape
    out = np.empty((L, H), dtype=np.int32)
    if _lib.oracle_group_labels(_p(values, _dp), L, H, int(M), int(scope), _p(out, _i32p)) != 0:
        raise ValueError("M must be between 1 and the size of the ranking set")
    return out


def majority_vote(erank, M: int, scope: int = 0):
    """Per-sample grouping and majority vote: erank [S, L, H] -> (votes int32 [L, H, M], labels int32 [L, H])."""
    erank = _f64(erank)
    S, L, H = erank.shape
    votes = np.empty((L, H, M), dtype=np.int32)
    labels = np.empty((L, H), dtype=np.int32)
    if _lib.oracle_majority_vote(_p(erank, _dp), S, L, H, int(M), int(scope), _p(votes, _i32p), _p(labels, _i32p)) != 0:
        raise ValueError("M must be between 1 and the size of the ranking set")
    return votes, labels


def entropy_wide(X, k_trunc: int = 32, center: bool = True, norm: int = 0, return_spectrum: bool = False):
    """(H_k, erank_k[, spectrum]) of a wide token matrix X [N, D] (hidden states, or a layer's heads side by
    side; Section 3.1 Eq. 1 and Section 3.2).  The same definition as `entropy`, with the two heavy steps
    handed to library routines so that D in the thousands finishes in seconds: the centred scatter matrix is a
    library matrix product of the centred rows, its eigenvalues come from the library's symmetric
    eigensolver; truncation and entropy are the oracle's own `truncated_entropy`."""
    X = _f64(X)
    if center:
        X = X - X.mean(axis=0, keepdims=True)
    lam = np.linalg.eigvalsh(X.T @ X)[::-1].copy()
    H, E = truncated_entropy(lam, k_trunc, norm)
    if return_spectrum:
        return H, E, lam
    return H, E


def decode_seed(score, idx) -> np.ndarray:
    """Cumulative scores of one head's cache after prefill: score [P] of the prefix positions, idx the kept
    positions (window positions are >= P) -> cum [len(idx)]."""
    score = _f64(score)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    cum = np.empty(len(idx), dtype=np.float64)
    _lib.oracle_decode_seed(_p(score, _dp), len(score), _p(idx, _i32p), len(idx), _p(cum, _dp))
    return cum


def retrieval_layer(values):
    """(layer, increase [L - 1]) for per-head values [L, H]: the layer after the largest rise of the layer mean."""
    values = _f64(values)
    L, H = values.shape
    inc = np.empty(L - 1, dtype=np.float64)
    return int(_lib.oracle_retrieval_layer(_p(values, _dp), L, H, _p(inc, _dp))), inc
