"""Thin ctypes binding over libuncomp.so: the same names as include/uncomp.h, argument marshalling only.

Every step of the pass runs in the CUDA library.  PyTorch supplies device memory and streams.  There is
no CPU fallback: if the library cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

UNCOMP_BF16, UNCOMP_FP32 = 0, 1
UNCOMP_OK = 0
UNCOMP_E_NULL, UNCOMP_E_SHAPE, UNCOMP_E_ALIGN, UNCOMP_E_WORKSPACE = -1, -2, -3, -4
UNCOMP_E_PARAM, UNCOMP_E_CUDA, UNCOMP_E_LIMIT = -5, -6, -7
UNCOMP_STATUS_NOT_CONVERGED, UNCOMP_STATUS_TIMEOUT, UNCOMP_STATUS_BOUNDS, UNCOMP_STATUS_NONFINITE = 1, 2, 4, 8


class uncomp_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "L", "H", "Hq", "N", "d", "w", "dtype")]


class uncomp_strides(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("sB", "sL", "sH", "sN")]


class uncomp_entropy_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("k_trunc", "center", "norm", "max_iters")]


class uncomp_budget_params(C.Structure):
    _fields_ = [("avg_budget", C.c_int32), ("M", C.c_int32), ("n_max", C.c_int32), ("scope", C.c_int32),
                ("eps", C.c_float), ("dn", C.c_int32), ("n_last", C.c_int32)]


class uncomp_score_params(C.Structure):
    _fields_ = [("pool_kernel", C.c_int32), ("pool_mode", C.c_int32), ("scale", C.c_float),
                ("reuse_stats", C.c_int32)]


def _load() -> C.CDLL:
    # UNCOMP_DEBUG_LIBRARY=1 selects the bounds-checked build of the same sources (libuncomp_debug.so)
    debug = os.environ.get("UNCOMP_DEBUG_LIBRARY") == "1"
    path = _build.LIB_DEBUG if debug else _build.LIB
    if not os.path.exists(path):
        path = _build.build(debug=debug)
    lib = C.CDLL(path)
    vp, i32p, i64p, fp, dp = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p
    lib.uncomp_version.restype = C.c_int
    lib.uncomp_strerror.restype = C.c_char_p
    lib.uncomp_strerror.argtypes = [C.c_int]
    lib.uncomp_workspace_bytes.restype = C.c_size_t
    lib.uncomp_workspace_bytes.argtypes = [C.POINTER(uncomp_shape)]
    lib.uncomp_create.restype = C.c_int
    lib.uncomp_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(uncomp_shape), vp, C.c_size_t]
    lib.uncomp_destroy.restype = None
    lib.uncomp_destroy.argtypes = [vp]
    lib.uncomp_last_cuda_error.restype = C.c_int
    lib.uncomp_last_cuda_error.argtypes = [vp]
    lib.uncomp_entropy.restype = C.c_int
    lib.uncomp_entropy.argtypes = [vp, vp, uncomp_strides, C.POINTER(uncomp_entropy_params), vp, C.c_float, fp, fp, dp, vp]
    lib.uncomp_gram.restype = C.c_int
    lib.uncomp_gram.argtypes = [vp, vp, uncomp_strides, dp, vp]
    lib.uncomp_gram_static.restype = C.c_int
    lib.uncomp_gram_static.argtypes = [C.POINTER(uncomp_shape), vp, uncomp_strides, dp, vp]
    lib.uncomp_gram_static_max_bytes.restype = C.c_size_t
    lib.uncomp_assign_budgets.restype = C.c_int
    lib.uncomp_assign_budgets.argtypes = [vp, fp, C.POINTER(uncomp_budget_params), i32p, i64p, i32p, i32p, vp]
    lib.uncomp_score_select.restype = C.c_int
    lib.uncomp_score_select.argtypes = [vp, vp, vp, uncomp_strides, fp, i32p, i64p, C.POINTER(uncomp_score_params),
                                        fp, i32p, vp]
    lib.uncomp_compress.restype = C.c_int
    lib.uncomp_compress.argtypes = [vp, vp, vp, uncomp_strides, uncomp_strides, vp, fp, C.POINTER(uncomp_entropy_params),
                                    C.POINTER(uncomp_budget_params), C.POINTER(uncomp_score_params), fp, fp, i32p, i64p,
                                    i32p, i32p, fp, i32p, vp, vp, vp]
    lib.uncomp_compact.restype = C.c_int
    lib.uncomp_compact.argtypes = [vp, vp, vp, uncomp_strides, uncomp_strides, i32p, i64p, vp, vp, vp]
    lib.uncomp_set_option.restype = C.c_int
    lib.uncomp_set_option.argtypes = [vp, C.c_int, C.c_int]
    lib.uncomp_profile_enable.restype = C.c_int
    lib.uncomp_profile_enable.argtypes = [vp, C.c_int]
    lib.uncomp_profile_slots.restype = C.c_int
    lib.uncomp_profile_slot_name.restype = C.c_char_p
    lib.uncomp_profile_slot_name.argtypes = [C.c_int]
    lib.uncomp_profile_read.restype = C.c_int
    lib.uncomp_profile_read.argtypes = [vp, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.uncomp_entropy_wide_scratch_bytes.restype = C.c_size_t
    lib.uncomp_entropy_wide_scratch_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.uncomp_entropy_wide.restype = C.c_int
    lib.uncomp_entropy_wide.argtypes = [vp, vp, C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                        C.POINTER(uncomp_entropy_params), vp, C.c_size_t, fp, fp, dp, vp]
    lib.uncomp_measure_l2_sweep.restype = C.c_int
    lib.uncomp_measure_l2_sweep.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, vp]
    lib.uncomp_eviction_plan.restype = C.c_int
    lib.uncomp_eviction_plan.argtypes = [vp, vp, C.c_int32, vp, vp]
    lib.uncomp_retrieval_layer.restype = C.c_int
    lib.uncomp_retrieval_layer.argtypes = [vp, fp, i32p, fp, vp]
    lib.uncomp_prepare_groups.restype = C.c_int
    lib.uncomp_prepare_groups.argtypes = [vp, fp, C.c_int32, C.c_int32, C.c_int32, fp, i32p, i32p, i32p, vp]
    lib.uncomp_decode_seed.restype = C.c_int
    lib.uncomp_decode_seed.argtypes = [vp, fp, i32p, i64p, fp, vp]
    lib.uncomp_decode_update.restype = C.c_int
    lib.uncomp_decode_update.argtypes = [vp, vp, vp, vp, i32p, i64p, i32p, C.c_int32, C.c_int64, C.c_int32, C.c_float,
                                         vp, vp, i32p, fp, fp, i32p, vp]
    lib.uncomp_evict_hidden.restype = C.c_int
    lib.uncomp_evict_hidden.argtypes = [vp, vp, vp, uncomp_strides, vp, C.c_int32, C.c_int32, C.c_float, fp, i32p, vp, vp]
    lib.uncomp_status.restype = C.c_int
    lib.uncomp_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    return lib


lib = _load()


class UncompError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.uncomp_strerror(code).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != UNCOMP_OK:
        raise UncompError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def make_shape(B, L, H, Hq, N, d, w, dtype) -> uncomp_shape:
    code = {torch.bfloat16: UNCOMP_BF16, torch.float32: UNCOMP_FP32, "bf16": UNCOMP_BF16, "fp32": UNCOMP_FP32}[dtype]
    return uncomp_shape(B, L, H, Hq, N, d, w, code)


def strides_of(t: torch.Tensor) -> uncomp_strides:
    """Element strides of a [B, L, H, N, d] tensor (d contiguous)."""
    if t.dim() != 5 or t.stride(4) != 1:
        raise ValueError("expected a [B, L, H, N, d] tensor with a contiguous last dimension")
    return uncomp_strides(t.stride(0), t.stride(1), t.stride(2), t.stride(3))


def uncomp_workspace_bytes(shape: uncomp_shape) -> int:
    return int(lib.uncomp_workspace_bytes(C.byref(shape)))


class Context:
    """uncomp_ctx plus the torch tensor that backs its workspace."""

    def __init__(self, shape: uncomp_shape, device: torch.device | str = "cuda"):
        self.shape = shape
        nbytes = uncomp_workspace_bytes(shape)
        if nbytes == 0:
            raise UncompError(UNCOMP_E_SHAPE, "uncomp_workspace_bytes")
        self.device = torch.device(device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.workspace_bytes = nbytes
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib.uncomp_create(C.byref(h), C.byref(shape), C.c_void_p(self._ws_ptr), nbytes), "uncomp_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib.uncomp_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def uncomp_entropy(ctx: Context, K: torch.Tensor, k_trunc: int = 32, center: int = 1, norm: int = 0,
                   max_iters: int = 0, entropy: Optional[torch.Tensor] = None, erank: Optional[torch.Tensor] = None,
                   spectrum: Optional[torch.Tensor] = None, stream=None, Qw: Optional[torch.Tensor] = None,
                   scale: float = 0.0):
    """Qw given: the scorer's row statistics are produced in the same sweep over K (see uncomp.h)."""
    s = ctx.shape
    if entropy is None:
        entropy = torch.empty(s.B, s.L, s.H, dtype=torch.float32, device=K.device)
    if erank is None:
        erank = torch.empty(s.B, s.L, s.H, dtype=torch.float32, device=K.device)
    p = uncomp_entropy_params(k_trunc, center, norm, max_iters)
    _check(lib.uncomp_entropy(ctx.handle, _ptr(K), strides_of(K), C.byref(p), _ptr(Qw), scale, _ptr(entropy),
                              _ptr(erank), _ptr(spectrum), _stream(stream)), "uncomp_entropy")
    return entropy, erank


def uncomp_gram(ctx: Context, K: torch.Tensor, gram: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    s = ctx.shape
    if gram is None:
        gram = torch.empty(s.B * s.L * s.H, s.d * s.d + s.d, dtype=torch.float64, device=K.device)
    _check(lib.uncomp_gram(ctx.handle, _ptr(K), strides_of(K), _ptr(gram), _stream(stream)), "uncomp_gram")
    return gram


def uncomp_gram_static(shape: uncomp_shape, K: torch.Tensor, gram: torch.Tensor, stream=None) -> torch.Tensor:
    """uncomp_gram without a context or workspace (scratch lives in a fixed array inside the library).
    `gram` is the caller's [units, d*d + d] float64 output; nothing is allocated here."""
    _check(lib.uncomp_gram_static(C.byref(shape), _ptr(K), strides_of(K), _ptr(gram), _stream(stream)),
           "uncomp_gram_static")
    return gram


def uncomp_assign_budgets(ctx: Context, erank: torch.Tensor, avg_budget: int, M: int, n_max: int, scope: int = 0,
                          eps: float = 0.0, dn: int = 0, n_last: int = 0, budgets=None, offsets=None,
                          layer_group=None, layer_ctx=None, stream=None):
    s = ctx.shape
    dev = erank.device
    units = s.B * s.L * s.H
    if budgets is None:
        budgets = torch.empty(s.B, s.L, s.H, dtype=torch.int32, device=dev)
    if offsets is None:
        offsets = torch.empty(units + 1, dtype=torch.int64, device=dev)
    if layer_group is None:
        layer_group = torch.empty(s.B, s.L, dtype=torch.int32, device=dev)
    if layer_ctx is None:
        layer_ctx = torch.empty(s.B, s.L, dtype=torch.int32, device=dev)
    p = uncomp_budget_params(avg_budget, M, n_max, scope, eps, dn, n_last)
    _check(lib.uncomp_assign_budgets(ctx.handle, _ptr(erank), C.byref(p), _ptr(budgets), _ptr(offsets),
                                     _ptr(layer_group), _ptr(layer_ctx), _stream(stream)), "uncomp_assign_budgets")
    return budgets, offsets, layer_group, layer_ctx


def uncomp_score_select(ctx: Context, Qw: torch.Tensor, K: torch.Tensor, budgets: torch.Tensor,
                        offsets: torch.Tensor, total_rows: int, pool_kernel: int = 7, pool_mode: int = 0,
                        scale: float = 0.0, scores: Optional[torch.Tensor] = None,
                        indices: Optional[torch.Tensor] = None, stream=None, lse: Optional[torch.Tensor] = None,
                        reuse_stats: bool = False):
    """lse [B, L, Hq, w] float32 (natural-log sum of exponentials of every window row's scaled logits): the
    caller's softmax normalisers, one sweep over K instead of two.  reuse_stats: take the statistics a preceding
    uncomp_entropy(..., Qw=Qw) left in the workspace."""
    if indices is None:
        indices = torch.empty(total_rows, dtype=torch.int32, device=K.device)
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous()):
        raise ValueError("lse must be a contiguous float32 tensor [B, L, Hq, w]")
    p = uncomp_score_params(pool_kernel, pool_mode, scale, int(reuse_stats))
    _check(lib.uncomp_score_select(ctx.handle, _ptr(Qw), _ptr(K), strides_of(K), _ptr(lse), _ptr(budgets),
                                   _ptr(offsets), C.byref(p), _ptr(scores), _ptr(indices), _stream(stream)),
           "uncomp_score_select")
    return indices


def uncomp_compress(ctx: Context, K: torch.Tensor, V: torch.Tensor, Qw: torch.Tensor, entropy_params, budget_params,
                    score_params, entropy: torch.Tensor, erank: torch.Tensor, budgets: torch.Tensor,
                    offsets: torch.Tensor, layer_group: Optional[torch.Tensor], layer_ctx: Optional[torch.Tensor],
                    scores: Optional[torch.Tensor], indices: torch.Tensor, Kc: torch.Tensor, Vc: torch.Tensor,
                    lse: Optional[torch.Tensor] = None, stream=None) -> None:
    """The whole pass in one call (every output pre-allocated by the caller).  entropy_params = (k_trunc, center,
    norm, max_iters), budget_params = (avg_budget, M, n_max, scope, eps, dn, n_last), score_params = (pool_kernel,
    pool_mode, scale).  With `lse` [B, L, Hq, w] float32 the keys are swept once."""
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous()):
        raise ValueError("lse must be a contiguous float32 tensor [B, L, Hq, w]")
    ep = uncomp_entropy_params(*entropy_params)
    bp = uncomp_budget_params(*budget_params)
    sp = uncomp_score_params(score_params[0], score_params[1], score_params[2], 0)
    _check(lib.uncomp_compress(ctx.handle, _ptr(K), _ptr(V), strides_of(K), strides_of(V), _ptr(Qw), _ptr(lse),
                               C.byref(ep), C.byref(bp), C.byref(sp), _ptr(entropy), _ptr(erank), _ptr(budgets),
                               _ptr(offsets), _ptr(layer_group), _ptr(layer_ctx), _ptr(scores), _ptr(indices), _ptr(Kc),
                               _ptr(Vc), _stream(stream)), "uncomp_compress")


def uncomp_measure_l2_sweep(A: torch.Tensor, passes: int = 1, stream=None) -> None:
    """A [rows, cols] float32 on the device (overwritten): `passes` read-modify-write sweeps, for timing."""
    if A.dtype != torch.float32 or A.dim() != 2 or not A.is_contiguous():
        raise ValueError("expected a contiguous float32 matrix")
    _check(lib.uncomp_measure_l2_sweep(_ptr(A), A.shape[0], A.shape[1], passes, _stream(stream)),
           "uncomp_measure_l2_sweep")


def uncomp_eviction_plan(layer_group, layer_ctx):
    """Host rows [L] of one sequence (lists, numpy or CPU tensors) -> [(layer, n_keep)]."""
    import numpy as np
    g = np.ascontiguousarray(np.asarray(layer_group, dtype=np.int32).reshape(-1))
    c = np.ascontiguousarray(np.asarray(layer_ctx, dtype=np.int32).reshape(-1))
    if g.shape != c.shape:
        raise ValueError("layer_group and layer_ctx must have the same length")
    L = int(g.shape[0])
    out_l, out_k = np.zeros(max(L, 1), dtype=np.int32), np.zeros(max(L, 1), dtype=np.int32)
    n = lib.uncomp_eviction_plan(C.c_void_p(g.ctypes.data), C.c_void_p(c.ctypes.data), L,
                                 C.c_void_p(out_l.ctypes.data), C.c_void_p(out_k.ctypes.data))
    if n < 0:
        raise UncompError(n, "uncomp_eviction_plan")
    return [(int(out_l[i]), int(out_k[i])) for i in range(n)]


def uncomp_compact(ctx: Context, K: torch.Tensor, V: torch.Tensor, indices: torch.Tensor, offsets: torch.Tensor,
                   total_rows: int, Kc: Optional[torch.Tensor] = None, Vc: Optional[torch.Tensor] = None, stream=None):
    d = ctx.shape.d
    if Kc is None:
        Kc = torch.empty(total_rows, d, dtype=K.dtype, device=K.device)
    if Vc is None:
        Vc = torch.empty(total_rows, d, dtype=V.dtype, device=V.device)
    _check(lib.uncomp_compact(ctx.handle, _ptr(K), _ptr(V), strides_of(K), strides_of(V), _ptr(indices),
                              _ptr(offsets), _ptr(Kc), _ptr(Vc), _stream(stream)), "uncomp_compact")
    return Kc, Vc


def uncomp_evict_hidden(ctx: Context, qlast: torch.Tensor, K_layer: torch.Tensor, X: torch.Tensor, n_keep: int,
                        scale: float = 0.0, scores: Optional[torch.Tensor] = None,
                        indices: Optional[torch.Tensor] = None, Xout: Optional[torch.Tensor] = None, stream=None):
    """qlast [B, Hq, d], K_layer [B, H, N, d] (any 16-byte aligned strides, d contiguous), X [B, N, D]."""
    B, N, D = X.shape
    if K_layer.dim() != 4 or K_layer.stride(3) != 1:
        raise ValueError("expected K_layer [B, H, N, d] with a contiguous last dimension")
    if indices is None:
        indices = torch.empty(B, n_keep, dtype=torch.int32, device=X.device)
    if Xout is None:
        Xout = torch.empty(B, n_keep, D, dtype=X.dtype, device=X.device)
    st = uncomp_strides(K_layer.stride(0), 0, K_layer.stride(1), K_layer.stride(2))
    _check(lib.uncomp_evict_hidden(ctx.handle, _ptr(qlast), _ptr(K_layer), st, _ptr(X), D, n_keep, scale, _ptr(scores),
                                   _ptr(indices), _ptr(Xout), _stream(stream)), "uncomp_evict_hidden")
    return indices, Xout


def uncomp_decode_seed(ctx: Context, scores: torch.Tensor, indices: torch.Tensor, offsets: torch.Tensor,
                       cum: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Cumulative scores of the ragged cache right after prefill, from the outputs of uncomp_score_select."""
    if cum is None:
        cum = torch.empty(indices.shape[0], dtype=torch.float32, device=indices.device)
    _check(lib.uncomp_decode_seed(ctx.handle, _ptr(scores), _ptr(indices), _ptr(offsets), _ptr(cum), _stream(stream)),
           "uncomp_decode_seed")
    return cum


def uncomp_decode_update(ctx: Context, qnew: torch.Tensor, knew: torch.Tensor, vnew: torch.Tensor,
                         new_pos: torch.Tensor, offsets: torch.Tensor, lens: torch.Tensor, max_cap: int,
                         Kc: torch.Tensor, Vc: torch.Tensor, pos: torch.Tensor, cum: torch.Tensor, protect: int = 1,
                         scale: float = 0.0, p: Optional[torch.Tensor] = None,
                         evicted: Optional[torch.Tensor] = None, stream=None):
    """One decode step on the ragged cache, in place: qnew [B, L, Hq, d], knew / vnew [B, L, H, d],
    new_pos [B] int32, offsets [units + 1] int64, lens [units] int32, Kc / Vc [total_cap, d], pos int32 and
    cum float32 [total_cap]; optional outputs p [total_cap + units] and evicted [units]."""
    _check(lib.uncomp_decode_update(ctx.handle, _ptr(qnew), _ptr(knew), _ptr(vnew), _ptr(new_pos), _ptr(offsets),
                                    _ptr(lens), max_cap, Kc.shape[0], protect, scale, _ptr(Kc), _ptr(Vc), _ptr(pos),
                                    _ptr(cum), _ptr(p), _ptr(evicted), _stream(stream)), "uncomp_decode_update")


def uncomp_entropy_wide(ctx: Context, X: torch.Tensor, k_trunc: int = 32, center: int = 1, norm: int = 0,
                        max_iters: int = 0, scratch: Optional[torch.Tensor] = None, spectrum: bool = False, stream=None):
    """X [count, N, D] bf16 (rows may be strided, features contiguous) -> (entropy [count], erank [count]
    [, spectrum [count, k]])."""
    if X.dim() != 3 or X.stride(2) != 1:
        raise ValueError("expected X [count, N, D] with a contiguous last dimension")
    count, N, D = X.shape
    need = lib.uncomp_entropy_wide_scratch_bytes(N, D)
    if scratch is None:
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=X.device)
    ent = torch.empty(count, dtype=torch.float32, device=X.device)
    er = torch.empty(count, dtype=torch.float32, device=X.device)
    spec = torch.empty(count, min(k_trunc, D), dtype=torch.float64, device=X.device) if spectrum else None
    params = uncomp_entropy_params(k_trunc, center, norm, max_iters)
    _check(lib.uncomp_entropy_wide(ctx.handle, _ptr(X), count, X.stride(0), X.stride(1), N, D, C.byref(params),
                                   _ptr(scratch), scratch.numel(), _ptr(ent), _ptr(er), _ptr(spec), _stream(stream)),
           "uncomp_entropy_wide")
    return (ent, er, spec) if spectrum else (ent, er)


def uncomp_retrieval_layer(ctx: Context, values: torch.Tensor, stream=None):
    """values [L, H] float32 -> (layer int32 [1], increase float32 [L - 1])."""
    L = values.shape[0]
    layer = torch.empty(1, dtype=torch.int32, device=values.device)
    inc = torch.empty(L - 1, dtype=torch.float32, device=values.device)
    _check(lib.uncomp_retrieval_layer(ctx.handle, _ptr(values), _ptr(layer), _ptr(inc), _stream(stream)),
           "uncomp_retrieval_layer")
    return layer, inc


def uncomp_prepare_groups(ctx: Context, erank: torch.Tensor, M: int, scope: int = 0, stream=None):
    """erank [S, L, H] float32 -> (mean [L, H], group_mean [L, H], votes [L, H, M], group_vote [L, H])."""
    S, L, H = erank.shape
    dev = erank.device
    mean = torch.empty(L, H, dtype=torch.float32, device=dev)
    gm = torch.empty(L, H, dtype=torch.int32, device=dev)
    votes = torch.empty(L, H, M, dtype=torch.int32, device=dev)
    gv = torch.empty(L, H, dtype=torch.int32, device=dev)
    _check(lib.uncomp_prepare_groups(ctx.handle, _ptr(erank), S, M, scope, _ptr(mean), _ptr(gm), _ptr(votes), _ptr(gv),
                                     _stream(stream)), "uncomp_prepare_groups")
    return mean, gm, votes, gv


def uncomp_status(ctx: Context, stream=None) -> int:
    bits = C.c_uint32(0)
    _check(lib.uncomp_status(ctx.handle, _stream(stream), C.byref(bits)), "uncomp_status")
    return int(bits.value)


UNCOMP_OPT_CUDA_CORES = 1


def uncomp_set_option(ctx: Context, option: int, value: int) -> None:
    _check(lib.uncomp_set_option(ctx.handle, option, value), "uncomp_set_option")


def uncomp_profile_enable(ctx: Context, on: bool) -> None:
    _check(lib.uncomp_profile_enable(ctx.handle, int(on)), "uncomp_profile_enable")


def uncomp_profile_read(ctx: Context) -> dict:
    """{kernel name: (total ms, launches)} since the last read; waits for the recorded events."""
    n = lib.uncomp_profile_slots()
    ms = (C.c_float * n)()
    cnt = (C.c_int32 * n)()
    _check(lib.uncomp_profile_read(ctx.handle, n, ms, cnt), "uncomp_profile_read")
    return {lib.uncomp_profile_slot_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}
