"""The whole compression pass as one call: the four C-ABI calls back to back on one stream."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import binding as ub
from .synth import Workload


@dataclass
class PassOutput:
    entropy: torch.Tensor      # [B, L, H] float32, H_k
    erank: torch.Tensor        # [B, L, H] float32, erank_k
    budgets: torch.Tensor      # [B, L, H] int32
    offsets: torch.Tensor      # [units + 1] int64
    layer_group: torch.Tensor  # [B, L] int32
    layer_ctx: torch.Tensor    # [B, L] int32
    scores: torch.Tensor       # [B, L, H, N - w] float32, pooled window scores
    indices: torch.Tensor      # [total_rows] int32
    Kc: torch.Tensor           # [total_rows, d]
    Vc: torch.Tensor           # [total_rows, d]


class CompressionPass:
    """Pre-allocates every output of a workload once; `run` launches the pass without host syncs."""

    def __init__(self, wl: Workload, device: torch.device | str = "cuda", fused: bool = True):
        self.wl = wl
        self.fused = fused    # entropy call also produces the scorer's row statistics (one sweep over K less)
        self.device = torch.device(device)
        self.shape = ub.make_shape(wl.B, wl.L, wl.H, wl.Hq, wl.N, wl.d, wl.w, wl.dtype)
        self.ctx = ub.Context(self.shape, self.device)
        dev, u = self.device, wl.units
        f32, i32 = torch.float32, torch.int32
        self.out = PassOutput(
            entropy=torch.empty(wl.B, wl.L, wl.H, dtype=f32, device=dev),
            erank=torch.empty(wl.B, wl.L, wl.H, dtype=f32, device=dev),
            budgets=torch.empty(wl.B, wl.L, wl.H, dtype=i32, device=dev),
            offsets=torch.empty(u + 1, dtype=torch.int64, device=dev),
            layer_group=torch.empty(wl.B, wl.L, dtype=i32, device=dev),
            layer_ctx=torch.empty(wl.B, wl.L, dtype=i32, device=dev),
            scores=torch.empty(wl.B, wl.L, wl.H, wl.N - wl.w, dtype=f32, device=dev),
            indices=torch.empty(wl.total_rows, dtype=i32, device=dev),
            Kc=torch.empty(wl.total_rows, wl.d, dtype=wl.torch_dtype, device=dev),
            Vc=torch.empty(wl.total_rows, wl.d, dtype=wl.torch_dtype, device=dev),
        )

    def score(self, K: torch.Tensor, Qw: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
              eps: float = 0.0, dn: int = 0, n_last: int = 0, scope: int = 0,
              lse: Optional[torch.Tensor] = None) -> PassOutput:
        """Everything that needs only the keys and the window queries: entropy, budgets, scores, kept positions.
        With `lse` (the caller's log-sum-exp of every window row, [B, L, Hq, w] float32) the scorer makes one sweep
        over K and the entropy call runs the Gram stage on its own."""
        wl, o, ctx = self.wl, self.out, self.ctx
        fuse = self.fused and lse is None and wl.dtype == "bf16"
        ub.uncomp_entropy(ctx, K, wl.k_trunc, 1, 0, 0, o.entropy, o.erank, None, stream, Qw=Qw if fuse else None)
        ub.uncomp_assign_budgets(ctx, o.erank, wl.avg_budget, wl.M, wl.n_max, scope, eps, dn, n_last,
                                 o.budgets, o.offsets, o.layer_group, o.layer_ctx, stream)
        ub.uncomp_score_select(ctx, Qw, K, o.budgets, o.offsets, wl.total_rows, wl.pool_kernel, wl.pool_mode, 0.0,
                               o.scores, o.indices, stream, lse=lse, reuse_stats=fuse)
        return o

    def compact(self, K: torch.Tensor, V: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> PassOutput:
        """The gather of the kept K and V rows; the only step that touches the values."""
        wl, o = self.wl, self.out
        ub.uncomp_compact(self.ctx, K, V, o.indices, o.offsets, wl.total_rows, o.Kc, o.Vc, stream)
        return o

    def run(self, K: torch.Tensor, V: torch.Tensor, Qw: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
            eps: float = 0.0, dn: int = 0, n_last: int = 0, scope: int = 0,
            lse: Optional[torch.Tensor] = None) -> PassOutput:
        self.score(K, Qw, stream, eps, dn, n_last, scope, lse)
        return self.compact(K, V, stream)

    def run_one_call(self, K: torch.Tensor, V: torch.Tensor, Qw: torch.Tensor,
                     stream: Optional[torch.cuda.Stream] = None, eps: float = 0.0, dn: int = 0, n_last: int = 0,
                     scope: int = 0, lse: Optional[torch.Tensor] = None) -> PassOutput:
        """The same pass through `uncomp_compress`.  With `lse` the library sweeps the keys once: window scores and
        the Gram stage of the entropy come out of one kernel."""
        wl, o = self.wl, self.out
        ub.uncomp_compress(self.ctx, K, V, Qw, (wl.k_trunc, 1, 0, 0),
                           (wl.avg_budget, wl.M, wl.n_max, scope, eps, dn, n_last), (wl.pool_kernel, wl.pool_mode, 0.0),
                           o.entropy, o.erank, o.budgets, o.offsets, o.layer_group, o.layer_ctx, o.scores, o.indices,
                           o.Kc, o.Vc, lse=lse, stream=stream)
        return o

    def status(self, stream=None) -> int:
        return ub.uncomp_status(self.ctx, stream)


def eviction_plan(layer_group, layer_ctx):
    """[(layer, n_keep)] for one sequence: marshals the two host rows into `uncomp_eviction_plan` (the rule itself,
    paper Section 3.3.2, lives in the library)."""
    return ub.uncomp_eviction_plan(layer_group, layer_ctx)


class DecodeCache:
    """The ragged per-head cache after a prefill pass plus what the decode-time update needs (positions, cumulative
    scores, fill levels); `step` runs one `uncomp_decode_update` in place."""

    def __init__(self, cp: CompressionPass, out: Optional[PassOutput] = None):
        o = cp.out if out is None else out
        self.ctx, self.wl = cp.ctx, cp.wl
        self.offsets = o.offsets
        self.Kc, self.Vc = o.Kc, o.Vc
        self.pos = o.indices.clone()
        self.lens = o.budgets.reshape(-1).clone()
        self.cum = ub.uncomp_decode_seed(cp.ctx, o.scores, o.indices, o.offsets)
        self.max_cap = int(self.lens.max())
        self.evicted = torch.empty(self.wl.units, dtype=torch.int32, device=self.Kc.device)

    def step(self, qnew: torch.Tensor, knew: torch.Tensor, vnew: torch.Tensor, new_pos: torch.Tensor, protect: int = 1,
             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """qnew [B, L, Hq, d], knew / vnew [B, L, H, d], new_pos [B] int32; returns the evicted positions [units]."""
        ub.uncomp_decode_update(self.ctx, qnew, knew, vnew, new_pos, self.offsets, self.lens, self.max_cap, self.Kc,
                                self.Vc, self.pos, self.cum, protect=protect, evicted=self.evicted, stream=stream)
        return self.evicted
