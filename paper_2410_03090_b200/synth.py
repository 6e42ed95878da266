"""Seeded synthetic inputs for the KV-compression pass.

This module only *makes data*: key/value caches and observation-window queries
with the shapes of the long-context models the paper evaluates (Llama-2/3 and
Mistral style, head_dim 128, grouped-query attention) and with the value
structure the paper reports for real heads: a few dominant eigen-directions
per head that differ from head to head (Section 3.2, "Observation"), a
minority of high-entropy heads, and heavy-hitter tokens.  It contains none of
the method's arithmetic (no entropy, budget, score or selection logic), so
both the CUDA library's tests and the CPU oracle's tests can draw their inputs
from it without sharing any code of the method.

Every unit (batch b, layer l, KV head h) is generated from its own counter
derived seed, so a single unit can be regenerated without its neighbours.
The stored tensor bytes are the single source of truth for both sides; values
differ between a CPU and a CUDA generator and that is fine, because whoever
consumes the data reads the same stored bytes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    """Shape, value recipe and hyper-parameters of one synthetic workload."""

    name: str
    B: int
    L: int
    H: int            # KV heads
    Hq: int           # query heads (Hq = G * H)
    N: int            # sequence length
    d: int            # head dimension
    w: int            # observation window (last w positions)
    dtype: str        # "bf16" or "fp32" (storage type of K, V, Qw)
    rank_rule: str    # "pow2_head": r = 2**h ; "loguniform": r log-uniform in [rank_lo, rank_hi]
    rank_lo: int
    rank_hi: int
    alpha: float      # scale of the low-rank part
    sigma: float      # scale of the iid noise part
    isotropic_every: int   # if > 0: the unit with h == l % isotropic_every has alpha = 0
    spike_frac: float      # fraction of positions whose K row is multiplied by spike_gain
    spike_gain: float
    avg_budget: int   # average tokens kept per head, window included
    M: int            # head groups
    n_max: int        # budget of the group with the largest truncated effective rank
    k_trunc: int      # entropy truncation k
    seed: int
    seed_per_sequence: bool = False
    pool_kernel: int = 7
    pool_mode: int = 0     # 0 = max, 1 = mean

    @property
    def G(self) -> int:
        return self.Hq // self.H

    @property
    def units(self) -> int:
        return self.B * self.L * self.H

    @property
    def total_rows(self) -> int:
        return self.units * self.avg_budget

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    def algorithmic_bytes(self) -> int:
        """Bytes the pass must move per the method's definition: K once, the
        window queries, the selected K/V rows read and written, the indices."""
        s = self.elem_bytes
        per_unit = (self.N * self.d * s + self.G * self.w * self.d * s
                    + 4 * self.avg_budget * self.d * s + 4 * self.avg_budget)
        return self.units * per_unit


def _budget(frac: float, N: int) -> Tuple[int, int]:
    b = int(round(frac * N))
    return b, int(round(5.0 * b / 3.0))


def _mk(name, B, L, H, Hq, N, w, dtype, rank_rule, lo, hi, alpha, sigma, iso, sf, sg,
        avg_budget, n_max, seed, per_seq=False) -> Workload:
    return Workload(name=name, B=B, L=L, H=H, Hq=Hq, N=N, d=128, w=w, dtype=dtype,
                    rank_rule=rank_rule, rank_lo=lo, rank_hi=hi, alpha=alpha, sigma=sigma,
                    isotropic_every=iso, spike_frac=sf, spike_gain=sg,
                    avg_budget=avg_budget, M=8, n_max=n_max, k_trunc=32, seed=seed,
                    seed_per_sequence=per_seq)


_b2, _n2 = _budget(0.05, 8192)        # 410, 683
_b3, _n3 = _budget(0.047, 32768)      # 1540, 2567
_b4, _n4 = _budget(0.094, 32768)      # 3080, 5133
_b5, _n5 = _budget(0.02, 131072)      # 2621, 4368

WORKLOADS: Dict[str, Workload] = {
    # single layer, fp32, head-specific rank 2**h plus 1e-3 noise
    "c1": _mk("c1", 1, 1, 8, 8, 512, 32, "fp32", "pow2_head", 1, 128, 1.0, 1e-3, 0, 0.0, 1.0,
              128, 213, 1001),
    # Llama-3-8B shape, 8K tokens
    "c2": _mk("c2", 1, 32, 8, 32, 8192, 32, "bf16", "loguniform", 4, 128, 2.0, 1.0, 0, 0.0, 1.0,
              _b2, _n2, 1002),
    # Llama-3-8B shape, 32K tokens, one near-isotropic head in eight
    "c3": _mk("c3", 1, 32, 8, 32, 32768, 64, "bf16", "loguniform", 4, 128, 2.0, 1.0, 8, 0.0, 1.0,
              _b3, _n3, 1003),
    # Mistral-7B shape, batch 4, norm spikes on 1 % of the positions
    "c4": _mk("c4", 4, 32, 8, 32, 32768, 32, "bf16", "loguniform", 4, 128, 2.0, 1.0, 0, 0.01, 8.0,
              _b4, _n4, 1004, per_seq=True),
    # Llama-3-70B shape, 128K tokens
    "c5": _mk("c5", 1, 80, 8, 64, 131072, 64, "bf16", "loguniform", 2, 128, 1.0, 0.1, 0, 0.0, 1.0,
              _b5, _n5, 1005),
}


def scaled(wl: Workload, *, N: int | None = None, L: int | None = None, B: int | None = None,
           name: str | None = None) -> Workload:
    """A smaller (or larger) copy of a workload with the same value recipe.
    The budget keeps its fraction of the sequence and the 5:3 ratio n_max : average."""
    N2 = wl.N if N is None else N
    frac = wl.avg_budget / wl.N
    b = max(wl.w + 8, int(round(frac * N2)))
    n_max = min(N2, int(round(5.0 * b / 3.0)))
    # keep the smallest group's target (2*avg - n_max for equal groups) at or above the window
    n_max = min(n_max, 2 * b - wl.w)
    return replace(wl, N=N2, L=wl.L if L is None else L, B=wl.B if B is None else B,
                   avg_budget=b, n_max=n_max,
                   name=name or f"{wl.name}_N{N2}")


# ----------------------------------------------------------------------------------------------
# seeds
# ----------------------------------------------------------------------------------------------
_MASK63 = (1 << 63) - 1


def _mix(*vals: int) -> int:
    """A 63-bit integer hash of a tuple of small integers (splitmix-style steps)."""
    x = 0x9E3779B97F4A7C15
    for v in vals:
        x = (x ^ (int(v) + 0x9E3779B97F4A7C15 + ((x << 6) & _MASK63) + (x >> 2))) & _MASK63
        x = (x * 0xBF58476D1CE4E5B9) & _MASK63
        x ^= x >> 31
    return x & _MASK63


def unit_seed(wl: Workload, b: int, l: int, h: int, stream: int) -> int:
    base = wl.seed + (b if wl.seed_per_sequence else 0)
    return _mix(base, b, l, h, stream)


def unit_rank(wl: Workload, b: int, l: int, h: int) -> int:
    if wl.rank_rule == "pow2_head":
        return min(wl.rank_hi, 1 << h)
    u = (_mix(wl.seed + (b if wl.seed_per_sequence else 0), b, l, h, 77) % (1 << 24)) / float(1 << 24)
    lo, hi = math.log(wl.rank_lo), math.log(wl.rank_hi)
    return int(max(wl.rank_lo, min(wl.rank_hi, round(math.exp(lo + u * (hi - lo))))))


def unit_alpha(wl: Workload, l: int, h: int) -> float:
    if wl.isotropic_every > 0 and h == l % wl.isotropic_every:
        return 0.0
    return wl.alpha


def spike_positions(wl: Workload, b: int, device: torch.device | str = "cpu") -> torch.Tensor | None:
    """Boolean [N] mask of the positions whose key rows are amplified; the same
    positions in every layer and head of sequence b."""
    if wl.spike_frac <= 0.0:
        return None
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(wl.seed + (b if wl.seed_per_sequence else 0), b, 991))
    u = torch.rand(wl.N, generator=g)
    return (u < wl.spike_frac).to(device)


# ----------------------------------------------------------------------------------------------
# generation
# ----------------------------------------------------------------------------------------------
def generate_unit(wl: Workload, b: int, l: int, h: int, device: torch.device | str = "cpu",
                  spikes: torch.Tensor | None = None):
    """K [N,d], V [N,d], Qw [G,w,d] of one unit, in the storage dtype.

    K = alpha * (A W) / sqrt(r) + sigma * E with A [N,r], W [r,d], E [N,d] iid N(0,1); the window
    queries of the G query heads that share this KV head use the same W (so the attention has
    structure) with their own A_q, E_q; V is iid N(0,1)."""
    dev = torch.device(device)
    r = unit_rank(wl, b, l, h)
    alpha = unit_alpha(wl, l, h)
    g = torch.Generator(device=dev)
    g.manual_seed(unit_seed(wl, b, l, h, 0))
    W = torch.randn(r, wl.d, generator=g, device=dev, dtype=torch.float32)
    A = torch.randn(wl.N, r, generator=g, device=dev, dtype=torch.float32)
    K = torch.randn(wl.N, wl.d, generator=g, device=dev, dtype=torch.float32) * wl.sigma
    if alpha != 0.0:
        K.addmm_(A, W, alpha=alpha / math.sqrt(r))
    if spikes is not None:
        K[spikes] *= wl.spike_gain
    del A
    Aq = torch.randn(wl.G * wl.w, r, generator=g, device=dev, dtype=torch.float32)
    Q = torch.randn(wl.G * wl.w, wl.d, generator=g, device=dev, dtype=torch.float32) * wl.sigma
    if alpha != 0.0:
        Q.addmm_(Aq, W, alpha=alpha / math.sqrt(r))
    V = torch.randn(wl.N, wl.d, generator=g, device=dev, dtype=torch.float32)
    dt = wl.torch_dtype
    return K.to(dt), V.to(dt), Q.view(wl.G, wl.w, wl.d).to(dt)


def generate(wl: Workload, device: torch.device | str = "cpu", pin: bool = False):
    """Whole workload: K, V [B,L,H,N,d] and Qw [B,L,Hq,w,d] (contiguous, storage dtype).
    Query head q of layer l belongs to KV head q // G."""
    dev = torch.device(device)
    dt = wl.torch_dtype
    kw = dict(dtype=dt, device=dev)
    if pin and dev.type == "cpu":
        kw["pin_memory"] = True
    K = torch.empty(wl.B, wl.L, wl.H, wl.N, wl.d, **kw)
    V = torch.empty(wl.B, wl.L, wl.H, wl.N, wl.d, **kw)
    Qw = torch.empty(wl.B, wl.L, wl.Hq, wl.w, wl.d, **kw)
    for b in range(wl.B):
        spikes = spike_positions(wl, b, dev)
        for l in range(wl.L):
            for h in range(wl.H):
                k, v, q = generate_unit(wl, b, l, h, dev, spikes)
                K[b, l, h] = k
                V[b, l, h] = v
                Qw[b, l, h * wl.G:(h + 1) * wl.G] = q
    return K, V, Qw


def hidden_states(wl: Workload, D: int, device: torch.device | str = "cpu") -> torch.Tensor:
    """X [B, N, D]: the residual-stream rows a hidden-state eviction moves (unit-variance noise in the
    storage dtype; the method only copies these rows, so their values carry no structure)."""
    g = torch.Generator(device=device).manual_seed(_mix(wl.seed, D, 7) & 0x7FFFFFFF)
    X = torch.empty(wl.B, wl.N, D, dtype=wl.torch_dtype, device=device)
    for b in range(wl.B):
        X[b] = torch.randn(wl.N, D, generator=g, device=device, dtype=torch.float32).to(wl.torch_dtype)
    return X


def unit_index(wl: Workload, u: int) -> Tuple[int, int, int]:
    """(b, l, h) of the flat unit number u (row-major over [B, L, H])."""
    h = u % wl.H
    l = (u // wl.H) % wl.L
    b = u // (wl.H * wl.L)
    return b, l, h
