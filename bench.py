#!/usr/bin/env python
"""Benchmark of the UNComp prefill-end KV-compression pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

One step = one whole pass (entropy -> budgets -> window scores + selection -> compaction) over one batch
of synthetic input.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own
replica-sized shard (its own sequence of the same shape: units are independent, no collective on the
data path) and the value is the sum over ranks divided by the slowest rank's time.

`--impl reference` times the plain fp64 CPU oracle (oracle/) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# Hardware counters of the two scorer kernels from one ncu capture of a smaller case of the same workload
# (80 units x 16384 tokens): DRAM bytes per (unit x token) of one launch (dram__bytes_read.sum +
# dram__bytes_write.sum; traffic grows with units x tokens, so a full-size launch is scaled by that product),
# tensor-pipe and exponential-unit (XU) activity in % of peak.  They describe the kernel source whose SHA-256 is
# recorded beside them: when the file has changed since the capture, the bench prints null instead.
NCU_COUNTERS = {
    "source": "paper_2410_03090_b200/csrc/scores_tc.cu",
    "sha256": "5d7704c735797925551e24bea29c1be8724667b424932621e0c8c7a1c44d4428",
    "capture": "ncu --set full, one launch per kernel, c3 scaled to N 16384 x 10 layers; summary in profiles/",
    "kernels": {
        "gram_score_stats": {"dram_bytes_per_unit_token": (342.482688e6 + 21.898496e6) / (80 * 16384),
                             "tensor_pipe_pct": 40.0, "xu_pipe_pct": 54.4},
        "score_colsum": {"dram_bytes_per_unit_token": (340.933120e6 + 7.131136e6) / (80 * 16384),
                         "tensor_pipe_pct": 33.9, "xu_pipe_pct": 67.9},
        "gram_score_colsum": {"dram_bytes_per_unit_token": (341.082880e6 + 24.134912e6) / (80 * 16384),
                              "tensor_pipe_pct": 42.8, "xu_pipe_pct": 57.1},
    },
}
EXP_KERNELS = ("score_stats", "score_colsum", "gram_score_stats", "gram_score_colsum")
METRIC = "compression_pass_tokens_per_s"
UNIT = "tokens/s"


def ncu_counters(kernel):
    """Counters recorded for `kernel`, or None when there are none or the kernel source has changed since."""
    import hashlib
    ent = NCU_COUNTERS["kernels"].get(kernel)
    if not ent or not NCU_COUNTERS["sha256"]:
        return None
    try:
        with open(os.path.join(ROOT, NCU_COUNTERS["source"]), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return ent if digest == NCU_COUNTERS["sha256"] else None


def tensor_peak(peaks, clocks, timed_s):
    """Which measured bf16 peak a kernel timed inside this run is held against.  The burst figure applies to a
    short timed region that ran at full clocks with no power cap; once the region lasts a second or more, or
    the clock record shows sw_power_cap, the GPU is in the regime the sustained figure was taken in."""
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    if timed_s < 1.0 and not capped:
        return peaks["bf16_burst"], "burst bf16"
    return peaks["bf16_sustained"], "sustained bf16"


def composite_bound(wl, qk_passes, hbm_gbs, tensor_tflops, sm_count, sm_mhz, ms_step):
    """Lower bounds of one pass of the whole workload and the fraction of the largest the pass reaches:
    t_hbm (algorithmic bytes at the copy peak), t_tensor (Gram + qk_passes window products at the bf16 peak),
    t_exp (qk_passes x rows x tokens exponentials at 16 per clock per SM)."""
    u, N, d, rows = wl.units, wl.N, wl.d, wl.G * wl.w
    flops = u * (2.0 * N * d * d + qk_passes * 2.0 * rows * d * N)
    exps = u * qk_passes * float(rows) * N
    t_hbm = wl.algorithmic_bytes() / (hbm_gbs * 1e9) * 1e3
    t_tensor = flops / (tensor_tflops * 1e12) * 1e3
    t_exp = exps / (sm_count * 16.0 * sm_mhz * 1e6) * 1e3
    t_min = max(t_hbm, t_tensor, t_exp)
    return {"qk_passes": qk_passes, "t_hbm_ms": round(t_hbm, 4), "t_tensor_ms": round(t_tensor, 4),
            "t_exp_ms": round(t_exp, 4), "t_min_ms": round(t_min, 4),
            "binding": "hbm" if t_min == t_hbm else ("tensor" if t_min == t_tensor else "exp"),
            "frac_of_t_min": round(t_min / ms_step, 4) if ms_step else None}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p["bf16_tflops_sustained"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.002)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s), "power_w_max": round(max(self.power), 1) if self.power else None}


# ------------------------------------------------------------------------------------- roofline per kernel
def kernel_specs(wl, peaks, sustained, D=None, n_keep=None, cache_rows=None):
    """Algorithmic work of one launch of each kernel of the pass (units of one rank).  D and n_keep (width of
    a hidden-state row, tokens kept) size the kernels of the hidden-state eviction step; without them those
    entries carry no work figure."""
    u, N, d, P = wl.units, wl.N, wl.d, wl.N - wl.w
    rows, s = wl.G * wl.w, wl.elem_bytes
    # `sustained`: True / False pick one of the measured bf16 peaks, a number is taken as the peak itself
    tens = float(sustained) if not isinstance(sustained, bool) else (
        peaks["bf16_sustained"] if sustained else peaks["bf16_burst"])
    if wl.dtype == "fp32":
        tens = tens / 2.0 / 16.0   # fp32 inputs run on the CUDA cores; no tensor peak applies
    hbm = peaks["hbm_gbs"]
    return {
        "gram": ("tensor", 2.0 * N * d * d * u / 1e12, tens, "TFLOP/s"),
        "gram_score_stats": ("tensor", (2.0 * N * d * d + 2.0 * rows * d * N) * u / 1e12, tens, "TFLOP/s"),
        "gram_score_colsum": ("tensor", (2.0 * N * d * d + 2.0 * rows * d * N) * u / 1e12, tens, "TFLOP/s"),
        "score_stats": ("tensor", 2.0 * rows * d * N * u / 1e12, tens, "TFLOP/s"),
        "score_colsum": ("tensor", 2.0 * rows * d * P * u / 1e12, tens, "TFLOP/s"),
        "pool_select": ("hbm", (2.0 * u * P * 4 + wl.total_rows * 4) / 1e9, hbm, "GB/s"),
        "compact": ("hbm", wl.total_rows * (4.0 * d * s + 4) / 1e9, hbm, "GB/s"),
        "eigen_entropy": ("alu", None, None, None),
        "budgets": ("alu", None, None, None),
        "stats_merge": ("hbm", None, None, None),
        # hidden-state eviction of one layer boundary: keys of one layer in, Hq logits per token out;
        # logits in, one score per token out; kept rows of the hidden state in and out
        "evict_logits": ("hbm", (wl.B * wl.H * N * (d * s + wl.G * 4.0)) / 1e9 if D else None, hbm, "GB/s"),
        "evict_scores": ("hbm", (wl.B * N * (wl.Hq * 4.0 + 4.0)) / 1e9 if D else None, hbm, "GB/s"),
        "evict_gather": ("hbm", (wl.B * n_keep * (2.0 * D * s + 4.0)) / 1e9 if D else None, hbm, "GB/s"),
        # decode-time update over cache_rows cached rows: keys in, G logits per row out; logits, cumulative
        # score and position in, cumulative score out; one new key and value row per unit
        "decode_logits": ("hbm", cache_rows * (d * s + wl.G * 4.0) / 1e9 if cache_rows else None, hbm, "GB/s"),
        "decode_accumulate": ("hbm", cache_rows * (wl.G * 4.0 + 12.0) / 1e9 if cache_rows else None, hbm, "GB/s"),
        "decode_commit": ("hbm", None, None, None),
        "prepare_vote": ("alu", None, None, None),
        "prepare_finish": ("alu", None, None, None),
        "wide_gram": ("tensor", None, None, None),
        "wide_assemble": ("hbm", None, None, None),
        "wide_tridiag": ("alu", None, None, None),
        "wide_eigen_entropy": ("alu", None, None, None),
    }


# ------------------------------------------------------------------------------------------ oracle timing
def time_oracle(wl, unit_list, fetch, threads, data=None):
    """Wall time of the oracle chain over the given units, one thread per unit where possible.
    The entropy and score stages (all the floating-point work) run in parallel over units; the budget
    rule needs every head of a layer and runs once per layer."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    if data is None:
        data = [fetch(u) for u in unit_list]
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        er = list(ex.map(lambda kvq: oracle.entropy(kvq[0], k_trunc=wl.k_trunc)[1], data))
    n = len(data)
    M = min(wl.M, n)
    n_max = wl.n_max
    bud, off, _, _ = oracle.budgets(np.array(er, dtype=np.float32).astype(np.float64).reshape(1, 1, n), wl.N, wl.w,
                                    wl.avg_budget, M, n_max)

    def rest(i):
        K, V, Q = data[i]
        sc = oracle.pool(oracle.window_scores(Q, K), wl.pool_kernel, wl.pool_mode)
        idx = oracle.select(sc, wl.w, int(bud[0, 0, i]))
        oracle.compact(np.ascontiguousarray(K).view(np.uint8).reshape(wl.N, -1), idx)
        oracle.compact(np.ascontiguousarray(V).view(np.uint8).reshape(wl.N, -1), idx)
        return len(idx)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(rest, range(n)))
    return time.perf_counter() - t0


def run_reference(args):
    """The oracle as the reference arm: rank 0 only, CPU only, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from paper_2410_03090_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    threads = min(os.cpu_count() or 1, 16)
    total_steps = args.steps + args.warmup
    per_step = wl.H if total_steps <= 30 else max(1, (30 * wl.H) // total_steps)
    per_step = max(1, min(per_step, wl.H))

    def fetch(u):
        b, l, h = synth.unit_index(wl, u)
        K, V, Q = synth.generate_unit(wl, b, l, h, "cpu", synth.spike_positions(wl, b))
        return K.double().numpy(), V.double().numpy(), Q.double().numpy()

    layer_units = list(range(per_step))
    data = [fetch(u) for u in layer_units]
    times = []
    for s in range(total_steps):
        t = time_oracle(wl, layer_units, fetch, threads, data)
        if s >= args.warmup:
            times.append(t)
    t_step = sum(times) / len(times)
    # tokens/s of the whole workload at this rate: the sample is per_step of wl.units units
    value = wl.B * wl.N / (t_step * wl.units / per_step)
    sample = f"{per_step} of {wl.units} units (heads 0..{per_step - 1} of layer 0) per step, whole oracle chain"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": _workload_name(wl), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def prefill_lse(wl, K, Qw):
    """[B, L, Hq, w] float32: the natural-log sum of exponentials of every window row's scaled, causally visible
    logits.  Stands in for what the prefill attention kernel keeps per row; an input of the timed call."""
    import torch
    P = wl.N - wl.w
    out = torch.empty(wl.B, wl.L, wl.Hq, wl.w, dtype=torch.float32, device=K.device)
    pos = torch.arange(wl.N, device=K.device)[None, :]
    hidden = (pos > (P + torch.arange(wl.w, device=K.device))[:, None])[None]
    for b in range(wl.B):
        for l in range(wl.L):
            for h in range(wl.H):
                q = Qw[b, l, h * wl.G:(h + 1) * wl.G].float()
                s = torch.einsum("gwd,nd->gwn", q, K[b, l, h].float()) / wl.d ** 0.5
                out[b, l, h * wl.G:(h + 1) * wl.G] = torch.logsumexp(s.masked_fill(hidden, float("-inf")), dim=-1)
    return out


def _workload_name(wl):
    return (f"{wl.name}: B{wl.B} L{wl.L} Hkv{wl.H} Hq{wl.Hq} N{wl.N} d{wl.d} w{wl.w} {wl.dtype}, "
            f"avg budget {wl.avg_budget}, M{wl.M}, n_max {wl.n_max}, k{wl.k_trunc}")


# ------------------------------------------------------------------------------- hidden-state eviction
def run_hidden(args):
    """One layer-group boundary of the prefill (paper Section 3.3.2): the attention of the last token, summed
    over the query heads, ranks the positions; the hidden state keeps the best n_keep rows.  Sequences are
    independent, so ranks are replicas, as for the KV pass."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200 import shard, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pass has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=dev)
    base = synth.scaled(synth.WORKLOADS[args.workload], N=args.scale_N or None, L=1, B=args.hidden_batch)
    wl = shard.rank_workload(base, rank)
    D, n_keep = args.hidden_width, wl.N // 2
    peaks = _peaks()
    K, _, Qw = synth.generate(wl, dev)
    Kl = K[:, 0]
    q = Qw[:, 0, :, -1, :].contiguous()
    X = synth.hidden_states(wl, D, dev)
    ctx = ub.Context(ub.make_shape(wl.B, 1, wl.H, wl.Hq, wl.N, wl.d, 1, wl.dtype))
    scores = torch.empty(wl.B, wl.N - 1, device=dev)
    idx = torch.empty(wl.B, n_keep, dtype=torch.int32, device=dev)
    Xout = torch.empty(wl.B, n_keep, D, dtype=X.dtype, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()

    def step(q_, K_, X_):
        ub.uncomp_evict_hidden(ctx, q_, K_, X_, n_keep, scores=scores, indices=idx, Xout=Xout)

    for _ in range(args.warmup):
        step(q, Kl, X)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    sampler = ClockSampler(local)
    sampler.start()
    ub.uncomp_profile_enable(ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(args.steps):
        step(q, Kl, X)
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    prof = ub.uncomp_profile_read(ctx)
    ub.uncomp_profile_enable(ctx, False)
    ms_step = shard.max_over_ranks(ev0.elapsed_time(ev1), dev, world) / args.steps
    tokens_step = wl.B * wl.N * world
    specs = kernel_specs(wl, peaks, True, D=D, n_keep=n_keep)
    kernels, launches = {}, 0
    total_ms = sum(v[0] for v in prof.values())
    for name, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        launches += cnt
        bound, work, peak, unit = specs[name]
        avg_ms = ms / cnt
        ent = {"launches_per_step": cnt // args.steps, "avg_ms": round(avg_ms, 5), "share": round(ms / total_ms, 4),
               "bound": bound}
        if work is not None:
            ach = work / (avg_ms / 1e3)
            ent.update({"achieved": round(ach, 2), "peak": peak, "unit": unit, "frac": round(ach / peak, 4)})
        kernels[name] = ent
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    kd = kernels[dom]
    roofline = {"kernel": dom, "bound": kd["bound"], "achieved": kd.get("achieved"), "peak": kd.get("peak"),
                "unit": kd.get("unit"), "frac": kd.get("frac"), "traffic": None,
                "peak_source": f"of {peaks['source']} (copy)", "avg_ms": kd["avg_ms"], "share": kd["share"]}
    alg_bytes = sum(specs[n][1] for n in ("evict_logits", "evict_scores", "evict_gather")) * 1e9

    e2e = None
    if args.e2e_steps > 0:
        hq = torch.empty(q.shape, dtype=q.dtype, pin_memory=True).copy_(q)
        hK = torch.empty(Kl.shape, dtype=K.dtype, pin_memory=True).copy_(Kl)
        hX = torch.empty(X.shape, dtype=X.dtype, pin_memory=True).copy_(X)
        outs = [idx, Xout]
        houts = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
        dq, dK, dX = torch.empty_like(hq, device=dev), torch.empty_like(hK, device=dev), torch.empty_like(X)

        # the results return on a second stream and overlap the next step's input copies (full-duplex link); the next
        # step waits for them before it overwrites the outputs
        out_stream = torch.cuda.Stream(device=dev)
        done_step, done_out = torch.cuda.Event(), torch.cuda.Event()

        def e2e_step(first=False):
            dq.copy_(hq, non_blocking=True)
            dK.copy_(hK, non_blocking=True)
            dX.copy_(hX, non_blocking=True)
            if not first:
                stream.wait_event(done_out)
            step(dq, dK, dX)
            done_step.record(stream)
            out_stream.wait_event(done_step)
            with torch.cuda.stream(out_stream):
                for h, t in zip(houts, outs):
                    h.copy_(t, non_blocking=True)
                done_out.record(out_stream)

        e2e_step(first=True)
        torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        stream.wait_event(done_out)
        e1.record(stream)
        torch.cuda.synchronize()
        barrier()
        ms_e = shard.max_over_ranks(e0.elapsed_time(e1), dev, world)
        e2e = {"value": tokens_step / (ms_e / args.e2e_steps / 1e3), "unit": UNIT,
               "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in (hq, hK, hX)),
               "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in outs), "steps": args.e2e_steps}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        qn, Kn = q[0].double().cpu().numpy(), Kl[0].double().cpu().numpy()
        rows = X[0].contiguous().view(torch.uint8).reshape(wl.N, -1).cpu().numpy()
        t0 = time.perf_counter()
        sc = oracle.last_token_scores(qn, Kn)
        keep = oracle.select(np.ascontiguousarray(sc[:-1]), 1, n_keep)
        oracle.compact(rows, keep)
        t_cpu = time.perf_counter() - t0
        cpu_baseline = {"value": wl.N / t_cpu, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"1 of {wl.B} sequences, whole oracle chain, {t_cpu:.2f} s wall"}

    if rank == 0:
        line = {"metric": "hidden_state_eviction_tokens_per_s", "value": tokens_step / (ms_step / 1e3), "unit": UNIT,
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
                "data": "synthetic",
                "config": {"workload": f"hidden-state eviction at one layer-group boundary: B{wl.B} Hkv{wl.H} "
                                       f"Hq{wl.Hq} N{wl.N} d{wl.d} D{D} {wl.dtype}, keep {n_keep}",
                           "l2": f"inputs larger than L2 (keys {Kl.numel() * K.element_size() / 1e9:.2f} GB + hidden "
                                 f"state {X.numel() * X.element_size() / 1e9:.2f} GB per step)",
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
                "hbm_pass": {"algorithmic_gb": round(alg_bytes / 1e9, 4),
                             "achieved_gbs": round(alg_bytes / 1e9 / (ms_step / 1e3), 1),
                             "frac_of_measured_copy": round(alg_bytes / 1e9 / (ms_step / 1e3) / peaks["hbm_gbs"], 4)},
                "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline, "e2e": e2e,
                "gpu_launches": launches, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ decode-time update
def run_decode(args):
    """One decode step over the compressed cache of every layer (paper Section 3.3.3, last sentence of "Dynamic
    KV Cache Eviction"): the prefill pass builds the ragged cache, then every timed step appends one token per
    sequence to every head's cache and evicts the entry with the lowest cumulative score."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200 import shard, synth
    from paper_2410_03090_b200.compress import CompressionPass

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pass has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=dev)
    base = synth.WORKLOADS[args.workload]
    if args.scale_N or args.scale_L:
        base = synth.scaled(base, N=args.scale_N or None, L=args.scale_L or None)
    wl = shard.rank_workload(base, rank)
    peaks = _peaks()
    K, V, Qw = synth.generate(wl, dev)
    cp = CompressionPass(wl, dev)
    o = cp.run(K, V, Qw)
    torch.cuda.synchronize()
    assert cp.status() == 0
    # state after prefill: full caches; cumulative scores seeded from the prefill scores
    offs = o.offsets.cpu().numpy()
    cum = ub.uncomp_decode_seed(cp.ctx, o.scores, o.indices, o.offsets)
    pos = o.indices.clone()
    lens = o.budgets.reshape(-1).clone()
    Kc, Vc = o.Kc, o.Vc
    max_cap = int(lens.max())
    qnew = Qw[:, :, :, -1, :].contiguous()
    knew = K[:, :, :, -1, :].contiguous()
    vnew = V[:, :, :, -1, :].contiguous()
    del K, V
    n_steps = args.warmup + args.steps + args.e2e_steps + 2
    new_pos = [torch.full((wl.B,), wl.N + i, dtype=torch.int32, device=dev) for i in range(n_steps)]
    evicted = torch.empty(wl.units, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    it = iter(new_pos)

    def barrier():
        if world > 1:
            dist.barrier()

    def step(q_, k_, v_):
        ub.uncomp_decode_update(cp.ctx, q_, k_, v_, next(it), o.offsets, lens, max_cap, Kc, Vc, pos, cum,
                                evicted=evicted)

    for _ in range(args.warmup):
        step(qnew, knew, vnew)
    torch.cuda.synchronize()
    assert cp.status() == 0
    sampler = ClockSampler(local)
    sampler.start()
    ub.uncomp_profile_enable(cp.ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(args.steps):
        step(qnew, knew, vnew)
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    prof = ub.uncomp_profile_read(cp.ctx)
    ub.uncomp_profile_enable(cp.ctx, False)
    ms_step = shard.max_over_ranks(ev0.elapsed_time(ev1), dev, world) / args.steps
    tokens_step = wl.B * world
    specs = kernel_specs(wl, peaks, True, cache_rows=wl.total_rows)
    kernels, launches = {}, 0
    total_ms = sum(v[0] for v in prof.values())
    for name, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        launches += cnt
        bound, work, peak, unit = specs[name]
        avg_ms = ms / cnt
        ent = {"launches_per_step": cnt // args.steps, "avg_ms": round(avg_ms, 5), "share": round(ms / total_ms, 4),
               "bound": bound}
        if work is not None:
            ach = work / (avg_ms / 1e3)
            ent.update({"achieved": round(ach, 2), "peak": peak, "unit": unit, "frac": round(ach / peak, 4)})
        kernels[name] = ent
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    kd = kernels[dom]
    roofline = {"kernel": dom, "bound": kd["bound"], "achieved": kd.get("achieved"), "peak": kd.get("peak"),
                "unit": kd.get("unit"), "frac": kd.get("frac"), "traffic": None,
                "peak_source": f"of {peaks['source']} (copy)", "avg_ms": kd["avg_ms"], "share": kd["share"]}
    alg_bytes = (specs["decode_logits"][1] + specs["decode_accumulate"][1]) * 1e9

    e2e = None
    if args.e2e_steps > 0:
        hin = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in (qnew, knew, vnew)]
        din = [torch.empty_like(t) for t in (qnew, knew, vnew)]
        hev = torch.empty(evicted.shape, dtype=evicted.dtype, pin_memory=True)

        def e2e_step():
            for h, t in zip(hin, din):
                t.copy_(h, non_blocking=True)
            step(*din)
            hev.copy_(evicted, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
        barrier()
        ms_e = shard.max_over_ranks(e0.elapsed_time(e1), dev, world)
        e2e = {"value": tokens_step / (ms_e / args.e2e_steps / 1e3), "unit": UNIT,
               "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in hin),
               "d2h_bytes_per_step": hev.numel() * hev.element_size(), "steps": args.e2e_steps}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        sample = list(range(0, wl.units, max(1, wl.units // 16)))[:16]
        data = []
        for u in sample:
            a, b = int(offs[u]), int(offs[u + 1])
            data.append((qnew.view(wl.units, wl.G, wl.d)[u].double().cpu().numpy(), Kc[a:b].double().cpu().numpy(),
                         Vc[a:b].double().cpu().numpy(), pos[a:b].cpu().numpy(), cum[a:b].double().cpu().numpy(),
                         knew.view(wl.units, wl.d)[u].double().cpu().numpy(),
                         vnew.view(wl.units, wl.d)[u].double().cpu().numpy(), b - a))
        t0 = time.perf_counter()
        for q_, K_, V_, p_, c_, kn_, vn_, cap in data:
            oracle.decode_update(q_, K_, V_, p_, c_, kn_, vn_, wl.N + n_steps, cap)
        t_cpu = time.perf_counter() - t0
        cpu_baseline = {"value": wl.B / (t_cpu * wl.units / len(sample)), "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"{len(sample)} of {wl.units} units, one decode step, {t_cpu:.2f} s wall"}

    if rank == 0:
        line = {"metric": "decode_cache_update_tokens_per_s", "value": tokens_step / (ms_step / 1e3), "unit": UNIT,
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
                "data": "synthetic",
                "config": {"workload": f"decode-time cache update after the prefill pass of {_workload_name(wl)}: "
                                       f"{wl.units} head caches, {wl.total_rows} cached rows, largest {max_cap}",
                           "l2": f"cached keys {wl.total_rows * wl.d * wl.elem_bytes / 1e9:.3f} GB read every step"
                                 + ("" if wl.total_rows * wl.d * wl.elem_bytes > 126e6 else " (fits in L2)"),
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
                "hbm_pass": {"algorithmic_gb": round(alg_bytes / 1e9, 4),
                             "achieved_gbs": round(alg_bytes / 1e9 / (ms_step / 1e3), 1),
                             "frac_of_measured_copy": round(alg_bytes / 1e9 / (ms_step / 1e3) / peaks["hbm_gbs"], 4)},
                "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline, "e2e": e2e,
                "gpu_launches": launches, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ preparation stage
def run_prepare(args):
    """Aggregation of the preparation stage (paper Section 3.3.1; Algorithm 1) over 500 samples' effective ranks
    for the workload's layers and heads: mean, grouping of the mean, per-sample grouping and majority vote.
    Latency-bound integer work on 0.5 MB; single GPU only."""
    import numpy as np
    import torch
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200 import synth

    if int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pass has no CPU path")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    wl = synth.WORKLOADS[args.workload]
    S, M = 500, min(8, wl.H)
    g = torch.Generator(device=dev).manual_seed(wl.seed)
    erank = (torch.rand(wl.L, wl.H, generator=g, device=dev) * 30 + 1)[None] + \
        torch.randn(S, wl.L, wl.H, generator=g, device=dev) * 2.0
    ctx = ub.Context(ub.make_shape(1, wl.L, wl.H, wl.Hq, 256, wl.d, 8, wl.dtype))
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        ub.uncomp_prepare_groups(ctx, erank, M, 0)
    sampler = ClockSampler(dev.index)
    sampler.start()
    ub.uncomp_profile_enable(ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(args.steps):
        out = ub.uncomp_prepare_groups(ctx, erank, M, 0)
    ev1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    prof = ub.uncomp_profile_read(ctx)
    ms_step = ev0.elapsed_time(ev1) / args.steps
    kernels = {n: {"launches_per_step": c // args.steps, "avg_ms": round(ms / c, 5), "bound": "alu"}
               for n, (ms, c) in prof.items() if c}
    launches = sum(c for _, c in prof.values())
    h = torch.empty(erank.shape, dtype=erank.dtype, pin_memory=True).copy_(erank)
    d_in = torch.empty_like(erank)
    houts = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in out]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(max(1, args.e2e_steps)):
        d_in.copy_(h, non_blocking=True)
        res = ub.uncomp_prepare_groups(ctx, d_in, M, 0)
        for a, b in zip(houts, res):
            a.copy_(b, non_blocking=True)
    e1.record(stream)
    torch.cuda.synchronize()
    ms_e = e0.elapsed_time(e1) / max(1, args.e2e_steps)
    import oracle
    e64 = erank.double().cpu().numpy()
    t0 = time.perf_counter()
    oracle.group_labels(oracle.prepare_mean(e64), M)
    oracle.majority_vote(e64, M)
    t_cpu = time.perf_counter() - t0
    dom = max(kernels, key=lambda n: kernels[n]["avg_ms"])
    line = {"metric": "preparation_aggregation_samples_per_s", "value": S / (ms_step / 1e3), "unit": "samples/s",
            "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"preparation-stage aggregation: S{S} samples x L{wl.L} x H{wl.H} effective ranks, "
                                   f"M{M} groups per layer", "l2": "0.5 MB of input: resident in L2, latency-bound"},
            "roofline": {"kernel": dom, "bound": "alu", "achieved": None, "peak": None, "unit": None, "frac": None,
                         "traffic": None, "avg_ms": kernels[dom]["avg_ms"],
                         "note": "two launches of a few microseconds each; no throughput roofline applies"},
            "kernels": kernels,
            "cpu_baseline": {"value": S / t_cpu, "unit": "samples/s", "cores": 1, "kind": "oracle",
                             "sample": f"the whole aggregation, {t_cpu * 1e3:.1f} ms wall"},
            "e2e": {"value": S / (ms_e / 1e3), "unit": "samples/s", "h2d_bytes_per_step": h.numel() * 4,
                    "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in out)},
            "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------- wide-matrix entropy
def run_wide(args):
    """Truncated entropy of hidden-state matrices [N, D] (paper Section 3.1 Eq. 1 with D = 4096, Section 3.2): a step
    is the entropy of `--wide-count` matrices (the hidden states of that many layers).  Single GPU."""
    import numpy as np
    import torch
    from paper_2410_03090_b200 import binding as ub

    if int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pass has no CPU path")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    peaks = _peaks()
    N, D, count, k = args.wide_N, args.hidden_width, args.wide_count, 32
    g = torch.Generator(device=dev).manual_seed(11)
    # hidden states: a few hundred strong directions with a decaying spectrum plus isotropic noise
    r = 256
    W = torch.randn(r, D, generator=g, device=dev) * (torch.arange(1, r + 1, device=dev) ** -0.7)[:, None]
    X = torch.empty(count, N, D, dtype=torch.bfloat16, device=dev)
    for i in range(count):
        X[i] = (torch.randn(N, r, generator=g, device=dev) @ W + 0.05 * torch.randn(N, D, generator=g, device=dev) + 0.3
                ).to(torch.bfloat16)
    ctx = ub.Context(ub.make_shape(1, 1, 1, 1, 256, 128, 8, "bf16"))
    scratch = torch.empty(ub.lib.uncomp_entropy_wide_scratch_bytes(N, D), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        ub.uncomp_entropy_wide(ctx, X, k, scratch=scratch)
    torch.cuda.synchronize()
    assert ub.uncomp_status(ctx) == 0
    sampler = ClockSampler(dev.index)
    sampler.start()
    ub.uncomp_profile_enable(ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(args.steps):
        ent, er = ub.uncomp_entropy_wide(ctx, X, k, scratch=scratch)
    ev1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    prof = ub.uncomp_profile_read(ctx)
    ub.uncomp_profile_enable(ctx, False)
    ms_step = ev0.elapsed_time(ev1) / args.steps
    dual = N < D                                   # fewer tokens than features: the N x N token-space matrix is used
    Dt = max(128, (N + 63) // 64 * 64) if dual else D
    # denominator of the tridiagonalisation: its own memory pattern on a matrix of the same size, alone on the GPU
    l2_passes = 20
    Am = torch.zeros(Dt, Dt, dtype=torch.float32, device=dev)
    ub.uncomp_measure_l2_sweep(Am, 2)
    torch.cuda.synchronize()
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0.record(stream)
    ub.uncomp_measure_l2_sweep(Am, l2_passes)
    l1.record(stream)
    torch.cuda.synchronize()
    l2_peak = 2.0 * Am.numel() * 4 * l2_passes / 1e9 / (l0.elapsed_time(l1) / 1e3)
    del Am
    nblk = (Dt + 255) // 256
    flops_gram = 2.0 * (D if dual else N) * 256 * 256 * (nblk * (nblk + 1) // 2)   # block pairs actually computed
    kernels = {}
    total_ms = sum(v[0] for v in prof.values())
    for name, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        avg = ms / cnt
        ent_k = {"launches_per_step": cnt // args.steps, "avg_ms": round(avg, 4), "share": round(ms / total_ms, 4)}
        if name == "wide_gram":
            ach = flops_gram / 1e12 / (avg / 1e3)
            ent_k.update({"bound": "tensor", "achieved": round(ach, 1), "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                          "frac": round(ach / peaks["bf16_sustained"], 4)})
        elif name == "wide_tridiag":
            # the trailing matrix is read and written once per column: (2/3) D^3 floats each way
            gb = 2.0 * (Dt ** 3) / 3.0 * 4 / 1e9
            ent_k.update({"bound": "l2", "achieved": round(gb / (avg / 1e3), 1), "peak": round(l2_peak, 1),
                          "unit": "GB/s of L2 traffic", "frac": round(gb / (avg / 1e3) / l2_peak, 4),
                          "peak_source": f"measured in this run: read-modify-write sweep of a {Dt} x {Dt} fp32 matrix "
                                         f"resident in L2 (uncomp_measure_l2_sweep, {l2_passes} passes)"})
        else:
            ent_k["bound"] = "alu"
        kernels[name] = ent_k
    launches = sum(c for _, c in prof.values())
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    kd = kernels[dom]
    roofline = {"kernel": dom, "bound": kd["bound"], "achieved": kd.get("achieved"), "peak": kd.get("peak"),
                "unit": kd.get("unit"), "frac": kd.get("frac"), "traffic": None, "avg_ms": kd["avg_ms"], "share": kd["share"],
                "peak_source": kd.get("peak_source") or f"of {peaks['source']} (sustained bf16)"}
    e2e = None
    if args.e2e_steps > 0:
        hX = torch.empty(X.shape, dtype=X.dtype, pin_memory=True).copy_(X)
        dX = torch.empty_like(X)
        hout = torch.empty(count, dtype=torch.float32, pin_memory=True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.e2e_steps):
            dX.copy_(hX, non_blocking=True)
            en, _ = ub.uncomp_entropy_wide(ctx, dX, k, scratch=scratch)
            hout.copy_(en, non_blocking=True)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e = {"value": count * N / (e0.elapsed_time(e1) / args.e2e_steps / 1e3), "unit": UNIT,
               "h2d_bytes_per_step": hX.numel() * 2, "d2h_bytes_per_step": count * 4, "steps": args.e2e_steps}
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        x0 = X[0].double().cpu().numpy()
        t0 = time.perf_counter()
        H, _ = oracle.entropy_wide(x0, k)
        t_cpu = time.perf_counter() - t0
        cpu_baseline = {"value": N / t_cpu, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                        "sample": f"1 of {count} matrices (library matmul and eigensolver threads), {t_cpu:.1f} s wall; "
                                  f"H = {H:.6f}, GPU {float(ent[0]):.6f}"}
    line = {"metric": "wide_entropy_tokens_per_s", "value": count * N / (ms_step / 1e3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"truncated entropy (k {k}) of {count} hidden-state matrices N{N} x D{D} bf16",
                       "l2": f"inputs {X.numel() * 2 / 1e9:.2f} GB, larger than L2"},
            "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-N", type=int, default=0, help="profiling aid: same recipe at a shorter sequence")
    ap.add_argument("--scale-L", type=int, default=0, help="profiling aid: same recipe with fewer layers")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lse", action="store_true", help="skip the second timed run with caller-supplied log-sum-exp")
    ap.add_argument("--path", default="kv", choices=["kv", "hidden", "decode", "prepare", "wide"],
                    help="kv: the KV-cache compression pass (the default and the headline); hidden: the "
                         "hidden-state eviction of one layer-group boundary; decode: one decode-time update of "
                         "the compressed cache of every layer; each reported on a line of its own")
    ap.add_argument("--hidden-width", type=int, default=4096)
    ap.add_argument("--hidden-batch", type=int, default=4)
    ap.add_argument("--wide-N", type=int, default=8192)
    ap.add_argument("--wide-count", type=int, default=4)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return
    if args.path == "hidden":
        run_hidden(args)
        return
    if args.path == "decode":
        run_decode(args)
        return
    if args.path == "prepare":
        run_prepare(args)
        return
    if args.path == "wide":
        run_wide(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2410_03090_b200 import binding as ub
    from paper_2410_03090_b200 import shard, synth
    from paper_2410_03090_b200.compress import CompressionPass

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pass has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=dev)

    base = synth.WORKLOADS[args.workload]
    if args.scale_N or args.scale_L:
        base = synth.scaled(base, N=args.scale_N or None, L=args.scale_L or None)
    wl = shard.rank_workload(base, rank)      # every rank compresses its own sequence(s)
    peaks = _peaks()
    K, V, Qw = synth.generate(wl, dev)
    cp = CompressionPass(wl, dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()

    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count

    def timed_passes(lse, one_call=False):
        """W warm-up and K timed passes (barrier + synchronize on both sides, CUDA events on the launching stream,
        max over ranks); returns the step time, the clock record and the per-kernel event times.  A pass is the four
        staged calls on one stream, or (one_call, and always with normalisers) one uncomp_compress call."""
        run = cp.run_one_call if (one_call or lse is not None) else cp.run
        for _ in range(args.warmup):
            run(K, V, Qw, lse=lse)
        torch.cuda.synchronize()
        assert cp.status() == 0
        sampler = ClockSampler(local)
        sampler.start()
        ub.uncomp_profile_enable(cp.ctx, True)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(args.steps):
            run(K, V, Qw, lse=lse)
        ev1.record(stream)
        torch.cuda.synchronize()
        barrier()
        clk = sampler.stop()
        ms_total = ev0.elapsed_time(ev1)
        prof_ = ub.uncomp_profile_read(cp.ctx)
        ub.uncomp_profile_enable(cp.ctx, False)
        return shard.max_over_ranks(ms_total, dev, world) / args.steps, clk, prof_

    def kernel_records(prof_, clk, ms_step_):
        """Per-kernel roofline entries from the events the library recorded inside the timed region."""
        tens, tens_name = tensor_peak(peaks, clk, ms_step_ * args.steps / 1e3)
        specs = kernel_specs(wl, peaks, tens)
        recs, n_launch = {}, 0
        for name, (ms, cnt) in prof_.items():
            if cnt == 0:
                continue
            n_launch += cnt
            bound, work, peak, unit = specs[name]
            avg_ms = ms / cnt
            ent = {"launches_per_step": cnt // args.steps, "avg_ms": round(avg_ms, 5), "share": None, "bound": bound}
            if work is not None:
                ach = work / (avg_ms / 1e3)
                ent.update({"achieved": round(ach, 2), "peak": peak, "unit": unit, "frac": round(ach / peak, 4)})
            if name in EXP_KERNELS:
                # second ceiling of the scorer kernels: the exponential unit, 16 ex2 per clock per SM
                n_exp = wl.units * wl.G * wl.w * (wl.N if name != "score_colsum" else wl.N - wl.w)   # tokens swept
                peak_exp = sm_count * 16 * (clk.get("sm_max_mhz") or 1965) * 1e6
                ent.update({"ex2_per_launch": n_exp,
                            "ex2_frac_of_unit_peak": round(n_exp / (avg_ms / 1e3) / peak_exp, 4)})
            recs[name] = ent
        total_kernel_ms = sum(v[0] for v in prof_.values())
        for name in recs:
            recs[name]["share"] = round(prof_[name][0] / total_kernel_ms, 4)
        return recs, n_launch, tens, tens_name

    ms_step, clocks, prof = timed_passes(None)
    tokens_step = wl.B * wl.N * world
    value = shard.whole_job_tokens_per_s(wl, world, ms_step)
    kernels, launches, tens_peak, tens_name = kernel_records(prof, clocks, ms_step)
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    kd = kernels[dom]
    ctr = ncu_counters(dom)
    roofline = {"kernel": dom, "bound": kd["bound"], "achieved": kd.get("achieved"), "peak": kd.get("peak"),
                "unit": kd.get("unit"), "frac": kd.get("frac"),
                "traffic": round(ctr["dram_bytes_per_unit_token"] * wl.units * wl.N / 1e9, 4) if ctr else None,
                "traffic_unit": "GB per launch (ncu dram bytes of a smaller case, scaled by units x tokens)",
                "tensor_pipe_pct": ctr["tensor_pipe_pct"] if ctr else None,
                "xu_pipe_pct": ctr["xu_pipe_pct"] if ctr else None,
                "counters_source": NCU_COUNTERS["capture"] if ctr else None,
                "peak_source": f"of {peaks['source']} ({tens_name if kd['bound'] == 'tensor' else 'copy'}; the timed "
                               f"region lasted {ms_step * args.steps / 1e3:.2f} s, power cap "
                               f"{'seen' if 'sw_power_cap' in (clocks.get('reasons') or []) else 'not seen'})",
                "avg_ms": kd["avg_ms"], "share": kd["share"]}
    sm_mhz = clocks.get("sm_max_mhz") or 1965
    bound2 = composite_bound(wl, 2, peaks["hbm_gbs"], tens_peak, sm_count, sm_mhz, ms_step)
    bound2["note"] = ("the softmax needs the row normalisers before the column sums, so the window product and its "
                      "exponentials run twice; t_exp at the maximum SM clock")

    # ---- the same pass with the caller's log-sum-exp (what a prefill attention kernel keeps per window row),
    # through uncomp_compress: the statistics sweep and the merge drop out and the Gram stage rides along with the
    # column sums, one sweep over K in all.  The normalisers are prepared once, outside the timed region, by a plain
    # matrix product and logsumexp on the device.
    # ---- the pass through uncomp_compress without normalisers: same kernels, eigenvalues and budgets on a second
    # stream beside the column sums (per-kernel event times then overlap, so only the step time is reported)
    one_call = None
    if wl.dtype == "bf16" and not args.no_lse:
        ms_oc, clocks_oc, _ = timed_passes(None, one_call=True)
        one_call = {"ms_per_step": ms_oc, "value": shard.whole_job_tokens_per_s(wl, world, ms_oc), "unit": UNIT,
                    "clocks": clocks_oc}
    with_lse = None
    if wl.dtype == "bf16" and not args.no_lse:
        lse = prefill_lse(wl, K, Qw)
        ms_lse, clocks_lse, prof_lse = timed_passes(lse)
        k_lse, launches_lse, tens_lse, tens_lse_name = kernel_records(prof_lse, clocks_lse, ms_lse)
        hb = wl.algorithmic_bytes() / 1e9 / (ms_lse / 1e3)
        with_lse = {"ms_per_step": ms_lse, "value": shard.whole_job_tokens_per_s(wl, world, ms_lse), "unit": UNIT,
                    "hbm_frac_of_measured_copy": round(hb / peaks["hbm_gbs"], 4), "achieved_gbs": round(hb, 1),
                    "composite_bound": composite_bound(wl, 1, peaks["hbm_gbs"], tens_lse, sm_count, sm_mhz, ms_lse),
                    "tensor_peak": tens_lse_name, "kernels": {n: {"avg_ms": v["avg_ms"], "frac": v.get("frac")}
                                                              for n, v in k_lse.items()},
                    "gpu_launches": launches_lse, "clocks": clocks_lse}
        del lse
    alg_bytes = wl.algorithmic_bytes()
    hbm_pass = alg_bytes / 1e9 / (ms_step / 1e3)

    # ---- end to end: host buffers in, results out, copies inside the timed region
    e2e = None
    if args.e2e_steps > 0:
        hK = torch.empty(K.shape, dtype=K.dtype, pin_memory=True).copy_(K)
        hV = torch.empty(V.shape, dtype=V.dtype, pin_memory=True).copy_(V)
        hQ = torch.empty(Qw.shape, dtype=Qw.dtype, pin_memory=True).copy_(Qw)
        o = cp.out
        outs = [o.Kc, o.Vc, o.indices, o.offsets, o.budgets, o.entropy]
        houts = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
        dK, dV, dQ = torch.empty_like(K), torch.empty_like(V), torch.empty_like(Qw)
        h2d = sum(t.numel() * t.element_size() for t in (hK, hV, hQ))
        d2h = sum(t.numel() * t.element_size() for t in outs)

        # Three streams.  The inputs arrive on the main stream, keys and window queries first; the pass runs on a
        # second stream and starts as soon as those two are there, so that everything but the final gather overlaps the
        # copy of the values; the results go back on a third stream and overlap the next step's input copies (the link
        # is full duplex).  Every step still moves all of its inputs and all of its results.
        pass_stream, out_stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        have_kq, have_v, done_pass, done_out = (torch.cuda.Event() for _ in range(4))

        def e2e_step(first=False):
            if not first:
                stream.wait_event(done_pass)          # the last pass no longer reads the input buffers
            dK.copy_(hK, non_blocking=True)
            dQ.copy_(hQ, non_blocking=True)
            have_kq.record(stream)
            dV.copy_(hV, non_blocking=True)
            have_v.record(stream)
            pass_stream.wait_event(have_kq)
            if not first:
                pass_stream.wait_event(done_out)      # the last results have left the output buffers
            cp.score(dK, dQ, stream=pass_stream)
            pass_stream.wait_event(have_v)
            cp.compact(dK, dV, stream=pass_stream)
            done_pass.record(pass_stream)
            out_stream.wait_event(done_pass)
            with torch.cuda.stream(out_stream):
                for h, t in zip(houts, outs):
                    h.copy_(t, non_blocking=True)
                done_out.record(out_stream)

        e2e_step(first=True)
        torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        stream.wait_event(done_out)           # the last results have arrived on the host
        e1.record(stream)
        torch.cuda.synchronize()
        barrier()
        ms_e = e0.elapsed_time(e1)
        ms_e = shard.max_over_ranks(ms_e, dev, world)
        e2e = {"value": tokens_step / (ms_e / args.e2e_steps / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}
        del hK, hV, hQ, dK, dV, dQ

    # ---- the oracle on the host cores, bounded sample (rank 0, single GPU only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        threads = min(os.cpu_count() or 1, 16)
        n_units = min(wl.units, 2 * wl.H)
        layers = [0] if wl.L == 1 else [0, wl.L // 2]
        unit_list = [l * wl.H + h for l in layers for h in range(wl.H)][:n_units]

        def fetch(u):
            b, l, h = synth.unit_index(wl, u)
            return (K[b, l, h].double().cpu().numpy(), V[b, l, h].double().cpu().numpy(),
                    Qw[b, l, h * wl.G:(h + 1) * wl.G].double().cpu().numpy())

        t_cpu = 0.0
        for l in layers:
            ul = [x for x in unit_list if x // wl.H == l]
            t_cpu += time_oracle(wl, ul, fetch, threads)
        v = wl.B * wl.N / (t_cpu * wl.units / len(unit_list))
        cpu_baseline = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"{len(unit_list)} of {wl.units} units (all heads of layers {layers}), whole oracle "
                                  f"chain, {t_cpu:.1f} s wall"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
                "config": {"workload": _workload_name(wl), "l2": "inputs larger than L2 (K+V = "
                           f"{2 * K.numel() * K.element_size() / 1e9:.2f} GB streamed every step)",
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
                "hbm_pass": {"algorithmic_gb": round(alg_bytes / 1e9, 4), "achieved_gbs": round(hbm_pass, 1),
                             "frac_of_measured_copy": round(hbm_pass / peaks["hbm_gbs"], 4),
                             "frac_of_nominal_8tbs": round(hbm_pass / 8000.0, 4)},
                "roofline": roofline, "composite_bound": bound2, "kernels": kernels,
                "one_call": one_call, "with_lse": with_lse,
                "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
