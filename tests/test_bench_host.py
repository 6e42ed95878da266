"""Host logic of the benchmark and of multi-GPU sharding, on CPU (gloo, world size 2)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2410_03090_b200 import shard, synth
    base = synth.scaled(synth.WORKLOADS["c2"], N=128, L=1)
    wl = shard.rank_workload(base, rank)
    K, _, _ = synth.generate_unit(wl, 0, 0, 0)
    ms = shard.max_over_ranks(10.0 + 5.0 * rank, "cpu", world)          # the slowest rank decides
    digest = torch.tensor([float(K.float().sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    dist.barrier()
    if rank == 0:
        out.put({"ms": ms, "seed0": wl.seed, "digests": [float(g) for g in gathered],
                 "value": shard.whole_job_tokens_per_s(wl, world, ms)})
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_agree_on_time():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    res = out.get()
    assert res["ms"] == 15.0
    assert res["digests"][0] != res["digests"][1]            # each rank compresses its own sequence
    assert abs(res["value"] - 2 * 128 / 0.015) < 1e-6          # tokens of both ranks over the slowest time


def test_rank_workload_keeps_shape_and_changes_data():
    from paper_2410_03090_b200 import shard, synth
    base = synth.WORKLOADS["c3"]
    w0, w1 = shard.rank_workload(base, 0), shard.rank_workload(base, 1)
    assert w0 == base and w1.seed != base.seed
    assert (w1.N, w1.L, w1.H, w1.avg_budget, w1.n_max) == (base.N, base.L, base.H, base.avg_budget, base.n_max)
    assert shard.max_over_ranks(3.5, "cpu", 1) == 3.5


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "tokens/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["higher_is_better"] is True and line["vs_baseline"] is None


def test_kernel_specs_cover_every_profiled_kernel():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2410_03090_b200 import binding as ub, synth
    specs = bench.kernel_specs(synth.WORKLOADS["c3"], bench._peaks(), True)
    names = {ub.lib.uncomp_profile_slot_name(i).decode() for i in range(ub.lib.uncomp_profile_slots())}
    assert names == set(specs)
    # algorithmic work of the c3 pass: 0.275 TFLOP of Gram, 2.57 GB of bytes
    assert abs(specs["gram"][1] - 0.2749) < 1e-3
    assert abs(synth.WORKLOADS["c3"].algorithmic_bytes() / 1e9 - 2.5695) < 1e-3


def test_eviction_plan_host_logic():
    sys.path.insert(0, ROOT)
    from paper_2410_03090_b200.compress import eviction_plan
    # three groups: full context, then two cuts; a boundary into a group that is not smaller needs no call
    assert eviction_plan([0, 0, 1, 1, 1, 2, 2], [4096, 4096, 1536, 1536, 1536, 1024, 1024]) == [(2, 1536), (5, 1024)]
    assert eviction_plan([0, 0, 0], [900, 900, 900]) == []
    assert eviction_plan([0, 1, 2], [500, 500, 300]) == [(2, 300)]
    assert eviction_plan([], []) == []


def _bench():
    sys.path.insert(0, ROOT)
    import bench
    return bench


def test_tensor_peak_follows_the_regime_of_the_timed_region():
    bench = _bench()
    peaks = {"bf16_burst": 1600.0, "bf16_sustained": 1400.0}
    assert bench.tensor_peak(peaks, {"reasons": []}, 0.1) == (1600.0, "burst bf16")
    assert bench.tensor_peak(peaks, {"reasons": ["sw_power_cap"]}, 0.1) == (1400.0, "sustained bf16")
    assert bench.tensor_peak(peaks, {"reasons": []}, 2.5) == (1400.0, "sustained bf16")
    assert bench.tensor_peak(peaks, {}, 0.999)[1] == "burst bf16"


def test_composite_bound_arithmetic():
    from paper_2410_03090_b200 import synth
    bench = _bench()
    wl = synth.WORKLOADS["c3"]
    rows, u = wl.G * wl.w, wl.units
    b = bench.composite_bound(wl, 2, hbm_gbs=6500.0, tensor_tflops=1400.0, sm_count=148, sm_mhz=1965, ms_step=2.0)
    t_hbm = wl.algorithmic_bytes() / 6500e9 * 1e3
    t_tensor = u * (2.0 * wl.N * 128 * 128 + 2 * 2.0 * rows * 128 * wl.N) / 1400e12 * 1e3
    t_exp = u * 2.0 * rows * wl.N / (148 * 16 * 1965e6) * 1e3
    assert abs(b["t_hbm_ms"] - t_hbm) < 1e-3 and abs(b["t_tensor_ms"] - t_tensor) < 1e-3
    assert abs(b["t_exp_ms"] - t_exp) < 1e-3
    assert b["t_min_ms"] == max(b["t_hbm_ms"], b["t_tensor_ms"], b["t_exp_ms"]) and b["binding"] == "tensor"
    assert abs(b["frac_of_t_min"] - b["t_min_ms"] / 2.0) < 1e-3
    # one window product instead of two: both the tensor and the exponential bound shrink, the byte bound does not
    b1 = bench.composite_bound(wl, 1, 6500.0, 1400.0, 148, 1965, 1.5)
    assert b1["t_hbm_ms"] == b["t_hbm_ms"] and b1["t_exp_ms"] < b["t_exp_ms"] and b1["t_tensor_ms"] < b["t_tensor_ms"]
    assert abs(b1["t_exp_ms"] * 2 - b["t_exp_ms"]) < 1e-3


def test_ncu_counters_are_dropped_when_the_kernel_source_changed(monkeypatch):
    import hashlib
    bench = _bench()
    src = os.path.join(ROOT, bench.NCU_COUNTERS["source"])
    with open(src, "rb") as f:
        digest = hashlib.sha256(f.read()).hexdigest()
    fake = {"source": bench.NCU_COUNTERS["source"], "sha256": digest, "capture": "x",
            "kernels": {"k": {"dram_bytes_per_unit_token": 1.0, "tensor_pipe_pct": 2.0, "xu_pipe_pct": 3.0}}}
    monkeypatch.setattr(bench, "NCU_COUNTERS", fake)
    assert bench.ncu_counters("k")["tensor_pipe_pct"] == 2.0 and bench.ncu_counters("other") is None
    monkeypatch.setattr(bench, "NCU_COUNTERS", dict(fake, sha256="0" * 64))
    assert bench.ncu_counters("k") is None
