#!/usr/bin/env python
"""MLA decode benchmark: TFLOPS of one pass of the whole hot path (schedule + decode + combine) on
synthetic decode workloads, with the roofline fraction of the decode kernel and the FP64 CPU oracle
timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config dsv3|mtp|stress|long|tiny]
    python bench.py --impl reference ...      # times the CPU oracle (the reference arm)

A step is one amla_mla_decode call.  FLOPs = 2 * sum_b Sq*H*N_b*(576+512).  With N > 1 (torchrun) every
rank runs the same configuration on its own GPU: sequences are independent problems, so the batch
shards without any collective ("weak" scaling); the value is total FLOPs over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_25224_b200 import synth  # noqa: E402

METRIC = "MLA decode TFLOPS on 1 B200 and % of BF16 tensor peak / KV-bytes roofline"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        for ln in out.strip().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def kernel_source_hash():
    """sha256 over the CUDA sources of the library (what the ncu counters in profiles/ were taken with)."""
    import glob
    import hashlib
    h = hashlib.sha256()
    for p in sorted(glob.glob(os.path.join(ROOT, "paper_2509_25224_b200", "csrc", "*.cu*"))):
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# --------------------------------------------------------------------------------------------------
def oracle_sample_rows(w, n_rows, seed=0):
    rng = np.random.default_rng(seed)
    return np.stack([rng.integers(0, w.B, n_rows), rng.integers(0, w.Sq, n_rows), rng.integers(0, w.H, n_rows)], 1).astype(np.int32)


def time_oracle(w, n_rows):
    """Times the FP64 oracle on a sample of query rows; returns (tflops, seconds, cores, sample description)."""
    from oracle import reference as R
    rows = oracle_sample_rows(w, n_rows)
    R.decode_rows(w.q, w.kv, w.block_table, w.seqlens, w.scale, rows[:8])          # load + warm
    t0 = time.perf_counter()
    R.decode_rows(w.q, w.kv, w.block_table, w.seqlens, w.scale, rows)
    dt = time.perf_counter() - t0
    vis = np.minimum(w.seqlens[rows[:, 0]], w.seqlens[rows[:, 0]] - w.Sq + rows[:, 1] + 1).clip(min=0)
    flops = 2.0 * float(vis.astype(np.int64).sum()) * (synth.D_QK + synth.D_V)
    return flops / dt / 1e12, dt, R.num_threads(), f"{n_rows} seeded (b,t,h) query rows of the {w.name} workload, all their keys"


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    w = synth.CONFIGS[args.config]()
    # size the per-step sample for roughly 2 s of oracle time (probe with a small sample first)
    tf, dt, cores, _ = time_oracle(w, 64)
    n_rows = int(max(64, min(w.B * w.Sq * w.H, 64 * 2.0 / max(dt, 1e-3))))
    for _ in range(args.warmup):
        time_oracle(w, min(n_rows, 64))
    times, tfl = [], []
    sample = ""
    for _ in range(args.steps):
        tf, dt, cores, sample = time_oracle(w, n_rows)
        times.append(dt); tfl.append(tf)
    value = float(np.mean(tfl))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(w), "sample_rows_per_step": n_rows},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_name(w):
    sl = w.seqlens
    n = f"N={int(sl[0])}" if int(sl.min()) == int(sl.max()) else f"N~U[{int(sl.min())},{int(sl.max())}]"
    return f"{w.name}: B={w.B} Sq={w.Sq} H={w.H} {n} d_qk=576 d_v=512 bf16 paged-64 scale=1/sqrt(192)"


# --------------------------------------------------------------------------------------------------
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2509_25224_b200 import binding

    rank, world, local = dist_env()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks, peak_kind = load_peaks()

    w = synth.CONFIGS[args.config]()
    B, Sq, H = w.B, w.Sq, w.H
    # input replicas rotated between steps so that no step finds its KV cache in L2 (126 MB)
    kv_bytes = w.kv.nbytes
    nrep = max(2, int(np.ceil(400e6 / kv_bytes))) if kv_bytes < 400e6 else 2
    nrep = min(nrep, 8)
    reps = []
    for _ in range(nrep):
        q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
        kv = torch.from_numpy(w.kv.view(np.int16)).to(dev).view(torch.bfloat16)
        bt = torch.from_numpy(w.block_table).to(dev)
        sl = torch.from_numpy(w.seqlens).to(dev)
        reps.append((q, kv, bt, sl))
    out = torch.empty((B, Sq, H, 512), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, Sq, H), dtype=torch.float32, device=dev)
    ws = torch.empty(binding.workspace_size(B, Sq, H, w.max_blocks_per_seq, local), dtype=torch.uint8, device=dev)
    flags = None if args.mode is None and args.tau is None else (
        {"alg2": 0, "fold": 1, "fmul": 2}[args.mode or "alg2"] | binding.lazy(binding.DEFAULT_TAU if args.tau is None else args.tau)
        | (binding.FLAG_UNGUARDED_ADD if args.unguarded else 0))
    eff = binding.DEFAULT_FLAGS if flags is None else flags

    def step(i):
        q, kv, bt, sl = reps[i % nrep]
        binding.mla_decode(q, kv, bt, sl, w.scale, out, lse, ws, flags)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    binding.check_status(ws)

    # ---- timed region: K steps, device-resident inputs
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    evs[0].record()
    for i in range(args.steps):
        step(i)
        evs[i + 1].record()
    barrier()
    launches = binding.last_launch_count() * args.steps
    total_ms = evs[0].elapsed_time(evs[-1])
    per_step = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]

    # ---- same K steps again with per-kernel events (decode kernel duration for the roofline)
    binding.profile_enable(True)
    kern_ms = []
    for i in range(args.steps):
        step(i)
        kern_ms.append(binding.profile_last_ms())
    binding.profile_enable(False)
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    binding.check_status(ws)

    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms_max = float(t.item())
    flops = w.flops()
    value = world * flops * args.steps / (total_ms_max * 1e-3) / 1e12

    # ---- end to end: host buffers, H2D + decode + D2H inside the timed region
    e2e_steps = max(2, min(args.steps, 5))
    sess = binding.HostSession(B, Sq, H, w.num_blocks, w.max_blocks_per_seq, local)
    sess.set_inputs(w.q, w.kv, w.block_table, w.seqlens)
    sess.run(w.scale, flags)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        sess.run(w.scale, flags, sync=True)
    e1.record()
    barrier()
    t2 = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t2, op=dist.ReduceOp.MAX)
    e2e_value = world * flops * e2e_steps / (float(t2.item()) * 1e-3) / 1e12

    if rank == 0:
        dec_ms = float(np.mean([k[1] for k in kern_ms]))
        plan_ms = float(np.mean([k[0] for k in kern_ms]))
        comb_ms = float(np.mean([k[2] for k in kern_ms]))
        alg_bytes = w.algorithmic_bytes()
        hbm_peak = float(peaks["hbm_gbs"])
        tc_peak = float(peaks["bf16_tflops"])
        t_bytes = alg_bytes / (hbm_peak * 1e9)
        t_flops = flops / (tc_peak * 1e12)
        if t_bytes >= t_flops:
            ach = alg_bytes / (dec_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak}
        else:
            ach = flops / (dec_ms * 1e-3) / 1e12
            roof = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak}
        roof.update({
            "traffic": None, "peak_kind": f"of {peak_kind} (burst)", "kernel": "decode_tc_kernel",
            "kernel_ms": dec_ms, "schedule_ms": plan_ms, "combine_ms": comb_ms,
            "kernel_tflops": flops / (dec_ms * 1e-3) / 1e12,
            "frac_of_bf16_measured": flops / (dec_ms * 1e-3) / 1e12 / tc_peak,
            "frac_of_bf16_nominal_2250": flops / (dec_ms * 1e-3) / 1e12 / 2250.0,
            "kernel_gbs": alg_bytes / (dec_ms * 1e-3) / 1e9,
            "algorithmic_bytes": alg_bytes, "flops": flops,
        })
        # DRAM bytes per launch from the committed ncu capture; only valid for the kernel sources it was taken with
        traffic_file = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(traffic_file):
            with open(traffic_file) as f:
                tr = json.load(f)
            if tr.get("source_sha256") == kernel_source_hash():
                roof["traffic"] = tr.get(w.name)
        n_rows = {"tiny": 16, "dsv3": 4096, "mtp": 2048, "stress": 1024, "long": 256}[w.name]
        tf, dt, cores, sample = time_oracle(w, n_rows)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(w), "l2": f"{nrep} input replicas rotated between steps "
                       f"({nrep * kv_bytes / 1e6:.0f} MB of KV) > 126 MB L2", "rescale": ["alg2", "fold", "fmul"][eff & 3] + f" tau={(eff >> 8) & 15}" + (" unguarded" if eff & 4 else ""),
                       "median_step_ms": statistics.median(per_step)},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": sess.h2d_bytes, "d2h_bytes_per_step": sess.d2h_bytes,
                    "steps": e2e_steps},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": roof,
            "cpu_baseline": {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": dt},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="dsv3", choices=list(synth.CONFIGS))
    ap.add_argument("--mode", default=None, choices=["alg2", "fold", "fmul"], help="rescale variant (default: the library's)")
    ap.add_argument("--tau", type=int, default=None, help="lazy-reference threshold in octaves, 0..15 (default: the library's)")
    ap.add_argument("--unguarded", action="store_true", help="literal single integer add (measurement only)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
