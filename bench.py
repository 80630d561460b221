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


def config_block(w, nrep=None, eff=None):
    """The `config` object of the JSON line; the same for both arms (it names the workload, not the arm)."""
    kv_bytes = w.kv.nbytes
    if nrep is None:
        nrep = replica_count(kv_bytes)
    if eff is None:
        eff = DEFAULT_FLAGS
    tot = nrep * kv_bytes / 1e6
    return {"workload": workload_name(w),
            "l2": f"{nrep} input replicas rotated between steps ({tot:.0f} MB of KV) " + ("> 126 MB L2" if tot > 126 else "(fits in L2: latency-bound case)"),
            "rescale": ["alg2", "fold", "fmul"][eff & 3] + f" tau={(eff >> 8) & 15}" + (" unguarded" if eff & 4 else "")}


DEFAULT_FLAGS = 0 | (8 << 8)      # AMLA_RESCALE_ALG2 | AMLA_LAZY(8): what amla_mla_decode uses


def replica_count(kv_bytes):
    """Input replicas rotated between steps so that no step finds its KV cache in L2 (126 MB)."""
    nrep = max(2, int(np.ceil(400e6 / kv_bytes))) if kv_bytes < 400e6 else 2
    return min(nrep, 8)


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
        "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)), "median_step_ms": 1e3 * float(np.median(times)),
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_block(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample + " per step"},
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
def roofline_of(w, dec_ms, peaks, peak_kind):
    """Roofline object for the decode kernel of one workload: the slower of (FLOPs at the measured bf16 peak) and
    (algorithmic bytes at the measured HBM peak) is the bound; achieved = that quantity / the kernel's duration."""
    flops, alg_bytes = w.flops(), w.algorithmic_bytes()
    hbm_peak, tc_peak = float(peaks["hbm_gbs"]), float(peaks["bf16_tflops"])
    if alg_bytes / (hbm_peak * 1e9) >= flops / (tc_peak * 1e12):
        ach = alg_bytes / (dec_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak}
    else:
        ach = flops / (dec_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak}
    roof.update({"traffic": None, "peak_kind": f"of {peak_kind} (burst)", "kernel_ms": dec_ms,
                 "kernel_tflops": flops / (dec_ms * 1e-3) / 1e12,
                 "frac_of_bf16_measured": flops / (dec_ms * 1e-3) / 1e12 / tc_peak,
                 "frac_of_bf16_nominal_2250": flops / (dec_ms * 1e-3) / 1e12 / 2250.0,
                 "kernel_gbs": alg_bytes / (dec_ms * 1e-3) / 1e9, "algorithmic_bytes": alg_bytes, "flops": flops})
    return roof


class DeviceRun:
    """One workload resident on the device (rotating input replicas) and the timing of its decode calls."""

    def __init__(self, w, dev, local, flags):
        import torch
        from paper_2509_25224_b200 import binding
        self.torch, self.binding, self.w, self.flags = torch, binding, w, flags
        self.nrep = replica_count(w.kv.nbytes)
        self.reps = []
        for _ in range(self.nrep):
            self.reps.append((torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16),
                              torch.from_numpy(w.kv.view(np.int16)).to(dev).view(torch.bfloat16),
                              torch.from_numpy(w.block_table).to(dev), torch.from_numpy(w.seqlens).to(dev)))
        self.out = torch.empty((w.B, w.Sq, w.H, 512), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((w.B, w.Sq, w.H), dtype=torch.float32, device=dev)
        self.ws = torch.empty(binding.workspace_size(w.B, w.Sq, w.H, w.max_blocks_per_seq, local), dtype=torch.uint8, device=dev)

    def step(self, i, flags="same"):
        q, kv, bt, sl = self.reps[i % self.nrep]
        self.binding.mla_decode(q, kv, bt, sl, self.w.scale, self.out, self.lse, self.ws, self.flags if flags == "same" else flags)

    def timed(self, steps, barrier, flags="same"):
        """(total ms, per-step ms list) of `steps` calls bracketed by barrier + synchronize, CUDA events per step."""
        torch = self.torch
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        evs[0].record()
        for i in range(steps):
            self.step(i, flags)
            evs[i + 1].record()
        barrier()
        return evs[0].elapsed_time(evs[-1]), [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]

    def kernel_times(self, steps, flags="same"):
        """Mean (schedule, decode, combine) ms from events the library records around its launches."""
        self.binding.profile_enable(True)
        ks = []
        for i in range(steps):
            self.step(i, flags)
            ks.append(self.binding.profile_last_ms())
        self.binding.profile_enable(False)
        self.torch.cuda.synchronize()
        return tuple(float(np.mean([k[j] for k in ks])) for j in range(3))


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
    flags = None if args.mode is None and args.tau is None and not args.rows128 else (
        {"alg2": 0, "fold": 1, "fmul": 2}[args.mode or "alg2"] | binding.lazy(binding.DEFAULT_TAU if args.tau is None else args.tau)
        | (binding.FLAG_UNGUARDED_ADD if args.unguarded else 0) | (binding.FLAG_KERNEL_ROWS128 if args.rows128 else 0))
    eff = binding.DEFAULT_FLAGS if flags is None else flags
    run = DeviceRun(w, dev, local, flags)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        run.step(i)
    binding.check_status(run.ws)

    # ---- timed region: K steps, device-resident inputs
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    # the W warm-up steps again, now directly in front of the timed ones: starting the sampler left the GPU idle for a
    # quarter of a second, and a GPU that comes out of idle takes twice as long for its first call and 3 % longer for
    # the next six
    for i in range(max(args.warmup, 3)):
        run.step(i)
    total_ms, per_step = run.timed(args.steps, barrier)
    launches = binding.last_launch_count() * args.steps
    # ---- same K steps again with per-kernel events (decode kernel duration for the roofline)
    plan_ms, dec_ms, comb_ms = run.kernel_times(args.steps)
    clocks = sampler.stop() if rank == 0 else None
    binding.check_status(run.ws)

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
    h2d, d2h = sess.h2d_bytes, sess.d2h_bytes
    del sess

    # ---- the other configurations, on rank 0 at N = 1 (roofline fraction for every configuration)
    per_config = {}
    if rank == 0 and world == 1 and not args.no_per_config:
        traffic = load_traffic()
        ksteps = max(10, min(args.steps, 100))

        def entry(r, wk, fl="same"):
            for i in range(5):
                r.step(i, fl)
            tot, per = r.timed(ksteps, barrier, fl)
            _, dms, cms = r.kernel_times(min(ksteps, 50), fl)
            rf = roofline_of(wk, dms, peaks, peak_kind)
            return {"ms_per_step": tot / ksteps, "median_step_ms": statistics.median(per), "tflops": wk.flops() * ksteps / (tot * 1e-3) / 1e12,
                    "kernel_ms": dms, "combine_ms": cms, "kernel_tflops": rf["kernel_tflops"], "bound": rf["bound"],
                    "frac": rf["frac"], "frac_of_bf16_measured": rf["frac_of_bf16_measured"], "steps": ksteps,
                    "traffic": traffic.get(wk.name), "workload": workload_name(wk)}

        per_config[w.name] = {"ms_per_step": total_ms / args.steps, "median_step_ms": statistics.median(per_step),
                              "tflops": flops * args.steps / (total_ms * 1e-3) / 1e12, "kernel_ms": dec_ms, "combine_ms": comb_ms,
                              **{k: v for k, v in roofline_of(w, dec_ms, peaks, peak_kind).items() if k in ("kernel_tflops", "bound", "frac", "frac_of_bf16_measured")},
                              "steps": args.steps, "traffic": traffic.get(w.name), "workload": workload_name(w)}
        tau0 = binding.RESCALE_ALG2 | binding.lazy(0)
        if w.name in ("dsv3", "long") and flags is None:
            per_config[w.name + " tau=0"] = entry(run, w, tau0)
        del run
        torch.cuda.empty_cache()
        per_config["dsv3 fp8-cache"] = fp8_entry(synth.CONFIGS["dsv3"]() if w.name != "dsv3" else w, dev, local, ksteps, barrier, peaks, peak_kind)
        for name in synth.CONFIGS:
            if name == w.name:
                continue
            wk = synth.CONFIGS[name]()
            r = DeviceRun(wk, dev, local, None)
            per_config[name] = entry(r, wk)
            if name in ("dsv3", "long"):
                per_config[name + " tau=0"] = entry(r, wk, tau0)
            binding.check_status(r.ws)
            del r
            torch.cuda.empty_cache()

    if rank == 0:
        roof = roofline_of(w, dec_ms, peaks, peak_kind)
        roof.update({"kernel": "decode_quad_kernel" if (Sq * H > 128 and not args.rows128) else "decode_tc_kernel",
                     "schedule_ms": plan_ms, "combine_ms": comb_ms})
        roof["traffic"] = load_traffic().get(w.name)
        n_rows = {"tiny": 16, "dsv3": 4096, "mtp": 2048, "stress": 1024, "long": 256}[w.name]
        tf, dt, cores, sample = time_oracle(w, n_rows)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps, "median_step_ms": statistics.median(per_step),
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_block(w, None, eff),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": roof,
            "cpu_baseline": {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": dt},
            "per_config": per_config,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def fp8_entry(w, dev, local, steps, barrier, peaks, peak_kind, kv_scale=1.0 / 64.0):
    """The same workload with an E4M3 cache (amla_mla_decode_fp8: widen the used pages, then the bf16 kernels): whole
    call, CUDA events; its algorithmic bytes count one byte per cache element."""
    import torch
    from paper_2509_25224_b200 import binding
    kv8 = synth.quantise_cache_e4m3(w, kv_scale)
    q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
    bt, sl = torch.from_numpy(w.block_table).to(dev), torch.from_numpy(w.seqlens).to(dev)
    caches = [torch.from_numpy(kv8).to(dev) for _ in range(max(2, int(np.ceil(200e6 / kv8.nbytes))))]
    out = torch.empty((w.B, w.Sq, w.H, 512), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.B, w.Sq, w.H), dtype=torch.float32, device=dev)
    ws = torch.empty(binding.fp8_workspace_size(w.B, w.Sq, w.H, w.max_blocks_per_seq, local), dtype=torch.uint8, device=dev)
    for i in range(5):
        binding.mla_decode_fp8(q, caches[i % len(caches)], kv_scale, bt, sl, w.scale, out, lse, ws)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    evs[0].record()
    for i in range(steps):
        binding.mla_decode_fp8(q, caches[i % len(caches)], kv_scale, bt, sl, w.scale, out, lse, ws)
        evs[i + 1].record()
    barrier()
    binding.check_status(ws)
    tot = evs[0].elapsed_time(evs[-1])
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    flops = w.flops()
    rows = w.B * w.Sq * w.H
    alg_bytes = float(w.seqlens.astype(np.int64).sum()) * synth.D_QK + rows * synth.D_QK * 2 + rows * (synth.D_V * 2 + 4)
    ms = tot / steps
    t_b, t_f = alg_bytes / (float(peaks["hbm_gbs"]) * 1e9), flops / (float(peaks["bf16_tflops"]) * 1e12)
    bound = "hbm" if t_b >= t_f else "tensor"
    frac = max(t_b, t_f) / (ms * 1e-3)
    return {"ms_per_step": ms, "median_step_ms": statistics.median(per), "tflops": flops / (ms * 1e-3) / 1e12, "bound": bound,
            "frac": frac, "frac_of": "whole call (widen + decode + combine) against the " + peak_kind + " peak", "steps": steps,
            "algorithmic_bytes": alg_bytes, "launches_per_step": binding.last_launch_count(),
            "workload": workload_name(w).replace("bf16 paged-64", "bf16 q, E4M3 cache (scale 1/64) paged-64")}


def load_traffic():
    """DRAM bytes per launch from the committed ncu captures; only valid for the kernel sources they were taken with."""
    traffic_file = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(traffic_file):
        with open(traffic_file) as f:
            tr = json.load(f)
        if tr.get("source_sha256") == kernel_source_hash():
            return {k: v for k, v in tr.items() if k != "source_sha256"}
    return {}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="dsv3", choices=list(synth.CONFIGS))
    ap.add_argument("--mode", default=None, choices=["alg2", "fold", "fmul"], help="rescale variant (default: the library's)")
    ap.add_argument("--tau", type=int, default=None, help="lazy-reference threshold in octaves, 0..15 (default: the library's)")
    ap.add_argument("--unguarded", action="store_true", help="literal single integer add (measurement only)")
    ap.add_argument("--rows128", action="store_true", help="A/B: independent 128-row blocks instead of the 256-row kernel (measurement only)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other configurations")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
