"""The paper's own benchmark grid on one B200 (Section 5.2, Table 5): batch 96, 128 heads, S_q in {1, 2},
S_k in {1024, 2048, 3072, 4096, 6144, 16384}, BF16, one latent KV head of 576 / 512 columns.

For every grid point: duration of the whole decode call (all its launches, CUDA events on the stream, inputs
resident in HBM, input replicas rotated so that no step finds its cache in L2) and FLOPS utilisation
FU = 2 * B * S_q * 128 * S_k * 1088 / t / peak, against the measured and the nominal dense BF16 peak.  The cache
is paged (64 keys per page, shuffled block table), which the paper's benchmark is not; the inputs are seeded
N(0, 1) values like everything else in this repository.

    python -m paper_2509_25224_b200.paper_grid [--steps 20] [--out table.txt]

The printed table puts the paper's Table 5 rows (another machine: context, not a target) beside the measured ones.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

from . import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# Table 5 of the paper: (S_q, S_k) -> ((duration us, FU %) on Ascend 910, (duration us, FU %) FlashMLA on the GPU it names)
TABLE5 = {
    (1, 1024): ((95, 40.9), (85, 32.6)), (1, 2048): ((140, 55.1), (128, 43.3)), (1, 3072): ((186, 62.4), (173, 48.0)),
    (1, 4096): ((241, 64.1), (215, 51.5)), (1, 6144): ((331, 70.2), (316, 52.6)), (1, 16384): ((830, 74.5), (766, 57.8)),
    (2, 1024): ((135, 57.3), (115, 48.1)), (2, 2048): ((219, 70.7), (196, 56.5)), (2, 3072): ((306, 75.8), (278, 59.8)),
    (2, 4096): ((388, 79.7), (374, 59.2)), (2, 6144): ((565, 82.2), (527, 63.0)), (2, 16384): ((1427, 86.8), (1314, 67.4)),
}
GRID_SK = (1024, 2048, 3072, 4096, 6144, 16384)
BATCH = 96
HEADS = 128


def grid_workload(Sq: int, Sk: int, B: int = BATCH) -> synth.Workload:
    """One grid point as a paged workload (seeded; the seed depends on the point)."""
    return synth.make_workload(f"grid_sq{Sq}_sk{Sk}", B, Sq, HEADS, [Sk] * B, seed=0x5A00 + 16 * Sq + Sk // 1024)


def measured_bf16_peak() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


def time_point(w: synth.Workload, steps: int, warmup: int, dev) -> float:
    """Median milliseconds of one decode call."""
    import torch

    kv_bytes = w.kv.nbytes
    nrep = 2 if kv_bytes >= 200e6 else min(8, int(np.ceil(400e6 / kv_bytes)))
    reps = []
    for _ in range(nrep):
        reps.append((torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16),
                     torch.from_numpy(w.kv.view(np.int16)).to(dev).view(torch.bfloat16),
                     torch.from_numpy(w.block_table).to(dev), torch.from_numpy(w.seqlens).to(dev)))
    out = torch.empty((w.B, w.Sq, w.H, 512), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.B, w.Sq, w.H), dtype=torch.float32, device=dev)
    ws = torch.empty(binding.workspace_size(w.B, w.Sq, w.H, w.max_blocks_per_seq, dev.index or 0), dtype=torch.uint8, device=dev)

    def step(i):
        q, kv, bt, sl = reps[i % nrep]
        binding.mla_decode(q, kv, bt, sl, w.scale, out, lse, ws)

    for i in range(warmup):
        step(i)
    binding.check_status(ws)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    torch.cuda.synchronize()
    evs[0].record()
    for i in range(steps):
        step(i)
        evs[i + 1].record()
    torch.cuda.synchronize()
    binding.check_status(ws)
    return float(np.median([evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]))


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--out", type=str, default=None, help="also write the table to this file")
    args = ap.parse_args(argv)

    import torch

    if not torch.cuda.is_available():
        print("paper_grid needs a GPU", file=sys.stderr)
        return 2
    dev = torch.device("cuda", 0)
    peak, kind = measured_bf16_peak()
    lines = [f"# paper grid (Section 5.2, Table 5): B={BATCH} H={HEADS} bf16 paged-64, whole decode call, median of {args.steps} steps",
             f"# FU here = TFLOP/s / {peak:.0f} ({kind} dense bf16 peak of this pool) and / 2250 (nominal); Table 5 columns: the paper's machines (context)",
             f"{'S_q':>3s} {'S_k':>6s} | {'us':>8s} {'TFLOP/s':>8s} {'FU meas':>8s} {'FU nom':>7s} | {'910 us':>7s} {'910 FU':>7s} | {'GPU us':>7s} {'GPU FU':>7s}"]
    print("\n".join(lines))
    for Sq in (1, 2):
        for Sk in GRID_SK:
            w = grid_workload(Sq, Sk)
            ms = time_point(w, args.steps, args.warmup, dev)
            tf = w.flops() / (ms * 1e-3) / 1e12
            (a_us, a_fu), (g_us, g_fu) = TABLE5[(Sq, Sk)]
            row = (f"{Sq:3d} {Sk:6d} | {ms * 1e3:8.1f} {tf:8.1f} {100 * tf / peak:7.1f}% {100 * tf / 2250.0:6.1f}% | "
                   f"{a_us:7d} {a_fu:6.1f}% | {g_us:7d} {g_fu:6.1f}%")
            print(row, flush=True)
            lines.append(row)
            del w
    if args.out:
        with open(args.out, "w") as f:
            f.write("\n".join(lines) + "\n")
    return 0


if __name__ == "__main__":
    sys.exit(main())
