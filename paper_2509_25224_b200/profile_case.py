"""Runs a few decode calls of one (possibly cut-down) workload: the command that profiler captures wrap.

    python -m paper_2509_25224_b200.profile_case --config mtp [--batch 32] [--calls 3] [--mode alg2|fold|fmul]
                                                 [--tau T] [--rows128] [--n N]

--batch keeps the first B sequences of the named configuration (its seeded lengths and values), --n overrides the
sequence length of the fixed-length configurations (stress: the staircase of logit offsets spans the new length).
One warm-up call, then --calls calls; the status word is checked and a checksum of the output printed, so that a
capture can be told from a run that did nothing.
"""
from __future__ import annotations

import argparse
import sys

import numpy as np

from . import binding, synth


def build_workload(name: str, batch: int | None, n: int | None) -> synth.Workload:
    if name == "dsv3":
        B = batch or 32
        return synth.make_workload("dsv3", B, 1, 128, [n or 4096] * B, synth.SEEDS["dsv3"])
    if name == "mtp":
        sl = synth.mtp_seqlens()
        B = batch or len(sl)
        return synth.make_workload("mtp", B, 2, 128, sl[:B], synth.SEEDS["mtp"])
    if name == "stress":
        return synth.config_stress(B=batch or 16, N=n or 16384)
    if name == "long":
        B = batch or 4
        return synth.make_workload("long", B, 2, 128, [n or 65536] * B, synth.SEEDS["long"])
    if name == "tiny":
        return synth.config_tiny()
    raise ValueError(name)


def main() -> int:
    import torch

    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="dsv3", choices=["tiny", "dsv3", "mtp", "stress", "long"])
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--mode", default=None, choices=["alg2", "fold", "fmul"])
    ap.add_argument("--tau", type=int, default=None)
    ap.add_argument("--rows128", action="store_true")
    a = ap.parse_args()
    w = build_workload(a.config, a.batch, a.n)
    flags = None
    if a.mode is not None or a.tau is not None or a.rows128:
        flags = ({"alg2": 0, "fold": 1, "fmul": 2}[a.mode or "alg2"] | binding.lazy(binding.DEFAULT_TAU if a.tau is None else a.tau)
                 | (binding.FLAG_KERNEL_ROWS128 if a.rows128 else 0))
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
    kv = torch.from_numpy(w.kv.view(np.int16)).to(dev).view(torch.bfloat16)
    bt = torch.from_numpy(w.block_table).to(dev)
    sl = torch.from_numpy(w.seqlens).to(dev)
    out = torch.empty((w.B, w.Sq, w.H, 512), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.B, w.Sq, w.H), dtype=torch.float32, device=dev)
    ws = torch.empty(binding.workspace_size(w.B, w.Sq, w.H, w.max_blocks_per_seq, 0), dtype=torch.uint8, device=dev)
    for _ in range(1 + a.calls):
        binding.mla_decode(q, kv, bt, sl, w.scale, out, lse, ws, flags)
    binding.check_status(ws)
    torch.cuda.synchronize()
    print(f"{a.config}: B={w.B} Sq={w.Sq} keys={int(w.seqlens.astype(np.int64).sum())} KV={w.kv.nbytes / 1e6:.0f} MB "
          f"flops/call={w.flops():.4g} algorithmic_bytes/call={w.algorithmic_bytes():.4g} checksum={float(out.float().abs().sum()):.6g}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
