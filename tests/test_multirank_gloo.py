"""Host-side logic of the N > 1 path, run as two `gloo` ranks on CPU: the batch is sharded with no data-path
collective (sequences are independent problems), per-rank results reassemble to the unsharded result, the step time
of a job is the maximum over its ranks, and under a multi-rank launch only rank 0 of the reference arm prints."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str) -> None:
    import torch
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    from oracle import reference as R
    from paper_2509_25224_b200 import synth

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        w = synth.make_workload("mr", 5, 2, 16, [130, 0, 64, 257, 31], seed=77)
        mine = list(synth.shard_batch(w.B, world, rank))
        # every rank decodes its own sequences only: a sub-batch with its rows of the block table
        sub_out, sub_lse = R.decode(w.q[mine], w.kv, w.block_table[mine], w.seqlens[mine], w.scale)
        gathered = [None] * world
        dist.all_gather_object(gathered, (mine, sub_out, sub_lse))
        # the job's step time is the slowest rank's
        t = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        if rank == 0:
            full_out, full_lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
            seen = []
            for idx, o, l in gathered:
                seen += idx
                assert np.array_equal(o, full_out[idx]) and np.array_equal(l, full_lse[idx], equal_nan=True)
            assert sorted(seen) == list(range(w.B))
            assert float(t.item()) == 10.0 + 5.0 * (world - 1)
            with open(os.path.join(out_dir, "ok"), "w") as f:
                f.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_the_batch_and_reassemble(tmp_path):
    import torch.multiprocessing as mp

    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()


def test_reference_arm_prints_once_under_a_two_rank_launch():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--config", "tiny"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["cpu_baseline"]["kind"] == "oracle"
