"""Helpers for the GPU parity tests: run a synth.Workload through the C-ABI and compare with the
FP64 oracle under the three tolerances (max |err| <= 2e-2 and relative L2 <= 5e-3 on the bf16
output, |lse err| <= 1e-3)."""
import numpy as np

from oracle import reference as R
from paper_2509_25224_b200 import binding

TOL_ABS = 2e-2
TOL_REL_L2 = 5e-3
TOL_LSE = 1e-3


def to_device(w):
    import torch
    dev = torch.device("cuda", 0)
    q = torch.from_numpy(w.q.view(np.int16)).to(dev).view(torch.bfloat16)
    kv = torch.from_numpy(w.kv.view(np.int16)).to(dev).view(torch.bfloat16)
    bt = torch.from_numpy(w.block_table).to(dev)
    sl = torch.from_numpy(w.seqlens).to(dev)
    return q, kv, bt, sl


def run_gpu(w, flags=None, poison=True, dev_inputs=None):
    """Returns (out float64 [B,Sq,H,512], lse float64 [B,Sq,H]) computed by the CUDA path."""
    import torch
    q, kv, bt, sl = dev_inputs if dev_inputs is not None else to_device(w)
    B, Sq, H = w.B, w.Sq, w.H
    out = torch.empty((B, Sq, H, 512), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((B, Sq, H), dtype=torch.float32, device=q.device)
    ws = torch.empty(binding.workspace_size(B, Sq, H, bt.shape[1], 0), dtype=torch.uint8, device=q.device)
    if poison:   # unwritten outputs / stale workspace must not go unnoticed
        out.view(torch.int16).fill_(0x7FC0)
        lse.fill_(float("nan"))
        ws.fill_(0xFF)
    binding.mla_decode(q, kv, bt, sl, w.scale, out, lse, ws, flags)
    binding.check_status(ws)
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), (out, lse)


def compare(out, lse, ref_out, ref_lse, what="", tol_abs=TOL_ABS):
    assert not np.isnan(out).any(), f"{what}: NaN in out"
    err = np.abs(out - ref_out)
    rel = np.linalg.norm(out - ref_out) / (np.linalg.norm(ref_out) + 1e-10)
    assert err.max() <= tol_abs, f"{what}: max|err| {err.max():.3e}"
    assert rel <= TOL_REL_L2, f"{what}: rel L2 {rel:.3e}"
    inf_ref = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(lse), inf_ref), f"{what}: -inf pattern of lse differs"
    if (~inf_ref).any():
        le = np.abs(lse[~inf_ref] - ref_lse[~inf_ref]).max()
        assert le <= TOL_LSE, f"{what}: |lse err| {le:.3e}"
    return float(err.max()), float(rel)


def check_full(w, flags=None, what="", tol_abs=TOL_ABS):
    out, lse, _ = run_gpu(w, flags)
    ro, rl = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    return compare(out, lse, ro, rl, what or w.name, tol_abs)


def check_sampled(w, n_rows=192, flags=None, seed=0, what="", dev_inputs=None):
    """Full-size workloads: compare a seeded sample of (b,t,h) rows, plus finiteness everywhere."""
    out, lse, _ = run_gpu(w, flags, dev_inputs=dev_inputs)
    assert np.isfinite(out).all()
    rng = np.random.default_rng(seed)
    rows = np.stack([rng.integers(0, w.B, n_rows), rng.integers(0, w.Sq, n_rows), rng.integers(0, w.H, n_rows)], 1)
    rows = rows.astype(np.int32)
    # always include the first and last row of the first and last sequence
    rows[:4] = [[0, 0, 0], [0, w.Sq - 1, w.H - 1], [w.B - 1, 0, 0], [w.B - 1, w.Sq - 1, w.H - 1]]
    ro, rl = R.decode_rows(w.q, w.kv, w.block_table, w.seqlens, w.scale, rows)
    go = out[rows[:, 0], rows[:, 1], rows[:, 2]]
    gl = lse[rows[:, 0], rows[:, 1], rows[:, 2]]
    return compare(go, gl, ro, rl, what or w.name)
