"""amla_mla_decode_static -- the decode call for callers that may not allocate device memory.

A serving loop that must stay out of the allocator, a process whose device memory was handed out completely at
start-up, or a plugin that only ever receives input and output buffers cannot provide the workspace that
amla_mla_decode asks for.  The static entry point runs the same kernels on a scratch array built into the library.
This test calls it through the C-ABI twice in a row, on two different problems (so the second call finds the first
call's leftovers in the shared scratch), and checks each result against the ordinary entry point and against the
FP64 oracle within the tolerances of the parity tests; the status word of the built-in scratch is read back after
each call.  The file name sorts last on purpose: a run that stops at the first failure has
then already executed every other test.
"""
import numpy as np
import pytest

from oracle import reference as R
from paper_2509_25224_b200 import binding, synth
from tests._gpu_util import TOL_ABS, TOL_LSE, TOL_REL_L2, compare, to_device

pytestmark = pytest.mark.gpu


def _both(w):
    import torch
    q, kv, bt, sl = to_device(w)
    shape_o, shape_l = (w.B, w.Sq, w.H, 512), (w.B, w.Sq, w.H)
    ref_o = torch.empty(shape_o, dtype=torch.bfloat16, device=q.device)
    ref_l = torch.empty(shape_l, dtype=torch.float32, device=q.device)
    binding.mla_decode(q, kv, bt, sl, w.scale, ref_o, ref_l)
    # outputs are made by the caller beforehand and poisoned; the static call itself allocates nothing
    out = torch.empty(shape_o, dtype=torch.bfloat16, device=q.device)
    lse = torch.empty(shape_l, dtype=torch.float32, device=q.device)
    out.view(torch.int16).fill_(0x7FC0)
    lse.fill_(float("nan"))
    torch.cuda.synchronize()
    binding.mla_decode_static(q, kv, bt, sl, w.scale, out, lse)
    binding.static_check_status()          # no bounded wait ran out inside the static call
    torch.cuda.synchronize()
    return (out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64),
            ref_o.float().cpu().numpy().astype(np.float64), ref_l.cpu().numpy().astype(np.float64))


def _check(w):
    o, l, ro, rl = _both(w)
    assert not np.isnan(o).any()
    assert np.abs(o - ro).max() <= TOL_ABS
    assert np.linalg.norm(o - ro) / (np.linalg.norm(ro) + 1e-10) <= TOL_REL_L2
    inf = np.isneginf(rl)
    assert np.array_equal(np.isneginf(l), inf)
    if (~inf).any():
        assert np.abs(l[~inf] - rl[~inf]).max() <= TOL_LSE
    # and against the FP64 oracle (CUDA against CUDA alone would not notice an error both entry points share)
    oo, ol = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    compare(o, l, oo, ol, "static entry vs oracle")


def test_static_entry_matches_workspace_entry_on_two_calls_in_a_row():
    # ragged batch: split sequences (partials in the scratch), an empty one, Sq = 2 causal rule
    _check(synth.make_workload("na1", 5, 2, 128, [3000, 0, 65, 1500, 700], seed=4101))
    # a different shape right after it, on the same (now dirty) scratch
    _check(synth.make_workload("na2", 3, 1, 64, [200, 4097, 1], seed=4102))


def test_static_entry_rejects_problems_beyond_its_scratch():
    import torch
    w = synth.config_tiny()
    q, kv, bt, sl = to_device(w)
    out = torch.empty((1, 1, 16, 512), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((1, 1, 16), dtype=torch.float32, device=q.device)
    # claim more (sequence, row block) pairs than AMLA_STATIC_MAX_ITEMS: refused before anything is launched
    rc = binding.lib().amla_mla_decode_static(q.data_ptr(), kv.data_ptr(), bt.data_ptr(), sl.data_ptr(), 0.1, 5000, 1, 16,
                                              kv.shape[0], bt.shape[1], out.data_ptr(), lse.data_ptr(), 0)
    assert rc == -6
    assert "scratch" in binding.status_string(rc)
