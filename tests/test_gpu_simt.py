"""GPU parity of the scalar bring-up kernel (AMLA_FLAG_KERNEL_SIMT) through the C-ABI: it shares the
schedule, the combine kernel and the per-row recurrence with the tensor-core kernel."""
import numpy as np
import pytest

from paper_2509_25224_b200 import binding, synth
from tests._gpu_util import check_full

pytestmark = pytest.mark.gpu
SIMT = binding.FLAG_KERNEL_SIMT


def test_simt_tiny_config():
    check_full(synth.config_tiny(), SIMT)


@pytest.mark.parametrize("mode", [binding.RESCALE_ALG2, binding.RESCALE_FOLD, binding.RESCALE_FMUL])
def test_simt_ragged_and_split(mode):
    # ragged lengths, empty sequence, Sq=2 causal rule, H=16 padding; few tiles => heavy splitting
    w = synth.make_workload("r", 5, 2, 16, [300, 0, 1, 65, 1000], seed=101)
    check_full(w, SIMT | mode)
    w = synth.make_workload("r", 3, 1, 128, [700, 64, 129], seed=102)
    check_full(w, SIMT | mode)


def test_simt_staircase_rescale():
    w = synth.config_stress(B=1, N=2048)
    check_full(w, SIMT)
