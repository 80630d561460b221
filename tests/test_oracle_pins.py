"""Pins for the FP64 oracle: everything here is fixed by the mathematics or by
the paper, not by the oracle itself (Eq. 1; MLA sharing of Section 2.2)."""
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import reference as R
from paper_2509_25224_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(path) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _dense(w, b):
    return synth.bf16_bits_to_f32(synth.logical_kv_rows(w, b)).astype(np.float64)


def _q(w):
    return synth.bf16_bits_to_f32(w.q).astype(np.float64)


def test_brute_force_tiny_pure_python():
    # Hand-loop evaluation with python floats and math.exp on an 8-key problem.
    w = synth.make_workload("t", 1, 1, 2, [8], seed=11)
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    kv = _dense(w, 0)
    q = _q(w)
    for h in range(2):
        s = [w.scale * sum(float(q[0, 0, h, d]) * float(kv[j, d]) for d in range(576)) for j in range(8)]
        m = max(s)
        p = [math.exp(x - m) for x in s]
        l = sum(p)
        for d in (0, 1, 17, 255, 511):
            ref = sum(p[j] * float(kv[j, d]) for j in range(8)) / l
            assert abs(out[0, 0, h, d] - ref) < 1e-13
        assert abs(lse[0, 0, h] - (m + math.log(l))) < 1e-13


@pytest.mark.parametrize("n", [1, 63, 64, 65, 200])
def test_matches_scipy_softmax_dense(n):
    # Special case that reduces to library routines: dense softmax(QK^T*scale) V and logsumexp.
    w = synth.make_workload("t", 2, 1, 3, [n, max(1, n - 1)], seed=5 + n)
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    q = _q(w)
    for b in range(2):
        kv = _dense(w, b)
        s = (q[b, 0] @ kv.T) * w.scale
        ref = softmax(s, axis=1) @ kv[:, :512]
        np.testing.assert_allclose(out[b, 0], ref, rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[b, 0], logsumexp(s, axis=1), rtol=0, atol=1e-12)


def test_v_is_first_512_columns_not_last():
    # A transposed/shifted V slice would fail: make columns 512.. huge and distinct.
    w = synth.make_workload("t", 1, 1, 1, [70], seed=3)
    w.q[...] = 0
    w.kv[:, :, 512:] = synth.f32_to_bf16_bits(np.full((w.kv.shape[0], 64, 64), 1000.0, np.float32))
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    kv = _dense(w, 0)
    np.testing.assert_allclose(out[0, 0, 0], kv[:, :512].mean(axis=0), atol=1e-13)


def test_uniform_logits_give_mean_of_v_and_log_count():
    w = synth.make_workload("t", 3, 1, 4, [5, 64, 131], seed=7)
    w.q[...] = 0  # all logits equal
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    for b, n in enumerate([5, 64, 131]):
        kv = _dense(w, b)
        for h in range(4):
            np.testing.assert_allclose(out[b, 0, h], kv[:, :512].mean(axis=0), atol=1e-13)
            assert abs(lse[b, 0, h] - math.log(n)) < 1e-13


def test_dominant_key_returns_its_v_row():
    n, jstar = 150, 97
    w = synth.make_workload("t", 1, 1, 2, [n], seed=9)
    off = np.zeros(n)
    off[jstar] = 200.0  # margin far above the random part (|random logit| < ~10)
    synth.apply_logit_offsets(w, [off])
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    kv = _dense(w, 0)
    q = _q(w)
    for h in range(2):
        np.testing.assert_allclose(out[0, 0, h], kv[jstar, :512], atol=1e-20)
        s_star = w.scale * float(q[0, 0, h] @ kv[jstar])
        assert abs(lse[0, 0, h] - s_star) < 1e-12


def test_page_permutation_invariance_bit_identical():
    w = synth.make_workload("t", 2, 1, 2, [300, 129], seed=21, shuffle_pages=False, spare_blocks=3)
    out0, lse0 = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    rng = np.random.default_rng(0)
    perm = rng.permutation(w.num_blocks)          # new physical location of old page p is perm[p]
    kv2 = np.empty_like(w.kv)
    kv2[perm] = w.kv
    bt2 = np.where(w.block_table >= 0, perm[np.maximum(w.block_table, 0)], -1).astype(np.int32)
    out1, lse1 = R.decode(w.q, kv2, bt2, w.seqlens, w.scale)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


def test_scale_is_an_argument():
    w = synth.make_workload("t", 1, 1, 2, [40], seed=2)
    out_a, lse_a = R.decode(w.q, w.kv, w.block_table, w.seqlens, 0.05)
    q = _q(w)
    kv = _dense(w, 0)
    s = (q[0, 0] @ kv.T) * 0.05
    np.testing.assert_allclose(lse_a[0, 0], logsumexp(s, axis=1), atol=1e-12)


def test_causal_rule_between_speculative_tokens():
    # Sq=2: token 1 sees all N keys, token 0 sees N-1.  Same rows as two Sq=1 problems.
    n = 100
    w2 = synth.make_workload("t", 1, 2, 3, [n], seed=31)
    out2, lse2 = R.decode(w2.q, w2.kv, w2.block_table, w2.seqlens, w2.scale)
    for t, nv in ((0, n - 1), (1, n)):
        q1 = np.ascontiguousarray(w2.q[:, t:t + 1])
        out1, lse1 = R.decode(q1, w2.kv, w2.block_table, np.array([nv], np.int32), w2.scale)
        assert np.array_equal(out2[0, t], out1[0, 0]) and np.array_equal(lse2[0, t], lse1[0, 0])


def test_rows_without_visible_keys():
    # N=1 with Sq=2: token 0 sees nothing; N=0: nobody sees anything.
    w = synth.make_workload("t", 2, 2, 2, [1, 0], seed=4)
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    assert np.all(out[0, 0] == 0) and np.all(np.isneginf(lse[0, 0]))
    kv = _dense(w, 0)
    np.testing.assert_allclose(out[0, 1, 0], kv[0, :512], atol=1e-15)
    assert np.all(out[1] == 0) and np.all(np.isneginf(lse[1]))


def test_constant_logit_shift_moves_lse_only():
    n = 90
    w = synth.make_workload("t", 1, 1, 2, [n], seed=13)
    synth.apply_logit_offsets(w, [np.zeros(n)])
    out0, lse0 = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    synth.apply_logit_offsets(w, [np.full(n, 8.0)])
    out1, lse1 = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    # the planted column is bf16-rounded, so the realised shift is 4*scale*bf16(8/(4*scale)) for every key
    planted = float(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.array([8.0 / (4 * w.scale)], np.float32)))[0])
    shift = 4.0 * w.scale * planted
    np.testing.assert_allclose(lse1 - lse0, shift, atol=1e-12)
    # out changes only through column 512 of V?  No: V is columns 0..511, untouched.
    np.testing.assert_allclose(out1, out0, atol=1e-13)


def test_rows_entry_point_equals_full():
    w = synth.make_workload("t", 3, 2, 4, [70, 5, 129], seed=17)
    out, lse = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    rows = np.array([[0, 0, 0], [2, 1, 3], [1, 1, 2], [1, 0, 0]], np.int32)
    o, l = R.decode_rows(w.q, w.kv, w.block_table, w.seqlens, w.scale, rows)
    for i, (b, t, h) in enumerate(rows):
        assert np.array_equal(o[i], out[b, t, h]) and l[i] == lse[b, t, h]


def test_bad_block_table_is_reported():
    w = synth.make_workload("t", 1, 1, 1, [70], seed=1)
    bt = w.block_table.copy()
    bt[0, 1] = w.num_blocks
    with pytest.raises(ValueError):
        R.decode(w.q, w.kv, bt, w.seqlens, w.scale)


def test_flop_and_intensity_formulas_match_the_paper():
    # Table 2: AI = N1*S1*(Dk+Dv)/Dk.
    for heads, sq, printed in _rows(os.path.join(GOLD, "table2_arithmetic_intensity.txt")):
        ai = int(heads) * int(sq) * (576 + 512) / 576
        assert abs(ai - float(printed)) < 1.0
    # Table 5 / abstract: 614 TFLOPS at 1427 us.
    (bsz, heads, sq, sk, us, tf), = _rows(os.path.join(GOLD, "table5_flops_pin.txt"))
    flops = 2.0 * int(bsz) * int(sq) * int(heads) * int(sk) * (576 + 512)
    assert abs(flops / (float(us) * 1e-6) / 1e12 - float(tf)) < 0.5
    # and synth.Workload.flops uses the same count
    w = synth.make_workload("t", 2, 2, 4, [10, 20], seed=1)
    assert w.flops() == 2.0 * 2 * 4 * 30 * 1088


# ----------------------------------------------------------------- FP8 (E4M3) cache oracle

def test_e4m3_widening_matches_the_library_conversion_on_all_bytes():
    # the oracle's own decoder of OCP E4M3 bytes against torch's float8_e4m3fn on every byte value
    import torch
    b = torch.arange(256, dtype=torch.uint8)
    want = b.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.array([R.e4m3_to_double(i) for i in range(256)])
    assert np.isnan(got[0x7F]) and np.isnan(got[0xFF]) and np.isnan(want[0x7F]) and np.isnan(want[0xFF])
    ok = ~np.isnan(want)
    assert ok.sum() == 254 and np.array_equal(got[ok], want[ok])
    # a few values of the format by hand: 1.0, the largest (448), the smallest subnormal (2^-9), the smallest normal (2^-6), -1.5
    assert got[0x38] == 1.0 and got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0xBC] == -1.5


def test_e4m3_quantiser_of_the_input_generator():
    import torch
    # every representable value maps to its own byte ...
    vals = np.array([R.e4m3_to_double(i) for i in range(256)])
    ok = ~np.isnan(vals)
    bits = synth.f32_to_e4m3_bits(vals[ok].astype(np.float32))
    assert np.array_equal(bits, np.arange(256, dtype=np.uint8)[ok])
    # ... in-range values round like the library's conversion (nearest even), out-of-range ones saturate at 448
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000) * 60, rng.standard_normal(2000) * 0.01, [17.0, 19.0, 1.0625, 2.0 ** -10, 3 * 2.0 ** -10]]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = synth.f32_to_e4m3_bits(x)
    nz = (want & 0x7F) != 0            # (the sign of a zero result is not compared)
    assert np.array_equal(got[nz], want[nz]) and np.all((got[~nz] & 0x7F) == 0)
    assert synth.f32_to_e4m3_bits(np.array([1e6, -1e6], np.float32)).tolist() == [0x7E, 0xFE]


def test_fp8_oracle_equals_the_bf16_oracle_on_the_widened_cache():
    # E4M3 values are exact in bf16, and a power-of-two scale keeps them exact: the FP8 oracle on (bytes, kv_scale)
    # must agree with the bf16 oracle on the cache of widened, scaled values to rounding order
    w = synth.make_workload("f8", 3, 2, 4, [130, 0, 65], seed=91)
    for kv_scale in (1.0, 1.0 / 64.0):
        kv8 = synth.quantise_cache_e4m3(w, kv_scale)
        wide = np.array([R.e4m3_to_double(i) for i in range(256)])[kv8] * kv_scale
        kv16 = synth.f32_to_bf16_bits(wide.astype(np.float32))
        assert np.array_equal(synth.bf16_bits_to_f32(kv16).astype(np.float64), wide)      # exact in bf16
        o8, l8 = R.decode_fp8(w.q, kv8, kv_scale, w.block_table, w.seqlens, w.scale)
        o16, l16 = R.decode(w.q, kv16, w.block_table, w.seqlens, w.scale)
        fin = ~np.isneginf(l16)
        assert np.array_equal(np.isneginf(l8), ~fin)
        assert np.abs(o8 - o16).max() <= 1e-12 and np.abs(l8[fin] - l16[fin]).max() <= 1e-12
