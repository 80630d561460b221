"""Pins for the CPU simulators of Algorithm 1 / Algorithm 2 and for the exponent-add
identity (Lemma 3.1, Example 3.1, Eq. 3, Appendix A)."""
import math
import os

import numpy as np
import pytest

from oracle import amla_sim as S
from oracle import reference as R
from paper_2509_25224_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _dense(w, b=0):
    kv = synth.bf16_bits_to_f32(synth.logical_kv_rows(w, b))
    q = synth.bf16_bits_to_f32(w.q[b, 0])
    return q, kv, kv[:, :512]


# ---------------------------------------------------------------- bf16 rounding used by the simulators

def test_bf16_round_ties_and_carries_by_hand():
    f = lambda bits: np.array([bits], np.uint32).view(np.float32)
    cases = [
        (0x3F800000, 0x3F800000),   # 1.0 is representable
        (0x3F808000, 0x3F800000),   # 1 + 2^-8: exactly half way between 1 and 1 + 2^-7 -> even (1.0)
        (0x3F818000, 0x3F820000),   # 1 + 3 * 2^-8... half way between 0x3F81 and 0x3F82 -> even (0x3F82)
        (0x3F808001, 0x3F810000),   # just above the half way point -> up
        (0x3F80C000, 0x3F810000),   # 1 + 3 * 2^-9 -> nearest is 1 + 2^-7
        (0x3F807FFF, 0x3F800000),   # just below half way -> down
        (0x3FFFFFFF, 0x40000000),   # mantissa carry into the exponent: 1.9999999 -> 2.0
        (0x7F7FFFFF, 0x7F800000),   # the largest finite float rounds to +inf in bf16
        (0xBF808000, 0xBF800000),   # sign is carried along
        (0x00000000, 0x00000000),
    ]
    for src, want in cases:
        got = S.bf16_round(f(src)).view(np.uint32)[0]
        assert got == want, (hex(src), hex(got), hex(want))


# ---------------------------------------------------------------- Lemma 3.1

def test_example_3_1_bit_pattern():
    with open(os.path.join(GOLD, "example_3_1.txt")) as f:
        bits, val, efield = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")][0]
    i = int(bits, 2)
    assert i == 0x3F000000 == int(efield) * 2 ** 23 == 1056964608
    assert np.array([i], np.uint32).view(np.float32)[0] == np.float32(float(val))
    # one step of the lemma on it: 0.5 * 2^3 = 4
    assert S.exponent_add(np.float32(0.5), 3 << 23)[()] == np.float32(4.0)


def test_exponent_add_bit_exact_vs_ldexp_all_reachable_exponents():
    mant = np.array([0, 1, 2, 0x155555, 1 << 22, (1 << 22) + 1, 0x7FFFFE, 0x7FFFFF], dtype=np.uint32)
    rng = np.random.default_rng(1)
    mant = np.concatenate([mant, rng.integers(0, 1 << 23, 24, dtype=np.uint32)])
    checked = 0
    for sign in (0, 1):
        for E in range(1, 255):
            bits = (np.uint32(sign) << np.uint32(31)) | (np.uint32(E) << np.uint32(23)) | mant
            F = bits.view(np.float32)
            ns = np.arange(max(-30, 1 - E), min(30, 254 - E) + 1)
            for n in ns:
                got = S.exponent_add(F, int(n) << 23) if n >= 0 else S.exponent_add(F, -((-int(n)) << 23))
                ref = np.ldexp(F, int(n)).astype(np.float32)
                assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), (sign, E, n)
                got_g = S.exponent_add(F, int(n) * (1 << 23), guard=True)
                assert np.array_equal(got_g.view(np.uint32), ref.view(np.uint32))
                checked += 1
    assert checked > 2 * 254 * 30


def test_unguarded_add_breaks_on_zero_and_guard_fixes_it():
    z = np.array([0.0, -0.0], np.float32)
    n = -(3 << 23)
    bad = S.exponent_add(z, n, guard=False)
    assert not np.all(bad == 0)                      # the literal integer add corrupts an exact zero
    good = S.exponent_add(z, n, guard=True)
    assert np.array_equal(good.view(np.uint32), z.view(np.uint32))
    # underflow below the normal range: magnitude collapses to < 2^-126, sign kept
    tiny = np.array([2.0 ** -120, -(2.0 ** -120)], np.float32)
    r = S.exponent_add(tiny, -(30 << 23), guard=True)
    assert np.all(np.abs(r) < 2.0 ** -126) and np.signbit(r[1]) and not np.signbit(r[0])


def test_residual_factor_error_bound():
    # Appendix A: (1+eps) applied as +round(1.5 * 2^23 * eps) on the bit pattern, using M ~ 2^22.
    # Without a mantissa carry the relative error is eps*(0.5-f)/(1+f) with f = M/2^23 in [0,1),
    # i.e. within [-0.25, 0.5] * |eps|.
    rng = np.random.default_rng(3)
    F = (rng.random(200000).astype(np.float32) + np.float32(1.0)) * np.float32(2.0) ** rng.integers(-20, 20, 200000)
    F = F.astype(np.float32) * np.where(rng.random(200000) < 0.5, -1, 1).astype(np.float32)
    for eps in (2.0 ** -8, -(2.0 ** -8), 1e-3, -3e-3, 2.0 ** -12):
        k = int(np.rint(1.5 * 2 ** 23 * eps))
        got = S.exponent_add(F, k, guard=True).astype(np.float64)
        true = F.astype(np.float64) * (1.0 + eps)
        rel = (got - true) / true
        f = (F.view(np.uint32) & np.uint32(0x7FFFFF)).astype(np.float64) / 2 ** 23
        no_carry = (f + 1.5 * eps < 1.0) & (f + 1.5 * eps >= 0.0)
        pred = eps * (0.5 - f) / ((1 + f) * (1 + eps))
        assert np.max(np.abs(rel[no_carry] - pred[no_carry])) < 3e-7
        lo, hi = sorted((-0.25 * eps, 0.5 * eps))
        assert rel[no_carry].min() >= lo - abs(eps) * 0.01 - 3e-7
        assert rel[no_carry].max() <= hi + abs(eps) * 0.01 + 3e-7
        assert np.max(np.abs(rel)) <= 0.8 * abs(eps) + 3e-7      # carries included


# ---------------------------------------------------------------- Algorithm 1

@pytest.mark.parametrize("tile", [1, 64, 512])
def test_algorithm1_tiling_invariance_vs_oracle(tile):
    w = synth.make_workload("t", 1, 1, 6, [777], seed=41)
    q, K, V = _dense(w)
    out, lse = S.flash_attention(q, K, V, w.scale, tile, dtype=np.float64)
    ro, rl = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    np.testing.assert_allclose(out, ro[0, 0], atol=1e-12)
    np.testing.assert_allclose(lse, rl[0, 0], atol=1e-12)


def test_algorithm1_with_visibility_mask_vs_oracle():
    n = 200
    w = synth.make_workload("t", 1, 2, 4, [n], seed=43)
    kv = synth.bf16_bits_to_f32(synth.logical_kv_rows(w, 0))
    q = synth.bf16_bits_to_f32(w.q[0]).reshape(8, 576)
    vis = np.array([n - 1] * 4 + [n] * 4)
    out, lse = S.flash_attention(q, kv, kv[:, :512], w.scale, 64, visible=vis)
    ro, rl = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    np.testing.assert_allclose(out, ro[0].reshape(8, 512), atol=1e-12)
    np.testing.assert_allclose(lse, rl[0].reshape(8), atol=1e-12)


# ---------------------------------------------------------------- Algorithm 2

def test_algorithm2_scalar_invariants():
    w = synth.config_stress(B=1, N=4096)
    q, K, V = _dense(w)
    q = q[:8]
    tr = []
    S.amla(q, K, V, w.scale, 64, trace=tr)
    n_prev = None
    c_prev = None
    for st in tr:
        assert np.all(st["S32"] >= 1 / math.sqrt(2) - 1e-6) and np.all(st["S32"] <= math.sqrt(2) + 1e-6)   # Eq. 3
        assert np.all(np.abs(st["c"] - 1) <= 2.0 ** -8 + 1e-7)
        if n_prev is not None:
            assert np.all(st["n"] <= n_prev)                      # m_i non-decreasing => n_i non-increasing
            assert np.all(np.abs(st["c"] / c_prev - 1) < 1 / 128)
            # the integer splits into a power-of-two part and a small residual
            dn = np.maximum(st["n"] - n_prev, -30)
            resid = st["N"] - (dn.astype(np.int64) << 23)
            nz = st["N"] != 0
            assert np.all(np.abs(resid[nz]) < 1.5 * 2 ** 23 / 128 + 16)
        n_prev, c_prev = st["n"], st["c"]
    assert sum(int(np.count_nonzero(st["N"])) for st in tr) > 20   # the staircase does trigger rescales


def test_algorithm2_matches_oracle_random_and_staircase():
    for w in (synth.make_workload("t", 1, 1, 16, [2048], seed=47), synth.config_stress(B=1, N=2048)):
        q, K, V = _dense(w)
        q = q[:16]
        out, lse = S.amla(q, K, V, w.scale, 64)
        rows = np.array([[0, 0, h] for h in range(16)], np.int32)
        ro, rl = R.decode_rows(w.q, w.kv, w.block_table, w.seqlens, w.scale, rows)
        assert S.rel_frobenius(out, ro) < 3e-3
        assert np.max(np.abs(out - ro)) < 2e-2
        assert np.max(np.abs(lse - rl)) < 1e-4


def test_reading_of_c_i_appendix_vs_listing():
    # Tables 3-4 say AMLA ~= Base.  With c_i = S16/S32 (Appendix A) the compensation cancels the bf16
    # rounding of 1/r_i; with the ratio as printed in Algorithm 2 line 9 it doubles it.
    errs = {"base": [], "appendix": [], "listing": [], "none": []}
    for seed in (51, 52, 53):
        w = synth.make_workload("t", 1, 1, 16, [8192], seed=seed)
        q, K, V = _dense(w)
        ro, _ = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
        ro = ro[0, 0]
        b, _ = S.flash_attention(q, K, V, w.scale, 64, dtype=np.float32, low_precision_matmul=True)
        errs["base"].append(S.rel_frobenius(b, ro))
        for mode in ("appendix", "listing", "none"):
            o, _ = S.amla(q, K, V, w.scale, 64, c_mode=mode)
            errs[mode].append(S.rel_frobenius(o, ro))
    e = {k: float(np.mean(v)) for k, v in errs.items()}
    assert e["appendix"] < 1.35 * e["base"], e          # AMLA ~= Base
    assert e["listing"] > 1.8 * e["appendix"], e        # the printed ratio makes it worse ...
    assert e["listing"] > e["none"], e                  # ... than no compensation at all
    # plausibility band against Tables 3-4 (bf16 output rounding adds ~1.6e-3 on top)
    ob = S.bf16_round(S.amla(q, K, V, w.scale, 64)[0])
    assert 1.0e-3 < S.rel_frobenius(ob, ro) < 3.0e-3


def test_clamp_on_a_60_nat_jump():
    # One +60 nat step in the middle: the max jumps by ~86 octaves, beyond the -30 clamp.  The stale
    # accumulator is then over-weighted by at most 2^-30 relative to the new tile -- invisible.
    n = 512
    w = synth.make_workload("t", 1, 1, 8, [n], seed=61)
    off = np.where(np.arange(n) < 256, -30.0, 30.0)
    synth.apply_logit_offsets(w, [off])
    q, K, V = _dense(w)
    tr = []
    out, lse = S.amla(q, K, V, w.scale, 64, trace=tr)
    assert min(int(st["N"].min()) for st in tr) < -(29 << 23)        # the clamp was hit
    assert min(int(st["N"].min()) for st in tr) >= -(30 << 23) - (1 << 18)
    ro, rl = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    assert np.max(np.abs(out - ro[0, 0])) < 2e-2 and S.rel_frobenius(out, ro[0, 0]) < 3e-3
    assert np.max(np.abs(lse - rl[0, 0])) < 1e-4


def test_falling_staircase_needs_no_rescale_after_first_tile():
    n = 1024
    w = synth.make_workload("t", 1, 1, 4, [n], seed=63)
    synth.apply_logit_offsets(w, [synth.staircase_offsets(n)[::-1].copy() * 3])   # +90 .. -90, falling
    q, K, V = _dense(w)
    tr = []
    out, _ = S.amla(q, K, V, w.scale, 64, trace=tr)
    assert all(np.all(st["N"] == 0) for st in tr[1:])
    ro, _ = R.decode(w.q, w.kv, w.block_table, w.seqlens, w.scale)
    assert S.rel_frobenius(out, ro[0, 0]) < 3e-3


def test_exact_zero_v_columns_survive_rescale():
    w = synth.config_stress(B=1, N=1024)
    w.kv[:, :, 100:110] = 0
    q, K, V = _dense(w)
    out, _ = S.amla(q[:4], K, V, w.scale, 64, guard=True)
    assert np.all(out[:, 100:110] == 0)
    out_bad, _ = S.amla(q[:4], K, V, w.scale, 64, guard=False)
    assert not np.all(out_bad[:, 100:110] == 0)        # the literal add corrupts exact zeros


def test_split_merge_equals_unsplit():
    w = synth.make_workload("t", 1, 1, 5, [700], seed=71)
    q, K, V = _dense(w)
    full, lse_full = S.flash_attention(q, K, V, w.scale, 64)
    cuts = [0, 64, 320, 700]
    outs, lses = zip(*[S.flash_attention(q, K[a:b], V[a:b], w.scale, 64) for a, b in zip(cuts[:-1], cuts[1:])])
    mo, ml = S.merge_splits(outs, lses)
    np.testing.assert_allclose(mo, full, atol=1e-12)
    np.testing.assert_allclose(ml, lse_full, atol=1e-12)
    # a split that saw no key (lse=-inf, out=0) is neutral
    mo2, ml2 = S.merge_splits(list(outs) + [np.zeros_like(full)], list(lses) + [np.full(5, -np.inf)])
    np.testing.assert_allclose(mo2, full, atol=1e-12)
    np.testing.assert_allclose(ml2, lse_full, atol=1e-12)
