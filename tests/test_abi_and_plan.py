"""CPU-side checks of the C-ABI library: it loads, exports what include/amla.h declares, and its
host logic (argument checks that need no device, the split-KV schedule mirror) behaves."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2509_25224_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
UNIT_OVERHEAD = 10      # kUnitOverheadTiles of the schedule


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_symbols():
    txt = open(os.path.join(ROOT, "include", "amla.h")).read()
    txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
    return sorted(set(re.findall(r"\b(amla_[a-z_0-9]+)\s*\(", txt)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(c) for c in range(-5, 1)}
    assert len(seen) == 6 and "unknown status" not in seen
    assert binding.status_string(-99) == "unknown status"


def test_null_and_bad_arguments_are_rejected_before_any_cuda_call(lib):
    z = ctypes.c_void_p(0)
    rc = lib.amla_mla_decode(z, z, z, z, 0.1, 1, 1, 16, 4, 4, z, z, z, 0, z)
    assert rc == -1
    one = ctypes.c_void_p(256)
    # Sq out of range -> unsupported, reported before the device is looked at
    rc = lib.amla_mla_decode(one, one, one, one, 0.1, 1, 9, 16, 4, 4, one, one, one, 1 << 30, z)
    assert rc == -2
    # misaligned q
    rc = lib.amla_mla_decode(ctypes.c_void_p(258), one, one, one, 0.1, 1, 1, 16, 4, 4, one, one, one, 1 << 30, z)
    assert rc == -1
    n = ctypes.c_size_t(0)
    assert lib.amla_mla_decode_workspace_size(0, 1, 16, 4, 0, ctypes.byref(n)) == -1
    assert lib.amla_mla_decode_workspace_size(1, 1, 16, 4, 0, None) == -1


def _check_plan(seqlens, Sq, H, P):
    units = binding.plan_host(seqlens, Sq, H, P)
    nrb = (Sq * H + 127) // 128
    n_items = len(seqlens) * nrb
    tiles = [(max(int(seqlens[it // nrb]), 0) + 63) // 64 for it in range(n_items)]
    cover = [np.zeros(t, dtype=np.int32) for t in tiles]
    per_part = np.zeros(P, dtype=np.int64)
    slots = set()
    nsplit_seen = {}
    last = (-1, -1, -1)
    for p, it, t0, t1, slot, ns in units:
        assert 0 <= p < P and 0 <= it < n_items and 0 <= t0 < t1 <= tiles[it]
        assert (p, it, t0) > last          # units come out in schedule order
        last = (p, it, t0)
        cover[it][t0:t1] += 1
        per_part[p] += t1 - t0
        nsplit_seen.setdefault(it, []).append((p, slot, ns))
        if slot >= 0:
            assert slot not in slots and slot // 2 == p
            slots.add(slot)
    for it in range(n_items):
        assert np.all(cover[it] == 1), "every tile exactly once"
        parts = nsplit_seen.get(it, [])
        assert len(parts) == (0 if tiles[it] == 0 else parts[0][2])
        if not parts:
            continue
        if len(parts) == 1:
            assert parts[0][1] == -1                    # unsplit items write their output directly
        else:
            assert all(s >= 0 for _, s, _ in parts)
            ps = [p for p, _, _ in parts]
            assert ps == list(range(ps[0], ps[0] + len(ps)))   # consecutive parts
    # balance: the schedule cuts a range in which every non-empty item but the first is preceded by UNIT_OVERHEAD positions
    # (the cost of starting an item) into equal parts, so no part holds more tiles than one such share
    Lv = sum(t + (UNIT_OVERHEAD if it else 0) for it, t in enumerate(tiles) if t)
    if Lv:
        assert per_part.max() <= -(-Lv // min(P, Lv))
        starts = np.zeros(P, dtype=np.int64)            # items whose first tile a part holds
        for p, it, t0, t1, slot, ns in units:
            starts[p] += t0 == 0
        assert (per_part + UNIT_OVERHEAD * starts).max() <= -(-Lv // min(P, Lv)) + UNIT_OVERHEAD
    return units


@pytest.mark.parametrize("P", [1, 2, 74, 148])
def test_plan_covers_every_tile_once_and_balances(lib, P):
    rng = np.random.default_rng(5)
    _check_plan(np.array([256]), 1, 16, P)
    _check_plan(np.array([4096] * 32), 1, 128, P)
    _check_plan(synth.mtp_seqlens(), 2, 128, P)
    _check_plan(np.array([65536] * 4), 2, 128, P)
    _check_plan(np.array([0, 1, 0, 64, 65, 0, 7000, 0]), 2, 128, P)
    _check_plan(np.array([0, 0, 0]), 1, 128, P)
    for _ in range(10):
        B = int(rng.integers(1, 40))
        _check_plan(rng.integers(0, 3000, B), int(rng.integers(1, 4)), int(rng.choice([16, 64, 128])), P)


def test_plan_small_case_by_hand(lib):
    # two sequences of 3 and 1 tiles, 2 parts: positions [tiles 0-2 | 10 overhead, tile 0] = 14; part 0 = [0,7) holds
    # the first item, part 1 = [7,14) the second
    u = binding.plan_host(np.array([129, 10]), 1, 128, 2)
    assert u.tolist() == [[0, 0, 0, 3, -1, 1], [1, 1, 0, 1, -1, 1]]


def test_batch_sharding_partitions_sequences():
    for B in (1, 7, 32, 64):
        for ws in (1, 2, 3, 8):
            got = [i for r in range(ws) for i in synth.shard_batch(B, ws, r)]
            assert got == list(range(B))
            sizes = [len(synth.shard_batch(B, ws, r)) for r in range(ws)]
            assert max(sizes) - min(sizes) <= 1
