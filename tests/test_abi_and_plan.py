"""CPU-side checks of the C-ABI library: it loads, exports what include/amla.h declares, and its
host logic (argument checks that need no device, the split-KV schedule mirror) behaves."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2509_25224_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _variant(Sq, H):
    """(rows per item, keys per tile, overhead positions) of the schedule for a shape: up to 128 query rows per
    sequence the items are 128-row blocks with one-page tiles, above that 256-row blocks with two-page tiles."""
    return (256, 128, 5) if Sq * H > 128 else (128, 64, 6)


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
    seen = {binding.status_string(c) for c in range(-6, 1)}
    assert len(seen) == 7 and "unknown status" not in seen
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
    item_rows, tile_keys, UNIT_OVERHEAD = _variant(Sq, H)
    nrb = (Sq * H + item_rows - 1) // item_rows
    n_items = len(seqlens) * nrb
    tiles = [(max(int(seqlens[it // nrb]), 0) + tile_keys - 1) // tile_keys for it in range(n_items)]
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
    # two sequences of 3 and 1 tiles, 2 parts: positions [tiles 0-2 | 6 overhead, tile 0] = 10; part 0 = [0,5) holds
    # the first item, part 1 = [5,10) the second
    u = binding.plan_host(np.array([129, 10]), 1, 128, 2)
    assert u.tolist() == [[0, 0, 0, 3, -1, 1], [1, 1, 0, 1, -1, 1]]


def test_plan_small_case_by_hand_256_row_items(lib):
    # Sq = 2, H = 128: one 256-row item per sequence, 128-key tiles, 5 overhead positions.  Lengths 300 and 100 give
    # 3 and 1 tiles: positions [tiles 0-2 | 5 overhead, tile 0] = 9; 3 parts own [0,3), [3,6), [6,9): the first
    # item is one unit of part 0, the second item's tile (position 8) falls into part 2
    u = binding.plan_host(np.array([300, 100]), 2, 128, 3)
    assert u.tolist() == [[0, 0, 0, 3, -1, 1], [2, 1, 0, 1, -1, 1]]
    # Sq = 3: 384 rows are two 256-row items per sequence (the second half filled)
    u = binding.plan_host(np.array([128]), 3, 128, 1)
    assert u.tolist() == [[0, 0, 0, 1, -1, 1], [0, 1, 0, 1, -1, 1]]


def test_paging_validation_names_the_bad_entry(lib):
    bt = np.array([[3, 1, -1], [0, 2, 7]], dtype=np.int32)
    assert binding.validate_paging_host(bt, [100, 192], 8) is None            # unused entries are ignored
    assert binding.validate_paging_host(bt, [129, 192], 8) == (0, 2)          # third page of sequence 0 is -1
    assert binding.validate_paging_host(bt, [100, 192], 7) == (1, 2)          # page 7 of a 7-page cache
    assert binding.validate_paging_host(bt, [100, 193], 8) == (1, -1)         # longer than the table allows
    assert binding.validate_paging_host(bt, [-1, 0], 8) == (0, -1)
    z = ctypes.c_void_p(0)
    assert lib.amla_validate_paging_host(z, z, 1, 1, 1, None, None) == -1


def test_wait_selftest_rejects_bad_arguments_without_a_device(lib):
    z = ctypes.c_void_p(0)
    assert lib.amla_wait_selftest(z, 1000, z) == -1
    assert lib.amla_wait_selftest(ctypes.c_void_p(256), 0, z) == -1
    assert lib.amla_wait_selftest(ctypes.c_void_p(256), 10**9, z) == -1       # limits above 0.1 s are refused
    assert lib.amla_wait_selftest(ctypes.c_void_p(258), 1000, z) == -1


def test_batch_sharding_partitions_sequences():
    for B in (1, 7, 32, 64):
        for ws in (1, 2, 3, 8):
            got = [i for r in range(ws) for i in synth.shard_batch(B, ws, r)]
            assert got == list(range(B))
            sizes = [len(synth.shard_batch(B, ws, r)) for r in range(ws)]
            assert max(sizes) - min(sizes) <= 1
