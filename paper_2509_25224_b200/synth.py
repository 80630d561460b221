"""Seeded synthetic MLA-decode workloads (inputs only).

This module builds the tensors that both the CUDA path and the CPU oracle
consume: bf16 bit patterns (as uint16), int32 block tables and sequence
lengths.  It contains none of the attention arithmetic; the only numeric
step is rounding float32 samples to bf16 (round to nearest even), which is
input preparation.  Random numbers come from numpy's Philox bit generator,
so the same seed gives the same bits on every machine.

Shapes follow the decode setting of the paper's Section 5.2 (128 query
heads, one latent KV head, d_qk = 576, d_v = 512, bf16) with a paged cache
of 64-token pages.  The paper's benchmark inputs are private; these stand in
for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

D_QK = 576
D_V = 512
PAGE = 64

# One 64-bit seed per named configuration.
SEEDS = {
    "tiny": 2509252241,
    "dsv3": 2509252242,
    "mtp": 2509252243,
    "stress": 2509252244,
    "long": 2509252245,
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to OCP FP8 E4M3 (nearest even, saturating at +-448); returns the uint8 bit patterns.
    Input preparation for the FP8-cache workloads: 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent
    field 0 holds the subnormals m * 2^-9; S.1111.111 (NaN) is never produced."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    sign = (np.signbit(x)).astype(np.uint8) << 7
    a = np.minimum(np.abs(x).astype(np.float64), 448.0)
    # spacing of the E4M3 grid at |x|: 2^(e-3) with e = max(floor(log2 |x|), -6)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)
    step = np.exp2(e - 3.0)
    k = np.rint(a / step)                 # nearest even multiple count (numpy rounds half to even)
    v = k * step                          # may land on the next binade (k = 16), still representable or 448+ -> clamp
    v = np.minimum(v, 448.0)
    # encode v exactly
    with np.errstate(divide="ignore"):
        ev = np.floor(np.log2(np.where(v > 0, v, 1.0)))
    ev = np.maximum(ev, -6.0)
    mant = v / np.exp2(ev)                # in [1, 2) for normals, [0, 1) for subnormals
    is_sub = v < 2.0 ** -6
    efield = np.where(is_sub, 0, ev + 7).astype(np.int64)
    mfield = np.where(is_sub, np.rint(v * 512.0), np.rint((mant - 1.0) * 8.0)).astype(np.int64)
    return (sign | (efield.astype(np.uint8) << 3) | mfield.astype(np.uint8)).astype(np.uint8)


@dataclass
class Workload:
    name: str
    B: int
    Sq: int
    H: int
    seqlens: np.ndarray          # int32 [B], KV length including the Sq new tokens
    q: np.ndarray                # uint16 (bf16 bits) [B, Sq, H, 576]
    kv: np.ndarray               # uint16 (bf16 bits) [num_blocks, 64, 576]; V = columns 0..511
    block_table: np.ndarray      # int32 [B, max_blocks_per_seq]; unused entries are -1
    scale: float
    meta: dict = field(default_factory=dict)

    @property
    def num_blocks(self) -> int:
        return int(self.kv.shape[0])

    @property
    def max_blocks_per_seq(self) -> int:
        return int(self.block_table.shape[1])

    def flops(self) -> float:
        """2 * sum_b Sq*H*N_b*(576+512): the paper's FLOP count (Section 2.4)."""
        return 2.0 * float(self.Sq) * self.H * float(self.seqlens.astype(np.int64).sum()) * (D_QK + D_V)

    def algorithmic_bytes(self) -> float:
        """KV read once + q + out + lse (bf16 tensors, fp32 lse)."""
        kvb = float(self.seqlens.astype(np.int64).sum()) * D_QK * 2
        rows = self.B * self.Sq * self.H
        return kvb + rows * D_QK * 2 + rows * (D_V * 2 + 4)


def _normal_bf16(rng: np.random.Generator, shape, sigma: float = 1.0, chunk: int = 1 << 24) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = rng.standard_normal(e - s, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        out[s:e] = f32_to_bf16_bits(x)
    return out.reshape(shape)


def _uniform_bf16(rng: np.random.Generator, shape, a: float) -> np.ndarray:
    x = rng.random(int(np.prod(shape)), dtype=np.float32)
    x = (x * np.float32(2.0 * a) - np.float32(a)).astype(np.float32)
    return f32_to_bf16_bits(x).reshape(shape)


def make_workload(name: str, B: int, Sq: int, H: int, seqlens, seed: int, *,
                  scale: float = 1.0 / math.sqrt(192.0), shuffle_pages: bool = True,
                  spare_blocks: int = 0, dist: str = "normal", sigma: float = 1.0,
                  max_blocks_per_seq: int | None = None) -> Workload:
    """Generic builder: random q and KV pages, block table from a page permutation."""
    seqlens = np.asarray(seqlens, dtype=np.int32).reshape(B)
    rng = np.random.Generator(np.random.Philox(seed))
    nblk = (seqlens.astype(np.int64) + PAGE - 1) // PAGE
    total = int(nblk.sum()) + int(spare_blocks)
    total = max(total, 1)
    mb = int(max(1, nblk.max() if B else 1))
    if max_blocks_per_seq is not None:
        assert max_blocks_per_seq >= mb
        mb = max_blocks_per_seq
    if dist == "normal":
        q = _normal_bf16(rng, (B, Sq, H, D_QK), sigma)
        kv = _normal_bf16(rng, (total, PAGE, D_QK), sigma)
    elif dist == "uniform":
        q = _uniform_bf16(rng, (B, Sq, H, D_QK), sigma)
        kv = _uniform_bf16(rng, (total, PAGE, D_QK), sigma)
    else:
        raise ValueError(dist)
    perm = rng.permutation(total).astype(np.int32) if shuffle_pages else np.arange(total, dtype=np.int32)
    bt = np.full((B, mb), -1, dtype=np.int32)
    off = 0
    for b in range(B):
        k = int(nblk[b])
        bt[b, :k] = perm[off:off + k]
        off += k
    return Workload(name, B, Sq, H, seqlens, q, kv, bt, float(scale),
                    meta={"seed": seed, "dist": dist, "sigma": sigma, "shuffled": shuffle_pages})


def quantise_cache_e4m3(w: Workload, kv_scale: float = 1.0 / 64.0) -> np.ndarray:
    """uint8 [num_blocks, 64, 576]: the workload's bf16 cache divided by kv_scale and rounded to E4M3 (the FP8-cache
    variant of the same workload; element value = decode(byte) * kv_scale).  With the default scale N(0,1) values
    land around +-64 in the E4M3 range (max 448)."""
    out = np.empty(w.kv.shape, dtype=np.uint8)
    flat_in = w.kv.reshape(-1)
    flat_out = out.reshape(-1)
    chunk = 1 << 24
    for s0 in range(0, flat_in.size, chunk):
        x = bf16_bits_to_f32(flat_in[s0:s0 + chunk]) / np.float32(kv_scale)
        flat_out[s0:s0 + chunk] = f32_to_e4m3_bits(x)
    return out


def logical_kv_rows(w: Workload, b: int) -> np.ndarray:
    """uint16 [N_b, 576]: the logical key rows of sequence b gathered through the block table."""
    n = int(w.seqlens[b])
    nb = (n + PAGE - 1) // PAGE
    pages = w.kv[w.block_table[b, :nb]]
    return pages.reshape(nb * PAGE, D_QK)[:n]


def staircase_offsets(n: int, lo: float = -30.0, hi: float = 30.0, steps: int = 32) -> np.ndarray:
    """Per-position logit offsets rising in `steps` equal steps from lo to hi."""
    j = np.arange(n, dtype=np.int64)
    return lo + (hi - lo) * ((steps * j) // n).astype(np.float64) / float(steps - 1)


def apply_logit_offsets(w: Workload, offsets_per_seq, q_gain: float = 4.0) -> None:
    """Plant a known additive logit offset per key position.

    Column 512 (first RoPE column) of every query row is set to q_gain and the
    same column of key j to bf16(offset_j / (q_gain * scale)), so that the
    scaled logit gains ~offset_j on top of the random part.
    """
    w.q[..., D_V] = f32_to_bf16_bits(np.full(w.q.shape[:-1], q_gain, dtype=np.float32))
    for b in range(w.B):
        n = int(w.seqlens[b])
        off = np.asarray(offsets_per_seq[b], dtype=np.float64)[:n]
        col = f32_to_bf16_bits((off / (q_gain * w.scale)).astype(np.float32))
        for i in range((n + PAGE - 1) // PAGE):
            lo, hi = i * PAGE, min(n, (i + 1) * PAGE)
            w.kv[w.block_table[b, i], : hi - lo, D_V] = col[lo:hi]


# ----------------------------------------------------------------------------
# The five named configurations.
# ----------------------------------------------------------------------------

def config_tiny() -> Workload:
    return make_workload("tiny", 1, 1, 16, [256], SEEDS["tiny"], shuffle_pages=False)


def config_dsv3() -> Workload:
    return make_workload("dsv3", 32, 1, 128, [4096] * 32, SEEDS["dsv3"])


def mtp_seqlens(B: int = 64, seed: int = SEEDS["mtp"]) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(seed ^ 0x5EED))
    return rng.integers(1024, 8193, size=B).astype(np.int32)


def config_mtp() -> Workload:
    return make_workload("mtp", 64, 2, 128, mtp_seqlens(), SEEDS["mtp"])


def config_stress(B: int = 16, N: int = 16384) -> Workload:
    w = make_workload("stress", B, 1, 128, [N] * B, SEEDS["stress"])
    apply_logit_offsets(w, [staircase_offsets(N)] * B)
    return w


def config_long() -> Workload:
    return make_workload("long", 4, 2, 128, [65536] * 4, SEEDS["long"])


CONFIGS = {
    "tiny": config_tiny,
    "dsv3": config_dsv3,
    "mtp": config_mtp,
    "stress": config_stress,
    "long": config_long,
}


def shard_batch(B: int, world_size: int, rank: int) -> range:
    """Contiguous slice of sequence indices owned by `rank` (no collective needed:
    sequences are independent problems)."""
    base, rem = divmod(B, world_size)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))
