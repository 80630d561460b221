"""TEST INFRASTRUCTURE -- not part of the product path.

CPU simulators, in numpy, of the two recurrences the paper states, in the
paper's notation so they can be checked against it by eye:

* ``flash_attention``  -- Algorithm 1 (tiled online softmax, "Base").
* ``amla``             -- Algorithm 2 (AMLA): power-of-two reference n_i,
  S32 = 1/r_i, S16 = bf16(S32), compensation factor c_i, the integer N added to
  the bit pattern of the FP32 accumulator (Lemma 3.1, Appendix A).
* ``exponent_add``     -- the Lemma 3.1 identity on raw bit patterns.

They are secondary references (the role of the paper's "Base" in Section 5.1):
the parity oracle is the FP64 definition in ``mla_decode_oracle.cpp``.  The
simulators pin the readings of the paper that the CUDA kernels implement and
are themselves pinned in tests/test_amla_sim.py (tiling invariance against the
FP64 oracle, bit-exactness against ldexp, Example 3.1's bit pattern, the
"AMLA ~= Base" relation of Tables 3-4).

Readings taken where the paper is ambiguous (each is an argument here so the
alternative can be evaluated):
  c_mode="appendix": c_i = S16/S32 (= r_i/r'_i, Appendix A); "listing" uses
      S32/S16 as printed in Algorithm 2 line 9; "none" sets eps = 0.
  skip_unchanged: add N only for rows whose running max changed (otherwise the
      true factor is exactly 1).
  guard: clamp the magnitude bits at zero so that 0.0 and tiny accumulators do
      not wrap when a negative N is added (Lemma 3.1 requires 0 < E + n).
"""
from __future__ import annotations

import numpy as np

LN2 = np.float32(np.log(2.0))


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest-even bf16 -> float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)) << np.uint32(16)
    return r.astype(np.uint32).view(np.float32)


def exponent_add(f: np.ndarray, n_int: np.ndarray, guard: bool = False) -> np.ndarray:
    """AS_FP32(AS_INT32(F) + N) elementwise (Lemma 3.1; N = n * 2**23 for a pure power of two).

    With ``guard`` the add is applied to the magnitude bits and clamped at zero,
    the sign bit is kept: exact zeros stay zero and results that would leave the
    normal range downwards become zero/denormal instead of wrapping.
    """
    i = np.ascontiguousarray(f, dtype=np.float32).view(np.int32).astype(np.int64)
    n = np.asarray(n_int, dtype=np.int64)
    if not guard:
        r = (i + n) & 0xFFFFFFFF
        return r.astype(np.uint32).view(np.float32)
    sign = i & 0x80000000
    mag = i & 0x7FFFFFFF
    mag = np.maximum(mag + n, 0)
    r = (mag | sign) & 0xFFFFFFFF
    return r.astype(np.uint32).view(np.float32)


def flash_attention(Q, K, V, scale, tile, dtype=np.float64, low_precision_matmul=False, visible=None):
    """Algorithm 1.  Q [G,Dk], K [S2,Dk], V [S2,Dv]; returns (O [G,Dv], lse [G]).

    ``visible`` (int array [G]) limits row g to keys 0..visible[g]-1 (masking is
    outside the paper; masked logits are -inf).  With ``low_precision_matmul`` P is
    rounded to bf16 before P@V, as on matrix hardware with bf16 inputs.
    """
    dt = dtype
    Q = np.asarray(Q, dtype=dt); K = np.asarray(K, dtype=dt); V = np.asarray(V, dtype=dt)
    G, S2 = Q.shape[0], K.shape[0]
    O = np.zeros((G, V.shape[1]), dtype=dt)
    m = np.full(G, -np.inf, dtype=dt)
    l = np.zeros(G, dtype=dt)
    for lo in range(0, S2, tile):
        hi = min(S2, lo + tile)
        S = (Q @ K[lo:hi].T) * dt(scale)                                   # C1 + scaling
        if visible is not None:
            S = np.where(np.arange(lo, hi)[None, :] < np.asarray(visible)[:, None], S, -np.inf)
        m_new = np.maximum(m, S.max(axis=1))
        m_safe = np.where(np.isneginf(m_new), dt(0), m_new)
        P = np.exp(S - m_safe[:, None])
        up = np.where(np.isneginf(m), dt(0), np.exp(m - m_safe))
        l = l * up + P.sum(axis=1)
        if low_precision_matmul:
            P = bf16_round(P.astype(np.float32)).astype(dt)
        T = P @ V[lo:hi]                                                   # C2
        O = O * up[:, None] + T                                            # V2
        m = m_new
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(l[:, None] > 0, O / np.where(l > 0, l, 1)[:, None], 0)
        lse = np.where(l > 0, m + np.log(np.where(l > 0, l, 1)), -np.inf)
    return out, lse


def amla(Q, K, V, scale, tile, c_mode="appendix", skip_unchanged=True, guard=True,
         clamp=-30.0, tiny=1e-6, visible=None, trace=None):
    """AMLA (Algorithm 2; Eq. 3, Lemma 3.1, Appendix A) in FP32 with bf16 P, organised around its quantities.

    Everything the rescaling needs depends on the running row maxima alone, so it is computed first, for all
    tiles at once: the power-of-two reference n_i = round(-m_i / ln 2) (Eq. 3), S32_i = 1/r_i = exp(n_i ln 2 + m_i)
    in [1/sqrt 2, sqrt 2], its bf16 rounding S16_i, the compensation c_i of Appendix A, the residual
    eps_i = 1.5 (c_i / c_{i-1} - 1), and from them the integer N_i that Lemma 3.1 adds to the bit pattern of the
    accumulator, (max(n_i - n_{i-1}, clamp) + eps_i + tiny) * 2^23 rounded.  The second part walks the tiles: P and the
    row sum against the reference, P~ = bf16(P * S16_i), the integer add on O, O += P~ V.  The result is
    O / (l * S16) of the last tile.

    Returns (O [G,Dv] float32, lse [G] float32).  ``trace``, if a list, receives one dict per tile with the per-row
    scalars (m, n, S32, S16, c, eps, N).
    """
    f = np.float32
    Q = np.asarray(Q, dtype=f); K = np.asarray(K, dtype=f); V = np.asarray(V, dtype=f)
    G, S2 = Q.shape[0], K.shape[0]
    bounds = [(lo, min(S2, lo + tile)) for lo in range(0, S2, tile)]
    T = len(bounds)
    if T == 0:
        return np.zeros((G, V.shape[1]), dtype=f), np.full(G, -np.inf, dtype=f)

    # ---- scores of every tile and the running maxima
    tiles = []
    for lo, hi in bounds:
        S = (Q @ K[lo:hi].T).astype(f) * f(scale)
        if visible is not None:
            S = np.where(np.arange(lo, hi)[None, :] < np.asarray(visible)[:, None], S, f(-np.inf)).astype(f)
        tiles.append(S)
    m = np.maximum.accumulate(np.stack([S.max(axis=1) for S in tiles]).astype(f), axis=0)      # [T, G]
    m_before = np.concatenate([np.full((1, G), -np.inf, dtype=f), m[:-1]])
    live = ~np.isneginf(m)                                   # the row has seen a key by tile i
    started = ~np.isneginf(m_before)                         # ... before tile i: O holds something to rescale
    m_safe = np.where(live, m, f(0)).astype(f)

    # ---- what the rescaling needs, for all tiles (Eq. 3, Appendix A)
    n = np.rint(-m_safe / LN2).astype(f)
    S32 = np.exp((LN2 * (n + m_safe / LN2)).astype(f)).astype(f)
    S16 = bf16_round(S32)
    if c_mode == "appendix":
        c = (S16 / S32).astype(f)                            # r_i / r'_i
    elif c_mode == "listing":
        c = (S32 / S16).astype(f)
    elif c_mode == "none":
        c = np.ones((T, G), dtype=f)
    else:
        raise ValueError(c_mode)
    # the scalars of the previous tile that had seen a key (n = 0, c = 1 before there is one)
    n_before = np.concatenate([np.zeros((1, G), dtype=f), n[:-1]])
    c_before = np.concatenate([np.ones((1, G), dtype=f), c[:-1]])
    n_before = np.where(started, n_before, f(0)).astype(f)
    c_before = np.where(started, c_before, f(1)).astype(f)
    eps = (f(1.5) * (c / c_before - f(1))).astype(f)
    dn = np.maximum(n - n_before, f(clamp)).astype(np.float64)
    N = np.rint((dn + eps.astype(np.float64) + tiny) * 2.0 ** 23).astype(np.int64)
    moved = (m != m_before) if skip_unchanged else np.ones((T, G), dtype=bool)
    N = np.where(started & live & moved, N, 0)
    l_up = np.where(started, np.exp((m_before - m_safe).astype(f)), f(0)).astype(f)       # exp(m_{i-1} - m_i)

    # ---- the tiles: row sum, P~, integer add on O, accumulation
    O = np.zeros((G, V.shape[1]), dtype=f)
    l = np.zeros(G, dtype=f)
    for i, (lo, hi) in enumerate(bounds):
        P = np.exp((tiles[i] - m_safe[i][:, None]).astype(f)).astype(f)
        l = (l * l_up[i] + P.sum(axis=1, dtype=f)).astype(f)
        Pt = bf16_round((P * S16[i][:, None]).astype(f))
        O = exponent_add(O, N[i][:, None], guard=guard)
        O = (O + (Pt @ V[lo:hi]).astype(f)).astype(f)
        if trace is not None:
            trace.append(dict(m=m[i].copy(), n=n[i].copy(), S32=S32[i].copy(), S16=S16[i].copy(),
                              c=c[i].copy(), eps=eps[i].copy(), N=N[i].copy()))
    with np.errstate(divide="ignore", invalid="ignore"):
        den = (l * S16[-1]).astype(f)
        out = np.where(l[:, None] > 0, O / np.where(l > 0, den, f(1))[:, None], f(0)).astype(f)
        lse = np.where(l > 0, m[-1] + np.log(np.where(l > 0, l, f(1))), f(-np.inf)).astype(f)
    return out, lse


def merge_splits(outs, lses):
    """Log-sum-exp merge of per-split normalised outputs (follows from the blockwise
    associativity of Algorithm 1's recurrence).  outs [S,G,Dv], lses [S,G] -> (out, lse)."""
    outs = np.asarray(outs, dtype=np.float64); lses = np.asarray(lses, dtype=np.float64)
    mx = lses.max(axis=0)
    mx_safe = np.where(np.isneginf(mx), 0.0, mx)
    w = np.exp(lses - mx_safe[None])
    tot = w.sum(axis=0)
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(tot[:, None] > 0, (w[:, :, None] * outs).sum(axis=0) / np.where(tot > 0, tot, 1)[:, None], 0.0)
        lse = np.where(tot > 0, mx_safe + np.log(np.where(tot > 0, tot, 1)), -np.inf)
    return out, lse


def rel_frobenius(A, B):
    """The paper's accuracy metric (Section 5.1): ||A-B||_F / (||B||_F + 1e-10)."""
    A = np.asarray(A, dtype=np.float64); B = np.asarray(B, dtype=np.float64)
    return float(np.linalg.norm(A - B) / (np.linalg.norm(B) + 1e-10))
