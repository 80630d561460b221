"""TEST INFRASTRUCTURE -- not part of the product path.

CPU simulators, in numpy, of the two recurrences the paper states, written in
the paper's order and notation so they can be checked against it by eye:

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
    """Algorithm 2 in FP32 with bf16 P (the mixed precision of Appendix A).

    Returns (O [G,Dv] float32, lse [G] float32).  ``trace``, if a list, receives one
    dict per tile with the per-row scalars (m, n, S32, S16, c, eps, N).
    """
    f = np.float32
    Q = np.asarray(Q, dtype=f); K = np.asarray(K, dtype=f); V = np.asarray(V, dtype=f)
    G, S2 = Q.shape[0], K.shape[0]
    O = np.zeros((G, V.shape[1]), dtype=f)
    m = np.full(G, -np.inf, dtype=f)
    l = np.zeros(G, dtype=f)
    n_prev = np.zeros(G, dtype=f)
    c_prev = np.ones(G, dtype=f)
    S16 = np.ones(G, dtype=f)
    started = np.zeros(G, dtype=bool)       # row has received at least one P V product ("i > 1" per row)
    for lo in range(0, S2, tile):
        hi = min(S2, lo + tile)
        S = (Q @ K[lo:hi].T).astype(f) * f(scale)                          # lines 4-5
        if visible is not None:
            S = np.where(np.arange(lo, hi)[None, :] < np.asarray(visible)[:, None], S, f(-np.inf)).astype(f)
        m_new = np.maximum(m, S.max(axis=1)).astype(f)
        live = ~np.isneginf(m_new)
        m_safe = np.where(live, m_new, f(0)).astype(f)
        M_up = np.where(np.isneginf(m), f(0), np.exp((m - m_safe).astype(f))).astype(f)
        n_i = np.rint(-m_safe / LN2).astype(f)                              # line 6
        P = np.exp((S - m_safe[:, None]).astype(f)).astype(f)
        l = (l * M_up + P.sum(axis=1, dtype=f)).astype(f)
        S32 = np.exp((LN2 * (n_i + m_safe / LN2)).astype(f)).astype(f)      # line 7: 1/r_i
        S16 = bf16_round(S32)                                               # line 8: 1/r'_i
        if c_mode == "appendix":
            c_i = (S16 / S32).astype(f)                                     # r_i / r'_i
        elif c_mode == "listing":
            c_i = (S32 / S16).astype(f)
        elif c_mode == "none":
            c_i = np.ones(G, dtype=f)
        else:
            raise ValueError(c_mode)
        eps = (f(1.5) * (c_i / c_prev - f(1))).astype(f)                    # line 9
        Pt = bf16_round((P * S16[:, None]).astype(f))                       # line 10
        Nf = np.maximum(n_i - n_prev, f(clamp)).astype(np.float64)          # line 11 (exact in fp64)
        N = np.rint((Nf + eps.astype(np.float64) + tiny) * 2.0 ** 23).astype(np.int64)   # line 12
        changed = m_new != m
        apply = started & live & (changed if skip_unchanged else True)
        N = np.where(apply, N, 0)
        O = exponent_add(O, N[:, None], guard=guard)                        # lines 13-16
        O = (O + (Pt @ V[lo:hi]).astype(f)).astype(f)                       # lines 17-18
        if trace is not None:
            trace.append(dict(m=m_new.copy(), n=n_i.copy(), S32=S32.copy(), S16=S16.copy(),
                              c=c_i.copy(), eps=eps.copy(), N=N.copy()))
        upd = live
        n_prev = np.where(upd, n_i, n_prev).astype(f)
        c_prev = np.where(upd, c_i, c_prev).astype(f)
        started = started | live
        m = m_new
    with np.errstate(divide="ignore", invalid="ignore"):
        den = (l * S16).astype(f)
        out = np.where(l[:, None] > 0, O / np.where(l > 0, den, f(1))[:, None], f(0)).astype(f)   # line 20
        lse = np.where(l > 0, m + np.log(np.where(l > 0, l, f(1))), f(-np.inf)).astype(f)
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
