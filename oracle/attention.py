"""Oracle: window-verify grouped-query attention and per-key attention mass.

The target model scores the gamma+1 window positions in one pass over the
whole multimodal prefix (Sec. 2.2: the drafted tokens are verified "in a
single, parallel forward pass"; Sec. 4.2 Stage II: verification uses the full
context V_{1:m}).  The arithmetic is standard scaled-dot-product attention:
s = scale * q.k, P = softmax over the visible keys, O = P V.  The attention
mass of key j is the sum of P over all query heads and window rows, i.e. the
"attention score" signal that attention-guided pruning ranks tokens by
(Sec. 3, Challenge 2).

Readings where the paper is silent: query head h uses KV head floor(h / G)
(contiguous groups); scale = 1/sqrt(D); window row r sees keys 0..n_ctx+r
(the context, then the window's own rows causally).
"""
from __future__ import annotations

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def verify_attn(q_bits, k_bits, v_bits, n_ctx: int, scale: float | None = None, heads=None):
    """q [R,Hq,D], k,v [T,Hkv,D] (bf16 bits), T = n_ctx + R.

    Returns (O fp64 [R,Hq,D], lse fp64 [Hq,R] natural log, mass fp64 [T]).
    `heads` restricts the work to a subset of query heads (sampled checks at
    full size); mass then only holds those heads' contribution.
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    R, Hq, D = q.shape
    T, Hkv, _ = k.shape
    assert T == n_ctx + R and Hq % Hkv == 0
    G = Hq // Hkv
    if scale is None or scale == 0.0:
        scale = 1.0 / np.sqrt(D)
    O = np.zeros((R, Hq, D))
    lse = np.full((Hq, R), -np.inf)
    mass = np.zeros(T)
    for h in (range(Hq) if heads is None else heads):
        g = h // G
        S = scale * (k[:, g, :] @ q[:, h, :].T)         # [T, R] scores of head h against every key
        for r in range(R):
            vis = n_ctx + r + 1                          # row r sees keys 0 .. n_ctx + r
            s = S[:vis, r]
            M = s.max()
            e = np.exp(s - M)
            Z = e.sum()
            P = e / Z
            lse[h, r] = M + np.log(Z)
            O[r, h, :] = P @ v[:vis, g, :]
            mass[:vis] += P
    return O, lse, mass
