"""Oracle: UV-Prune score (layer-to-layer variation), Top-K, and the gather
that builds the draft's pruned context.

Eq. 2 scores visual token i by the sum over layers of the change of its
relevance signal between consecutive layers (already summed over the text /
query side); the rationale (Appendix E) is that the position-induced part of
the signal is the same at every layer and cancels in the difference, and the
paper reports that this variation step helps the attention criterion as well
as the similarity one.  Here the per-layer signal is the attention mass of the
verify pass.  Eq. 3 keeps the Top-K scores; Eq. 5 fixes K as the 1 - alpha
fraction.  Sec. 4.2 (Stage I) defines the draft context as the kept visual
tokens V* followed by all text tokens.

Readings: ties go to the lower index (so the result is unique); the kept
indices are reported in ascending order (V* stays a subsequence of the
video); -0.0 equals +0.0; inputs are finite.
"""
from __future__ import annotations

import numpy as np


def cosine_similarity(hidden_bits, vis_start: int, m: int, text_start: int, n: int) -> np.ndarray:
    """Eq. 1: S_ij = V_i . X_j / (|V_i| |X_j|) between the m visual rows and the n text rows of one
    layer's token representations (bf16 bits [rows, d]).  Returns the full fp64 matrix [m, n].
    A zero vector has similarity 0 with everything."""
    b = np.ascontiguousarray(hidden_bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    h = b.view(np.float32).astype(np.float64)
    V = h[vis_start:vis_start + m]
    X = h[text_start:text_start + n]
    nv = np.sqrt((V * V).sum(axis=1))
    nx = np.sqrt((X * X).sum(axis=1))
    S = V @ X.T
    denom = nv[:, None] * nx[None, :]
    return np.divide(S, denom, out=np.zeros_like(S), where=denom > 0)


def similarity_sum(hidden_bits, vis_start: int, m: int, text_start: int, n: int) -> np.ndarray:
    """sum_j S_ij: the per-layer relevance signal of visual token i (the inner sum of Eq. 2)."""
    return cosine_similarity(hidden_bits, vis_start, m, text_start, n).sum(axis=1)


def similarity_variation(hidden_layers, vis_start: int, m: int, text_start: int, n: int) -> np.ndarray:
    """Eq. 2 as printed: sum over text tokens j and over layers l = 1..L of (S^l_ij - S^{l-1}_ij);
    hidden_layers[0] is layer 0."""
    S = [cosine_similarity(h, vis_start, m, text_start, n) for h in hidden_layers]
    score = np.zeros(m)
    for j in range(n):
        for l in range(1, len(S)):
            score += S[l][:, j] - S[l - 1][:, j]
    return score


def variation_score(mass_layers, vis_start: int, m: int) -> np.ndarray:
    """Eq. 2 as printed: sum over consecutive-layer differences, in fp64.

    mass_layers: sequence of per-layer mass arrays (layer 0 first)."""
    ml = [np.asarray(x, dtype=np.float64)[vis_start:vis_start + m] for x in mass_layers]
    score = np.zeros(m)
    for l in range(1, len(ml)):
        score += ml[l] - ml[l - 1]
    return score


def score_fp32(mass_cur, mass_ref, vis_start: int, m: int) -> np.ndarray:
    """The canonical score the selection ranks by: Eq. 2 telescoped to its two
    end layers and evaluated as ONE fp32 subtraction (round to nearest); with
    no reference layer it is the raw mass (the attention-guided criterion)."""
    cur = np.asarray(mass_cur, dtype=np.float32)[vis_start:vis_start + m]
    if mass_ref is None:
        return cur.copy()
    ref = np.asarray(mass_ref, dtype=np.float32)[vis_start:vis_start + m]
    return (cur - ref).astype(np.float32)


def select_topk(score: np.ndarray, k: int) -> np.ndarray:
    """Eq. 3: indices of the k largest scores, ties to the lower index,
    returned ascending (int32)."""
    score = np.asarray(score)
    m = score.shape[0]
    assert 0 <= k <= m
    s = score + 0.0                                   # -0.0 -> +0.0
    order = np.argsort(-s, kind="stable")             # descending, stable => lower index first
    return np.sort(order[:k]).astype(np.int32)


def gather_rows(src: np.ndarray, vis_start: int, m: int, idx: np.ndarray) -> np.ndarray:
    """src [L, S, ...] -> [L, S - m + k, ...]: rows before the visual span,
    the kept visual rows (vis_start + idx), then everything after the span."""
    idx = np.asarray(idx, dtype=np.int64)
    return np.concatenate([src[:, :vis_start], src[:, vis_start + idx], src[:, vis_start + m:]], axis=1)
