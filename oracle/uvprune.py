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
