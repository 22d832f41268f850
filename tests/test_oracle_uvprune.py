"""Pins for the UV-Prune oracle: Eq. 2's telescoping, Top-K against brute
force and a library routine, the tie rule, gather against explicit loops, and
the direction of the debiasing effect."""
import numpy as np
import pytest

from oracle.attention import verify_attn
from oracle.uvprune import gather_rows, score_fp32, select_topk, variation_score
from paper_2603_19610_b200 import workloads as wl


def test_eq2_telescopes():
    rng = np.random.default_rng(1)
    L, T, v0, m = 7, 50, 3, 40
    layers = [rng.random(T).astype(np.float32) for _ in range(L)]
    full = variation_score(layers, v0, m)
    ends = layers[-1].astype(np.float64)[v0:v0 + m] - layers[0].astype(np.float64)[v0:v0 + m]
    np.testing.assert_allclose(full, ends, rtol=0, atol=1e-12)
    s32 = score_fp32(layers[-1], layers[0], v0, m)
    assert s32.dtype == np.float32
    np.testing.assert_allclose(s32, full, rtol=0, atol=1e-6 * (np.abs(layers[-1]).max() + np.abs(layers[0]).max()))
    np.testing.assert_array_equal(score_fp32(layers[-1], None, v0, m), layers[-1][v0:v0 + m])


def brute_topk(score, k):
    order = sorted(range(len(score)), key=lambda i: (-float(score[i]), i))
    return np.array(sorted(order[:k]), dtype=np.int32)


@pytest.mark.parametrize("m,k", [(1, 1), (17, 5), (100, 0), (100, 100), (257, 31), (1000, 250)])
def test_topk_brute_force(m, k):
    rng = np.random.default_rng(m * 31 + k)
    distinct = rng.standard_normal(m).astype(np.float32)
    np.testing.assert_array_equal(select_topk(distinct, k), brute_topk(distinct, k))
    if 0 < k < m:                                   # distinct scores: equals the argpartition set
        part = np.sort(np.argpartition(-distinct, k - 1)[:k])
        np.testing.assert_array_equal(select_topk(distinct, k), part)
    tied = (np.round(distinct * 2) / 2).astype(np.float32)      # heavy ties
    got = select_topk(tied, k)
    np.testing.assert_array_equal(got, brute_topk(tied, k))
    assert (np.diff(got) > 0).all()
    if 0 < k < m:
        kept = np.zeros(m, bool)
        kept[got] = True
        thr = tied[kept].min()
        assert tied[~kept].max() <= thr
        eq = np.flatnonzero(tied == thr)
        n_eq_kept = kept[eq].sum()
        np.testing.assert_array_equal(np.flatnonzero(kept[eq]), np.arange(n_eq_kept))  # lowest indices among equals


def test_topk_special_cases():
    np.testing.assert_array_equal(select_topk(np.zeros(10, np.float32), 4), [0, 1, 2, 3])
    z = np.array([0.0, -0.0, 0.0, -0.0, 1.0], dtype=np.float32)       # -0.0 == +0.0
    np.testing.assert_array_equal(select_topk(z, 3), [0, 1, 4])
    assert select_topk(np.arange(5, dtype=np.float32), 0).size == 0
    np.testing.assert_array_equal(select_topk(np.arange(5, dtype=np.float32), 5), np.arange(5))
    np.testing.assert_array_equal(select_topk(np.array([1, 3, 2, 3, 0], np.float32), 2), [1, 3])
    np.testing.assert_array_equal(select_topk(np.array([-1, -3, -2, -3, -5], np.float32), 3), [0, 1, 2])


def test_gather_explicit_loops():
    rng = np.random.default_rng(4)
    L, S, row, v0, m = 3, 40, 6, 4, 25
    src = rng.integers(0, 65535, size=(L, S, row)).astype(np.uint16)
    idx = np.sort(rng.choice(m, size=9, replace=False)).astype(np.int32)
    dst = gather_rows(src, v0, m, idx)
    assert dst.shape == (L, S - m + 9, row)
    for l in range(L):
        rows = [src[l, j] for j in range(v0)] + [src[l, v0 + i] for i in idx] + [src[l, j] for j in range(v0 + m, S)]
        for a, b in zip(dst[l], rows):
            assert a.tobytes() == b.tobytes()
    assert gather_rows(src, v0, m, np.arange(m)).tobytes() == src.tobytes()          # k = m: identity
    assert gather_rows(src, v0, m, np.zeros(0, np.int32)).shape[1] == S - m          # k = 0: text only


def test_variation_reduces_positional_concentration():
    """Direction only (Fig. 2 / Appendix E): raw-mass picks pile onto the late
    positions favoured by the recency ramp; the variation score against a
    reference layer with the same positional bias is less concentrated."""
    cfg = wl.CONFIGS[0]
    q, k, v = wl.attn_layer(cfg, 0)
    qr, kr, vr = wl.attn_layer(cfg, 0, role="ref")
    _, _, mass_cur = verify_attn(q, k, v, cfg.n_ctx)
    _, _, mass_ref = verify_attn(qr, kr, vr, cfg.n_ctx)
    kk = cfg.k_keep
    raw = select_topk(score_fp32(mass_cur, None, 0, cfg.m), kk)
    var = select_topk(score_fp32(mass_cur, mass_ref, 0, cfg.m), kk)
    last_q = 3 * cfg.m // 4
    share_raw = (raw >= last_q).mean()
    share_var = (var >= last_q).mean()
    assert share_raw > 0.5
    assert share_var < share_raw - 0.15
