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


def _hidden(m, n, d, seed):
    rng = np.random.default_rng(seed)
    return wl.f32_to_bf16_bits(rng.standard_normal((m + n, d)).astype(np.float32))


def test_cosine_brute_force_and_bounds():
    """Eq. 1 against scalar loops; |S_ij| <= 1; scaling a row leaves its cosines unchanged."""
    import math
    from oracle.attention import bf16_bits_to_f64
    from oracle.uvprune import cosine_similarity, similarity_sum
    m, n, d = 7, 5, 16
    hb = _hidden(m, n, d, 1)
    S = cosine_similarity(hb, 0, m, m, n)
    h = bf16_bits_to_f64(hb)
    for i in range(m):
        for j in range(n):
            dot = sum(float(h[i, c]) * float(h[m + j, c]) for c in range(d))
            ni = math.sqrt(sum(float(h[i, c]) ** 2 for c in range(d)))
            nj = math.sqrt(sum(float(h[m + j, c]) ** 2 for c in range(d)))
            assert abs(S[i, j] - dot / (ni * nj)) < 1e-12
    assert np.abs(S).max() <= 1 + 1e-12
    h2 = bf16_bits_to_f64(hb).astype(np.float32)
    h2[2] *= 4.0                                             # exact in bf16
    h2[m + 1] *= 0.5
    S2 = cosine_similarity(wl.f32_to_bf16_bits(h2), 0, m, m, n)
    np.testing.assert_allclose(S2, S, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(similarity_sum(hb, 0, m, m, n), S.sum(axis=1), rtol=1e-13)
    # identical rows => cosine 1; opposite => -1; zero row => 0
    h3 = h2.copy()
    h3[0] = h3[m]
    h3[1] = -h3[m]
    h3[3] = 0.0
    S3 = cosine_similarity(wl.f32_to_bf16_bits(h3), 0, m, m, n)
    assert abs(S3[0, 0] - 1) < 1e-12 and abs(S3[1, 0] + 1) < 1e-12 and (S3[3] == 0).all()
    # library routine: sklearn / scipy cosine distance
    from scipy.spatial.distance import cdist
    np.testing.assert_allclose(S, 1.0 - cdist(h[:m], h[m:], metric="cosine"), atol=1e-12)


def test_similarity_variation_telescopes_to_end_layers():
    """Eq. 2's double sum equals (sum_j S^L_ij) - (sum_j S^0_ij)."""
    from oracle.uvprune import similarity_sum, similarity_variation
    m, n, d, L = 30, 9, 32, 6
    layers = [_hidden(m, n, d, 10 + l) for l in range(L + 1)]
    full = similarity_variation(layers, 0, m, m, n)
    ends = similarity_sum(layers[-1], 0, m, m, n) - similarity_sum(layers[0], 0, m, m, n)
    np.testing.assert_allclose(full, ends, rtol=0, atol=1e-11)


def test_similarity_variation_cancels_positional_component():
    """Direction only: on the synthetic representations, raw similarity picks pile onto the text-side
    end of the video; the variation between the first and the 20th layer does not."""
    from oracle.uvprune import similarity_sum
    cfg = wl.CONFIGS[0]
    h0 = wl.hidden_layer(cfg, 0)
    hL = wl.hidden_layer(cfg, 20)
    s0 = similarity_sum(h0, 0, cfg.m, cfg.m, cfg.n_text)
    sL = similarity_sum(hL, 0, cfg.m, cfg.m, cfg.n_text)
    k = cfg.k_keep
    raw = select_topk(sL.astype(np.float32), k)
    var = select_topk((sL - s0).astype(np.float32), k)
    last_q = 3 * cfg.m // 4
    assert (raw >= last_q).mean() > 0.6
    assert (var >= last_q).mean() < 0.45
    # and the variation finds the tokens whose alignment grew with depth
    sem = wl.rng_for(cfg.cid, wl.S_HIDDEN, 0).choice(cfg.m, size=max(1, cfg.m // 10), replace=False)
    assert np.isin(sem, var).mean() > 0.7
