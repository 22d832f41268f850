"""Pins for the attention oracle: brute force, closed forms, a library routine,
and invariants.  None of these re-use the oracle's own formula path."""
import math

import numpy as np
import pytest
import torch

from oracle.attention import bf16_bits_to_f64, verify_attn
from paper_2603_19610_b200 import workloads as wl


def brute_force(q, k, v, n_ctx, scale):
    """Pure-Python scalar loops (math.exp), no numpy reductions."""
    R, Hq, D = q.shape
    T, Hkv, _ = k.shape
    G = Hq // Hkv
    O = [[[0.0] * D for _ in range(Hq)] for _ in range(R)]
    lse = [[0.0] * R for _ in range(Hq)]
    mass = [0.0] * T
    for h in range(Hq):
        g = h // G
        for r in range(R):
            s = []
            for j in range(n_ctx + r + 1):
                acc = 0.0
                for d in range(D):
                    acc += float(q[r, h, d]) * float(k[j, g, d])
                s.append(acc * scale)
            mx = max(s)
            e = [math.exp(x - mx) for x in s]
            z = sum(e)
            lse[h][r] = mx + math.log(z)
            for j, ej in enumerate(e):
                pj = ej / z
                mass[j] += pj
                for d in range(D):
                    O[r][h][d] += pj * float(v[j, g, d])
    return np.array(O), np.array(lse), np.array(mass)


@pytest.mark.parametrize("Hq,Hkv,D,n_ctx,R", [(4, 2, 8, 5, 3), (3, 1, 4, 0, 4), (2, 2, 16, 9, 1)])
def test_brute_force_tiny(Hq, Hkv, D, n_ctx, R):
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, n_ctx + R, sink=True, seed=11 + n_ctx)
    O, lse, mass = verify_attn(qb, kb, vb, n_ctx)
    Ob, lb, mb = brute_force(bf16_bits_to_f64(qb), bf16_bits_to_f64(kb), bf16_bits_to_f64(vb),
                             n_ctx, 1.0 / math.sqrt(D))
    np.testing.assert_allclose(O, Ob, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, lb, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(mass, mb, rtol=1e-12, atol=1e-13)


def test_bf16_widening_exact():
    vals = np.array([0.0, 1.0, -2.5, 3.140625, 2.0 ** -100, -65280.0], dtype=np.float32)
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)     # these are exactly representable
    np.testing.assert_array_equal(bf16_bits_to_f64(bits), vals.astype(np.float64))
    # generator rounding is round-to-nearest-even: 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    got = bf16_bits_to_f64(wl.f32_to_bf16_bits(x))
    np.testing.assert_array_equal(got, [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7])


def test_total_mass_and_positivity_config0():
    cfg = wl.CONFIGS[0]
    q, k, v = wl.attn_layer(cfg, 0)
    O, lse, mass = verify_attn(q, k, v, cfg.n_ctx)
    assert mass.min() >= 0.0
    assert abs(mass.sum() - cfg.Hq * cfg.R) < 1e-9          # every softmax row sums to 1
    # window key N+r' is visible to rows r >= r' only: its mass is at most Hq * (R - r')
    for rp in range(cfg.R):
        assert mass[cfg.n_ctx + rp] <= cfg.Hq * (cfg.R - rp) + 1e-12
    # O is a convex combination of V rows
    vf = bf16_bits_to_f64(v)
    assert (O.max(axis=(0, 1)) <= vf.max(axis=(0, 1)) + 1e-12).all()
    assert (O.min(axis=(0, 1)) >= vf.min(axis=(0, 1)) - 1e-12).all()


def test_closed_form_identical_keys():
    """All keys equal => P uniform over the visible keys."""
    Hq, Hkv, D, n_ctx, R = 6, 2, 16, 37, 4
    T = n_ctx + R
    qb, _, vb = wl.make_qkv(Hq, Hkv, D, R, T, sink=False, seed=5, bias=False)
    krow = wl.f32_to_bf16_bits(np.linspace(-1, 1, Hkv * D, dtype=np.float32).reshape(1, Hkv, D))
    kb = np.repeat(krow, T, axis=0)
    O, lse, mass = verify_attn(qb, kb, vb, n_ctx)
    expect = np.array([Hq * sum(1.0 / (n_ctx + r + 1) for r in range(R) if j <= n_ctx + r) for j in range(T)])
    np.testing.assert_allclose(mass, expect, rtol=1e-12)
    vf = bf16_bits_to_f64(vb)
    G = Hq // Hkv
    for r in range(R):
        for h in range(Hq):
            np.testing.assert_allclose(O[r, h], vf[:n_ctx + r + 1, h // G].mean(axis=0), rtol=1e-11, atol=1e-13)
    # lse = s + log(#visible): s is the common score
    qf, kf = bf16_bits_to_f64(qb), bf16_bits_to_f64(kb)
    for h in range(Hq):
        for r in range(R):
            s = (qf[r, h] * kf[0, h // G]).sum() / math.sqrt(D)
            assert abs(lse[h, r] - (s + math.log(n_ctx + r + 1))) < 1e-11


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (5, 5), (7, 1)])
def test_against_torch_sdpa_gqa(Hq, Hkv):
    """Independent library routine: torch SDPA in fp64 with an explicit mask and
    KV heads expanded by repeat_interleave (contiguous query-head groups)."""
    D, n_ctx, R = 32, 50, 6
    T = n_ctx + R
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, T, sink=True, seed=77)
    O, lse, mass = verify_attn(qb, kb, vb, n_ctx)
    G = Hq // Hkv
    tq = torch.from_numpy(bf16_bits_to_f64(qb)).permute(1, 0, 2)[None]              # [1,Hq,R,D]
    tk = torch.from_numpy(bf16_bits_to_f64(kb)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    tv = torch.from_numpy(bf16_bits_to_f64(vb)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    mask = (torch.arange(T)[None, :] <= (n_ctx + torch.arange(R))[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)[0]
    np.testing.assert_allclose(O, ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    # lse and mass against torch's own softmax / logsumexp
    s = (tq[0] @ tk[0].transpose(1, 2)) / math.sqrt(D)
    s = s.masked_fill(~mask[None], float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), rtol=1e-12)
    np.testing.assert_allclose(mass, torch.softmax(s, dim=-1).sum(dim=(0, 1)).numpy(), rtol=1e-10, atol=1e-13)


def test_shift_invariance_and_permutation():
    Hq, Hkv, D, n_ctx, R = 4, 2, 16, 40, 3
    T = n_ctx + R
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, T, sink=False, seed=3)
    O, lse, mass = verify_attn(qb, kb, vb, n_ctx)
    # adding a constant to every key's bias channel shifts all scores of a row equally
    kf = bf16_bits_to_f64(kb).astype(np.float32)
    kf[:, :, D - 1] = np.round(kf[:, :, D - 1] * 4) / 4          # keep exact in bf16
    kb0 = wl.f32_to_bf16_bits(kf)
    kf[:, :, D - 1] += 0.5
    kb1 = wl.f32_to_bf16_bits(kf)
    O0, l0, m0 = verify_attn(qb, kb0, vb, n_ctx)
    O1, l1, m1 = verify_attn(qb, kb1, vb, n_ctx)
    np.testing.assert_allclose(O0, O1, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(m0, m1, rtol=1e-10, atol=1e-13)
    assert np.abs(l1 - l0).min() > 0                              # lse does move
    # permuting context keys permutes mass, leaves O unchanged
    perm = np.random.default_rng(0).permutation(n_ctx)
    full = np.concatenate([perm, np.arange(n_ctx, T)])
    O2, l2, m2 = verify_attn(qb, kb[full], vb[full], n_ctx)
    np.testing.assert_allclose(O2, O, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(m2, mass[full], rtol=1e-10, atol=1e-13)


def test_window_causality():
    """Changing window row r' (its K and V) must not move O of rows r < r'."""
    Hq, Hkv, D, n_ctx, R = 4, 2, 16, 20, 5
    T = n_ctx + R
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, T, sink=False, seed=9)
    O, _, mass = verify_attn(qb, kb, vb, n_ctx)
    rp = 3
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[n_ctx + rp] = wl.f32_to_bf16_bits(np.full((Hkv, D), 2.0, dtype=np.float32))
    vb2[n_ctx + rp] = wl.f32_to_bf16_bits(np.full((Hkv, D), -7.0, dtype=np.float32))
    O2, _, mass2 = verify_attn(qb, kb2, vb2, n_ctx)
    np.testing.assert_array_equal(O2[:rp], O[:rp])
    assert np.abs(O2[rp:] - O[rp:]).max() > 1e-3
    # a key with an overwhelming score (through the bias channel, where every query
    # carries sqrt(D)) collects ~all the mass of exactly the rows that can see it
    kf = bf16_bits_to_f64(kb).astype(np.float32)
    kf[n_ctx + rp, :, D - 1] = 200.0
    _, _, mass3 = verify_attn(qb, wl.f32_to_bf16_bits(kf), vb, n_ctx)
    assert abs(mass3[n_ctx + rp] - Hq * (R - rp)) < 1e-9


def test_config0_bias_shows_in_mass():
    """The synthetic recency ramp must make late visual tokens heavier on
    average (the positional bias the variation score is meant to cancel)."""
    cfg = wl.CONFIGS[0]
    q, k, v = wl.attn_layer(cfg, 0)
    _, _, mass = verify_attn(q, k, v, cfg.n_ctx)
    vis = mass[:cfg.m]
    assert vis[-cfg.m // 4:].mean() > 2.0 * vis[:cfg.m // 4].mean()
