"""Parity of pvlm_uvprune_similarity (the paper's hidden-state criterion, Eq. 1 summed over the text
tokens) against the oracle, and the whole paper-faithful UV-Prune: similarity variation between two
layers (Eq. 2) -> Top-K (Eq. 3) -> gather."""
import numpy as np
import pytest
import torch

from oracle.attention import bf16_bits_to_f64
from oracle.uvprune import gather_rows, score_fp32, select_topk, similarity_sum
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import bf16_cuda, bits_of

pytestmark = pytest.mark.gpu


def text_direction_norm(hb, text_start, n):
    """|u| with u = sum_j X_j/|X_j|: the scale of the fp32 rounding error of one dot product."""
    x = bf16_bits_to_f64(hb)[text_start:text_start + n]
    nx = np.sqrt((x * x).sum(axis=1))
    u = (x / np.where(nx > 0, nx, 1.0)[:, None]).sum(axis=0)
    return float(np.sqrt((u * u).sum()))


def check(hb, vis_start, m, text_start, n):
    sim = binding.uvprune_similarity(bf16_cuda(hb), vis_start, m, text_start, n)
    torch.cuda.synchronize()
    ref = similarity_sum(hb, vis_start, m, text_start, n)
    # fp32 accumulation of d bf16 products against fp64: |err| <= ~sqrt(d) 2^-24 |u| (+ 1e-4 relative)
    d = hb.shape[1]
    tol = 1e-4 * np.abs(ref) + 8.0 * np.sqrt(d) * 2.0 ** -24 * max(text_direction_norm(hb, text_start, n), 1.0)
    err = np.abs(sim.cpu().numpy().astype(np.float64) - ref)
    assert (err <= tol).all(), (err.max(), tol.min())
    return sim, ref


@pytest.mark.parametrize("m,n,d,v0", [(1, 1, 8, 0), (7, 5, 16, 0), (100, 33, 256, 3), (1000, 257, 3584, 0),
                                      (513, 17, 5120, 0), (64, 2048, 8192, 0), (300, 40, 16384, 5)])
def test_similarity_shapes(m, n, d, v0):
    rng = np.random.default_rng(m + n + d)
    h = rng.standard_normal((v0 + m + n + 2, d)).astype(np.float32)
    h[v0 + m:] += 0.3                                            # text rows share a direction
    check(wl.f32_to_bf16_bits(h), v0, m, v0 + m, n)


def test_zero_rows_and_strided_rows():
    rng = np.random.default_rng(5)
    m, n, d = 40, 9, 64
    h = rng.standard_normal((m + n, d)).astype(np.float32)
    h[3] = 0.0                                                   # zero visual row: similarity 0
    h[m + 2] = 0.0                                               # zero text row: contributes nothing
    hb = wl.f32_to_bf16_bits(h)
    sim, ref = check(hb, 0, m, m, n)
    assert float(sim[3]) == 0.0 and ref[3] == 0.0
    wide = torch.zeros((m + n, d + 24), dtype=torch.bfloat16, device="cuda")      # padded row stride
    wide[:, :d] = bf16_cuda(hb)
    sim2 = binding.uvprune_similarity(wide[:, :d], 0, m, m, n)
    torch.cuda.synchronize()
    assert torch.equal(sim2, sim)
    with pytest.raises(binding.PvlmError) as e:
        binding.uvprune_similarity(bf16_cuda(hb)[:, :12], 0, m, m, n)              # d % 8 != 0
    assert e.value.status in (1, 2)


def test_several_layers_in_one_call_equal_single_calls():
    """Two and three layers through one call (one launch of each kernel for all of them): every layer's result is
    bitwise what a call on that layer alone gives, and matches the oracle; a padded layer stride is honoured."""
    rng = np.random.default_rng(41)
    for L, m, n, d in [(2, 700, 90, 1024), (3, 33, 5, 64), (2, 1, 1, 8)]:
        hb = [wl.f32_to_bf16_bits(rng.standard_normal((m + n + 3, d)).astype(np.float32) + (0.2 if l else 0.0)) for l in range(L)]
        stack = torch.zeros((L, m + n + 7, d), dtype=torch.bfloat16, device="cuda")         # rows beyond the last are padding
        for l in range(L):
            stack[l, :m + n + 3] = bf16_cuda(hb[l])
        sims = binding.uvprune_similarity(stack, 0, m, m, n)
        torch.cuda.synchronize()
        assert sims.shape == (L, m)
        for l in range(L):
            one, ref = check(hb[l], 0, m, m, n)
            assert torch.equal(sims[l], one)


def test_several_layers_with_offsets_and_strided_views():
    """Layers that are views of a larger buffer (padded row stride, layer stride larger than a layer, rows before the
    visual span and between the spans), results into a strided output: each layer against the oracle."""
    rng = np.random.default_rng(43)
    L, v0, m, gap, n, d = 2, 5, 300, 4, 37, 192
    rows = v0 + m + gap + n + 2
    big = torch.zeros((L, rows + 9, d + 16), dtype=torch.bfloat16, device="cuda")
    hb = [wl.f32_to_bf16_bits(rng.standard_normal((rows, d)).astype(np.float32)) for _ in range(L)]
    for l in range(L):
        big[l, :rows, :d] = bf16_cuda(hb[l])
    out = torch.full((L, m + 11), -7.0, dtype=torch.float32, device="cuda")
    sims = binding.uvprune_similarity(big[:, :rows, :d], v0, m, v0 + m + gap, n, out=out[:, :m])
    torch.cuda.synchronize()
    assert (out[:, m:] == -7.0).all()                                     # nothing written past a layer's m results
    for l in range(L):
        one, ref = check(hb[l], v0, m, v0 + m + gap, n)
        assert torch.equal(sims[l], one)


@pytest.mark.parametrize("cid", [0, 1])
def test_paper_uvprune_end_to_end(cid):
    """Eq. 1 -> Eq. 2 (layers 0 and 20) -> Eq. 3 -> gather, GPU against oracle."""
    cfg = wl.CONFIGS[cid]
    h0, hL = wl.hidden_layer(cfg, 0), wl.hidden_layer(cfg, 20)
    m, n = cfg.m, cfg.n_text
    s0, sL = binding.uvprune_similarity(torch.stack([bf16_cuda(h0), bf16_cuda(hL)]), 0, m, m, n)     # both end layers, one call
    _, k, v = wl.attn_layer(cfg, 0)
    kept, score, dk, dv = binding.uvprune_select_gather(sL, s0, 0, m, cfg.k_keep, bf16_cuda(k), bf16_cuda(v), want_score=True)
    torch.cuda.synchronize()
    # bit-exact from the GPU's own fp32 signals
    g0, gL = s0.cpu().numpy(), sL.cpu().numpy()
    np.testing.assert_array_equal(kept.cpu().numpy(), select_topk(score_fp32(gL, g0, 0, m), cfg.k_keep))
    assert bits_of(dk).tobytes() == gather_rows(k[None], 0, m, kept.cpu().numpy())[0].tobytes()
    # end to end against the oracle's signals: differences only next to the k-th score
    r0, rL = similarity_sum(h0, 0, m, m, n), similarity_sum(hL, 0, m, m, n)
    s_or = (rL - r0).astype(np.float32)
    idx_or = select_topk(s_or, cfg.k_keep)
    tau = np.sort(s_or)[::-1][cfg.k_keep - 1]
    band = 1e-4 * max(abs(float(tau)), 1e-30) + 64.0 * np.sqrt(cfg.d_model) * 2.0 ** -24 * text_direction_norm(hL, m, n)
    for i in np.setxor1d(kept.cpu().numpy(), idx_or):
        assert abs(float(s_or[i]) - float(tau)) <= band, (i, s_or[i], tau, band)
