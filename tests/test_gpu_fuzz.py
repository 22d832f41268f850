"""Seeded random-geometry sweeps of every call (GPU) against the CPU oracle: the attention over ragged
shapes, CTA counts, both cache layouts and mass-layer subsets (every case against the oracle, and against
the mma.sync implementation as an extra); selection, gather and the accept path.  PVLM_FUZZ_CASES scales the number of cases
(default 60 per call; a few hundred take about a minute)."""
import os

import numpy as np
import pytest
import torch

from oracle.attention import verify_attn as oracle_attn
from oracle.pipeline import parallel_decode as oracle_decode
from oracle.uvprune import gather_rows, score_fp32, select_topk
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import assert_o_close, assert_rel_close, bits_of
from test_gpu_accept import check_against_oracle
from test_gpu_decode import first_token_mismatch_is_a_rounding_band_event, gpu_decode, log_rows, make_case
from test_gpu_prune import gpu_select
from test_gpu_rate import run_case as rate_case
from test_gpu_similarity import check as similarity_check

pytestmark = pytest.mark.gpu
CASES = int(os.environ.get("PVLM_FUZZ_CASES", "60"))


ORACLE_ROW_KEYS = 5_000_000      # query rows x keys of one layer the oracle finishes in about a second


def test_attention_random_geometries(pvlm_option):
    rng = np.random.default_rng(11)
    for case in range(CASES):
        D = int(rng.choice([64, 128]))
        Hkv = int(rng.integers(1, 9))
        G = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 12, 16]))
        R = int(rng.integers(1, max(2, 128 // G + 1)))
        n_ctx = int(rng.choice([0, 1, 2, 63, 64, 127, 128, 129, 255, 256, 257, 700, 2500, int(rng.integers(0, 9000))]))
        L = int(rng.integers(1, 6))
        ctas = int(rng.choice([0, 0, 1, 2, 5, 37, 148]))
        head_major = bool(rng.integers(0, 2))
        Hq = G * Hkv
        # every case is checked against the oracle: keep one layer within its budget (still tens of ragged tiles)
        n_ctx = min(n_ctx, max(0, ORACLE_ROW_KEYS // (Hq * R) - R))
        T = n_ctx + R
        g = torch.Generator(device="cuda")
        g.manual_seed(case)
        mk = lambda *sh: torch.randn(sh, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        q, k, v = mk(L, R, Hq, D), mk(L, T, Hkv, D), mk(L, T, Hkv, D)
        if rng.integers(0, 3) == 0:                      # a sink-like first key now and then
            k[:, 0] *= 4
        if head_major:                                   # [layer][kv_head][token][D] storage behind the same view
            k = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            v = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        ml = None
        if L > 1 and rng.integers(0, 2):
            ml = sorted(set(int(x) for x in rng.integers(0, L, size=2)))
        pvlm_option("attn_mma_sync", 0)
        pvlm_option("attn_max_ctas", ctas)
        o1, l1, m1 = binding.verify_attn(q, k, v, n_ctx, want_mass=True, check=True, mass_layers=ml)
        pvlm_option("attn_max_ctas", 0)
        pvlm_option("attn_mma_sync", 1)
        o2, l2, m2 = binding.verify_attn(q, k, v, n_ctx, want_mass=True, mass_layers=ml)
        torch.cuda.synchronize()
        tag = (case, L, Hq, Hkv, D, n_ctx, R, ctas, head_major, ml)
        assert bool(torch.isfinite(o1.float()).all()), tag
        # the oracle: a mass layer if there is a choice, every layer while the whole call stays within the budget
        layers = range(L) if L * Hq * R * T <= ORACLE_ROW_KEYS else [ml[-1] if ml else int(rng.integers(0, L))]
        for l in layers:
            O, Lr, M = oracle_attn(np.ascontiguousarray(bits_of(q[l])), np.ascontiguousarray(bits_of(k[l])),
                                   np.ascontiguousarray(bits_of(v[l])), n_ctx)
            assert_o_close(o1[l], O)
            assert np.abs(l1[l].cpu().numpy() - Lr).max() <= 1e-4, tag
            if ml is None or l in ml:
                row = m1[l] if ml is None else m1[ml.index(l)]
                assert_rel_close(row.cpu().numpy(), M, what="mass")
        # extra: the second implementation over ALL layers
        err = (o1.float() - o2.float()).abs()
        assert bool((err <= 1e-2 + 2e-2 * o2.float().abs()).all()), tag
        assert float((l1 - l2).abs().max()) <= 1e-4, tag
        assert bool(((m1 - m2).abs() <= 1e-4 * m2.abs() + 1e-30).all()), tag


def test_select_random_sizes_and_score_distributions():
    rng = np.random.default_rng(5)
    for case in range(CASES):
        m = int(rng.choice([1, 2, 31, 32, 33, 1000, 4095, 4096, 4097, int(rng.integers(1, 200000))]))
        k = int(rng.choice([0, 1, m, max(0, m - 1), int(rng.integers(0, m + 1))]))
        v0 = int(rng.integers(0, 40))
        T = v0 + m + int(rng.integers(0, 20))
        kind = int(rng.integers(0, 4))
        if kind == 0:
            cur = rng.random(T).astype(np.float32)
        elif kind == 1:
            cur = (np.round(rng.standard_normal(T) * 4) / 4).astype(np.float32)        # heavy ties
        elif kind == 2:
            cur = np.full(T, 0.5, dtype=np.float32)                                    # all equal
        else:
            cur = (rng.standard_normal(T) * 10.0 ** rng.integers(-30, 30)).astype(np.float32)
        ref = rng.random(T).astype(np.float32) if rng.integers(0, 2) else None
        kept, score = gpu_select(cur, ref, v0, m, k)
        s_ref = score_fp32(cur, ref, v0, m)
        tag = (case, m, k, v0, kind, ref is not None)
        assert (score.view(np.uint32) == s_ref.view(np.uint32)).all(), tag
        assert (kept == select_topk(s_ref, k)).all(), tag


def test_gather_random_shapes():
    rng = np.random.default_rng(6)
    for case in range(max(10, CASES // 3)):
        L, Hkv, D = int(rng.integers(1, 5)), int(rng.choice([1, 2, 4, 8])), int(rng.choice([64, 128]))
        S = int(rng.integers(2, 3000))
        v0 = int(rng.integers(0, S))
        m = int(rng.integers(0, S - v0 + 1))
        k = int(rng.integers(0, m + 1))
        kb = rng.integers(0, 65536, size=(L, S, Hkv, D), dtype=np.uint16)
        vb = rng.integers(0, 65536, size=(L, S, Hkv, D), dtype=np.uint16)
        mass = rng.random(S).astype(np.float32)
        to_dev = lambda b: torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).cuda()
        kept, _, dk, dv = binding.uvprune_select_gather(torch.from_numpy(mass).cuda(), None, v0, m, k, to_dev(kb), to_dev(vb))
        torch.cuda.synchronize()
        idx = kept.cpu().numpy()
        tag = (case, L, S, Hkv, D, v0, m, k)
        assert (idx == select_topk(mass[v0:v0 + m], k)).all(), tag
        assert bits_of(dk).tobytes() == gather_rows(kb, v0, m, idx).tobytes(), tag
        assert bits_of(dv).tobytes() == gather_rows(vb, v0, m, idx).tobytes(), tag


def test_accept_random_vocab_window_and_temperature():
    rng = np.random.default_rng(8)
    for case in range(CASES):
        V = int(rng.choice([1, 2, 3, 17, 255, 256, 257, 1000, 4096, 5000, int(rng.integers(1, 40000))]))
        gamma = int(rng.integers(1, 65 if V < 3000 else 17))
        sig = float(rng.choice([0.0, 0.1, 0.5, 2.0]))
        temp = float(rng.choice([1.0, 1.0, 0.7, 1.5]))
        tl = (rng.standard_normal((gamma + 1, V)) * 3).astype(np.float32)
        dl = (tl[:gamma] + sig * rng.standard_normal((gamma, V))).astype(np.float32)
        tok = rng.integers(0, V, size=gamma).astype(np.int32)
        if rng.integers(0, 2):                           # the draft row's most likely token: usually accepted
            tok = dl.argmax(1).astype(np.int32)
        u = rng.random(gamma + 1).astype(np.float32)
        check_against_oracle(tl, dl, tok, u, temp)


def test_step_overlap_mode_random_gather_splits():
    """pvlm_verify_step in overlap mode (rows outside the visual span copied on the second stream, selected rows on
    the main one) against the one-call select + gather: empty spans on either side, k = 0 and k = m included."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(9)
    cs, ea, eb = torch.cuda.Stream(), torch.cuda.Event(), torch.cuda.Event()
    ea.record()
    eb.record()
    torch.cuda.synchronize()
    for case in range(max(10, CASES // 2)):
        L, Hkv, D = int(rng.integers(1, 4)), int(rng.choice([1, 2, 4, 8])), int(rng.choice([64, 128]))
        S = int(rng.integers(2, 2500))
        v0 = int(rng.choice([0, 0, int(rng.integers(0, S))]))
        m = int(rng.choice([S - v0, int(rng.integers(0, S - v0 + 1))]))
        k = int(rng.choice([0, m, int(rng.integers(0, m + 1))]))
        g = torch.Generator(device="cuda")
        g.manual_seed(1000 + case)
        src_k = torch.randn((L, S, Hkv, D), generator=g, device=dev).to(torch.bfloat16)
        src_v = torch.randn((L, S, Hkv, D), generator=g, device=dev).to(torch.bfloat16)
        cur = torch.rand(S, generator=g, device=dev)
        ref = torch.rand(S, generator=g, device=dev)
        kept_e, _, dk_e, dv_e = binding.uvprune_select_gather(cur, ref, v0, m, k, src_k, src_v)
        kept = torch.full((max(k, 1),), -7, dtype=torch.int32, device=dev)
        dk = torch.zeros((L, S - m + k, Hkv, D), dtype=torch.bfloat16, device=dev)
        dv = torch.zeros_like(dk)
        pp = binding.prune_params(cur, ref, v0, m, k, kept, None, src_k, src_v, dk, dv)
        binding.verify_step(None, pp, None, device=dev, overlap=(cs, ea, eb))
        torch.cuda.current_stream().synchronize()
        tag = (case, L, S, Hkv, D, v0, m, k)
        assert torch.equal(kept[:k], kept_e[:k]), tag
        assert torch.equal(dk, dk_e) and torch.equal(dv, dv_e), tag


def test_parallel_decode_random_windows_vocabularies_and_temperatures():
    """Tokens, round count and round log equal the oracle's.  A draw that lands within the rounding band of a step of
    the cumulative weights (about one in 1e4 cases; none among the default 60) may give the neighbouring token, after
    which the two runs differ legitimately: such a case is checked to be exactly that, and at most one in 500 may be."""
    rng = np.random.default_rng(2)
    banded = 0
    for case in range(CASES):
        V = int(rng.choice([2, 3, 17, 50, 257, 1000, 4099, int(rng.integers(2, 20000))]))
        K, gamma = int(rng.integers(1, 60)), int(rng.integers(1, 17))
        sigma = float(rng.choice([0.0, 0.2, 0.6, 1.5]))
        temp = float(rng.choice([1.0, 1.0, 0.8]))
        tl, dl, ud, ua, ur = make_case(V, K, gamma, sigma, 100 + case)
        ref = oracle_decode(tl, dl, gamma, K, ud, ua, ur, temp)
        for serial in (False, True):
            out = gpu_decode(tl, dl, gamma, K, ud, ua, ur, serial=serial, temperature=temp)
            tag = (case, V, K, gamma, sigma, temp, serial)
            got = out["tokens"].numpy()
            if len(got) == len(ref["tokens"]) and (got == ref["tokens"]).all():
                assert out["rounds"] == ref["rounds"], tag
                assert out["log"].tolist() == log_rows(ref["log"]), tag
            else:
                assert first_token_mismatch_is_a_rounding_band_event(got, ref["tokens"], tl, dl, ud, ua, ur, temp), tag
                banded += 1
    assert banded <= max(1, 2 * CASES // 500), banded


def test_acceptance_rate_random_sizes_and_strides():
    rng = np.random.default_rng(3)
    for case in range(CASES):
        N = int(rng.choice([0, 1, 2, 33, 100, int(rng.integers(1, 600))]))
        V = int(rng.choice([1, 2, 17, 255, 256, 1000, 4099, int(rng.integers(1, 30000))]))
        rate_case(N, V, float(rng.choice([0.0, 0.3, 1.0])), 500 + case, float(rng.choice([1.0, 0.7, 1.3])),
                  int(rng.choice([0, 0, 1, 2, 4])))


def test_similarity_random_shapes():
    rng = np.random.default_rng(4)
    for case in range(CASES):
        m = int(rng.choice([1, 7, 8, 9, 100, int(rng.integers(1, 3000))]))
        n = int(rng.choice([0, 1, 7, 8, 9, 17, int(rng.integers(1, 600))]))
        d = int(rng.choice([8, 16, 256, 264, 1000, 2560, 2568, 3584, 5120, 8192]))
        v0 = int(rng.integers(0, 5))
        h = rng.standard_normal((v0 + m + n + 2, d)).astype(np.float32)
        h[v0 + m:] += 0.3                                # text rows share a direction
        if m > 2 and rng.integers(0, 4) == 0:
            h[v0 + 1] = 0                                # a zero visual row
        hb = wl.f32_to_bf16_bits(h)
        one, _ = similarity_check(hb, v0, m, v0 + m, n)
        if case % 3 == 0:                                # the same layer inside a two- or three-layer call: bitwise the same result
            L = 2 + case % 2
            stack = torch.zeros((L, h.shape[0] + int(rng.integers(0, 4)), d), dtype=torch.bfloat16, device="cuda")
            for l in range(L):
                other = wl.f32_to_bf16_bits(rng.standard_normal(h.shape).astype(np.float32))
                stack[l, :h.shape[0]] = torch.from_numpy((hb if l == L - 1 else other).view(np.int16)).view(torch.bfloat16).cuda()
            sims = binding.uvprune_similarity(stack, v0, m, v0 + m, n)
            torch.cuda.synchronize()
            assert torch.equal(sims[L - 1], one), (case, m, n, d, v0, L)
