"""Parity of pvlm_uvprune_select_gather against the CPU oracle: bit-exact
indices and bytes."""
import numpy as np
import pytest
import torch

from oracle.attention import verify_attn as oracle_attn
from oracle.uvprune import gather_rows, score_fp32, select_topk
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import bf16_cuda, bits_of

pytestmark = pytest.mark.gpu


def gpu_select(cur, ref, v0, m, k, want_score=True):
    c = torch.from_numpy(cur).cuda()
    r = torch.from_numpy(ref).cuda() if ref is not None else None
    kept, score, _, _ = binding.uvprune_select_gather(c, r, v0, m, k, want_score=want_score)
    torch.cuda.synchronize()
    return kept.cpu().numpy(), (score.cpu().numpy() if score is not None else None)


@pytest.mark.parametrize("m,k,v0", [(1, 1, 0), (1, 0, 0), (17, 5, 3), (1024, 256, 0), (1025, 1025, 2),
                                    (5000, 617, 7), (30720, 3072, 0), (131072, 6553, 0), (70000, 69999, 1)])
def test_select_matches_oracle(m, k, v0):
    rng = np.random.default_rng(m + 7 * k)
    T = v0 + m + 9
    cur = rng.random(T).astype(np.float32)
    ref = rng.random(T).astype(np.float32)
    kept, score = gpu_select(cur, ref, v0, m, k)
    s_ref = score_fp32(cur, ref, v0, m)
    np.testing.assert_array_equal(score.view(np.uint32), s_ref.view(np.uint32))     # one fp32 subtraction: bit-exact
    np.testing.assert_array_equal(kept, select_topk(s_ref, k))
    kept2, _ = gpu_select(cur, None, v0, m, k, want_score=False)                     # raw-mass criterion
    np.testing.assert_array_equal(kept2, select_topk(cur[v0:v0 + m], k))


def test_ties_zeros_negatives_nan_free():
    rng = np.random.default_rng(5)
    m = 40000
    q = (np.round(rng.standard_normal(m) * 8) / 8).astype(np.float32)      # heavy ties, both signs
    q[rng.integers(0, m, 500)] = 0.0
    q[rng.integers(0, m, 500)] = -0.0
    for k in (1, 100, 12345, m // 2, m - 1):
        kept, _ = gpu_select(q, None, 0, m, k, want_score=False)
        np.testing.assert_array_equal(kept, select_topk(q, k))
    same = np.full(5000, 0.25, dtype=np.float32)
    kept, _ = gpu_select(same, None, 0, 5000, 777, want_score=False)
    np.testing.assert_array_equal(kept, np.arange(777))
    # extremes: +-inf and denormals order correctly
    x = np.array([np.inf, -np.inf, 1e-45, -1e-45, 0.0, 3.4e38, -3.4e38, 1.0], dtype=np.float32)
    for k in range(9):
        kept, _ = gpu_select(x, None, 0, 8, k, want_score=False)
        np.testing.assert_array_equal(kept, select_topk(x, k))


@pytest.mark.parametrize("L,S,Hkv,D,v0,m,k", [(1, 300, 2, 64, 0, 250, 31), (3, 1029, 4, 128, 5, 896, 224),
                                              (2, 200, 8, 128, 0, 150, 0), (2, 200, 8, 128, 10, 150, 150)])
def test_gather_bytes(L, S, Hkv, D, v0, m, k):
    rng = np.random.default_rng(S + k)
    src_k = rng.integers(0, 65536, size=(L, S, Hkv, D)).astype(np.uint16)
    src_v = rng.integers(0, 65536, size=(L, S, Hkv, D)).astype(np.uint16)
    cur = rng.random(v0 + m).astype(np.float32)
    kept, _, dk, dv = binding.uvprune_select_gather(torch.from_numpy(cur).cuda(), None, v0, m, k,
                                                    bf16_cuda(src_k), bf16_cuda(src_v))
    torch.cuda.synchronize()
    idx = select_topk(cur[v0:v0 + m], k)
    np.testing.assert_array_equal(kept.cpu().numpy(), idx)
    assert dk.shape == (L, S - m + k, Hkv, D)
    assert bits_of(dk).tobytes() == gather_rows(src_k, v0, m, idx).tobytes()
    assert bits_of(dv).tobytes() == gather_rows(src_v, v0, m, idx).tobytes()


def test_gather_layer_strides_and_single_layer_form():
    rng = np.random.default_rng(11)
    L, S, Hkv, D, m, k = 2, 120, 2, 64, 100, 17
    big_k = torch.from_numpy(rng.integers(0, 30000, size=(L, S + 8, Hkv, D)).astype(np.int16)).view(torch.bfloat16).cuda()
    big_v = torch.from_numpy(rng.integers(0, 30000, size=(L, S + 8, Hkv, D)).astype(np.int16)).view(torch.bfloat16).cuda()
    cur = torch.from_numpy(rng.random(m).astype(np.float32)).cuda()
    kept, _, dk, dv = binding.uvprune_select_gather(cur, None, 0, m, k, big_k[:, :S], big_v[:, :S])
    torch.cuda.synchronize()
    idx = kept.cpu().numpy()
    assert bits_of(dk).tobytes() == gather_rows(bits_of(big_k[:, :S].contiguous()), 0, m, idx).tobytes()
    assert bits_of(dv).tobytes() == gather_rows(bits_of(big_v[:, :S].contiguous()), 0, m, idx).tobytes()
    kept1, _, dk1, _ = binding.uvprune_select_gather(cur, None, 0, m, k, big_k[0, :S], big_v[0, :S])
    torch.cuda.synchronize()
    assert torch.equal(dk1, dk[0])


def test_select_from_oracle_masses_config0():
    """Kept indices from the ORACLE's masses (as fp32) are bit-exact."""
    cfg = wl.CONFIGS[0]
    _, _, m_cur = oracle_attn(*wl.attn_layer(cfg, 0), cfg.n_ctx)
    _, _, m_ref = oracle_attn(*wl.attn_layer(cfg, 0, role="ref"), cfg.n_ctx)
    cur, ref = m_cur.astype(np.float32), m_ref.astype(np.float32)
    kept, _ = gpu_select(cur, ref, 0, cfg.m, cfg.k_keep)
    np.testing.assert_array_equal(kept, select_topk(score_fp32(cur, ref, 0, cfg.m), cfg.k_keep))


def test_single_cta_kernels_still_match(pvlm_option):
    """The select_one_cta switch keeps the selection on the single-CTA kernels (register-resident up to
    32,768 scores, global-memory keys above): the second implementation of the same selection."""
    pvlm_option("select_one_cta", 1)
    rng = np.random.default_rng(77)
    for m, k in [(30720, 3072), (131072, 6553), (5000, 4999)]:
        cur = (np.round(rng.random(m) * 4096) / 4096).astype(np.float32)       # ties included
        ref = rng.random(m).astype(np.float32)
        kept, _ = gpu_select(cur, ref, 0, m, k, want_score=False)
        np.testing.assert_array_equal(kept, select_topk(score_fp32(cur, ref, 0, m), k))
        kept, _ = gpu_select(cur, None, 0, m, k, want_score=False)
        np.testing.assert_array_equal(kept, select_topk(cur, k))


def test_cluster_select_boundaries():
    """Sizes around the per-CTA and per-variant boundaries of the 8-CTA cluster kernel, heavy ties."""
    rng = np.random.default_rng(78)
    for m in (4095, 4096, 4097, 32768, 32769, 131071, 131073, 262144):
        cur = (np.round(rng.random(m) * 64) / 64).astype(np.float32)
        for k in (1, m // 3, m - 1):
            kept, _ = gpu_select(cur, None, 0, m, k, want_score=False)
            np.testing.assert_array_equal(kept, select_topk(cur, k))
