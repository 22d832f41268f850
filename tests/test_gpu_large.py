"""Maximum-size cases of the calls other than the attention (GPU): sizes at which element counts and byte offsets
leave 32 bits, and the capacity limits the header states.  Where the oracle would take minutes on the whole input it
checks the rows behind the large offsets; byte-exact work is checked in full against torch indexing."""
import numpy as np
import pytest
import torch

from oracle.accept import tokenwise_acceptance
from oracle.uvprune import score_fp32, select_topk, similarity_sum
from paper_2603_19610_b200 import binding
from test_gpu_accept import check_against_oracle

pytestmark = pytest.mark.gpu


def test_gather_with_a_layer_stride_beyond_2_32_bytes():
    dev = torch.device("cuda")
    L, S, rowb = 2, 2_200_000, 2048
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    mk = lambda: torch.randint(-32768, 32767, (L, S, 1, rowb // 2), generator=g, dtype=torch.int16, device=dev).view(torch.bfloat16)
    src_k, src_v = mk(), mk()
    assert src_k.stride(0) * 2 > 2 ** 32
    v0, m, k = 1000, 2_000_000, 150_000
    mass = torch.rand(S, generator=g, device=dev)
    kept, _, dk, dv = binding.uvprune_select_gather(mass, None, v0, m, k, src_k, src_v)
    torch.cuda.synchronize()
    idx = select_topk(mass[v0:v0 + m].cpu().numpy(), k)
    np.testing.assert_array_equal(kept.cpu().numpy(), idx)
    rows = torch.cat([torch.arange(0, v0, device=dev), v0 + torch.from_numpy(idx.astype(np.int64)).to(dev),
                      torch.arange(v0 + m, S, device=dev)])
    assert torch.equal(dk.view(torch.int16), src_k.view(torch.int16).index_select(1, rows))
    assert torch.equal(dv.view(torch.int16), src_v.view(torch.int16).index_select(1, rows))


def test_select_at_its_capacity_of_2_24_tokens():
    dev = torch.device("cuda")
    m, k = 1 << 24, 1_000_003
    g = torch.Generator(device=dev)
    g.manual_seed(2)
    cur = torch.rand(m + 5, generator=g, device=dev)
    ref = torch.rand(m + 5, generator=g, device=dev)
    kept, score, _, _ = binding.uvprune_select_gather(cur, ref, 3, m, k, want_score=True)
    torch.cuda.synchronize()
    s_ref = score_fp32(cur.cpu().numpy(), ref.cpu().numpy(), 3, m)
    np.testing.assert_array_equal(score.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    np.testing.assert_array_equal(kept.cpu().numpy(), select_topk(s_ref, k))
    with pytest.raises(binding.PvlmError):                    # one more token than the capacity
        binding.uvprune_select_gather(torch.zeros(m + 1, device=dev), None, 0, m + 1, 1)


def test_acceptance_rate_over_more_than_2_31_logits():
    dev = torch.device("cuda")
    N, V = 15000, 152064
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    tl = torch.randn((N, V), generator=g, device=dev).mul_(1.5)
    dl = tl + 0.5 * torch.randn((N, V), generator=g, device=dev)
    tok = torch.randint(0, V, (N,), generator=g, device=dev, dtype=torch.int32)
    u = torch.rand(N, generator=g, device=dev)
    assert N * V > 2 ** 31
    out = binding.acceptance_rate(tl, dl, tok, u)
    torch.cuda.synchronize()
    sl = slice(N - 40, N)                                      # the rows behind the large offsets
    ref = tokenwise_acceptance(tl[sl].cpu().numpy(), dl[sl].cpu().numpy(), tok[sl].cpu().numpy(), u[sl].cpu().numpy())
    assert np.allclose(out["p_tok"][sl].cpu().numpy(), ref["p_tok"], rtol=1e-4, atol=1e-30)
    assert np.allclose(out["q_tok"][sl].cpu().numpy(), ref["q_tok"], rtol=1e-4, atol=1e-30)
    assert (out["accepted"][sl].cpu().numpy().astype(bool) == ref["accepted"]).all()
    assert int(out["n_accepted"].item()) == int(out["accepted"].sum().item())


def test_similarity_over_more_than_2_31_elements():
    dev = torch.device("cuda")
    m, n, d = 270_000, 64, 8192
    g = torch.Generator(device=dev)
    g.manual_seed(4)
    h = torch.randn((m + n, d), generator=g, device=dev).to(torch.bfloat16)
    assert (m + n) * d > 2 ** 31
    sim = binding.uvprune_similarity(h, 0, m, m, n)
    torch.cuda.synchronize()
    hb = torch.cat([h[m - 50:m], h[m:]]).cpu().view(torch.int16).numpy().view(np.uint16)   # last visual rows + the text rows
    ref = similarity_sum(hb, 0, 50, 50, n)
    assert np.abs(sim[m - 50:].cpu().numpy() - ref).max() <= 1e-3


def test_accept_with_a_four_million_entry_vocabulary():
    V, gamma = 4_000_003, 3
    rng = np.random.default_rng(1)
    tl = (rng.standard_normal((gamma + 1, V)) * 3).astype(np.float32)
    dl = (tl[:gamma] + 0.5 * rng.standard_normal((gamma, V))).astype(np.float32)
    check_against_oracle(tl, dl, dl.argmax(1).astype(np.int32), rng.random(gamma + 1).astype(np.float32))
