"""Parity of pvlm_spec_accept against the CPU oracle, plus the distributional
test on the GPU path itself."""
import numpy as np
import pytest
import torch
from scipy.stats import chi2

from oracle.accept import softmax64, spec_accept as oracle_accept, spec_accept_trials
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import assert_rel_close

pytestmark = pytest.mark.gpu


def gpu_accept(tl, dl, tok, u, temperature=1.0, want_probs=False):
    out = binding.spec_accept(torch.from_numpy(tl).cuda(), torch.from_numpy(dl).cuda(),
                              torch.from_numpy(np.asarray(tok, dtype=np.int32)).cuda(),
                              torch.from_numpy(np.asarray(u, dtype=np.float32)).cuda(), temperature,
                              want_probs=want_probs)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def check_against_oracle(tl, dl, tok, u, temperature=1.0):
    g = gpu_accept(tl, dl, tok, u, temperature, want_probs=True)
    r = oracle_accept(tl, dl, tok, u, temperature)
    gamma = dl.shape[0]
    assert_rel_close(g["probs_p"], r["p"], what="p")
    assert_rel_close(g["probs_q"], r["q"], what="q")
    assert_rel_close(g["p_tok"], r["p_tok"].astype(np.float64), what="p_tok")
    assert_rel_close(g["q_tok"], r["q_tok"].astype(np.float64), what="q_tok")
    assert np.abs(g["lse_p"] - r["lse_p"]).max() <= 1e-4 and np.abs(g["lse_q"] - r["lse_q"]).max() <= 1e-4
    # the accept decision recomputed on the host from the GPU's own fp32 probabilities is bit-exact
    n_from_gpu_probs = gamma
    for t in range(gamma):
        if not (np.float32(np.float32(u[t]) * g["q_tok"][t]) < g["p_tok"][t]):
            n_from_gpu_probs = t
            break
    assert int(g["n_accept"]) == n_from_gpu_probs
    # end to end: accepted length may differ from the oracle's only where u is within 1e-5 of p/q
    n_g, n_r = int(g["n_accept"]), r["n_accept"]
    if n_g != n_r:
        t = min(n_g, n_r)
        assert abs(float(u[t]) - float(r["p"][t, tok[t]] / r["q"][t, tok[t]])) <= 1e-5
        return g, r
    out = g["out_tokens"]
    assert (out[:n_g] == np.asarray(tok)[:n_g]).all() and (out[n_g + 1:] == -1).all()
    if out[n_g] != r["out_tokens"][n_r]:
        # the drawn token may differ only when u * Z sits within 1e-5 * Z of the CDF step between them
        w = r["resample_weights"]
        c = np.cumsum(w)
        lo, hi = sorted((int(out[n_g]), int(r["out_tokens"][n_r])))
        assert w[lo + 1:hi].sum() == 0.0 and abs(float(u[gamma]) * c[-1] - c[lo]) <= 1e-5 * c[-1]
    return g, r


@pytest.mark.parametrize("cid", [0, 1, 2, 3, 4])
def test_accepted_length_from_the_oracles_probabilities(cid):
    """The accept decision on its own (pvlm_accept_from_probs), fed the ORACLE's fp32 p(x_t), q(x_t): the accepted
    length is bit-exact on every workload config, several steps each, and on the edges of the uniform's range."""
    cfg = wl.CONFIGS[cid]
    for step in range(3):
        tl, dl, tok, u = wl.accept_inputs(cfg, step)
        r = oracle_accept(tl, dl, tok, u)
        p_d, q_d = torch.from_numpy(r["p_tok"]).cuda(), torch.from_numpy(r["q_tok"]).cuda()
        assert int(binding.accept_from_probs(p_d, q_d, torch.from_numpy(u).cuda())) == r["n_accept"]
        for edge in (0.0, 1.0 - 2.0 ** -24):                   # smallest and largest uniform there is
            ue = np.full_like(u, edge)
            want = oracle_accept(tl, dl, tok, ue)["n_accept"]
            assert int(binding.accept_from_probs(p_d, q_d, torch.from_numpy(ue).cuda())) == want
            if edge == 0.0:
                assert want == cfg.gamma                       # u = 0 accepts every token with p > 0


def test_accepted_length_from_probabilities_random_trials():
    """1e5 random trials of the decision alone against the rule written out in numpy fp32 (one rounded multiply,
    strict compare, first failure), a third of them placed ON the boundary u * q == p and one ulp either side."""
    rng = np.random.default_rng(99)
    B, gamma = 100_000, 6
    q = rng.random((B, gamma)).astype(np.float32) * np.float32(0.9) + np.float32(1e-3)
    u = wl.unit_uniforms(rng, (B, gamma + 1))
    p = (q * rng.random((B, gamma)).astype(np.float32) * np.float32(2.5)).astype(np.float32)       # ratios in [0, 2.5)
    on = rng.random((B, gamma)) < 1 / 3
    uq = (u[:, :gamma] * q).astype(np.float32)
    side = rng.integers(-1, 2, size=(B, gamma))
    edge = np.where(side < 0, np.nextafter(uq, np.float32(-1)), np.where(side > 0, np.nextafter(uq, np.float32(2)), uq))
    p = np.where(on, edge, p).astype(np.float32)
    ok = (u[:, :gamma] * q).astype(np.float32) < p
    want = np.where(ok.all(axis=1), gamma, np.argmin(ok, axis=1)).astype(np.int32)
    got = binding.accept_from_probs(torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(), torch.from_numpy(u).cuda())
    np.testing.assert_array_equal(got.cpu().numpy(), want)
    assert 0 < (want == gamma).sum() < B and (want == 0).any()
    # the oracle's trial routine agrees on the same decision when given logits whose softmax it computes itself
    V = 16
    tl = (1.5 * rng.standard_normal((gamma + 1, V))).astype(np.float32)
    dl = (tl[:gamma] + 0.7 * rng.standard_normal((gamma, V))).astype(np.float32)
    x = rng.integers(0, V, size=(B, gamma))
    n_ref, _ = spec_accept_trials(tl, dl, x, u)
    P, Q = softmax64(tl), softmax64(dl)
    t_idx = np.arange(gamma)[None, :]
    got = binding.accept_from_probs(torch.from_numpy(P[t_idx, x].astype(np.float32)).cuda(),
                                    torch.from_numpy(Q[t_idx, x].astype(np.float32)).cuda(), torch.from_numpy(u).cuda())
    np.testing.assert_array_equal(got.cpu().numpy(), n_ref)
    # gamma = 0: nothing to test
    z = torch.empty((3, 0), dtype=torch.float32, device="cuda")
    assert binding.accept_from_probs(z, z, torch.zeros((3, 1), device="cuda")).tolist() == [0, 0, 0]


def test_config0():
    tl, dl, tok, u = wl.accept_inputs(wl.CONFIGS[0])
    check_against_oracle(tl, dl, tok, u)


@pytest.mark.parametrize("cid", [1, 2, 3, 4])
def test_full_vocab_configs(cid):
    cfg = wl.CONFIGS[cid]
    for step in range(3):
        tl, dl, tok, u = wl.accept_inputs(cfg, step)
        check_against_oracle(tl, dl, tok, u)


@pytest.mark.parametrize("V,gamma", [(1, 1), (2, 3), (3, 1), (5, 2), (16, 4), (17, 64), (1023, 5), (1025, 7), (4097, 2),
                                     # around the sizes at which the tail team grows to 2, 4 and 8 CTAs, and a vocabulary whose
                                     # warp ranges are longer than the steps kept in registers (the recomputing walk)
                                     (20480, 3), (20481, 3), (40961, 2), (81921, 2), (200003, 1), (600001, 1)])
def test_small_and_ragged_vocab(V, gamma):
    rng = np.random.default_rng(V * 100 + gamma)
    for trial in range(4):
        tl, dl = wl.make_logits(V, gamma, 0.7, rng, rng, target_std=2.0)
        tok = wl.gumbel_draft_tokens(dl, rng)
        u = wl.unit_uniforms(rng, gamma + 1)
        check_against_oracle(tl, dl, tok, u)


def test_forced_outcomes_and_temperature():
    rng = np.random.default_rng(3)
    V, gamma = 3000, 6
    tl, dl = wl.make_logits(V, gamma, 0.5, rng, rng)
    tok = wl.gumbel_draft_tokens(dl, rng)
    g, r = check_against_oracle(tl, dl, tok, np.zeros(gamma + 1, np.float32))          # u = 0: accept all (p > 0)
    assert int(g["n_accept"]) == gamma
    g, r = check_against_oracle(tl, tl[:gamma].copy(), tok, np.full(gamma + 1, 1 - 2.0 ** -24, np.float32))
    assert int(g["n_accept"]) == gamma                                                 # q == p: ratio 1 always accepts
    u = np.full(gamma + 1, 0.999999, np.float32)
    g, r = check_against_oracle(tl, dl + np.float32(3.0) * (np.arange(V) % 7 == 0), tok, u)
    for temp in (0.5, 2.0):
        check_against_oracle(tl, dl, tok, wl.unit_uniforms(rng, gamma + 1), temperature=temp)
    # masked vocabulary entries (-inf logits) carry zero probability and are never drawn
    tl2, dl2 = tl.copy(), dl.copy()
    tl2[:, ::2] = -np.inf
    dl2[:, 1::2] = -np.inf
    tok2 = (np.asarray(tok) // 2 * 2).astype(np.int32)        # even tokens: q > 0, p = 0 => reject at 0
    g, r = check_against_oracle(tl2, dl2, tok2, wl.unit_uniforms(rng, gamma + 1))
    assert int(g["n_accept"]) == 0 and g["out_tokens"][0] % 2 == 1


def test_batched_matches_single_calls():
    rng = np.random.default_rng(8)
    B, V, gamma = 5, 2000, 4
    tls, dls, toks, us = [], [], [], []
    for b in range(B):
        tl, dl = wl.make_logits(V, gamma, 0.6, rng, rng)
        tls.append(tl); dls.append(dl); toks.append(wl.gumbel_draft_tokens(dl, rng)); us.append(wl.unit_uniforms(rng, gamma + 1))
    gb = gpu_accept(np.stack(tls), np.stack(dls), np.stack(toks), np.stack(us))
    for b in range(B):
        g1 = gpu_accept(tls[b], dls[b], toks[b], us[b])
        assert int(gb["n_accept"][b]) == int(g1["n_accept"])
        np.testing.assert_array_equal(gb["out_tokens"][b], g1["out_tokens"])
        np.testing.assert_array_equal(gb["p_tok"][b], g1["p_tok"])


def test_chi_square_on_gpu_path():
    """1e6 trials, V = 16, gamma = 4, run as batches through the C ABI: the first emitted
    token follows the target p (df = 15, p-value 1e-4), and every trial matches the oracle."""
    V, gamma, B = 16, 4, 1_000_000
    rng = np.random.default_rng(123)
    tl = (1.5 * rng.standard_normal((gamma + 1, V))).astype(np.float32)
    dl = (tl[:gamma] + 0.7 * rng.standard_normal((gamma, V))).astype(np.float32)
    g = np.random.Generator(np.random.Philox(key=2024))
    x = np.stack([wl.gumbel_draft_tokens(np.repeat(dl[t][None], B, axis=0), g) for t in range(gamma)], axis=1)
    u = wl.unit_uniforms(g, (B, gamma + 1))
    n_ref, tok_ref = spec_accept_trials(tl, dl, x, u)
    tl_d = torch.from_numpy(tl).cuda()
    dl_d = torch.from_numpy(dl).cuda()
    n_gpu = np.empty(B, np.int32)
    tok_gpu = np.empty(B, np.int32)
    step = 50_000
    for s in range(0, B, step):
        e = s + step
        out = binding.spec_accept(tl_d[None].expand(step, -1, -1), dl_d[None].expand(step, -1, -1),
                                  torch.from_numpy(x[s:e].astype(np.int32)).cuda(), torch.from_numpy(u[s:e]).cuda())
        n = out["n_accept"].cpu().numpy()
        n_gpu[s:e] = n
        tok_gpu[s:e] = out["out_tokens"].cpu().numpy()[np.arange(step), n]
    first = np.where(n_gpu >= 1, x[:, 0], tok_gpu)
    counts = np.bincount(first, minlength=V).astype(np.float64)
    p0 = softmax64(tl)[0]
    stat = ((counts - B * p0) ** 2 / (B * p0)).sum()
    assert stat < chi2.isf(1e-4, V - 1), stat
    mism = np.flatnonzero((n_gpu != n_ref) | (tok_gpu != tok_ref))
    assert mism.size <= 20, mism.size          # only trials sitting on a decision boundary may differ
    p, q = softmax64(tl), softmax64(dl)
    for b in mism:
        if n_gpu[b] != n_ref[b]:
            t = min(n_gpu[b], n_ref[b])
            assert abs(float(u[b, t]) - p[t, x[b, t]] / q[t, x[b, t]]) <= 1e-5


def test_sample_gamma_zero_matches_inverse_cdf():
    """gamma = 0 through the same entry point is plain sampling (the draft's own decoding step): the token is
    the oracle's inverse-CDF draw from softmax(logits / T); tokens that differ must sit on a CDF boundary."""
    from oracle.accept import inverse_cdf
    rng = np.random.default_rng(31)
    for V, B, T in [(151_936, 6, 1.0), (4099, 9, 0.7), (16, 64, 1.3), (1, 3, 1.0)]:
        lg = (2.0 * rng.standard_normal((B, V))).astype(np.float32)
        u = wl.unit_uniforms(rng, B)
        tok = binding.sample(torch.from_numpy(lg).cuda(), torch.from_numpy(u).cuda(), T).cpu().numpy()
        for b in range(B):
            p = softmax64(lg[b][None], T)[0]
            ref = inverse_cdf(p, float(u[b]))
            if tok[b] != ref:
                c = np.cumsum(p)
                lo, hi = sorted((int(tok[b]), int(ref)))
                assert hi - lo == 1 and abs(c[lo] - float(u[b]) * c[-1]) <= 1e-6, (V, b, tok[b], ref)
    o = oracle_accept(lg[0][None], np.zeros((0, V), np.float32), np.zeros(0, np.int32), u[:1])
    assert o["n_accept"] == 0 and o["out_tokens"][0] == binding.sample(torch.from_numpy(lg[0]).cuda(), torch.from_numpy(u[:1]).cuda()).item()


def test_sample_gamma_zero_chi_square():
    """4e5 draws from one row (stride-0 batch): counts follow softmax (df = 15, p-value 1e-4)."""
    V, B = 16, 400_000
    rng = np.random.default_rng(77)
    lg = (1.5 * rng.standard_normal(V)).astype(np.float32)
    u = wl.unit_uniforms(np.random.Generator(np.random.Philox(key=99)), B)
    lg_d, step = torch.from_numpy(lg).cuda(), 50_000                      # one call takes at most 65535 rows
    tok = np.concatenate([binding.sample(lg_d[None].expand(step, -1), torch.from_numpy(u[s:s + step]).cuda()).cpu().numpy()
                          for s in range(0, B, step)])
    counts = np.bincount(tok, minlength=V).astype(np.float64)
    p = softmax64(lg[None])[0]
    stat = ((counts - B * p) ** 2 / (B * p)).sum()
    assert stat < chi2.isf(1e-4, V - 1), stat
