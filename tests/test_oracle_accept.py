"""Pins for the accept/reject oracle: exact output law by integrating over the
uniforms on tiny vocabularies, closed-form acceptance, Lemma 1's truncated
geometric law, a 1e6-trial chi-square that the emitted token follows the
target p, and special cases."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.stats import chi2

from oracle.accept import inverse_cdf, softmax64, spec_accept, spec_accept_trials, window_size
from paper_2603_19610_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_softmax_rows():
    rng = np.random.default_rng(0)
    x = (3 * rng.standard_normal((5, 1000))).astype(np.float32)
    p = softmax64(x)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    # against explicit exponentials (no max subtraction needed at this range)
    e = np.array([[math.exp(float(v)) for v in row] for row in x])
    np.testing.assert_allclose(p, e / e.sum(axis=1, keepdims=True), rtol=1e-12)
    np.testing.assert_allclose(softmax64(x, 2.0), softmax64(x / np.float32(2.0)), rtol=1e-6)
    # shift invariance incl. values that would overflow without max subtraction
    np.testing.assert_allclose(softmax64(x + np.float32(1000.0)), p, rtol=1e-3)


@pytest.mark.parametrize("temperature", [1.0, 0.5, 2.0])
def test_lse_rows(temperature):
    """log-sum-exp of logits / temperature, pinned four ways: scalar math.exp / math.log loops, the identity
    lse = x_j / T - log softmax_j at the argmax and at every j, the shift law lse(x + c) = lse(x) + c / T
    (also where exp(x) alone would overflow), and the closed form log(n) + a / T for n equal logits."""
    from oracle.accept import lse64
    rng = np.random.default_rng(11)
    x = (3 * rng.standard_normal((4, 700))).astype(np.float32)
    got = lse64(x, temperature)
    assert got.shape == (4,) and got.dtype == np.float64
    want = np.array([math.log(sum(math.exp(float(v) / temperature) for v in row)) for row in x])
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    p = softmax64(x, temperature)
    j = p.argmax(axis=1)
    np.testing.assert_allclose(got, x[np.arange(4), j].astype(np.float64) / temperature - np.log(p[np.arange(4), j]), atol=1e-12)
    np.testing.assert_allclose(got[:, None] - x.astype(np.float64) / temperature, -np.log(p), atol=1e-9)
    np.testing.assert_allclose(lse64(x + np.float32(900.0), temperature),
                               lse64((x + np.float32(900.0)).astype(np.float64) - 900.0, temperature) + 900.0 / temperature, atol=1e-9)
    np.testing.assert_allclose(lse64(np.full((2, 37), 1.25, np.float32), temperature), math.log(37) + 1.25 / temperature, atol=1e-13)
    # a masked entry (-inf) adds nothing; a single entry is its own lse
    y = x.copy()
    y[:, 5] = -np.inf
    np.testing.assert_allclose(lse64(y, temperature), lse64(np.delete(x, 5, axis=1), temperature), atol=1e-12)
    np.testing.assert_allclose(lse64(x[:, :1], temperature), x[:, 0].astype(np.float64) / temperature, atol=1e-13)
    # the values spec_accept reports are these
    r = spec_accept(x, x[:3] + np.float32(0.5), [0, 1, 2], np.full(4, 0.5, np.float32), temperature)
    np.testing.assert_array_equal(r["lse_p"], got)
    np.testing.assert_allclose(r["lse_q"], got[:3] + 0.5 / temperature, atol=1e-6)


def test_inverse_cdf_rule():
    w = np.array([0.0, 0.2, 0.0, 0.3, 0.5, 0.0])
    assert inverse_cdf(w, 0.0) == 1            # zero-weight token 0 is never chosen
    assert inverse_cdf(w, 0.19999) == 1
    assert inverse_cdf(w, 0.2) == 3            # boundary belongs to the next token (strict >)
    assert inverse_cdf(w, 0.5) == 4
    assert inverse_cdf(w, 0.999999) == 4       # trailing zero-weight token never chosen
    assert inverse_cdf(3.0 * w, 0.49) == 3     # unnormalised weights


def exact_first_token_law(p0, q0):
    """Law of the token emitted at position 0 under draft x ~ q0: accept with
    min(1, p/q), else resample from norm(max(0, p - q))."""
    V = len(p0)
    out = np.zeros(V)
    res = np.maximum(0.0, p0 - q0)
    rej = 0.0
    for x in range(V):
        a = min(1.0, p0[x] / q0[x]) if q0[x] > 0 else 1.0
        out[x] += q0[x] * a
        rej += q0[x] * (1 - a)
    if res.sum() > 0:
        out += rej * res / res.sum()
    return out


@pytest.mark.parametrize("V", [2, 3, 4])
def test_exact_law_equals_target_on_tiny_vocab(V):
    """Integrate the oracle over a fine grid of (u_accept, u_sample) for every
    draft token, weight by q(x): the emitted first token must follow p."""
    rng = np.random.default_rng(V)
    tl = rng.standard_normal((2, V)).astype(np.float32)
    dl = rng.standard_normal((1, V)).astype(np.float32)
    p, q = softmax64(tl), softmax64(dl)
    np.testing.assert_allclose(exact_first_token_law(p[0], q[0]), p[0], atol=1e-12)   # the rule itself is lossless
    Nu = 400
    grid = ((np.arange(Nu) + 0.5) / Nu).astype(np.float32)
    law = np.zeros(V)
    for x in range(V):
        for ua in grid:
            # the sampling uniform only matters after a rejection; integrate it too
            r = spec_accept(tl, dl, [x], [ua, 0.5])
            if r["n_accept"] == 1:
                law[x] += q[0, x] / Nu
            else:
                for us in grid[::8]:
                    tok = spec_accept(tl, dl, [x], [ua, us])["out_tokens"][0]
                    law[tok] += q[0, x] / Nu / len(grid[::8])
    np.testing.assert_allclose(law, p[0], atol=2.5 / Nu * 8)


def _trial_inputs(V, gamma, B, seed, std=1.5, sigma=0.7):
    rng = np.random.default_rng(seed)
    tl = (std * rng.standard_normal((gamma + 1, V))).astype(np.float32)
    dl = (tl[:gamma] + sigma * rng.standard_normal((gamma, V))).astype(np.float32)
    q = softmax64(dl)
    # drafts ~ q by inverse CDF with their own uniforms (independent of the accept uniforms)
    ud = rng.random((B, gamma))
    x = np.stack([np.minimum(np.searchsorted(np.cumsum(q[t]), ud[:, t], side="right"), V - 1)
                  for t in range(gamma)], axis=1)
    u = wl.unit_uniforms(np.random.Generator(np.random.Philox(key=seed)), (B, gamma + 1))
    return tl, dl, x.astype(np.int32), u


def test_trials_match_single_calls():
    tl, dl, x, u = _trial_inputs(16, 4, 3000, seed=5)
    n, tok = spec_accept_trials(tl, dl, x, u)
    for b in range(3000):
        r = spec_accept(tl, dl, x[b], u[b])
        assert r["n_accept"] == n[b]
        assert r["out_tokens"][n[b]] == tok[b]
        assert (r["out_tokens"][:n[b]] == x[b, :n[b]]).all()
        assert (r["out_tokens"][n[b] + 1:] == -1).all()


def test_chi_square_first_token_follows_target():
    """1e6 trials, V = 16: the first emitted token (accepted draft or its
    replacement) is distributed as p_0.  df = 15, reject at p-value 1e-4."""
    V, gamma, B = 16, 4, 1_000_000
    tl, dl, x, u = _trial_inputs(V, gamma, B, seed=123)
    n, tok = spec_accept_trials(tl, dl, x, u)
    first = np.where(n >= 1, x[:, 0], tok)
    counts = np.bincount(first, minlength=V).astype(np.float64)
    p0 = softmax64(tl)[0]
    stat = ((counts - B * p0) ** 2 / (B * p0)).sum()
    assert stat < chi2.isf(1e-4, V - 1), stat
    # empirical acceptance at position 0 equals sum_x min(p, q) (closed form)
    tau = np.minimum(p0, softmax64(dl)[0]).sum()
    acc = (n >= 1).mean()
    assert abs(acc - tau) < 4.9 * math.sqrt(tau * (1 - tau) / B)
    # every emitted sequence position also follows its target row given the prefix was accepted:
    # position 1 token among trials with n >= 1
    sel = n >= 1
    second = np.where(n[sel] >= 2, x[sel, 1], tok[sel])
    second = second[(n[sel] >= 2) | (n[sel] == 1)]
    c2 = np.bincount(second, minlength=V).astype(np.float64)
    p1 = softmax64(tl)[1]
    stat2 = ((c2 - c2.sum() * p1) ** 2 / (c2.sum() * p1)).sum()
    assert stat2 < chi2.isf(1e-4, V - 1), stat2


def test_lemma1_truncated_geometric():
    """Identical (p, q) at every position => n_accept ~ TruncGeo(tau, gamma):
    P(k) = (1 - tau) tau^k for k < gamma, tau^gamma at k = gamma, and
    E = tau (1 - tau^gamma) / (1 - tau)  (Lemma 1)."""
    V, B = 16, 400_000
    for line in open(os.path.join(GOLD, "truncgeo.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tau_target, gamma = float(line.split()[0]), int(line.split()[1])
        rng = np.random.default_rng(int(tau_target * 100))
        t_row = (1.5 * rng.standard_normal(V)).astype(np.float32)
        # pick a draft row whose overlap with the target is near the printed tau
        best = None
        for sig in np.linspace(0.5, 6.0, 60):
            d_row = (t_row + sig * rng.standard_normal(V)).astype(np.float32)
            tau = np.minimum(softmax64(t_row[None])[0], softmax64(d_row[None])[0]).sum()
            if best is None or abs(tau - tau_target) < abs(best[0] - tau_target):
                best = (tau, d_row)
        tau, d_row = best
        tl = np.repeat(t_row[None], gamma + 1, axis=0)
        dl = np.repeat(d_row[None], gamma, axis=0)
        q = softmax64(dl)
        ud = rng.random((B, gamma))
        x = np.minimum(np.searchsorted(np.cumsum(q[0]), ud, side="right"), V - 1).astype(np.int32)
        u = wl.unit_uniforms(np.random.Generator(np.random.Philox(key=gamma)), (B, gamma + 1))
        n, _ = spec_accept_trials(tl, dl, x, u)
        pmf = np.array([(1 - tau) * tau ** k for k in range(gamma)] + [tau ** gamma])
        mean_closed = tau * (1 - tau ** gamma) / (1 - tau)
        assert abs((pmf * np.arange(gamma + 1)).sum() - mean_closed) < 1e-12     # the lemma's algebra
        assert abs(n.mean() - mean_closed) < 5 * n.std() / math.sqrt(B)
        counts = np.bincount(n, minlength=gamma + 1).astype(np.float64)
        keep = B * pmf >= 5
        stat = ((counts[keep] - B * pmf[keep]) ** 2 / (B * pmf[keep])).sum()
        assert stat < chi2.isf(1e-4, int(keep.sum()) - 1), (tau, stat)


def test_special_cases():
    rng = np.random.default_rng(2)
    V, gamma = 12, 5
    tl = rng.standard_normal((gamma + 1, V)).astype(np.float32)
    x = rng.integers(0, V, gamma)
    for _ in range(50):                          # q == p: ratio 1, always accepted, bonus from row gamma
        u = rng.random(gamma + 1).astype(np.float32)
        r = spec_accept(tl, tl[:gamma], x, u)
        assert r["n_accept"] == gamma
        assert r["out_tokens"][gamma] == inverse_cdf(softmax64(tl)[gamma], float(u[gamma]))
    # disjoint supports: draft mass only on tokens the target excludes => always reject at 0, emit ~ p
    tl2 = tl.copy()
    tl2[:, :6] = -1e4
    dl2 = tl[:gamma].copy()
    dl2[:, 6:] = -1e4
    r = spec_accept(tl2, dl2, np.full(gamma, 2), np.full(gamma + 1, 1e-6, dtype=np.float32))
    assert r["n_accept"] == 0 and r["out_tokens"][0] >= 6 and (r["out_tokens"][1:] == -1).all()
    # one-hot target: emitted first token is always that token
    tl3 = np.full((gamma + 1, V), -1e4, dtype=np.float32)
    tl3[:, 7] = 0.0
    for xx in (3, 7):
        for ua in (0.0, 0.3, 0.99):
            r = spec_accept(tl3, tl[:gamma], np.full(gamma, xx), np.array([ua] * gamma + [0.5], np.float32))
            assert r["out_tokens"][0] == 7
    # strictness: ratio >= 1 accepts for every u in [0,1); p = 0 never accepts (u = 0 included)
    r = spec_accept(tl3, tl[:gamma], np.full(gamma, 7), np.array([1 - 2.0 ** -24] * (gamma + 1), np.float32))
    assert r["n_accept"] == gamma
    r = spec_accept(tl3, tl[:gamma], np.full(gamma, 3), np.zeros(gamma + 1, np.float32))
    assert r["n_accept"] == 0
    # p_tok / q_tok are reported for every position, accepted or not
    r = spec_accept(tl, tl[:gamma] + 1.0, x, np.full(gamma + 1, 0.999, np.float32))
    np.testing.assert_allclose(r["p_tok"], softmax64(tl)[np.arange(gamma), x], rtol=1e-6)


def test_expected_accept_equals_sum_min_pq_sequence():
    """P(n_accept >= t) = prod_{s<t} sum_x min(p_s, q_s) when drafts ~ q."""
    V, gamma, B = 16, 4, 300_000
    tl, dl, x, u = _trial_inputs(V, gamma, B, seed=99)
    n, _ = spec_accept_trials(tl, dl, x, u)
    p, q = softmax64(tl), softmax64(dl)
    prod = 1.0
    for t in range(gamma):
        prod *= np.minimum(p[t], q[t]).sum()
        emp = (n >= t + 1).mean()
        assert abs(emp - prod) < 4.9 * math.sqrt(prod * (1 - prod) / B)


def test_window_rule_printed_examples():
    """Eq. 6 with the forward times the paper prints reproduces its printed ratios."""
    for line in open(os.path.join(GOLD, "window_rule.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tp, tq, printed = (float(s) for s in line.split())
        c = window_size(tp, tq)
        tol = 0.5 if printed == round(printed) and "." not in line.split()[2] else 0.1
        assert abs(c - printed) <= tol, (tp, tq, c, printed)


def test_window_choice_reproduces_the_papers_gammas():
    """Nearest-integer rounding of c* on the paper's printed forward times gives the window sizes the
    paper uses for its five model pairs; the other two modes bracket it."""
    from oracle.accept import window_size_rounded
    for line in open(os.path.join(GOLD, "window_choice.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tp, tq, gamma = line.split()
        assert window_size_rounded(float(tp), float(tq)) == int(gamma), line
        assert window_size_rounded(float(tp), float(tq), "down") <= int(gamma) <= window_size_rounded(float(tp), float(tq), "up")
    assert window_size_rounded(420, 78, "down") == 5 and window_size_rounded(420, 47, "down") == 8
    assert window_size_rounded(420, 47, "up") == 9 and window_size_rounded(10, 50) == 1


def test_gamma_zero_is_plain_sampling():
    rng = np.random.default_rng(0)
    tl = rng.standard_normal((1, 50)).astype(np.float32)
    r = spec_accept(tl, np.zeros((0, 50), np.float32), np.zeros(0, np.int32), np.array([0.37], np.float32))
    assert r["n_accept"] == 0 and r["out_tokens"].shape == (1,)
    assert r["out_tokens"][0] == inverse_cdf(softmax64(tl)[0], 0.37)


def test_tokenwise_acceptance_pins():
    """(1) position by position it is the gamma = 1 accept rule; (2) with tokens drawn from q the acceptance
    frequency is sum_x min(p, q) = 1 - TV(p, q); (3) identical models accept everything, a token outside the
    target's support is rejected."""
    from oracle.accept import tokenwise_acceptance
    rng = np.random.default_rng(17)
    N, V = 40, 37
    tl = (1.5 * rng.standard_normal((N, V))).astype(np.float32)
    dl = (tl + rng.standard_normal((N, V))).astype(np.float32)
    x = wl.gumbel_draft_tokens(dl, rng)
    u = wl.unit_uniforms(rng, N)
    out = tokenwise_acceptance(tl, dl, x, u)
    for n in range(N):
        one = spec_accept(np.stack([tl[n], tl[n]]), dl[n][None], x[n:n + 1], np.array([u[n], 0.5], np.float32))
        assert int(one["n_accept"]) == int(out["accepted"][n])
        assert one["p_tok"][0] == out["p_tok"][n] and one["q_tok"][0] == out["q_tok"][n]
    B = 200_000
    g = np.random.Generator(np.random.Philox(key=5))
    xs = wl.gumbel_draft_tokens(np.repeat(dl[:1], B, axis=0), g)
    rate = tokenwise_acceptance(np.repeat(tl[:1], B, axis=0), np.repeat(dl[:1], B, axis=0), xs, wl.unit_uniforms(g, B))["rate"]
    want = np.minimum(softmax64(tl[:1]), softmax64(dl[:1])).sum()
    assert abs(rate - want) < 4 * np.sqrt(want * (1 - want) / B), (rate, want)
    assert tokenwise_acceptance(tl, tl, x, u)["accepted"].all()
    tl2 = tl.copy()
    tl2[np.arange(N), x] = -np.inf
    assert not tokenwise_acceptance(tl2, dl, x, u)["accepted"].any()
