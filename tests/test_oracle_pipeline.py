"""CPU pins of the parallel-decoding oracle: the paper's worked example, closed forms, an independent
Markov-chain solution of the mode machine, Theorem 6's two-round count, and losslessness."""
import os

import numpy as np
from scipy.stats import chi2

from oracle.accept import inverse_cdf, softmax64
from oracle.pipeline import (POST, PRE, Schedule, expected_accepted, parallel_decode, simulate_iid,
                             simulate_vanilla_sd, t_psd, t_psd_rollback, t_sd)
from paper_2603_19610_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_worked_example_of_the_appendix():
    cfg, rounds, cache_after = {}, [], {}
    for line in open(os.path.join(GOLD, "pipeline_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        if parts[0] == "round":
            rounds.append(tuple(int(x) for x in parts[1:3] + parts[4:6]))
        elif parts[0] == "draft_cache_after_round":
            cache_after[int(parts[1])] = int(parts[2])
        else:
            cfg[parts[0]] = int(parts[1])
    s = Schedule(cfg["gamma"], cfg["start_mode"], cfg["start_pending"], cfg["start_committed"])
    run, longest = cfg["start_committed"], 0            # the pre-verified first token opens the run
    for i, (verified, accepted, committed, next_mode) in enumerate(rounds, start=1):
        assert s.n_verify() == verified
        before = s.committed
        rec = s.advance(accepted)
        assert (rec["emitted"], rec["next_mode"]) == (committed, next_mode)
        # cache lengths: the verification's context is what was committed; the draft keeps one row per generated
        # token it restarts AFTER, so "k generated tokens stay in its cache" reads draft_keep = k + 1
        assert rec["target_ctx"] == before
        if i in cache_after:
            assert rec["draft_keep"] - 1 == cache_after[i] and accepted < verified
        else:
            assert rec["draft_keep"] == rec["draft_ctx"] + cfg["gamma"]          # nothing dropped: gamma more rows
        run += accepted
        longest = max(longest, run)
        if accepted < verified:
            run = 0
    assert len(cache_after) == 2
    assert s.committed == cfg["total_committed"] and len(s.log) == cfg["total_rounds"]
    assert len(s.log) * max(cfg["gamma"], cfg["gamma"]) == cfg["total_time_in_t"]      # c = gamma: a round lasts 3t
    assert longest == cfg["longest_accepted_run"]


def test_round_sequence_from_a_pre_verify_start_under_this_builds_reading():
    """The mode machine started in Pre-verify mode, against a hand-written round table that records this build's
    READING of the Pre -> Post transition (gamma - 1 drafts stay pending); the fixture says so itself."""
    gamma, rounds, total = None, [], None
    for line in open(os.path.join(GOLD, "pipeline_from_pre_reading.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        if parts[0] == "gamma":
            gamma = int(parts[1])
        elif parts[0] == "total_committed":
            total = int(parts[1])
        else:
            rounds.append(tuple(int(x) for x in parts[1:4] + parts[5:9]))
    s = Schedule(gamma)
    for mode, verified, accepted, committed, dropped, next_mode, pending_after in rounds:
        assert (s.mode if s.pending else PRE, s.n_verify()) == (mode, verified)
        rec = s.advance(accepted)
        assert (rec["mode"], rec["emitted"], rec["dropped"], rec["next_mode"], s.pending) == (mode, committed, dropped, next_mode, pending_after)
    assert s.committed == total


def test_closed_forms_and_their_stated_consequences():
    for c in (3.0, 5.0, 9.0):
        g = c
        assert abs(c / t_psd(g, c) - c) < 1e-12                                  # V_PSD = c at gamma = c
        assert abs((c / t_psd(g, c)) / (c / t_sd(g, c)) - 2 * c / (c + 1)) < 1e-12   # V_PSD / V_SD = 2c / (c + 1)
        for tau in (0.27, 0.41, 0.8):
            assert abs(c / t_psd(g, c, tau=tau) - tau * c) < 1e-12               # practical: tau * c
            assert abs(c / t_sd(g, c, tau=tau) - c * (tau * g + 1) / (g + c)) < 1e-12
            # Theorem 6 at gamma = c: speedup = 1/2 * sum_{k=1}^{2c} tau^k
            ci = int(c)
            assert abs(c / t_psd_rollback(ci, c, tau) - 0.5 * sum(tau ** k for k in range(1, 2 * ci + 1))) < 1e-12
    assert t_psd(4, 9) == 9 / 4 and t_psd(12, 9) == 1.0                          # the two branches of the max
    # Lemma 1's closed form against the defining sum used by the oracle
    for tau, g in ((0.41, 9), (0.9, 5), (0.5, 1)):
        assert abs(expected_accepted(tau, g) - tau * (1 - tau ** g) / (1 - tau)) < 1e-12


def _stationary_rate(tau, g):
    """Committed tokens per round of the mode machine, from the stationary distribution of its three
    states (Pre, Post with gamma-1 pending, Post with gamma pending): linear algebra, no simulation."""
    def post_reward(n):
        return sum((k + 1) * (1 - tau) * tau ** k for k in range(n)) + n * tau ** n
    P = np.zeros((3, 3))
    P[0, 1], P[0, 0] = tau, 1 - tau
    P[1, 2], P[1, 0] = tau ** (g - 1), 1 - tau ** (g - 1)
    P[2, 2], P[2, 0] = tau ** g, 1 - tau ** g
    A = np.vstack([P.T - np.eye(3), np.ones(3)])
    pi = np.linalg.lstsq(A, np.array([0, 0, 0, 1.0]), rcond=None)[0]
    return float(pi @ np.array([1.0, post_reward(g - 1), post_reward(g)]))


def test_mode_machine_matches_its_markov_chain():
    rng = np.random.default_rng(5)
    for tau, g in ((0.41, 9), (0.8, 5), (0.3, 3), (0.95, 12)):
        log = simulate_iid(tau, g, 200_000, rng)
        rate = sum(r["emitted"] for r in log) / len(log)
        assert abs(rate - _stationary_rate(tau, g)) < 0.02 * _stationary_rate(tau, g), (tau, g, rate)
    # all accepted: one Pre round, then gamma tokens per round (Theorem 3: per-token time max(gamma t, c t) / gamma)
    log = simulate_iid(1.0, 6, 50, rng)
    assert [r["emitted"] for r in log[:3]] == [1, 5, 6] and all(r["emitted"] == 6 for r in log[2:])
    # nothing accepted: every round is a Pre-verify round that commits the target's own token
    log = simulate_iid(0.0, 6, 20, rng)
    assert all(r["mode"] == PRE and r["emitted"] == 1 and r["dropped"] == 6 for r in log)
    # gamma = 1 never leaves Pre-verify
    assert all(r["mode"] == PRE for r in simulate_iid(0.7, 1, 50, rng))


def test_two_round_count_of_theorem_6():
    """Two rounds that start in Post-verify with a full window accept (1 + tau^gamma) E[X] drafted
    tokens in their Post-verify verifications (the retry round after a rejection adds none)."""
    rng = np.random.default_rng(11)
    for tau, g in ((0.41, 9), (0.8, 4)):
        tot, n = 0, 60_000
        for _ in range(n):
            log = simulate_iid(tau, g, 2, rng, POST, g)
            tot += sum(r["accepted"] for r in log if r["mode"] == POST)
        want = (1 + tau ** g) * expected_accepted(tau, g)
        assert abs(tot / n - want) < 0.02 * want, (tot / n, want)


def test_vanilla_sd_rounds():
    rng = np.random.default_rng(2)
    assert simulate_vanilla_sd(1.0, 5, 10, rng) == [6] * 10                     # Theorem 2: gamma + 1 tokens per round
    m = np.mean(simulate_vanilla_sd(0.6, 5, 100_000, rng))
    assert abs(m - (expected_accepted(0.6, 5) + 1)) < 0.02


def _inputs(V, K, gamma, sigma, seed):
    rng = np.random.default_rng(seed)
    P = K + 2 * gamma + 1
    tl = (1.5 * rng.standard_normal((P, V))).astype(np.float32)
    dl = (tl + sigma * rng.standard_normal((P, V))).astype(np.float32)
    return tl, dl


def test_token_level_pipeline_basic_properties():
    V, K, gamma = 50, 40, 4
    tl, dl = _inputs(V, K, gamma, 0.8, 3)
    g = np.random.Generator(np.random.Philox(key=9))
    ud, ua, ur = wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, K)
    out = parallel_decode(tl, dl, gamma, K, ud, ua, ur)
    assert out["tokens"].shape == (K,) and out["rounds"] == len(out["log"]) <= K
    assert sum(r["emitted"] for r in out["log"]) >= K and out["log"][0]["mode"] == PRE
    starts = np.cumsum([0] + [r["emitted"] for r in out["log"]])[:-1]
    assert [r["start"] for r in out["log"]] == list(starts)
    again = parallel_decode(tl, dl, gamma, K, ud, ua, ur)
    np.testing.assert_array_equal(out["tokens"], again["tokens"])
    # identical models: everything is accepted and the output is the draft's own inverse-CDF draws
    same = parallel_decode(tl, tl, gamma, K, ud, ua, ur)
    assert all(r["accepted"] == r["verified"] for r in same["log"])
    q = softmax64(tl)
    r0 = same["log"]
    assert same["tokens"][0] == inverse_cdf(q[0], float(ud[0, 0]))               # round 0 drafts positions 0..3
    assert same["tokens"][1] == inverse_cdf(q[1], float(ud[0, 1]))
    assert same["tokens"][gamma] == inverse_cdf(q[gamma], float(ud[1, 0]))       # round 1 drafts positions 4..7
    assert [r["emitted"] for r in r0[:3]] == [1, gamma - 1, gamma]


def test_token_level_pipeline_is_lossless():
    """Whatever the draft model, position i of the output follows the target's p_i (chi-square,
    V = 6, positions 0..4, 20000 runs; p-value 1e-4 per position)."""
    V, K, gamma, runs = 6, 5, 3, 20_000
    tl, dl = _inputs(V, K, gamma, 1.2, 21)
    p = softmax64(tl)
    g = np.random.Generator(np.random.Philox(key=4))
    counts = np.zeros((K, V))
    for _ in range(runs):
        ud, ua, ur = wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, K)
        tok = parallel_decode(tl, dl, gamma, K, ud, ua, ur)["tokens"]
        counts[np.arange(K), tok] += 1
    for i in range(K):
        stat = ((counts[i] - runs * p[i]) ** 2 / (runs * p[i])).sum()
        assert stat < chi2.isf(1e-4, V - 1), (i, stat)
