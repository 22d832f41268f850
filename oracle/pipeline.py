"""Oracle: the parallel decoding pipeline (Stage II; Algorithm 1 and the appendix
"Parallel Pipeline Details") and the per-token-time formulas of the appendix
"Theoretical Analysis" (Theorems 2-6, Lemma 1).  TEST INFRASTRUCTURE ONLY.

One ROUND is one target forward running beside `gamma` draft forwards; it lasts
max(gamma * t, c * t) with t = T_q and c = T_p / T_q.

Readings where the paper (which defers to Parallel SD for the two modes) is
silent:
* Pre-verify round: the target runs on the committed prefix only, the draft
  writes gamma fresh tokens d_0..d_{gamma-1}; then d_0 alone is tested against
  the target's distribution for that position.  Accepted: d_0 is committed, the
  other gamma-1 drafts stay pending, mode becomes Post-verify.  Rejected: the
  replacement drawn from norm(max(0, p - q)) is committed, every draft is
  dropped (the draft cache rolls back to the committed prefix), mode stays
  Pre-verify.
* Post-verify round: the target verifies all pending drafts in one batch while
  the draft writes gamma more tokens behind them.  All accepted: they are
  committed, the gamma new drafts become pending (no bonus token: the draft has
  already written its own token for that position), mode stays Post-verify.
  Otherwise the accepted prefix and the replacement token are committed, all
  other drafts are dropped, mode becomes Pre-verify.
* A Post-verify round with nothing pending (gamma = 1) is a Pre-verify round.
* Random numbers are indexed by (round, slot) so that every implementation
  consumes the same ones: u_draft[r, s] draws the s-th token drafted in round
  r, u_accept[r, s] tests the s-th token verified in round r, u_resample[r]
  draws round r's replacement token.
* Synthetic stand-in for the two models: row i of `target_logits` /
  `draft_logits` is the model's distribution for generated position i,
  whatever the prefix (the pipeline's control flow does not depend on how the
  rows come about).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .accept import inverse_cdf, softmax64, spec_accept

PRE, POST = 0, 1


# ----------------------------------------------------------------------------------------------
# Closed forms (appendix "Theoretical Analysis"); t = T_q, c = T_p / T_q
# ----------------------------------------------------------------------------------------------
def t_sd(gamma: float, c: float, t: float = 1.0, tau: float = 1.0) -> float:
    """Per-token time of vanilla SD: Theorem 2 (tau = 1) and Theorem 4."""
    return (gamma + c) / (tau * gamma + 1.0) * t


def t_psd(gamma: float, c: float, t: float = 1.0, tau: float = 1.0) -> float:
    """Per-token time of parallel SD in Post-verify mode: Theorem 3 (tau = 1) and Theorem 5."""
    return max(gamma * t, c * t) / (tau * gamma)


def expected_accepted(tau: float, gamma: int) -> float:
    """Lemma 1, written as the defining sum over the truncated geometric distribution."""
    return sum(k * (1.0 - tau) * tau ** k for k in range(gamma)) + gamma * tau ** gamma


def t_psd_rollback(gamma: int, c: float, tau: float, t: float = 1.0) -> float:
    """Theorem 6: two rounds yield (1 + tau^gamma) E[X] accepted tokens."""
    return 2.0 * max(gamma * t, c * t) / ((1.0 + tau ** gamma) * expected_accepted(tau, gamma))


# ----------------------------------------------------------------------------------------------
# The mode machine of Algorithm 1
# ----------------------------------------------------------------------------------------------
@dataclass
class Schedule:
    gamma: int
    mode: int = PRE
    pending: int = 0            # drafts written in earlier rounds, not yet verified
    committed: int = 0          # generated tokens committed so far
    log: list = field(default_factory=list)

    def n_verify(self) -> int:
        """Tokens the target tests in the coming round."""
        return self.pending if (self.mode == POST and self.pending > 0) else 1

    def advance(self, n_accept: int) -> dict:
        """Applies one round's verification outcome; returns what was committed and dropped, and the cache
        lengths of the round, counted in rows beyond each model's context before the first generated token
        (a model's forward takes its newest token as input, so a cache that "holds k generated tokens and
        restarts from the next one" is k + 1 rows here):
        target_ctx = context rows of the round's verification (the committed tokens; its window holds the last
        committed token and the tokens under test); draft_ctx = context rows of the draft's first forward of the
        round (committed and pending tokens); draft_keep = the same count after the round: everything the draft
        has written if all was accepted, the committed prefix alone after a rejection (the cache rolls back and
        the replacement token is the draft's next input)."""
        g = self.gamma
        post = self.mode == POST and self.pending > 0
        lengths = dict(target_ctx=self.committed, draft_ctx=self.committed + (self.pending if post else 0))
        if post:
            nv = self.pending
            assert 0 <= n_accept <= nv
            if n_accept == nv:
                rec = dict(mode=POST, verified=nv, accepted=nv, emitted=nv, dropped=0, next_mode=POST)
                self.pending = g
            else:
                rec = dict(mode=POST, verified=nv, accepted=n_accept, emitted=n_accept + 1,
                           dropped=nv - n_accept + g, next_mode=PRE)
                self.pending, self.mode = 0, PRE
        else:
            assert n_accept in (0, 1)
            if n_accept == 1 and g > 1:
                rec = dict(mode=PRE, verified=1, accepted=1, emitted=1, dropped=0, next_mode=POST)
                self.pending, self.mode = g - 1, POST
            elif n_accept == 1:
                rec = dict(mode=PRE, verified=1, accepted=1, emitted=1, dropped=0, next_mode=PRE)
                self.pending, self.mode = 0, PRE
            else:
                rec = dict(mode=PRE, verified=1, accepted=0, emitted=1, dropped=g, next_mode=PRE)
                self.pending, self.mode = 0, PRE
        self.committed += rec["emitted"]
        rec.update(lengths, draft_keep=self.committed + self.pending)
        self.log.append(rec)
        return rec


def simulate_iid(tau: float, gamma: int, rounds: int, rng, start_mode: int = PRE, start_pending: int = 0):
    """Runs the mode machine with every verified token accepted independently with probability tau.
    Returns the round log."""
    s = Schedule(gamma, start_mode, start_pending)
    for _ in range(rounds):
        nv = s.n_verify()
        ok = rng.random(nv) < tau
        s.advance(nv if ok.all() else int(np.argmin(ok)))
    return s.log


def simulate_vanilla_sd(tau: float, gamma: int, rounds: int, rng):
    """Vanilla SD for comparison (Theorems 2 and 4): a round drafts gamma tokens, then verifies them;
    it lasts gamma * t + c * t and commits the accepted prefix plus one token of the target's."""
    out = []
    for _ in range(rounds):
        ok = rng.random(gamma) < tau
        out.append((gamma if ok.all() else int(np.argmin(ok))) + 1)
    return out


# ----------------------------------------------------------------------------------------------
# Token-level reference of the pipeline
# ----------------------------------------------------------------------------------------------
def parallel_decode(target_logits, draft_logits, gamma: int, K: int, u_draft, u_accept, u_resample,
                    temperature: float = 1.0):
    """Generates K tokens.  target_logits / draft_logits fp32 [P, V] with P >= K + 2 * gamma + 1 rows;
    u_draft, u_accept fp32 [rounds, gamma]; u_resample fp32 [rounds].
    Returns dict(tokens int32 [K], rounds, log (one record per round, as `Schedule.advance` plus
    `start` = committed length at the round's start; the cache lengths target_ctx, draft_ctx, draft_keep of
    `Schedule.advance` are checked against the token lists kept here))."""
    tl = np.asarray(target_logits, dtype=np.float32)
    dl = np.asarray(draft_logits, dtype=np.float32)
    q = softmax64(dl, temperature)
    s = Schedule(gamma)
    tokens: list[int] = []
    pending: list[int] = []
    r = 0
    while len(tokens) < K:
        L = len(tokens)
        post = s.mode == POST and s.pending > 0
        # the draft model's gamma new tokens of this round, behind whatever is pending
        base = L + (len(pending) if post else 0)
        fresh = [inverse_cdf(q[base + j], float(u_draft[r, j])) for j in range(gamma)]
        verify = pending if post else fresh[:1]
        nv = len(verify)
        res = spec_accept(tl[L:L + nv + 1], dl[L:L + nv], np.asarray(verify, dtype=np.int64),
                          np.concatenate([np.asarray(u_accept[r, :nv], dtype=np.float32),
                                          np.asarray(u_resample[r:r + 1], dtype=np.float32)]), temperature)
        n = int(res["n_accept"])
        rec = s.advance(n)
        rec["start"] = L
        assert rec["target_ctx"] == L and rec["draft_ctx"] == base      # the token lists and the schedule agree
        tokens.extend(int(x) for x in verify[:n])
        if n < nv:
            tokens.append(int(res["out_tokens"][n]))          # the replacement token
            pending = []                                      # rollback: the draft keeps the committed prefix only
        else:
            pending = fresh if post else fresh[1:]            # no bonus token: the draft has moved on
        assert rec["draft_keep"] == len(tokens) + len(pending)
        r += 1
    return dict(tokens=np.asarray(tokens[:K], dtype=np.int32), rounds=r, log=s.log)
