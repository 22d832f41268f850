"""Oracle: vocab softmax, the lossless accept/reject rule and residual
resampling (Sec. 2.2), plus the window-size rule (Eq. 6).

A drafted token x_t is accepted with probability min{1, p_t(x_t)/q_t(x_t)};
at the first rejection a replacement is drawn from norm(max(0, p - q)); if
every drafted token is accepted one more token is drawn from the target's
next-position distribution.  The output is then distributed exactly as the
target model's.

Readings where the paper is silent: temperature 1 unless given; accept test
`u < p/q` taken strictly with u in [0,1) and evaluated division-free in fp32
as `u * q32 < p32`; the replacement / bonus token is drawn by inverse CDF in
vocabulary order with one uniform (smallest j whose cumulative weight exceeds
u * Z); gamma accept uniforms then one sampling uniform per step.
"""
from __future__ import annotations

import numpy as np


def softmax64(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """Row-wise softmax in fp64 with max subtraction."""
    x = np.asarray(logits, dtype=np.float64)
    if temperature not in (0.0, 1.0):
        x = x / temperature
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=-1, keepdims=True)


def lse64(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    x = np.asarray(logits, dtype=np.float64)
    if temperature not in (0.0, 1.0):
        x = x / temperature
    M = x.max(axis=-1)
    return M + np.log(np.exp(x - M[..., None]).sum(axis=-1))


def inverse_cdf(w: np.ndarray, u: float) -> int:
    """Smallest j with sum_{i<=j} w_i > u * sum(w); if rounding leaves none,
    the largest j with w_j > 0."""
    c = np.cumsum(w)                                   # sequential, index order
    Z = c[-1]
    j = int(np.searchsorted(c, np.float64(u) * Z, side="right"))
    if j >= w.shape[0]:
        j = int(np.flatnonzero(w > 0)[-1])
    return j


def spec_accept(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0):
    """target_logits fp32 [gamma+1, V], draft_logits fp32 [gamma, V],
    draft_tokens int [gamma], uniforms fp32 [gamma+1].

    Returns dict(n_accept, out_tokens[gamma+1] (-1 padded), p_tok, q_tok (fp32,
    all gamma positions), lse_p, lse_q, p, q (fp64 matrices), ratio_margin)."""
    tl = np.asarray(target_logits, dtype=np.float32)
    dl = np.asarray(draft_logits, dtype=np.float32)
    gamma, V = dl.shape
    assert tl.shape == (gamma + 1, V)
    u = np.asarray(uniforms, dtype=np.float32)
    p = softmax64(tl, temperature)
    q = softmax64(dl, temperature)
    x = np.asarray(draft_tokens, dtype=np.int64)
    p_tok = p[np.arange(gamma), x].astype(np.float32)
    q_tok = q[np.arange(gamma), x].astype(np.float32)
    n = gamma
    for t in range(gamma):
        if not (np.float32(u[t] * q_tok[t]) < p_tok[t]):   # one rounded fp32 multiply, strict compare
            n = t
            break
    if n < gamma:
        w = np.maximum(0.0, p[n] - q[n])
        if w.sum() == 0.0:
            w = p[n]
    else:
        w = p[gamma]
    tok = inverse_cdf(w, float(u[gamma]))
    out = np.full(gamma + 1, -1, dtype=np.int32)
    out[:n] = x[:n]
    out[n] = tok
    return dict(n_accept=n, out_tokens=out, p_tok=p_tok, q_tok=q_tok,
                lse_p=lse64(tl, temperature), lse_q=lse64(dl, temperature), p=p, q=q,
                resample_weights=w)


def window_size(T_p: float, T_q: float) -> float:
    """Eq. 6: the draft window equals the pruned speed ratio c* = T_p / T_q(alpha)."""
    return T_p / T_q


def window_size_rounded(T_p: float, T_q: float, mode: str = "nearest") -> int:
    """Integer window from c* = T_p / T_q.  The paper leaves the rounding direction to the user (down for
    windows that are aggressive relative to the accepted length, up for narrow windows with high accepted
    lengths, Appendix A); the five windows it uses itself equal c* rounded to the nearest integer."""
    import math
    c = window_size(T_p, T_q)
    g = {"nearest": math.floor(c + 0.5), "down": math.floor(c + 1e-9), "up": math.ceil(c - 1e-9)}[mode]
    return max(1, int(g))


def spec_accept_trials(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0):
    """The same rule as `spec_accept`, applied to B independent trials that
    share one set of logits: draft_tokens int [B, gamma], uniforms fp32
    [B, gamma+1].  Returns (n_accept int32 [B], emitted token int32 [B]) where
    the emitted token is the replacement / bonus token of each trial.
    Used for the distributional tests (1e6 trials)."""
    tl = np.asarray(target_logits, dtype=np.float32)
    dl = np.asarray(draft_logits, dtype=np.float32)
    gamma, V = dl.shape
    p = softmax64(tl, temperature)
    q = softmax64(dl, temperature)
    x = np.asarray(draft_tokens, dtype=np.int64)
    u = np.asarray(uniforms, dtype=np.float32)
    B = x.shape[0]
    t_idx = np.arange(gamma)[None, :]
    p_tok = p[t_idx, x].astype(np.float32)
    q_tok = q[t_idx, x].astype(np.float32)
    ok = (u[:, :gamma] * q_tok).astype(np.float32) < p_tok
    n = np.where(ok.all(axis=1), gamma, np.argmin(ok, axis=1)).astype(np.int32)
    # one weight row per possible stopping position
    W = np.empty((gamma + 1, V))
    for t in range(gamma):
        w = np.maximum(0.0, p[t] - q[t])
        W[t] = w if w.sum() != 0.0 else p[t]
    W[gamma] = p[gamma]
    tok = np.empty(B, dtype=np.int32)
    for t in range(gamma + 1):
        sel = np.flatnonzero(n == t)
        if sel.size == 0:
            continue
        c = np.cumsum(W[t])
        j = np.searchsorted(c, u[sel, gamma].astype(np.float64) * c[-1], side="right")
        last = int(np.flatnonzero(W[t] > 0)[-1])
        tok[sel] = np.where(j >= V, last, j)
    return n, tok


def tokenwise_acceptance(target_logits, draft_logits, tokens, uniforms, temperature: float = 1.0):
    """Token-wise speculative sampling of a given text (appendix "Tasks and Metrics": the acceptance
    rate A of a saved output under the full-context target): token x_n, drawn by a model with
    distribution q_n, is accepted iff u_n < p_n(x_n) / q_n(x_n), every position on its own.
    target_logits, draft_logits fp32 [N, V]; tokens int [N]; uniforms fp32 [N].
    Returns dict(accepted bool [N], p_tok, q_tok fp32 [N], rate = mean(accepted)).
    Same strictness and precision as `spec_accept`: u * q32 < p32 in fp32."""
    p = softmax64(np.asarray(target_logits, dtype=np.float32), temperature)
    q = softmax64(np.asarray(draft_logits, dtype=np.float32), temperature)
    x = np.asarray(tokens, dtype=np.int64)
    n = np.arange(x.shape[0])
    p_tok = p[n, x].astype(np.float32)
    q_tok = q[n, x].astype(np.float32)
    u = np.asarray(uniforms, dtype=np.float32)
    accepted = (u * q_tok).astype(np.float32) < p_tok
    return dict(accepted=accepted, p_tok=p_tok, q_tok=q_tok, rate=float(accepted.mean()) if x.size else 0.0)
