"""Parity of pvlm_parallel_decode (Algorithm 1 on two streams) with the pipeline oracle: committed tokens and
the per-round log (mode, verified, accepted, committed, dropped, start, and the three cache lengths: tokens in the
verification's context, in the draft's cache before the round, in the draft's cache after commit / rollback) must be
identical."""
import numpy as np
import pytest
import torch

from oracle.pipeline import parallel_decode as oracle_decode
from paper_2603_19610_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def make_case(V, K, gamma, sigma, seed):
    rng = np.random.default_rng(seed)
    P = K + 2 * gamma + 1
    tl = (1.5 * rng.standard_normal((P, V))).astype(np.float32)
    dl = (tl + sigma * rng.standard_normal((P, V))).astype(np.float32)
    g = np.random.Generator(np.random.Philox(key=seed + 1000))
    ud, ua, ur = wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, (K, gamma)), wl.unit_uniforms(g, K)
    return tl, dl, ud, ua, ur


def gpu_decode(tl, dl, gamma, K, ud, ua, ur, **kw):
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return binding.parallel_decode(d(tl), d(dl), gamma, K, d(ud), d(ua), d(ur), **kw)


def first_token_mismatch_is_a_rounding_band_event(gpu_tokens, ref_tokens, tl, dl, ud, ua, ur, temperature=1.0):
    """Where the library's tokens leave the oracle's, the FIRST differing token must be a draw whose u * Z lies within
    1e-5 * Z of the step of the cumulative weights between the two tokens, with no weight between them (the documented
    band of the fp32-weight / fp64-sum inverse CDF against the fp64 oracle); what follows such a draw may differ freely.
    The weights are those of the position's three possible draws: the draft's q, the residual max(0, p - q), the target's p."""
    from oracle.accept import softmax64
    n = min(len(gpu_tokens), len(ref_tokens))
    bad = np.nonzero(np.asarray(gpu_tokens[:n]) != np.asarray(ref_tokens[:n]))[0]
    assert len(bad) > 0
    i = int(bad[0])
    a, b = sorted((int(gpu_tokens[i]), int(ref_tokens[i])))
    p = softmax64(np.asarray(tl)[i], temperature)
    q = softmax64(np.asarray(dl)[i], temperature)
    us = np.concatenate([np.asarray(x, dtype=np.float64).ravel() for x in (ud, ua, ur)])
    for w in (q, np.maximum(0.0, p - q), p):
        c = np.cumsum(w)
        if w[a + 1:b].sum() == 0.0 and np.abs(us * c[-1] - c[a]).min() <= 1e-5 * c[-1]:
            return True
    return False


def log_rows(log):
    return [[r["mode"], r["verified"], r["accepted"], r["emitted"], r["dropped"], r["start"],
             r["target_ctx"], r["draft_ctx"], r["draft_keep"]] for r in log]


@pytest.mark.parametrize("V,K,gamma,sigma,seed", [(50, 40, 4, 0.8, 3), (1000, 64, 9, 0.5, 7), (4099, 33, 1, 0.7, 11),
                                                   (32000, 24, 5, 0.3, 5), (17, 80, 12, 1.5, 9), (152064, 12, 3, 0.4, 2),
                                                   (300, 200, 64, 0.05, 1), (300, 200, 64, 0.6, 2),      # the widest window
                                                   (1000, 500, 33, 0.2, 3), (5, 1000, 2, 0.3, 4),        # long runs
                                                   # windows whose gamma - 1 pending drafts need MORE accept scratch than
                                                   # the full window (fewer rows, more statistics chunks per row)
                                                   (152064, 16, 7, 0.1, 6), (50000, 16, 13, 0.1, 8), (16384, 20, 13, 0.1, 9)])
def test_tokens_and_round_log_match_the_oracle(V, K, gamma, sigma, seed):
    tl, dl, ud, ua, ur = make_case(V, K, gamma, sigma, seed)
    ref = oracle_decode(tl, dl, gamma, K, ud, ua, ur)
    out = gpu_decode(tl, dl, gamma, K, ud, ua, ur)
    assert out["rounds"] == ref["rounds"]
    assert out["log"].tolist() == log_rows(ref["log"])
    np.testing.assert_array_equal(out["tokens"].numpy(), ref["tokens"])


def test_serial_order_and_attention_payloads_do_not_change_the_tokens():
    V, K, gamma = 2000, 48, 6
    tl, dl, ud, ua, ur = make_case(V, K, gamma, 0.6, 21)
    ref = oracle_decode(tl, dl, gamma, K, ud, ua, ur)
    ser = gpu_decode(tl, dl, gamma, K, ud, ua, ur, serial=True)
    np.testing.assert_array_equal(ser["tokens"].numpy(), ref["tokens"])
    # the two models' attention over their caches: a target context of 3000 tokens, a compacted draft context of 400;
    # every round's calls follow the caches (committed tokens become context, the draft's cache grows and rolls back)
    dev = torch.device("cuda")
    mk = lambda *s: torch.randn(s, device=dev, dtype=torch.float32).to(torch.bfloat16)
    R = gamma + 1
    rows_t, rows_d = 3000 + K + 2 * gamma + 1, 400 + K + 2 * gamma + 1
    qt, kt, vt = mk(2, R, 8, 128), mk(2, rows_t, 2, 128), mk(2, rows_t, 2, 128)
    qd, kd, vd = mk(2, 1, 8, 128), mk(2, rows_d, 2, 128), mk(2, rows_d, 2, 128)
    ws_t = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
    ws_d = torch.empty(64 << 20, dtype=torch.uint8, device=dev)
    pt = binding.attn_params(qt, kt[:, :3000 + R], vt[:, :3000 + R], 3000, torch.empty_like(qt), None, None, workspace=ws_t)
    pd = binding.attn_params(qd, kd[:, :401], vd[:, :401], 400, torch.empty_like(qd), None, None, workspace=ws_d)
    out = gpu_decode(tl, dl, gamma, K, ud, ua, ur, target_attn=pt, draft_attn=pd, want_ms=True)
    np.testing.assert_array_equal(out["tokens"].numpy(), ref["tokens"])
    assert out["log"].tolist() == log_rows(ref["log"])
    assert out["round_ms"].shape[0] == out["rounds"] and float(out["round_ms"].min()) > 0.0


def test_cache_lengths_follow_commit_and_rollback():
    """The logged cache lengths against their definition, round by round: the verification's context is what is
    committed; the draft starts a round with the committed and pending tokens in its cache, ends it with gamma more,
    and keeps either all of them (everything accepted) or the committed prefix alone (a rejection: the replacement
    token is not in the cache yet, it is the next forward's input)."""
    V, K, gamma = 500, 120, 5
    tl, dl, ud, ua, ur = make_case(V, K, gamma, 0.7, 33)
    out = gpu_decode(tl, dl, gamma, K, ud, ua, ur)
    log = out["log"].tolist()
    committed, pending, rollbacks = 0, 0, 0
    for mode, verified, accepted, emitted, dropped, start, t_ctx, d_ctx, d_keep in log:
        assert start == committed == t_ctx
        assert d_ctx == committed + (pending if mode == 1 else 0)
        committed += emitted
        if accepted < verified:
            pending = 0
            rollbacks += 1
            assert d_keep == committed and d_keep < d_ctx + gamma          # the cache was truncated
        else:
            pending = gamma if mode == 1 else gamma - 1
            assert d_keep == committed + pending == d_ctx + gamma          # nothing dropped
    assert rollbacks > 3 and committed >= K


def test_argument_errors():
    V, K, gamma = 64, 8, 3
    tl, dl, ud, ua, ur = make_case(V, K, gamma, 0.5, 1)
    with pytest.raises(binding.PvlmError, match="TOO_LARGE"):
        gpu_decode(tl[:K + gamma], dl[:K + gamma], gamma, K, ud, ua, ur)           # too few positions
    with pytest.raises(binding.PvlmError, match="INVALID_ARG"):
        gpu_decode(tl, dl, gamma, K, ud, ua, ur, draft_stream=torch.cuda.current_stream())   # needs two streams
    with pytest.raises(binding.PvlmError, match="TOO_LARGE"):
        gpu_decode(tl, dl, gamma, K, ud[:2], ua[:2], ur[:2])                       # round tables exhausted
