"""Parity of pvlm_acceptance_rate (token-wise acceptance of a given text) with the oracle."""
import numpy as np
import pytest
import torch

from oracle.accept import tokenwise_acceptance
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import assert_rel_close

pytestmark = pytest.mark.gpu


def run_case(N, V, sigma, seed, temperature=1.0, stride_pad=0):
    rng = np.random.default_rng(seed)
    tl = (1.5 * rng.standard_normal((N, V))).astype(np.float32)
    dl = (tl + sigma * rng.standard_normal((N, V))).astype(np.float32)
    x = wl.gumbel_draft_tokens(dl, rng) if N else np.zeros(0, np.int32)
    u = wl.unit_uniforms(rng, N)
    ref = tokenwise_acceptance(tl, dl, x, u, temperature)
    dev = torch.device("cuda")
    if stride_pad:
        t_d = torch.zeros((N, V + stride_pad), device=dev)[:, :V]
        d_d = torch.zeros((N, V + stride_pad), device=dev)[:, :V]
        t_d.copy_(torch.from_numpy(tl)); d_d.copy_(torch.from_numpy(dl))
    else:
        t_d, d_d = torch.from_numpy(tl).to(dev), torch.from_numpy(dl).to(dev)
    out = binding.acceptance_rate(t_d, d_d, torch.from_numpy(x.astype(np.int32)).to(dev), torch.from_numpy(u).to(dev), temperature)
    acc = out["accepted"].cpu().numpy().astype(bool)
    if N:
        assert_rel_close(out["p_tok"].cpu().numpy(), ref["p_tok"], 1e-4, "p_tok")
        assert_rel_close(out["q_tok"].cpu().numpy(), ref["q_tok"], 1e-4, "q_tok")
    diff = np.flatnonzero(acc != ref["accepted"])
    for n in diff:                      # only a test sitting on the decision boundary may differ
        assert abs(float(u[n]) * ref["q_tok"][n] - ref["p_tok"][n]) <= 1e-4 * ref["p_tok"][n], n
    assert diff.size <= max(1, N // 1000)
    assert int(out["n_accepted"].item()) == int(acc.sum())
    return out, ref


@pytest.mark.parametrize("N,V,sigma,seed", [(1, 1, 0.5, 1), (7, 17, 1.0, 2), (33, 4099, 0.7, 3), (300, 2048, 0.4, 4),
                                             (64, 152064, 0.3, 5), (0, 100, 0.5, 6), (1000, 333, 1.5, 7)])
def test_matches_oracle(N, V, sigma, seed):
    run_case(N, V, sigma, seed)


def test_temperature_padded_rows_and_unaligned_stride():
    run_case(50, 5000, 0.6, 11, temperature=0.7)
    run_case(50, 5000, 0.6, 12, stride_pad=4)         # 16-byte path with a padded stride
    run_case(50, 5001, 0.6, 13, stride_pad=2)         # odd stride: scalar path


def test_degenerate_rows():
    dev = torch.device("cuda")
    N, V = 6, 300
    rng = np.random.default_rng(3)
    tl = rng.standard_normal((N, V)).astype(np.float32)
    x = rng.integers(0, V, N).astype(np.int32)
    u = wl.unit_uniforms(rng, N)
    same = binding.acceptance_rate(torch.from_numpy(tl).to(dev), torch.from_numpy(tl).to(dev), torch.from_numpy(x).to(dev),
                                   torch.from_numpy(u).to(dev))
    assert int(same["n_accepted"].item()) == N                        # p = q: u * q < p for every u < 1
    tl2 = tl.copy(); tl2[np.arange(N), x] = -np.inf                    # outside the target's support
    none = binding.acceptance_rate(torch.from_numpy(tl2).to(dev), torch.from_numpy(tl).to(dev), torch.from_numpy(x).to(dev),
                                   torch.from_numpy(u).to(dev))
    assert int(none["n_accepted"].item()) == 0
    bad = x.copy(); bad[0] = -1; bad[1] = V
    o = binding.acceptance_rate(torch.from_numpy(tl).to(dev), torch.from_numpy(tl).to(dev), torch.from_numpy(bad).to(dev),
                                torch.from_numpy(u).to(dev))
    assert o["accepted"].cpu().tolist() == [0, 0, 1, 1, 1, 1]
