"""The selection entry point for callers that cannot allocate device memory
(pvlm_uvprune_select_static) against the workspace-taking entry point.

Collected last on purpose: a run that stops at the first failure has then already
executed every other test.  It must pass alone in a fresh process and after the rest."""
import numpy as np
import pytest
import torch

from oracle.uvprune import score_fp32, select_topk
from paper_2603_19610_b200 import binding

pytestmark = pytest.mark.gpu


def _case(m, k, v0, seed, ties):
    rng = np.random.default_rng(seed)
    cur = rng.random(v0 + m + 3).astype(np.float32)
    ref = rng.random(v0 + m + 3).astype(np.float32)
    if ties:                                     # coarse values: many equal scores, tie rule matters
        cur = (np.round(cur * 16) / 16).astype(np.float32)
        ref = (np.round(ref * 16) / 16).astype(np.float32)
    return torch.from_numpy(cur).cuda(), torch.from_numpy(ref).cuda()


def test_static_scratch_select_matches_workspace_select_twice_in_a_row():
    # two calls in a row share the built-in buffer: the second is smaller, so keys of the
    # first call remain behind it in the buffer and must not influence the result
    cases = [(131072, 6553, 0, 1, False), (30720, 3072, 5, 2, True)]
    for m, k, v0, seed, ties in cases:
        cur, ref = _case(m, k, v0, seed, ties)
        want_idx, want_score, _, _ = binding.uvprune_select_gather(cur, ref, v0, m, k, want_score=True)
        got_idx = torch.full((k,), -7, dtype=torch.int32, device="cuda")      # outputs are the caller's
        got_score = torch.zeros(m, dtype=torch.float32, device="cuda")
        binding.uvprune_select_static(cur, ref, v0, m, k, got_idx, got_score)
        torch.cuda.synchronize()
        assert torch.equal(got_idx, want_idx)                                  # indices: bit-exact
        assert torch.equal(got_score, want_score)
        # and both against the CPU oracle (score bits, kept indices)
        s_ref = score_fp32(cur.cpu().numpy(), ref.cpu().numpy(), v0, m)
        assert (got_score.cpu().numpy().view(np.uint32) == s_ref.view(np.uint32)).all()
        np.testing.assert_array_equal(got_idx.cpu().numpy(), select_topk(s_ref, k))
    # raw-signal mode (no reference layer) and the empty selection
    cur, _ = _case(1000, 10, 0, 3, True)
    want_idx, _, _, _ = binding.uvprune_select_gather(cur, None, 0, 1000, 10)
    got_idx = torch.empty(10, dtype=torch.int32, device="cuda")
    binding.uvprune_select_static(cur, None, 0, 1000, 10, got_idx)
    torch.cuda.synchronize()
    assert torch.equal(got_idx, want_idx)
    np.testing.assert_array_equal(got_idx.cpu().numpy(), select_topk(cur.cpu().numpy()[:1000], 10))
    binding.uvprune_select_static(cur, None, 0, 1000, 0, torch.empty(0, dtype=torch.int32, device="cuda"))


def test_static_scratch_select_rejects_oversize_before_launching():
    m = binding.SELECT_STATIC_MAX_M + 1
    cur = torch.zeros(m, dtype=torch.float32, device="cuda")
    out = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.PvlmError) as e:
        binding.uvprune_select_static(cur, None, 0, m, 4, out)
    assert e.value.status == 5
    torch.cuda.synchronize()
    assert (out == -1).all()
