"""End to end: verify attention -> mass -> UV-Prune -> gather -> accept on the five
workload configurations, GPU against oracle, with the tolerance bands for decisions that
floating point can flip; the whole-step C-ABI entry with host buffers; two streams."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle.accept import spec_accept as oracle_accept
from oracle.attention import verify_attn as oracle_attn
from oracle.uvprune import gather_rows, score_fp32, select_topk
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import assert_o_close, assert_rel_close, bf16_cuda, bits_of

pytestmark = pytest.mark.gpu


def layers_for(cfg):
    """(reference layer inputs, current layer inputs) of a config."""
    if cfg.n_layers > 1:
        return wl.attn_layer(cfg, cfg.ref_layer), wl.attn_layer(cfg, cfg.cur_layer)
    return wl.attn_layer(cfg, 0, role="ref"), wl.attn_layer(cfg, 0)


@pytest.mark.parametrize("cid", [0, 1, 2, 3, 4])
def test_config_end_to_end(cid):
    cfg = wl.CONFIGS[cid]
    ref_in, cur_in = layers_for(cfg)
    # ---- GPU: both mass layers in one batched launch, then prune (2-layer cache), then accept
    q = torch.stack([bf16_cuda(ref_in[0]), bf16_cuda(cur_in[0])])
    k = torch.stack([bf16_cuda(ref_in[1]), bf16_cuda(cur_in[1])])
    v = torch.stack([bf16_cuda(ref_in[2]), bf16_cuda(cur_in[2])])
    o, lse, mass = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True, mass_layers=[0, 1])
    kept, score, dk, dv = binding.uvprune_select_gather(mass[1], mass[0], 0, cfg.m, cfg.k_keep, k, v, want_score=True)
    tl, dl, tok, u = wl.accept_inputs(cfg)
    acc = binding.spec_accept(torch.from_numpy(tl).cuda(), torch.from_numpy(dl).cuda(),
                              torch.from_numpy(tok).cuda(), torch.from_numpy(u).cuda())
    torch.cuda.synchronize()

    # ---- oracle
    O_ref, L_ref, M_ref = oracle_attn(*ref_in, cfg.n_ctx)
    O_cur, L_cur, M_cur = oracle_attn(*cur_in, cfg.n_ctx)
    assert_o_close(o[0], O_ref)
    assert_o_close(o[1], O_cur)
    assert_rel_close(mass[0].cpu().numpy(), M_ref, what="mass(ref)")
    assert_rel_close(mass[1].cpu().numpy(), M_cur, what="mass(cur)")
    assert abs(float(mass[1].double().sum()) - cfg.Hq * cfg.R) < 1e-4 * cfg.Hq * cfg.R

    # kept indices are bit-exact when computed from the GPU's own fp32 masses ...
    g_cur, g_ref = mass[1].cpu().numpy(), mass[0].cpu().numpy()
    np.testing.assert_array_equal(kept.cpu().numpy(), select_topk(score_fp32(g_cur, g_ref, 0, cfg.m), cfg.k_keep))
    np.testing.assert_array_equal(score.cpu().numpy(), score_fp32(g_cur, g_ref, 0, cfg.m))
    # ... bit-exact from the ORACLE's fp32 scores through the scores-only entry point ...
    s_or = score_fp32(M_cur.astype(np.float32), M_ref.astype(np.float32), 0, cfg.m)
    idx_or = select_topk(s_or, cfg.k_keep)
    np.testing.assert_array_equal(binding.select_from_scores(torch.from_numpy(s_or).cuda(), cfg.k_keep).cpu().numpy(), idx_or)
    # ... and end to end may differ from the oracle's only where a score sits within 1e-4 relative of the k-th score.
    # A score is a difference of two masses, so where it is much smaller than they are the masses' own error
    # (measured in this run as eps, itself asserted <= 1e-4 above) can exceed that band: an index outside the band
    # must lie within the cancellation bound eps * (cur + ref) of both scores involved.  Each is printed.
    diff = np.setxor1d(kept.cpu().numpy(), idx_or)
    order = np.argsort(-s_or, kind="stable")
    i_tau = int(order[cfg.k_keep - 1])
    tau = float(s_or[i_tau])
    eps = max(float(np.abs(g_cur - M_cur).max() / np.abs(M_cur).max()), float(np.abs(g_ref - M_ref).max() / np.abs(M_ref).max()),
              float((np.abs(g_cur - M_cur) / np.abs(M_cur)).max()), float((np.abs(g_ref - M_ref) / np.abs(M_ref)).max()))
    for i in diff:
        gap = abs(float(s_or[i]) - tau)
        band = 1e-4 * max(abs(float(s_or[i])), abs(tau), 1e-30)
        if gap > band:
            bound = eps * float(M_cur[i] + M_ref[i] + M_cur[i_tau] + M_ref[i_tau])
            print(f"config {cid}: index {i} outside the relative band: |s - tau| = {gap:.3e}, band {band:.3e}, "
                  f"cancellation bound {bound:.3e} (eps {eps:.2e})")
            assert gap <= bound, (i, s_or[i], tau, gap, band, bound)
    assert diff.size <= max(4, cfg.k_keep // 100)

    # gather is byte exact for the indices the GPU selected
    idx = kept.cpu().numpy()
    src_k = np.stack([ref_in[1], cur_in[1]])
    src_v = np.stack([ref_in[2], cur_in[2]])
    assert bits_of(dk).tobytes() == gather_rows(src_k, 0, cfg.m, idx).tobytes()
    assert bits_of(dv).tobytes() == gather_rows(src_v, 0, cfg.m, idx).tobytes()
    assert dk.shape[1] == cfg.T - cfg.m + cfg.k_keep

    # accept / resample
    r = oracle_accept(tl, dl, tok, u)
    # accepted length bit-exact from the ORACLE's fp32 probabilities through the probabilities-only entry point
    n_from_oracle = binding.accept_from_probs(torch.from_numpy(r["p_tok"]).cuda(), torch.from_numpy(r["q_tok"]).cuda(),
                                              torch.from_numpy(u).cuda())
    assert int(n_from_oracle) == r["n_accept"]
    n_g = int(acc["n_accept"])
    if n_g != r["n_accept"]:
        t = min(n_g, r["n_accept"])
        assert abs(float(u[t]) - float(r["p"][t, tok[t]] / r["q"][t, tok[t]])) <= 1e-5
    else:
        np.testing.assert_array_equal(acc["out_tokens"].cpu().numpy()[:n_g], tok[:n_g])
        assert acc["out_tokens"].cpu().numpy()[n_g] == r["out_tokens"][n_g]


def test_verify_step_host_buffers_config0():
    """The single-call step with host inputs/outputs gives the same results as the three calls."""
    cfg = wl.CONFIGS[0]
    ref_in, cur_in = layers_for(cfg)
    dev = torch.device("cuda", 0)
    q = torch.stack([bf16_cuda(ref_in[0]), bf16_cuda(cur_in[0])])
    k = torch.stack([bf16_cuda(ref_in[1]), bf16_cuda(cur_in[1])])
    v = torch.stack([bf16_cuda(ref_in[2]), bf16_cuda(cur_in[2])])
    tl, dl, tok, u = wl.accept_inputs(cfg)
    # expected: separate calls
    o_e, lse_e, mass_e = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
    kept_e, _, dk_e, dv_e = binding.uvprune_select_gather(mass_e[1], mass_e[0], 0, cfg.m, cfg.k_keep, k, v)
    acc_e = binding.spec_accept(torch.from_numpy(tl).cuda(), torch.from_numpy(dl).cuda(),
                                torch.from_numpy(tok).cuda(), torch.from_numpy(u).cuda())
    torch.cuda.synchronize()
    # step call: device buffers start zeroed / scrambled, inputs arrive from the host
    q2 = torch.zeros_like(q)
    k2, v2 = k.clone(), v.clone()
    k2[:, cfg.n_ctx:] = 0
    v2[:, cfg.n_ctx:] = 0
    o2 = torch.zeros_like(q)
    mass2 = torch.zeros((2, cfg.T), dtype=torch.float32, device=dev)
    kept2 = torch.zeros(cfg.k_keep, dtype=torch.int32, device=dev)
    S2 = cfg.T - cfg.m + cfg.k_keep
    dk2 = torch.zeros((2, S2, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device=dev)
    dv2 = torch.zeros_like(dk2)
    tl2 = torch.zeros(tl.shape, device=dev)
    dl2 = torch.zeros(dl.shape, device=dev)
    tok2 = torch.zeros(cfg.gamma, dtype=torch.int32, device=dev)
    u2 = torch.zeros(cfg.gamma + 1, device=dev)
    outs = dict(n_accept=torch.zeros(1, dtype=torch.int32, device=dev),
                out_tokens=torch.zeros((1, cfg.gamma + 1), dtype=torch.int32, device=dev))
    pa = binding.attn_params(q2, k2, v2, cfg.n_ctx, o2, None, mass2)
    pp = binding.prune_params(mass2[1], mass2[0], 0, cfg.m, cfg.k_keep, kept2, None, k2, v2, dk2, dv2)
    pc = binding.accept_params(tl2, dl2, tok2, u2, 1.0, outs)
    pin = lambda t: t.contiguous().cpu().pin_memory()
    h_in = dict(h_q=pin(q), h_k_window=pin(k[:, cfg.n_ctx:]), h_v_window=pin(v[:, cfg.n_ctx:]),
                h_target_logits=torch.from_numpy(tl).pin_memory(), h_draft_logits=torch.from_numpy(dl).pin_memory(),
                h_draft_tokens=torch.from_numpy(tok).pin_memory(), h_uniforms=torch.from_numpy(u).pin_memory())
    h_out = dict(h_o=torch.zeros(q.shape, dtype=torch.bfloat16).pin_memory(),
                 h_n_accept=torch.zeros(1, dtype=torch.int32).pin_memory(),
                 h_out_tokens=torch.zeros(cfg.gamma + 1, dtype=torch.int32).pin_memory(),
                 h_kept_idx=torch.zeros(cfg.k_keep, dtype=torch.int32).pin_memory())
    binding.verify_step(pa, pp, pc, host_in=h_in, host_out=h_out)
    torch.cuda.synchronize()
    first = {k: v.clone() for k, v in h_out.items()}
    # the same step with the accept-input upload and the o download overlapped on a copy stream
    for host_t in h_out.values():
        host_t.zero_()
    tl2.zero_(); dl2.zero_(); q2.zero_(); o2.zero_()
    dk2.zero_(); dv2.zero_(); kept2.zero_(); mass2.zero_()   # everything the step writes must be written again
    outs["n_accept"].fill_(-7); outs["out_tokens"].fill_(-7)
    cs, ea, eb = torch.cuda.Stream(), torch.cuda.Event(), torch.cuda.Event()
    ea.record(); eb.record()
    torch.cuda.synchronize()
    binding.verify_step(pa, pp, pc, host_in=h_in, host_out=h_out, overlap=(cs, ea, eb))
    torch.cuda.current_stream().synchronize()              # the caller's stream alone
    for name in first:
        assert torch.equal(first[name], h_out[name]), name
    assert torch.equal(h_out["h_o"], o_e.cpu())
    assert torch.equal(k2, k) and torch.equal(v2, v)                     # window rows landed in the cache
    assert torch.equal(h_out["h_kept_idx"], kept_e.cpu())
    assert torch.equal(dk2, dk_e) and torch.equal(dv2, dv_e)
    assert int(h_out["h_n_accept"]) == int(acc_e["n_accept"])
    assert torch.equal(h_out["h_out_tokens"], acc_e["out_tokens"].cpu())


def test_verify_step_host_buffers_head_major_cache():
    """The step call with a head-major cache ([layer][kv_head][token][D]): the window's K/V rows arrive from a host
    buffer laid out [layer][kv_head][R][D], the gather sees layer * kv_head pseudo-layers of D-element rows; results
    equal those of the token-major calls."""
    dev = torch.device("cuda", 0)
    L, R, Hq, Hkv, D, n_ctx, m, k_keep = 3, 5, 8, 2, 128, 700, 600, 150
    T = n_ctx + R
    g = torch.Generator(device=dev); g.manual_seed(8)
    mk = lambda *sh: torch.randn(sh, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q, k, v = mk(L, R, Hq, D), mk(L, T, Hkv, D), mk(L, T, Hkv, D)
    o_e, lse_e, mass_e = binding.verify_attn(q, k, v, n_ctx, want_mass=True, mass_layers=[0, 2])
    kept_e, _, dk_e, dv_e = binding.uvprune_select_gather(mass_e[1], mass_e[0], 0, m, k_keep, k, v)
    torch.cuda.synchronize()
    kb = k.permute(0, 2, 1, 3).contiguous()                      # [L][Hkv][T][D]
    vb = v.permute(0, 2, 1, 3).contiguous()
    h_kw, h_vw = kb[:, :, n_ctx:].contiguous().cpu().pin_memory(), vb[:, :, n_ctx:].contiguous().cpu().pin_memory()
    kb[:, :, n_ctx:] = 0; vb[:, :, n_ctx:] = 0
    q2, o2 = torch.zeros_like(q), torch.zeros_like(q)
    mass2 = torch.zeros_like(mass_e)
    kept2 = torch.zeros(k_keep, dtype=torch.int32, device=dev)
    S2 = T - m + k_keep
    dk2 = torch.zeros((L * Hkv, S2, 1, D), dtype=torch.bfloat16, device=dev)
    dv2 = torch.zeros_like(dk2)
    pa = binding.attn_params(q2, kb.permute(0, 2, 1, 3), vb.permute(0, 2, 1, 3), n_ctx, o2, None, mass2, mass_layers=[0, 2])
    pp = binding.prune_params(mass2[1], mass2[0], 0, m, k_keep, kept2, None, kb.view(L * Hkv, T, 1, D), vb.view(L * Hkv, T, 1, D), dk2, dv2)
    h_in = dict(h_q=q.cpu().pin_memory(), h_k_window=h_kw, h_v_window=h_vw)
    h_out = dict(h_o=torch.zeros(q.shape, dtype=torch.bfloat16).pin_memory(), h_kept_idx=torch.zeros(k_keep, dtype=torch.int32).pin_memory())
    cs, ea, eb = torch.cuda.Stream(), torch.cuda.Event(), torch.cuda.Event()
    ea.record(); eb.record()
    torch.cuda.synchronize()
    for overlap in (None, (cs, ea, eb)):
        o2.zero_(); dk2.zero_(); dv2.zero_(); kept2.zero_(); kb[:, :, n_ctx:] = 0; vb[:, :, n_ctx:] = 0
        binding.verify_step(pa, pp, None, host_in=h_in, host_out=h_out, device=dev, overlap=overlap)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(kb.permute(0, 2, 1, 3), k) and torch.equal(vb.permute(0, 2, 1, 3), v)     # window rows landed
        assert torch.equal(h_out["h_o"], o_e.cpu()) and torch.equal(h_out["h_kept_idx"], kept_e.cpu())
        # compacted cache: [L * Hkv][S2][D] head-major against the token-major result [L][S2][Hkv][D]
        assert torch.equal(dk2.view(L, Hkv, S2, D).permute(0, 2, 1, 3), dk_e)
        assert torch.equal(dv2.view(L, Hkv, S2, D).permute(0, 2, 1, 3), dv_e)


def test_verify_step_overlap_mode_splits_the_gather_correctly():
    """Overlap mode copies the rows outside the visual span on the second stream and the selected rows on the
    main stream: with rows before AND after the visual span the compacted caches must equal the one-call result."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(77)
    L, S, Hkv, D, v0, m, k = 3, 1029, 4, 128, 5, 896, 224
    src_k = torch.randn((L, S, Hkv, D), device=dev).to(torch.bfloat16)
    src_v = torch.randn((L, S, Hkv, D), device=dev).to(torch.bfloat16)
    cur = torch.from_numpy(rng.random(S).astype(np.float32)).to(dev)
    ref = torch.from_numpy(rng.random(S).astype(np.float32)).to(dev)
    kept_e, _, dk_e, dv_e = binding.uvprune_select_gather(cur, ref, v0, m, k, src_k, src_v)
    kept = torch.zeros(k, dtype=torch.int32, device=dev)
    dk = torch.zeros((L, S - m + k, Hkv, D), dtype=torch.bfloat16, device=dev)
    dv = torch.zeros_like(dk)
    pp = binding.prune_params(cur, ref, v0, m, k, kept, None, src_k, src_v, dk, dv)
    cs, ea, eb = torch.cuda.Stream(), torch.cuda.Event(), torch.cuda.Event()
    ea.record(); eb.record()
    torch.cuda.synchronize()
    for _ in range(2):                                            # twice: events and streams are reused across steps
        dk.zero_(); dv.zero_(); kept.zero_()
        binding.verify_step(None, pp, None, device=dev, overlap=(cs, ea, eb))
        torch.cuda.current_stream().synchronize()
        assert torch.equal(kept, kept_e) and torch.equal(dk, dk_e) and torch.equal(dv, dv_e)


def test_draft_and_verify_streams_run_concurrently_and_agree():
    """Draft-side decode attention (R = 1 over the compacted cache) on one stream while the
    verify pass runs on another: each stream has its own workspace; results equal the
    serial ones bit for bit."""
    cfg = wl.CONFIGS[0]
    q, k, v = (bf16_cuda(x) for x in wl.attn_layer(cfg, 0))
    qd, kd, vd = (bf16_cuda(x) for x in wl.make_qkv(8, 2, 64, 1, 400, sink=False, seed=77))
    o_s, lse_s, mass_s = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
    od_s, lsed_s, _ = binding.verify_attn(qd, kd, vd, 399)
    torch.cuda.synchronize()
    sv, sd = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(5):
        with torch.cuda.stream(sv):
            o_c, lse_c, mass_c = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
        with torch.cuda.stream(sd):
            od_c, lsed_c, _ = binding.verify_attn(qd, kd, vd, 399)
    torch.cuda.synchronize()
    assert torch.equal(o_c, o_s) and torch.equal(mass_c, mass_s) and torch.equal(lse_c, lse_s)
    assert torch.equal(od_c, od_s) and torch.equal(lsed_c, lsed_s)


@pytest.mark.parametrize("cid", [0, 1])
def test_the_three_calls_replay_from_a_cuda_graph(cid):
    """pvlm_verify_attn -> pvlm_uvprune_select_gather -> pvlm_spec_accept on device-resident inputs
    make no host round trip, so a stream capture records them; the replayed graph, fed new contents in
    the same buffers, gives what the direct calls give, bit for bit, and matches the oracle."""
    cfg = wl.CONFIGS[cid]
    ref_in, cur_in = layers_for(cfg)
    q = torch.stack([bf16_cuda(ref_in[0]), bf16_cuda(cur_in[0])])
    k = torch.stack([bf16_cuda(ref_in[1]), bf16_cuda(cur_in[1])])
    v = torch.stack([bf16_cuda(ref_in[2]), bf16_cuda(cur_in[2])])
    tl, dl, tok, u = (torch.from_numpy(x).cuda() for x in wl.accept_inputs(cfg))

    def run():
        o, lse, mass = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True, mass_layers=[0, 1])
        kept, _, dk, dv = binding.uvprune_select_gather(mass[1], mass[0], 0, cfg.m, cfg.k_keep, k, v)
        acc = binding.spec_accept(tl, dl, tok, u)
        return o, lse, mass, kept, dk, dv, acc["n_accept"], acc["out_tokens"]

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):                       # warm-up: workspaces and function attributes exist before the capture
        run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        outs = run()
    for rnd in range(2):
        if rnd == 1:                                 # new contents, same buffers: the window rows of another seed, swapped logits
            q2, k2, v2 = (bf16_cuda(x) for x in wl.make_qkv(cfg.Hq, cfg.Hkv, cfg.D, cfg.R, cfg.T, sink=True, seed=4242 + cid))
            q[1].copy_(q2); k[1].copy_(k2); v[1].copy_(v2)
            u.copy_(torch.flip(u, [0]))
        for t in outs:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        got = [t.clone() for t in outs]
        want = run()
        torch.cuda.synchronize()
        for a, b in zip(got, want):
            assert torch.equal(a, b)
    # the second replay against the oracle
    O, L, M = oracle_attn(bits_of(q[1]), bits_of(k[1]), bits_of(v[1]), cfg.n_ctx)
    assert_o_close(got[0][1], O)
    assert_rel_close(got[2][1].cpu().numpy(), M, what="mass")
    r = oracle_accept(tl.cpu().numpy(), dl.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy())
    assert int(got[6]) == r["n_accept"]


def test_step_call_reports_the_attention_status_word():
    """The status word of the attention stage comes back with the step's other host results.  No GPU wait is made
    to expire: the word is poisoned from the host after a clean call and read back through a step that runs no stage."""
    qb, kb, vb = wl.make_qkv(8, 2, 128, 3, 303, sink=False, seed=3)
    q, k, v = bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb)
    pa = binding.attn_params(q, k, v, 300, torch.empty_like(q), None, None)
    status = torch.full((1,), 77, dtype=torch.int32).pin_memory()
    binding.verify_step(pa, None, None, host_out=dict(h_attn_status=status))
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    need = binding.lib().pvlm_verify_attn_workspace_bytes(C.byref(pa))
    pa._keep[6][need - 8192:need - 8188] = torch.tensor([1, 0, 0, 0], dtype=torch.uint8, device="cuda")
    sp = binding.StepParams()
    sp.attn = pa
    sp.h_attn_status = C.c_void_p(status.data_ptr())
    assert binding.lib().pvlm_verify_step(C.byref(sp), C.c_void_p(torch.cuda.current_stream().cuda_stream)) == 0
    torch.cuda.synchronize()
    assert int(status[0]) == 1
    binding.verify_step(pa, None, None, host_out=dict(h_attn_status=status))          # a new attention call clears it
    torch.cuda.synchronize()
    assert int(status[0]) == 0


def test_step_call_with_an_idle_side_stream_is_capturable():
    """Overlap handles given but nothing for the side stream to do (attention only, select without a gather):
    the side stream is still joined back, so a stream capture of the call closes and replays."""
    cfg = wl.CONFIGS[0]
    ref_in, cur_in = layers_for(cfg)
    q = torch.stack([bf16_cuda(ref_in[0]), bf16_cuda(cur_in[0])])
    k = torch.stack([bf16_cuda(ref_in[1]), bf16_cuda(cur_in[1])])
    v = torch.stack([bf16_cuda(ref_in[2]), bf16_cuda(cur_in[2])])
    o = torch.empty_like(q)
    mass = torch.empty((2, cfg.T), dtype=torch.float32, device="cuda")
    kept = torch.empty(cfg.k_keep, dtype=torch.int32, device="cuda")
    s, side = torch.cuda.Stream(), torch.cuda.Stream()
    evs = [torch.cuda.Event(), torch.cuda.Event()]
    for e in evs:
        e.record()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        pa = binding.attn_params(q, k, v, cfg.n_ctx, o, None, mass, mass_layers=[0, 1])
        pp = binding.prune_params(mass[1], mass[0], 0, cfg.m, cfg.k_keep, kept, None, None, None, None, None)
        for blocks in ((pa, None), (pa, pp)):
            binding.verify_step(blocks[0], blocks[1], None, overlap=(side, evs[0], evs[1]))      # warm-up, direct
            torch.cuda.synchronize()
            want = (o.clone(), mass.clone(), kept.clone())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                binding.verify_step(blocks[0], blocks[1], None, overlap=(side, evs[0], evs[1]))
            o.zero_(); mass.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(o, want[0]) and torch.equal(mass, want[1]) and torch.equal(kept, want[2])


def test_similarity_and_acceptance_rate_replay_from_a_cuda_graph():
    """The hidden-state criterion (three kernels chained by programmatic dependent launch) and the acceptance-rate
    pass are capturable too: a replay equals the direct calls bit for bit."""
    dev = torch.device("cuda")
    g0 = torch.Generator(device="cpu").manual_seed(31)
    hidden = torch.randn((700 + 90, 1024), generator=g0).to(torch.bfloat16).to(dev)
    N, V = 40, 3001
    tl = torch.randn((N, V), generator=g0).mul_(3).to(dev)
    dl = (tl.cpu() + 0.5 * torch.randn((N, V), generator=g0)).to(dev)
    tok = torch.randint(0, V, (N,), generator=g0, dtype=torch.int32).to(dev)
    u = torch.rand(N, generator=g0).to(dev)

    def run():
        sim = binding.uvprune_similarity(hidden, 0, 700, 700, 90)
        r = binding.acceptance_rate(tl, dl, tok, u)
        return sim, r["accepted"], r["n_accepted"], r["p_tok"], r["q_tok"]

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        outs = run()
    hidden.copy_(torch.randn(hidden.shape, generator=g0).to(torch.bfloat16))
    u.copy_(torch.rand(N, generator=g0))
    for t in outs:
        t.zero_()
    g.replay()
    torch.cuda.synchronize()
    want = run()
    torch.cuda.synchronize()
    for a, b in zip(outs, want):
        assert torch.equal(a, b)
    assert float(outs[0].abs().max()) > 0


def test_step_call_rejects_bad_arguments_before_queuing_anything():
    """A bad argument in any stage of pvlm_verify_step is reported before the call touches either stream:
    the second stream is not left waiting on a half-built step, and the next (valid) call is unaffected."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(5)
    L, S, Hkv, D, v0, m, k = 2, 500, 2, 64, 3, 400, 100
    src_k = torch.randn((L, S, Hkv, D), device=dev).to(torch.bfloat16)
    src_v = torch.randn((L, S, Hkv, D), device=dev).to(torch.bfloat16)
    cur = torch.from_numpy(rng.random(S).astype(np.float32)).to(dev)
    kept_e, _, dk_e, dv_e = binding.uvprune_select_gather(cur, None, v0, m, k, src_k, src_v)
    kept = torch.zeros(k, dtype=torch.int32, device=dev)
    dk = torch.zeros((L, S - m + k, Hkv, D), dtype=torch.bfloat16, device=dev)
    dv = torch.zeros_like(dk)
    pp = binding.prune_params(cur, None, v0, m, k, kept, None, src_k, src_v, dk, dv)
    cs, ea, eb = torch.cuda.Stream(), torch.cuda.Event(), torch.cuda.Event()
    ea.record(); eb.record()
    torch.cuda.synchronize()
    pp.k = m + 1                                              # more kept tokens than visual tokens
    with pytest.raises(binding.PvlmError) as err:
        binding.verify_step(None, pp, None, device=dev, overlap=(cs, ea, eb))
    assert "INVALID_ARG" in str(err.value)
    assert cs.query() and torch.cuda.current_stream().query()  # nothing was queued
    pp.k = k
    binding.verify_step(None, pp, None, device=dev, overlap=(cs, ea, eb))
    torch.cuda.current_stream().synchronize()
    assert torch.equal(kept, kept_e) and torch.equal(dk, dk_e) and torch.equal(dv, dv_e)


def test_config2_full_step_in_the_bench_configuration():
    """The step bench.py times, at full size: ONE pvlm_verify_step call in overlap mode over all 64 layers of
    config 2 (head-major cache; the gather sees layer x kv_head pseudo-layers of 256-byte rows).  Selection is
    checked against the oracle's rule on the call's own masses, every gathered byte against torch indexing, the
    current layer's attention and the accept outcome against the oracle."""
    cfg = wl.CONFIGS[2]
    L, T, R, Hkv, D = cfg.n_layers, cfg.T, cfg.R, cfg.Hkv, cfg.D
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev)
    g.manual_seed(123)
    k_base = torch.empty((L, Hkv, T, D), dtype=torch.bfloat16, device=dev)
    v_base = torch.empty_like(k_base)
    q = torch.empty((L, R, cfg.Hq, D), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        k_base[l].copy_(torch.randn((Hkv, T, D), generator=g, device=dev))
        v_base[l].copy_(torch.randn((Hkv, T, D), generator=g, device=dev))
        q[l].copy_(torch.randn((R, cfg.Hq, D), generator=g, device=dev))
    k, v = k_base.permute(0, 2, 1, 3), v_base.permute(0, 2, 1, 3)
    host = {l: wl.attn_layer(cfg, l) for l in (cfg.ref_layer, cfg.cur_layer)}
    for l, (qb, kb, vb) in host.items():
        q[l].copy_(bf16_cuda(qb)); k[l].copy_(bf16_cuda(kb)); v[l].copy_(bf16_cuda(vb))
    o = torch.empty_like(q)
    lse = torch.empty((L, cfg.Hq, R), dtype=torch.float32, device=dev)
    mass = torch.empty((2, T), dtype=torch.float32, device=dev)
    S2 = T - cfg.m + cfg.k_keep
    src_k, src_v = k_base.view(L * Hkv, T, 1, D), v_base.view(L * Hkv, T, 1, D)
    dk = torch.zeros((L * Hkv, S2, 1, D), dtype=torch.bfloat16, device=dev)
    dv = torch.zeros_like(dk)
    kept = torch.zeros(cfg.k_keep, dtype=torch.int32, device=dev)
    tl, dl, tok, u = wl.accept_inputs(cfg)
    outs = dict(n_accept=torch.zeros(1, dtype=torch.int32, device=dev),
                out_tokens=torch.zeros((1, cfg.gamma + 1), dtype=torch.int32, device=dev),
                p_tok=torch.zeros((1, cfg.gamma), dtype=torch.float32, device=dev),
                q_tok=torch.zeros((1, cfg.gamma), dtype=torch.float32, device=dev))
    pa = binding.attn_params(q, k, v, cfg.n_ctx, o, lse, mass, mass_layers=[cfg.ref_layer, cfg.cur_layer])
    pp = binding.prune_params(mass[1], mass[0], 0, cfg.m, cfg.k_keep, kept, None, src_k, src_v, dk, dv)
    pc = binding.accept_params(*(torch.from_numpy(x).to(dev) for x in (tl, dl, tok, u)), 1.0, outs)
    cs, ea, eb = torch.cuda.Stream(device=dev), torch.cuda.Event(), torch.cuda.Event()
    ea.record(); eb.record()
    torch.cuda.synchronize()
    for _ in range(2):
        binding.verify_step(pa, pp, pc, device=dev, overlap=(cs, ea, eb))
    torch.cuda.current_stream().synchronize()
    assert binding.lib().pvlm_verify_attn_check(C.byref(pa), None) == 0
    # selection: the oracle's rule on the call's own fp32 masses, bit for bit
    g_ref, g_cur = mass[0].cpu().numpy(), mass[1].cpu().numpy()
    idx = select_topk(score_fp32(g_cur, g_ref, 0, cfg.m), cfg.k_keep)
    np.testing.assert_array_equal(kept.cpu().numpy(), idx)
    # gather: every byte of both compacted caches (torch indexing as the independent routine)
    rows = torch.cat([torch.from_numpy(idx.astype(np.int64)).to(dev), torch.arange(cfg.m, T, device=dev)])
    assert torch.equal(dk, src_k.index_select(1, rows)) and torch.equal(dv, src_v.index_select(1, rows))
    # the current layer's attention and the accept outcome against the oracle
    O, Lr, M = oracle_attn(*host[cfg.cur_layer], cfg.n_ctx)
    assert_o_close(o[cfg.cur_layer], O)
    assert np.abs(lse[cfg.cur_layer].cpu().numpy() - Lr).max() <= 1e-4
    assert_rel_close(g_cur, M, what="mass")
    r = oracle_accept(tl, dl, tok, u)
    assert int(outs["n_accept"].item()) == r["n_accept"]
    assert (outs["out_tokens"].cpu().numpy().ravel()[:r["n_accept"] + 1] == r["out_tokens"][:r["n_accept"] + 1]).all()
