"""Parity of pvlm_verify_attn (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle.attention import verify_attn as oracle_attn
from paper_2603_19610_b200 import binding, workloads as wl
from helpers import assert_o_close, assert_rel_close, bf16_cuda, bits_of

pytestmark = pytest.mark.gpu


def run_case(qb, kb, vb, n_ctx, scale=0.0):
    o, lse, mass = binding.verify_attn(bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb), n_ctx,
                                       want_lse=True, want_mass=True, scale=scale)
    torch.cuda.synchronize()
    O, L, M = oracle_attn(qb, kb, vb, n_ctx, scale if scale else None)
    assert_o_close(o, O)
    # lse: probabilities exp(s - lse) within 1e-4 relative <=> |dlse| <= 1e-4
    assert np.abs(lse.cpu().numpy().astype(np.float64) - L).max() <= 1e-4
    assert_rel_close(mass.cpu().numpy(), M, what="mass")
    R, Hq = qb.shape[0], qb.shape[1]
    assert abs(float(mass.double().sum()) - Hq * R) <= 1e-4 * Hq * R
    return o, lse, mass


def test_config0():
    cfg = wl.CONFIGS[0]
    q, k, v = wl.attn_layer(cfg, 0)
    run_case(q, k, v, cfg.n_ctx)


@pytest.mark.parametrize("Hq,Hkv,D,n_ctx,R", [
    (8, 2, 128, 300, 3),      # ragged tail, several tiles
    (7, 7, 64, 0, 4),         # empty context: row r sees r + 1 keys
    (4, 4, 128, 0, 1),        # a single key
    (6, 2, 64, 70, 1),        # decode-style single row
    (28, 4, 128, 1000, 9),    # 63 rows per KV head
    (16, 2, 128, 129, 16),    # 128 rows per KV head (the maximum)
    (40, 8, 128, 2500, 13),   # several key splits with a ragged last split
    (1, 1, 64, 63, 70),       # window longer than a key tile: rows that see nothing of the last tile's tail
    (4, 1, 64, 60, 10),       # window straddles a tile boundary
])
def test_shapes(Hq, Hkv, D, n_ctx, R):
    if (Hq // Hkv) * R > 128:
        pytest.skip("outside the supported set")
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, n_ctx + R, sink=True, seed=1000 + n_ctx + R)
    run_case(qb, kb, vb, n_ctx)


def test_window_too_long_is_unsupported():
    qb, kb, vb = wl.make_qkv(5, 1, 64, 70, 133, sink=False, seed=1)
    with pytest.raises(binding.PvlmError) as e:
        binding.verify_attn(bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb), 63)
    assert e.value.status == 2


def test_running_max_keeps_growing():
    """Scores that increase steeply with position force a rescale at every tile."""
    Hq, Hkv, D, n_ctx, R = 8, 2, 128, 5000, 5
    T = n_ctx + R
    rq, rk, rv = (np.random.Generator(np.random.Philox(key=[7, i])) for i in range(3))
    q, k, v = wl.make_qkv_f32(Hq, Hkv, D, R, T, False, rq, rk, rv)
    k[:, :, D - 1] = (40.0 * np.arange(T) / T).astype(np.float32)[:, None]       # +40 logits over the range
    run_case(wl.f32_to_bf16_bits(q), wl.f32_to_bf16_bits(k), wl.f32_to_bf16_bits(v), n_ctx)
    k[:, :, D - 1] = (40.0 - 40.0 * np.arange(T) / T).astype(np.float32)[:, None]  # and decreasing
    run_case(wl.f32_to_bf16_bits(q), wl.f32_to_bf16_bits(k), wl.f32_to_bf16_bits(v), n_ctx)


def test_extreme_score_ranges_stay_finite():
    """Scores of magnitude ~1e3 (nearly one-hot rows) and a sudden jump of several hundred log2 units inside one
    tile: the reference is replaced before anything is exponentiated, so nothing overflows."""
    Hq, Hkv, D, n_ctx, R = 8, 2, 128, 1500, 5
    T = n_ctx + R
    rq, rk, rv = (np.random.Generator(np.random.Philox(key=[11, i])) for i in range(3))
    q, k, v = wl.make_qkv_f32(Hq, Hkv, D, R, T, False, rq, rk, rv)
    o, lse, mass = run_case(wl.f32_to_bf16_bits(8 * q), wl.f32_to_bf16_bits(8 * k), wl.f32_to_bf16_bits(v), n_ctx)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all() and torch.isfinite(mass).all()
    k2 = k.copy()
    k2[700:703, :, :] *= 60.0                     # three keys whose scores dwarf everything seen before
    o, lse, mass = run_case(wl.f32_to_bf16_bits(q), wl.f32_to_bf16_bits(k2), wl.f32_to_bf16_bits(v), n_ctx)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all() and torch.isfinite(mass).all()


def test_custom_scale_and_no_mass():
    qb, kb, vb = wl.make_qkv(8, 4, 64, 3, 203, sink=False, seed=21)
    run_case(qb, kb, vb, 200, scale=0.07)
    o, lse, mass = binding.verify_attn(bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb), 200, want_lse=False)
    assert lse is None and mass is None
    O, _, _ = oracle_attn(qb, kb, vb, 200)
    assert_o_close(o, O)


def test_batched_layers_with_strides():
    """n_layers = 3 in one launch; K/V live in a larger buffer (padded token and layer strides)."""
    Hq, Hkv, D, n_ctx, R, L = 12, 4, 128, 700, 6, 3
    T = n_ctx + R
    layers = [wl.make_qkv(Hq, Hkv, D, R, T, True, seed=300 + l) for l in range(L)]
    q = torch.stack([bf16_cuda(x[0]) for x in layers])
    kbuf = torch.zeros(L, T + 5, Hkv + 1, D + 64, dtype=torch.bfloat16, device="cuda")
    vbuf = torch.zeros_like(kbuf)
    for l, (_, kb, vb) in enumerate(layers):
        kbuf[l, :T, :Hkv, :D] = bf16_cuda(kb)
        vbuf[l, :T, :Hkv, :D] = bf16_cuda(vb)
    k, v = kbuf[:, :T, :Hkv, :D], vbuf[:, :T, :Hkv, :D]
    o, lse, mass = binding.verify_attn(q, k, v, n_ctx, want_mass=True)
    torch.cuda.synchronize()
    for l, (qb, kb, vb) in enumerate(layers):
        O, Lr, M = oracle_attn(qb, kb, vb, n_ctx)
        assert_o_close(o[l], O)
        assert np.abs(lse[l].cpu().numpy() - Lr).max() <= 1e-4
        assert_rel_close(mass[l].cpu().numpy(), M, what="mass")


def test_deterministic():
    cfg = wl.CONFIGS[0]
    q, k, v = (bf16_cuda(x) for x in wl.attn_layer(cfg, 0))
    a = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
    b = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_config1_full_size():
    cfg = wl.CONFIGS[1]
    q, k, v = wl.attn_layer(cfg, 0)
    run_case(q, k, v, cfg.n_ctx)


@pytest.mark.parametrize("layout", ["head", "token"])
def test_config2_full_size_batched_launch(layout):
    """Config-2 geometry at full context in the multi-layer launch configuration the bench
    times (4 of the 64 layers here; each layer checked in full against the oracle)."""
    cfg = wl.CONFIGS[2]
    L = 4
    layers = [wl.attn_layer(cfg, l) for l in (0, 19, 20, 63)]
    q = torch.stack([bf16_cuda(x[0]) for x in layers])
    k = torch.stack([bf16_cuda(x[1]) for x in layers])
    v = torch.stack([bf16_cuda(x[2]) for x in layers])
    if layout == "head":                  # [layer][kv_head][token][D] storage (the bench's layout), passed through the strides
        k = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        v = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        assert k.stride(1) == cfg.D and k.stride(2) == cfg.T * cfg.D
    o, lse, mass = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True)
    torch.cuda.synchronize()
    for l in range(L):
        O, Lr, M = oracle_attn(*layers[l], cfg.n_ctx)
        assert_o_close(o[l], O)
        assert np.abs(lse[l].cpu().numpy() - Lr).max() <= 1e-4
        assert_rel_close(mass[l].cpu().numpy(), M, what="mass")


def test_config3_and_4_geometry_full_context():
    for cid in (3, 4):
        cfg = wl.CONFIGS[cid]
        q, k, v = wl.attn_layer(cfg, 0)
        run_case(q, k, v, cfg.n_ctx)


@pytest.mark.parametrize("ctas", [1, 3, 7])
def test_tensor_core_path_long_tile_runs(ctas, pvlm_option):
    """The tcgen05 kernel with few CTAs: long tile runs, several (layer, KV head) segments per CTA,
    segments split between CTAs (the library reads the switch when it plans a call)."""
    pvlm_option("attn_max_ctas", ctas)
    for (Hq, Hkv, D, n_ctx, R) in [(40, 8, 128, 2500, 13), (8, 2, 128, 1500, 5), (12, 4, 128, 700, 6)]:
        qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, n_ctx + R, sink=True, seed=5 + n_ctx)
        run_case(qb, kb, vb, n_ctx)


def test_tensor_core_path_rescales_inside_long_runs(pvlm_option):
    """Steeply growing scores inside one CTA's run: the lazy reference must be replaced many times,
    rescaling the TMEM accumulator of each softmax group."""
    pvlm_option("attn_max_ctas", 2)
    Hq, Hkv, D, n_ctx, R = 8, 2, 128, 5000, 5
    T = n_ctx + R
    rq, rk, rv = (np.random.Generator(np.random.Philox(key=[17, i])) for i in range(3))
    q, k, v = wl.make_qkv_f32(Hq, Hkv, D, R, T, False, rq, rk, rv)
    k[:, :, D - 1] = (60.0 * np.arange(T) / T).astype(np.float32)[:, None]
    run_case(wl.f32_to_bf16_bits(q), wl.f32_to_bf16_bits(k), wl.f32_to_bf16_bits(v), n_ctx)


def test_mma_sync_path_still_matches(pvlm_option):
    """The attn_mma_sync switch forces the mma.sync kernel for D = 128 as well (the second implementation)."""
    pvlm_option("attn_mma_sync", 1)
    for (Hq, Hkv, D, n_ctx, R) in [(40, 8, 128, 2500, 13), (28, 4, 128, 1000, 9), (6, 2, 64, 700, 5), (14, 2, 64, 70, 1)]:
        qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, n_ctx + R, sink=True, seed=9 + n_ctx)
        run_case(qb, kb, vb, n_ctx)


@pytest.mark.parametrize("Hq,Hkv,R", [(16, 2, 13), (16, 2, 16), (14, 2, 15), (16, 2, 11), (16, 2, 12), (14, 2, 12)])
def test_wide_row_groups_on_the_tensor_core_path(Hq, Hkv, R, pvlm_option):
    """81..128 query rows per KV head: 96 and 128 padded rows run in split-column mode (both softmax groups on every tile,
    half of the rows each; 84, 88, 96 and 128 rows here), 112 padded rows (104, 105 rows) on alternate tiles with 3 ring
    slots and 2 score buffers.  Long tile runs with several segments per CTA."""
    pvlm_option("attn_max_ctas", 3)
    n_ctx = 2100
    qb, kb, vb = wl.make_qkv(Hq, Hkv, 128, R, n_ctx + R, sink=True, seed=500 + R)
    run_case(qb, kb, vb, n_ctx)


def test_head_dim_64_on_the_tensor_core_path(pvlm_option):
    """D = 64 runs the tcgen05 kernels on channels padded to 128 by the TMA's out-of-range fill: several layers,
    long tile runs on few CTAs (many segments per CTA), batched launch with mass rows."""
    pvlm_option("attn_max_ctas", 5)
    L, Hq, Hkv, D, n_ctx, R = 3, 14, 2, 64, 1500, 4
    layers = [wl.make_qkv(Hq, Hkv, D, R, n_ctx + R, sink=True, seed=300 + l) for l in range(L)]
    q = torch.stack([bf16_cuda(x[0]) for x in layers])
    k = torch.stack([bf16_cuda(x[1]) for x in layers])
    v = torch.stack([bf16_cuda(x[2]) for x in layers])
    o, lse, mass = binding.verify_attn(q, k, v, n_ctx, want_mass=True, mass_layers=[0, 2], check=True)
    for i, l in enumerate([0, 2]):
        O, Lr, M = oracle_attn(*layers[l], n_ctx)
        assert_o_close(o[l], O)
        assert_rel_close(lse[l].cpu().numpy(), Lr, 1e-4, "lse")
        assert_rel_close(mass[i].cpu().numpy(), M, 1e-4, "mass")
    O1, L1, _ = oracle_attn(*layers[1], n_ctx)
    assert_o_close(o[1], O1)


@pytest.mark.parametrize("Hq,R", [(16, 11), (16, 16), (14, 15)])
def test_head_dim_64_with_wide_row_groups(Hq, R, pvlm_option):
    """D = 64 together with 88 / 128 rows per KV head (split-column mode) and 105 rows (alternate tiles, 3 ring slots)."""
    pvlm_option("attn_max_ctas", 4)
    n_ctx = 1700
    qb, kb, vb = wl.make_qkv(Hq, 2, 64, R, n_ctx + R, sink=True, seed=640 + R)
    run_case(qb, kb, vb, n_ctx)


def test_head_major_cache_layout():
    """K/V stored [Hkv][T][D] and passed through the strides."""
    Hq, Hkv, D, n_ctx, R = 16, 4, 128, 900, 7
    T = n_ctx + R
    qb, kb, vb = wl.make_qkv(Hq, Hkv, D, R, T, sink=True, seed=44)
    k = bf16_cuda(kb).permute(1, 0, 2).contiguous().permute(1, 0, 2)      # [T,Hkv,D] view of head-major storage
    v = bf16_cuda(vb).permute(1, 0, 2).contiguous().permute(1, 0, 2)
    assert k.stride(0) == D and k.stride(1) == T * D
    o, lse, mass = binding.verify_attn(bf16_cuda(qb), k, v, n_ctx, want_mass=True, check=True)
    torch.cuda.synchronize()
    O, L, M = oracle_attn(qb, kb, vb, n_ctx)
    assert_o_close(o, O)
    assert_rel_close(mass.cpu().numpy(), M, what="mass")


def test_timeout_status_is_reported_from_the_workspace_word():
    """Failure reporting without making a GPU wait: the status word a bounded on-device wait would
    set is poisoned from the host, and the health check must report PVLM_ERR_TIMEOUT."""
    import ctypes as C
    qb, kb, vb = wl.make_qkv(8, 2, 128, 3, 303, sink=False, seed=3)
    q, k, v = bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb)
    o = torch.empty_like(q)
    p = binding.attn_params(q, k, v, 300, o, None, None)
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert binding.lib().pvlm_verify_attn(C.byref(p), st) == 0
    assert binding.lib().pvlm_verify_attn_check(C.byref(p), st) == 0
    need = binding.lib().pvlm_verify_attn_workspace_bytes(C.byref(p))
    ws = p._keep[6]
    ws[need - 8192:need - 8188] = torch.tensor([1, 0, 0, 0], dtype=torch.uint8, device="cuda")   # the status word
    assert binding.lib().pvlm_verify_attn_check(C.byref(p), st) == 6
    assert binding.lib().pvlm_verify_attn(C.byref(p), st) == 0                                    # a new call clears it
    assert binding.lib().pvlm_verify_attn_check(C.byref(p), st) == 0


def test_first_attention_calls_from_two_host_threads_at_once():
    """Two host threads make their FIRST call into the library at the same moment (a fresh process, so the one-time
    look-ups inside the first call really race); both must succeed and give what a later single call gives."""
    import os
    import subprocess
    import sys
    prog = r"""
import sys, threading, numpy as np, torch
sys.path.insert(0, %r)
from paper_2603_19610_b200 import binding, workloads as wl
binding.lib()                                         # load (and if need be build) the library before the race
dev = torch.device("cuda")
to_dev = lambda b: torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).to(dev)
cases = [tuple(to_dev(x) for x in wl.make_qkv(8, 2, 128, 3, 1003, True, seed=s)) for s in (1, 2)]
gate, out, err = threading.Barrier(2), [None, None], []
def work(i):
    try:
        with torch.cuda.stream(torch.cuda.Stream()):
            q, k, v = cases[i]
            gate.wait()
            out[i] = binding.verify_attn(q, k, v, 1000, want_mass=True, check=True)
    except Exception as e:                            # noqa: BLE001
        err.append(repr(e))
ts = [threading.Thread(target=work, args=(i,)) for i in range(2)]
[t.start() for t in ts]; [t.join() for t in ts]
torch.cuda.synchronize()
assert not err, err
for i in range(2):
    want = binding.verify_attn(*cases[i], 1000, want_mass=True, check=True)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(out[i], want))
print("ok")
""" % os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", prog], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and res.stdout.strip().endswith("ok"), res.stdout[-2000:] + res.stderr[-2000:]


def test_tensor_core_path_is_deterministic():
    """Same inputs twice through the tcgen05 kernels: bitwise equal O, lse and mass (no float atomics,
    fixed-order merges)."""
    qb, kb, vb = wl.make_qkv(40, 8, 128, 13, 6013, sink=True, seed=123)
    q, k, v = bf16_cuda(qb), bf16_cuda(kb), bf16_cuda(vb)
    a = binding.verify_attn(q, k, v, 6000, want_mass=True)
    a = [x.clone() for x in a]
    for _ in range(3):
        b = binding.verify_attn(q, k, v, 6000, want_mass=True)
        torch.cuda.synchronize()
        for x, y in zip(a, b):
            assert torch.equal(x, y)


def test_random_shapes_against_the_oracle_and_the_second_implementation(pvlm_option):
    """24 seeded random geometries (both head dimensions, 1..128 rows per KV head, contexts from empty to
    several tiles, 1..3 layers).  EVERY case is checked against the oracle (every layer: O within the bf16
    tolerance, lse and mass within 1e-4); the mma.sync implementation is compared as an extra."""
    rng = np.random.default_rng(2024)
    for case in range(24):
        D = int(rng.choice([64, 128]))
        Hkv = int(rng.integers(1, 5))
        G = int(rng.integers(1, 9))
        R = int(rng.integers(1, max(2, 128 // G + 1)))
        n_ctx = int(rng.choice([0, 1, 127, 128, 129, 700, 2500]))
        L = int(rng.integers(1, 4))
        Hq, T = G * Hkv, n_ctx + R
        g = torch.Generator(device="cuda"); g.manual_seed(case)
        mk = lambda *sh: torch.randn(sh, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        q, k, v = mk(L, R, Hq, D), mk(L, T, Hkv, D), mk(L, T, Hkv, D)
        pvlm_option("attn_mma_sync", 0)
        o1, l1, m1 = binding.verify_attn(q, k, v, n_ctx, want_mass=True, check=True)
        pvlm_option("attn_mma_sync", 1)
        o2, l2, m2 = binding.verify_attn(q, k, v, n_ctx, want_mass=True)
        torch.cuda.synchronize()
        tag = (case, L, Hq, Hkv, D, n_ctx, R)
        for l in range(L):
            O, Lr, M = oracle_attn(np.ascontiguousarray(bits_of(q[l])), np.ascontiguousarray(bits_of(k[l])),
                                   np.ascontiguousarray(bits_of(v[l])), n_ctx)
            for o, ls, ms in ((o1, l1, m1), (o2, l2, m2)):
                assert_o_close(o[l], O)
                assert np.abs(ls[l].cpu().numpy() - Lr).max() <= 1e-4, tag
                assert_rel_close(ms[l].cpu().numpy(), M, what="mass")
        err = (o1.float() - o2.float()).abs()
        assert bool((err <= 1e-2 + 2e-2 * o2.float().abs()).all()), tag


@pytest.mark.parametrize("cid", [2, 3])
def test_all_layers_in_the_bench_launch_configuration(cid):
    """The launch bench.py times: all layers of a multi-layer config in ONE call (head-major cache, mass on the
    reference and the current layer; config 2: 64 layers, 889 tiles and 3.5 items per persistent CTA; config 3: 80
    layers of 88 rows per KV head).  Three layers hold the host-generated data of the workload recipe and are checked
    in full against the oracle; the others are device-drawn filler of the same shape."""
    cfg = wl.CONFIGS[cid]
    L, T, R = cfg.n_layers, cfg.T, cfg.R
    dev = torch.device("cuda")
    g = torch.Generator(device=dev)
    g.manual_seed(99)
    k_base = torch.empty((L, cfg.Hkv, T, cfg.D), dtype=torch.bfloat16, device=dev)
    v_base = torch.empty_like(k_base)
    q = torch.empty((L, R, cfg.Hq, cfg.D), dtype=torch.bfloat16, device=dev)
    for l in range(L):
        k_base[l].copy_(torch.randn((cfg.Hkv, T, cfg.D), generator=g, device=dev))
        v_base[l].copy_(torch.randn((cfg.Hkv, T, cfg.D), generator=g, device=dev))
        q[l].copy_(torch.randn((R, cfg.Hq, cfg.D), generator=g, device=dev))
    k, v = k_base.permute(0, 2, 1, 3), v_base.permute(0, 2, 1, 3)          # the [layer][token][kv_head][D] view
    checked = {l: wl.attn_layer(cfg, l) for l in (cfg.ref_layer, cfg.cur_layer, L - 1)}
    for l, (qb, kb, vb) in checked.items():
        q[l].copy_(bf16_cuda(qb)); k[l].copy_(bf16_cuda(kb)); v[l].copy_(bf16_cuda(vb))
    mass_layers = [cfg.ref_layer, cfg.cur_layer]
    o, lse, mass = binding.verify_attn(q, k, v, cfg.n_ctx, want_mass=True, mass_layers=mass_layers, check=True)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(o.float()).all()) and bool(torch.isfinite(lse).all())
    for l, (qb, kb, vb) in checked.items():
        O, Lr, M = oracle_attn(qb, kb, vb, cfg.n_ctx)
        assert_o_close(o[l], O)
        assert np.abs(lse[l].cpu().numpy() - Lr).max() <= 1e-4
        if l in mass_layers:
            row = mass[mass_layers.index(l)]
            assert_rel_close(row.cpu().numpy(), M, what="mass")
            assert abs(float(row.double().sum()) - cfg.Hq * R) <= 1e-4 * cfg.Hq * R


@pytest.mark.parametrize("layout", ["token", "head"])
def test_two_million_token_context_with_layer_strides_beyond_2_31_elements(layout):
    """Maximum-size case: 2.1 M context tokens, 8 KV heads, two layers, so that a layer of K is 2.15 G elements
    (offsets need 64 bits) and a head-major KV head alone is 0.5 GB.  The oracle would take minutes here, so the
    reference is the definition written with plain torch fp64 ops on the device, for two heads of the last layer
    (the one behind the large offset); total mass must still equal heads x rows."""
    dev = torch.device("cuda")
    L, Hq, Hkv, D, R = 2, 16, 8, 128, 4
    n_ctx = 2_100_000
    T = n_ctx + R
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    if layout == "token":
        k = torch.empty((L, T, Hkv, D), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k)
    else:
        kb = torch.empty((L, Hkv, T, D), dtype=torch.bfloat16, device=dev)
        vb = torch.empty_like(kb)
        k, v = kb.permute(0, 2, 1, 3), vb.permute(0, 2, 1, 3)
    for l in range(L):
        for h in range(Hkv):
            k[l, :, h].copy_(torch.randn((T, D), generator=g, device=dev))
            v[l, :, h].copy_(torch.randn((T, D), generator=g, device=dev))
    q = torch.randn((L, R, Hq, D), generator=g, device=dev).to(torch.bfloat16)
    assert k.stride(0) > 2 ** 31
    o, lse, mass = binding.verify_attn(q, k, v, n_ctx, want_mass=True, check=True)
    torch.cuda.synchronize()
    for row in mass:
        assert abs(float(row.double().sum()) - Hq * R) <= 1e-4 * Hq * R
    l = L - 1
    for h in (0, Hq - 1):
        kv = h // (Hq // Hkv)
        s = (q[l, :, h].double() @ k[l, :, kv].double().T) / np.sqrt(D)       # [R, T]
        for r in range(R):
            s[r, n_ctx + r + 1:] = -float("inf")
        lse_ref = torch.logsumexp(s, dim=1)
        o_ref = torch.exp(s - lse_ref[:, None]) @ v[l, :, kv].double()
        assert bool(((o[l, :, h].double() - o_ref).abs() <= 1e-2 + 2e-2 * o_ref.abs()).all())
        assert float((lse[l, h].double() - lse_ref).abs().max()) <= 1e-4
