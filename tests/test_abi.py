"""The C-ABI library loads without a GPU, exports every symbol the header
declares, the header is valid C99, and the ctypes mirrors match its layout."""
import ctypes as C
import os
import re
import subprocess
import sys
import tempfile

import pytest

from paper_2603_19610_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "pvlm.h")


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(pvlm_[a-z_0-9]+)\s*\(", src)))


def test_exports_every_declared_symbol():
    L = binding.lib()
    names = declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), n
    assert set(binding.EXPORTS) <= set(names)
    assert L.pvlm_version() >= 1000
    assert L.pvlm_status_string(0) == b"PVLM_OK"
    assert L.pvlm_status_string(3) == b"PVLM_ERR_WORKSPACE"


def test_header_is_c99_and_layouts_match():
    fields = {"pvlm_attn_params": binding.AttnParams, "pvlm_prune_params": binding.PruneParams,
              "pvlm_accept_params": binding.AcceptParams, "pvlm_step_params": binding.StepParams,
              "pvlm_similarity_params": binding.SimilarityParams, "pvlm_decode_params": binding.DecodeParams,
              "pvlm_rate_params": binding.RateParams}
    prog = ['#include <stdio.h>', '#include <stddef.h>', '#include "pvlm.h"', 'int main(void){']
    for cname, st in fields.items():
        prog.append(f'printf("{cname} %zu\\n", sizeof({cname}));')
        for fname, _ in st._fields_:
            prog.append(f'printf("{cname}.{fname} %zu\\n", offsetof({cname}, {fname}));')
    prog.append("return 0;}")
    with tempfile.TemporaryDirectory() as td:
        src = os.path.join(td, "layout.c")
        open(src, "w").write("\n".join(prog))
        exe = os.path.join(td, "layout")
        subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                        src, "-o", exe], check=True)
        out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout
    got = dict(line.split() for line in out.strip().splitlines())
    for cname, st in fields.items():
        assert int(got[cname]) == C.sizeof(st)
        for fname, _ in st._fields_:
            assert int(got[f"{cname}.{fname}"]) == getattr(st, fname).offset, (cname, fname)


def test_workspace_queries_and_argument_errors_need_no_gpu():
    L = binding.lib()
    p = binding.AttnParams()
    p.n_layers, p.R, p.Hq, p.Hkv, p.D, p.n_ctx = 64, 13, 40, 8, 128, 32768
    ws = L.pvlm_verify_attn_workspace_bytes(C.byref(p))
    assert 0 < ws < (1 << 30)
    p.D = 96
    assert L.pvlm_verify_attn_workspace_bytes(C.byref(p)) == 0
    assert L.pvlm_verify_attn(C.byref(p), None) == 1                    # NULL tensors: invalid before any launch
    p.q = p.k = p.v = p.o = 4096
    assert L.pvlm_verify_attn(C.byref(p), None) == 2                    # D = 96 unsupported
    p.D = 128
    p.kv_head_stride, p.kv_token_stride = 128, 8 * 128
    p.kv_layer_stride, p.q_layer_stride = 32781 * 1024, 13 * 40 * 128
    assert L.pvlm_verify_attn(C.byref(p), None) == 3                    # no workspace
    p.Hq = 41
    assert L.pvlm_verify_attn(C.byref(p), None) == 2                    # Hq % Hkv != 0
    # a listed-mass-layers count out of range makes the workspace query answer 0 (never a wrapped size)
    p.Hq = 40
    p.mass = 4096
    layers = (C.c_int * 9)(*range(9))
    p.mass_layers = layers
    for bad in (0, -3, 9):
        p.n_mass_layers = bad
        assert L.pvlm_verify_attn_workspace_bytes(C.byref(p)) == 0
    p.n_mass_layers = 2
    assert 0 < L.pvlm_verify_attn_workspace_bytes(C.byref(p)) < (1 << 30)

    a = binding.AcceptParams()
    a.batch, a.gamma, a.V = 1, 12, 152064
    assert L.pvlm_spec_accept_workspace_bytes(C.byref(a)) > 0
    assert L.pvlm_spec_accept(C.byref(a), None) == 1
    a.gamma = 65
    assert L.pvlm_spec_accept_workspace_bytes(C.byref(a)) == 0

    u = binding.PruneParams()
    u.m, u.k = 100, 101
    assert L.pvlm_uvprune_select_gather(C.byref(u), None) == 1          # k > m
    u.k = 10
    assert L.pvlm_uvprune_workspace_bytes(C.byref(u)) >= 400
    assert L.pvlm_uvprune_select_gather(C.byref(u), None) == 1          # no mass pointer

    # similarity: the workspace grows with the layers of the call; bad layer counts and strides are refused before any launch
    sm = binding.SimilarityParams()
    sm.m, sm.n, sm.d, sm.hidden_row_stride = 1000, 100, 1024, 1024
    one = L.pvlm_uvprune_similarity_workspace_bytes(C.byref(sm))
    sm.n_layers = 2
    assert one > 0 and L.pvlm_uvprune_similarity_workspace_bytes(C.byref(sm)) > one
    sm.n_layers = -1
    assert L.pvlm_uvprune_similarity_workspace_bytes(C.byref(sm)) == 0
    sm.hidden = sm.sim = 4096
    assert L.pvlm_uvprune_similarity(C.byref(sm), None) == 1
    sm.n_layers, sm.hidden_layer_stride, sm.sim_layer_stride = 2, 1100 * 1024, 999
    assert L.pvlm_uvprune_similarity(C.byref(sm), None) == 1            # the layers' outputs would overlap
    sm.hidden_layer_stride, sm.sim_layer_stride = 1100 * 1024 + 4, 1000
    assert L.pvlm_uvprune_similarity(C.byref(sm), None) == 1            # layer stride not a multiple of 8 elements
    sm.hidden_layer_stride = 1100 * 1024
    assert L.pvlm_uvprune_similarity(C.byref(sm), None) == 3            # no workspace

    # the decision-only entry points
    assert L.pvlm_select_from_scores(None, 100, 101, None, None, 0, None) == 1    # k > m
    assert L.pvlm_select_from_scores(None, 100, 10, None, None, 0, None) == 1     # no scores
    assert L.pvlm_accept_from_probs(None, None, None, 3, 4, 1, None, None) == 1   # fewer uniforms than tokens
    assert L.pvlm_accept_from_probs(None, None, None, 5, 4, 1, 4096, None) == 1   # no probabilities
    assert L.pvlm_accept_from_probs(None, None, None, 5, 4, 0, 4096, None) == 1   # empty batch
    # process-wide switches: unknown option or negative value refused, previous value returned
    assert L.pvlm_set_option(99, 1) == -1 and L.pvlm_set_option(0, -1) == -1
    prev = L.pvlm_set_option(2, 7)
    assert L.pvlm_set_option(2, prev) == 7

    # the step call checks every stage before it queues anything (so this needs no GPU either)
    sp = binding.StepParams()
    assert L.pvlm_verify_step(None, None) == 1
    sp.run_prune = 1
    sp.prune.m, sp.prune.k = 100, 101
    assert L.pvlm_verify_step(C.byref(sp), None) == 1                   # k > m in the prune stage
    sp.run_prune, sp.run_accept = 0, 1
    sp.accept.batch, sp.accept.gamma, sp.accept.V = 1, 12, 152064
    assert L.pvlm_verify_step(C.byref(sp), None) == 1                   # accept stage without logits
    sp.run_accept, sp.run_attn = 0, 1
    sp.attn.n_layers, sp.attn.R, sp.attn.Hq, sp.attn.Hkv, sp.attn.D, sp.attn.n_ctx = 1, 13, 40, 8, 96, 1000
    sp.attn.q = sp.attn.k = sp.attn.v = sp.attn.o = 4096
    assert L.pvlm_verify_step(C.byref(sp), None) == 2                   # D = 96 in the attention stage
    sp.copy_stream = 1                                                   # overlap mode needs the stream AND both events
    assert L.pvlm_verify_step(C.byref(sp), None) == 1


def test_no_cpu_fallback():
    import torch
    q = torch.zeros(2, 4, 64, dtype=torch.bfloat16)
    with pytest.raises(RuntimeError):
        binding.verify_attn(q, torch.zeros(10, 1, 64, dtype=torch.bfloat16), torch.zeros(10, 1, 64, dtype=torch.bfloat16), 8)


def test_window_size_host_function_matches_oracle():
    from oracle.accept import window_size_rounded
    for tp, tq in [(420, 46.6), (203, 39.8), (78.3, 25.8), (78.3, 46.6), (420, 78), (10, 50), (63.7, 39.8)]:
        for mode in ("nearest", "down", "up"):
            assert binding.window_size(tp, tq, mode) == window_size_rounded(tp, tq, mode)
    assert binding.window_size(0, 1) == 0 and binding.window_size(1, -1) == 0
