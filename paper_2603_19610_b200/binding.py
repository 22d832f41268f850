"""Thin ctypes binding over libpvlm.so: argument marshalling only.

Function names and argument meaning follow include/pvlm.h.  torch is used for
device memory and streams; every step of the path runs in the library's CUDA
kernels.  There is no CPU fallback: if the shared library cannot be loaded or
built, or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes as C
import os
import threading

import torch

from . import build as _build

_LIB = None
_LOCK = threading.Lock()

STATUS_NAMES = {0: "PVLM_OK", 1: "PVLM_ERR_INVALID_ARG", 2: "PVLM_ERR_UNSUPPORTED",
                3: "PVLM_ERR_WORKSPACE", 4: "PVLM_ERR_CUDA", 5: "PVLM_ERR_TOO_LARGE", 6: "PVLM_ERR_TIMEOUT"}
SELECT_STATIC_MAX_M = 262144
DECODE_LOG_COLS = 9


class PvlmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class AttnParams(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("o", C.c_void_p),
                ("lse", C.c_void_p), ("mass", C.c_void_p),
                ("mass_layers", C.POINTER(C.c_int)), ("n_mass_layers", C.c_int),
                ("n_layers", C.c_int), ("R", C.c_int), ("Hq", C.c_int), ("Hkv", C.c_int), ("D", C.c_int),
                ("n_ctx", C.c_int),
                ("q_layer_stride", C.c_longlong), ("kv_layer_stride", C.c_longlong),
                ("kv_token_stride", C.c_longlong), ("kv_head_stride", C.c_longlong),
                ("mass_layer_stride", C.c_longlong),
                ("softmax_scale", C.c_float),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("prof_event_begin", C.c_void_p), ("prof_event_end", C.c_void_p), ("max_ctas", C.c_int)]


class PruneParams(C.Structure):
    _fields_ = [("mass_cur", C.c_void_p), ("mass_ref", C.c_void_p),
                ("vis_start", C.c_int), ("m", C.c_int), ("k", C.c_int),
                ("kept_idx", C.c_void_p), ("score", C.c_void_p),
                ("src_k", C.c_void_p), ("src_v", C.c_void_p), ("dst_k", C.c_void_p), ("dst_v", C.c_void_p),
                ("n_layers", C.c_int), ("src_len", C.c_int),
                ("row_bytes", C.c_longlong), ("src_layer_stride_bytes", C.c_longlong),
                ("dst_layer_stride_bytes", C.c_longlong),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class AcceptParams(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
                ("target_row_stride", C.c_longlong), ("draft_row_stride", C.c_longlong),
                ("target_batch_stride", C.c_longlong), ("draft_batch_stride", C.c_longlong),
                ("draft_tokens", C.c_void_p), ("uniforms", C.c_void_p),
                ("batch", C.c_int), ("gamma", C.c_int), ("V", C.c_int), ("temperature", C.c_float),
                ("n_accept", C.c_void_p), ("out_tokens", C.c_void_p),
                ("p_tok", C.c_void_p), ("q_tok", C.c_void_p), ("lse_p", C.c_void_p), ("lse_q", C.c_void_p),
                ("probs_p", C.c_void_p), ("probs_q", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class SimilarityParams(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("hidden_row_stride", C.c_longlong),
                ("vis_start", C.c_int), ("m", C.c_int), ("text_start", C.c_int), ("n", C.c_int), ("d", C.c_int),
                ("sim", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("n_layers", C.c_int), ("hidden_layer_stride", C.c_longlong), ("sim_layer_stride", C.c_longlong)]


class StepParams(C.Structure):
    _fields_ = [("attn", AttnParams), ("prune", PruneParams), ("accept", AcceptParams),
                ("run_attn", C.c_int), ("run_prune", C.c_int), ("run_accept", C.c_int),
                ("h_q", C.c_void_p), ("h_k_window", C.c_void_p), ("h_v_window", C.c_void_p),
                ("h_target_logits", C.c_void_p), ("h_draft_logits", C.c_void_p),
                ("h_draft_tokens", C.c_void_p), ("h_uniforms", C.c_void_p),
                ("h_o", C.c_void_p), ("h_n_accept", C.c_void_p), ("h_out_tokens", C.c_void_p),
                ("h_kept_idx", C.c_void_p),
                ("copy_stream", C.c_void_p), ("event_a", C.c_void_p), ("event_b", C.c_void_p),
                ("h_attn_status", C.c_void_p)]


class DecodeParams(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("draft_logits", C.c_void_p), ("row_stride", C.c_longlong),
                ("P", C.c_int), ("V", C.c_int), ("gamma", C.c_int), ("K", C.c_int), ("temperature", C.c_float),
                ("u_draft", C.c_void_p), ("u_accept", C.c_void_p), ("u_resample", C.c_void_p), ("max_rounds", C.c_int),
                ("tokens", C.c_void_p), ("round_log", C.c_void_p), ("n_rounds", C.c_void_p), ("round_ms", C.c_void_p),
                ("target_attn", C.POINTER(AttnParams)), ("draft_attn", C.POINTER(AttnParams)), ("serial", C.c_int),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class RateParams(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
                ("target_row_stride", C.c_longlong), ("draft_row_stride", C.c_longlong),
                ("tokens", C.c_void_p), ("uniforms", C.c_void_p), ("N", C.c_int), ("V", C.c_int),
                ("temperature", C.c_float), ("accepted", C.c_void_p), ("p_tok", C.c_void_p), ("q_tok", C.c_void_p),
                ("n_accepted", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


EXPORTS = ("pvlm_status_string", "pvlm_last_cuda_error", "pvlm_version",
           "pvlm_verify_attn_workspace_bytes", "pvlm_verify_attn", "pvlm_verify_attn_check",
           "pvlm_uvprune_workspace_bytes", "pvlm_uvprune_select_gather",
           "pvlm_spec_accept_workspace_bytes", "pvlm_spec_accept", "pvlm_verify_step",
           "pvlm_uvprune_select_static", "pvlm_uvprune_similarity_workspace_bytes", "pvlm_uvprune_similarity", "pvlm_window_size",
           "pvlm_parallel_decode_workspace_bytes", "pvlm_parallel_decode",
           "pvlm_acceptance_rate_workspace_bytes", "pvlm_acceptance_rate",
           "pvlm_select_from_scores", "pvlm_accept_from_probs", "pvlm_set_option")


def lib() -> C.CDLL:
    """Load (building it first if absent or stale) the C-ABI library."""
    global _LIB
    with _LOCK:
        if _LIB is None:
            path = os.environ.get("PVLM_LIB") or _build.build()     # PVLM_LIB: use a library built elsewhere
            L = C.CDLL(path)
            L.pvlm_status_string.restype = C.c_char_p
            L.pvlm_status_string.argtypes = [C.c_int]
            L.pvlm_last_cuda_error.restype = C.c_int
            L.pvlm_version.restype = C.c_int
            for name, st in (("verify_attn", AttnParams), ("uvprune", PruneParams), ("spec_accept", AcceptParams)):
                f = getattr(L, f"pvlm_{name}_workspace_bytes")
                f.restype = C.c_size_t
                f.argtypes = [C.POINTER(st)]
            for name, st in (("pvlm_verify_attn", AttnParams), ("pvlm_uvprune_select_gather", PruneParams),
                             ("pvlm_spec_accept", AcceptParams), ("pvlm_verify_step", StepParams),
                             ("pvlm_verify_attn_check", AttnParams)):
                f = getattr(L, name)
                f.restype = C.c_int
                f.argtypes = [C.POINTER(st), C.c_void_p]
            L.pvlm_uvprune_similarity_workspace_bytes.restype = C.c_size_t
            L.pvlm_uvprune_similarity_workspace_bytes.argtypes = [C.POINTER(SimilarityParams)]
            L.pvlm_uvprune_similarity.restype = C.c_int
            L.pvlm_uvprune_similarity.argtypes = [C.POINTER(SimilarityParams), C.c_void_p]
            L.pvlm_parallel_decode_workspace_bytes.restype = C.c_size_t
            L.pvlm_parallel_decode_workspace_bytes.argtypes = [C.POINTER(DecodeParams)]
            L.pvlm_parallel_decode.restype = C.c_int
            L.pvlm_parallel_decode.argtypes = [C.POINTER(DecodeParams), C.c_void_p, C.c_void_p]
            L.pvlm_acceptance_rate_workspace_bytes.restype = C.c_size_t
            L.pvlm_acceptance_rate_workspace_bytes.argtypes = [C.POINTER(RateParams)]
            L.pvlm_acceptance_rate.restype = C.c_int
            L.pvlm_acceptance_rate.argtypes = [C.POINTER(RateParams), C.c_void_p]
            L.pvlm_uvprune_select_static.restype = C.c_int
            L.pvlm_uvprune_select_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                                     C.c_void_p, C.c_void_p, C.c_void_p]
            L.pvlm_set_option.restype = C.c_int
            L.pvlm_set_option.argtypes = [C.c_int, C.c_int]
            L.pvlm_select_from_scores.restype = C.c_int
            L.pvlm_select_from_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
            L.pvlm_accept_from_probs.restype = C.c_int
            L.pvlm_accept_from_probs.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                                 C.c_void_p]
            _LIB = L
    return _LIB


_WS: dict = {}


def _workspace(dev: torch.device, key: str, nbytes: int) -> torch.Tensor:
    """A per-(device, stream, call kind) scratch buffer that only grows."""
    k = (dev.index, torch.cuda.current_stream(dev).cuda_stream, key)
    buf = _WS.get(k)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
        _WS[k] = buf
    return buf


OPTIONS = {"attn_mma_sync": 0, "select_one_cta": 1, "attn_max_ctas": 2}


def set_option(name: str, value: int) -> int:
    """Process-wide test / A-B switch (see pvlm_set_option).  Returns the previous value."""
    prev = lib().pvlm_set_option(OPTIONS[name], int(value))
    if prev < 0:
        raise ValueError(f"pvlm_set_option({name}, {value}) refused")
    return prev


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise RuntimeError("pvlm: tensors must live on a CUDA device (there is no CPU path)")


def _stream(dev):
    return C.c_void_p(torch.cuda.current_stream(dev).cuda_stream)


def attn_params(q, k, v, n_ctx, o, lse, mass, scale=0.0, workspace=None, mass_layers=None, max_ctas=0) -> AttnParams:
    """Fill an AttnParams from torch tensors: q/o [L,R,Hq,D] or [R,Hq,D]; k/v [L,T,Hkv,D] or [T,Hkv,D]."""
    if q.dim() == 3:
        q, k, v, o = q[None], k[None], v[None], o[None]
    L, R, Hq, D = q.shape
    _, T, Hkv, _ = k.shape
    assert T == n_ctx + R, "k/v must hold n_ctx + R rows"
    assert q.dtype == torch.bfloat16 and k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16
    assert q.stride(-1) == 1 and k.stride(-1) == 1 and v.stride() == k.stride() and o.stride() == q.stride()
    assert q.stride(2) == D and q.stride(1) == Hq * D
    p = AttnParams()
    p.q, p.k, p.v, p.o = _ptr(q), _ptr(k), _ptr(v), _ptr(o)
    p.lse, p.mass = _ptr(lse), _ptr(mass)
    ml = None
    if mass is not None and mass_layers is not None:
        ml = (C.c_int * len(mass_layers))(*[int(x) for x in mass_layers])
        p.mass_layers, p.n_mass_layers = ml, len(mass_layers)
    p.n_layers, p.R, p.Hq, p.Hkv, p.D, p.n_ctx = L, R, Hq, Hkv, D, n_ctx
    p.q_layer_stride = q.stride(0)
    p.kv_layer_stride, p.kv_token_stride, p.kv_head_stride = k.stride(0), k.stride(1), k.stride(2)
    p.mass_layer_stride = mass.stride(0) if (mass is not None and mass.dim() == 2) else T
    p.softmax_scale = float(scale)
    p.max_ctas = int(max_ctas)
    need = lib().pvlm_verify_attn_workspace_bytes(C.byref(p))
    ws = workspace if workspace is not None else _workspace(q.device, "attn", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    p._keep = (q, k, v, o, lse, mass, ws, ml)
    return p


def verify_attn(q, k, v, n_ctx: int, *, want_lse: bool = True, want_mass: bool = False, scale: float = 0.0,
                out=None, workspace=None, mass_layers=None, check: bool = False, max_ctas: int = 0):
    """Window-verify GQA attention (see pvlm_verify_attn).  Returns (o, lse, mass).

    mass_layers (batched form only): list of layer indices whose mass is wanted;
    mass then has one row per listed layer."""
    _need_cuda(q, k, v)
    batched = q.dim() == 4
    L = q.shape[0] if batched else 1
    R, Hq = q.shape[-3], q.shape[-2]
    T = k.shape[-3]
    o = out if out is not None else torch.empty_like(q)
    lse = torch.empty((L, Hq, R) if batched else (Hq, R), dtype=torch.float32, device=q.device) if want_lse else None
    n_mass = len(mass_layers) if mass_layers is not None else L
    mass = torch.empty((n_mass, T) if batched else (T,), dtype=torch.float32, device=q.device) if want_mass else None
    p = attn_params(q, k, v, n_ctx, o, lse, mass, scale, workspace, mass_layers if want_mass else None, max_ctas)
    st = lib().pvlm_verify_attn(C.byref(p), _stream(q.device))
    if st != 0:
        raise PvlmError(st, "pvlm_verify_attn")
    if check:                                    # synchronises: did any bounded on-device wait expire?
        st = lib().pvlm_verify_attn_check(C.byref(p), _stream(q.device))
        if st != 0:
            raise PvlmError(st, "pvlm_verify_attn_check")
    return o, lse, mass


def prune_params(mass_cur, mass_ref, vis_start, m, k, kept_idx, score, src_k, src_v, dst_k, dst_v,
                 workspace=None) -> PruneParams:
    p = PruneParams()
    p.mass_cur, p.mass_ref = _ptr(mass_cur), _ptr(mass_ref)
    p.vis_start, p.m, p.k = vis_start, m, k
    p.kept_idx, p.score = _ptr(kept_idx), _ptr(score)
    if src_k is not None:
        if src_k.dim() == 3:
            src_k, src_v, dst_k, dst_v = src_k[None], src_v[None], dst_k[None], dst_v[None]
        L, S = src_k.shape[0], src_k.shape[1]
        es = src_k.element_size()
        row_bytes = src_k.shape[2] * src_k.shape[3] * es
        assert src_k.stride(1) * es == row_bytes and dst_k.stride(1) * es == row_bytes, "rows must be dense"
        assert src_v.stride() == src_k.stride() and dst_v.stride() == dst_k.stride()
        p.src_k, p.src_v, p.dst_k, p.dst_v = _ptr(src_k), _ptr(src_v), _ptr(dst_k), _ptr(dst_v)
        p.n_layers, p.src_len, p.row_bytes = L, S, row_bytes
        p.src_layer_stride_bytes = src_k.stride(0) * es
        p.dst_layer_stride_bytes = dst_k.stride(0) * es
    need = lib().pvlm_uvprune_workspace_bytes(C.byref(p))
    dev = mass_cur.device
    ws = workspace if workspace is not None else _workspace(dev, "prune", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    p._keep = (mass_cur, mass_ref, kept_idx, score, src_k, src_v, dst_k, dst_v, ws)
    return p


def uvprune_select_gather(mass_cur, mass_ref, vis_start: int, m: int, k: int, src_k=None, src_v=None, *,
                          want_score: bool = False, workspace=None):
    """UV-Prune select (+ gather if src_k/src_v given; see pvlm_uvprune_select_gather).

    src_k/src_v: [L,S,Hkv,D] or [S,Hkv,D].  Returns (kept_idx int32 [k], score or None, dst_k, dst_v)."""
    _need_cuda(mass_cur, mass_ref, src_k, src_v)
    dev = mass_cur.device
    kept = torch.empty(k, dtype=torch.int32, device=dev)
    score = torch.empty(m, dtype=torch.float32, device=dev) if want_score else None
    dst_k = dst_v = None
    if src_k is not None:
        shp = list(src_k.shape)
        shp[-3] = shp[-3] - m + k
        dst_k = torch.empty(shp, dtype=src_k.dtype, device=dev)
        dst_v = torch.empty(shp, dtype=src_v.dtype, device=dev)
    p = prune_params(mass_cur, mass_ref, vis_start, m, k, kept, score, src_k, src_v, dst_k, dst_v, workspace)
    st = lib().pvlm_uvprune_select_gather(C.byref(p), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_uvprune_select_gather")
    return kept, score, dst_k, dst_v


def accept_params(target_logits, draft_logits, draft_tokens, uniforms, temperature, outs: dict,
                  workspace=None) -> AcceptParams:
    tl, dl = target_logits, draft_logits
    if tl.dim() == 2:
        tl, dl = tl[None], dl[None]
    B, R, V = tl.shape
    gamma = R - 1
    assert dl.shape == (B, gamma, V) and tl.dtype == torch.float32 and dl.dtype == torch.float32
    assert tl.stride(2) == 1 and dl.stride(2) == 1
    assert draft_tokens.dtype == torch.int32 and uniforms.dtype == torch.float32
    assert draft_tokens.is_contiguous() and uniforms.is_contiguous()
    p = AcceptParams()
    p.target_logits, p.draft_logits = _ptr(tl), _ptr(dl)
    p.target_row_stride, p.draft_row_stride = tl.stride(1), dl.stride(1)
    p.target_batch_stride, p.draft_batch_stride = tl.stride(0), dl.stride(0)
    p.draft_tokens, p.uniforms = _ptr(draft_tokens), _ptr(uniforms)
    p.batch, p.gamma, p.V, p.temperature = B, gamma, V, float(temperature)
    for name in ("n_accept", "out_tokens", "p_tok", "q_tok", "lse_p", "lse_q", "probs_p", "probs_q"):
        setattr(p, name, _ptr(outs.get(name)))
    need = lib().pvlm_spec_accept_workspace_bytes(C.byref(p))
    ws = workspace if workspace is not None else _workspace(tl.device, "accept", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    p._keep = (tl, dl, draft_tokens, uniforms, outs, ws)
    return p


def spec_accept(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0, *,
                want_probs: bool = False, workspace=None) -> dict:
    """Vocab softmax + accept/reject + residual resampling (see pvlm_spec_accept).

    Shapes [gamma+1,V]/[gamma,V]/[gamma]/[gamma+1], or with a leading batch dimension."""
    _need_cuda(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    batched = target_logits.dim() == 3
    B = target_logits.shape[0] if batched else 1
    gamma = target_logits.shape[-2] - 1
    f32, i32 = torch.float32, torch.int32
    outs = dict(n_accept=torch.empty(B, dtype=i32, device=dev),
                out_tokens=torch.empty((B, gamma + 1), dtype=i32, device=dev),
                p_tok=torch.empty((B, gamma), dtype=f32, device=dev),
                q_tok=torch.empty((B, gamma), dtype=f32, device=dev),
                lse_p=torch.empty((B, gamma + 1), dtype=f32, device=dev),
                lse_q=torch.empty((B, gamma), dtype=f32, device=dev))
    if want_probs:
        outs["probs_p"] = torch.empty_like(target_logits)
        outs["probs_q"] = torch.empty_like(draft_logits)
    p = accept_params(target_logits, draft_logits, draft_tokens, uniforms, temperature, outs, workspace)
    st = lib().pvlm_spec_accept(C.byref(p), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_spec_accept")
    if not batched:
        outs = {k: (v[0] if k not in ("probs_p", "probs_q") else v) for k, v in outs.items()}
    return outs


def verify_step(attn: AttnParams | None, prune: PruneParams | None, accept: AcceptParams | None, *,
                host_in: dict | None = None, host_out: dict | None = None, device=None, overlap=None) -> StepParams:
    """One whole verify -> prune -> accept step through pvlm_verify_step.

    attn / prune / accept are parameter blocks built by attn_params / prune_params /
    accept_params (None skips the stage).  host_in maps h_q, h_k_window, h_v_window,
    h_target_logits, h_draft_logits, h_draft_tokens, h_uniforms to (pinned) CPU tensors
    copied to the device first; host_out maps h_o, h_n_accept, h_out_tokens, h_kept_idx, h_attn_status to
    CPU tensors filled at the end.  overlap = (torch.cuda.Stream, torch.cuda.Event, torch.cuda.Event)
    lets the library overlap the accept-input upload and the output download with compute (the
    events must have been recorded once so that their handles exist).
    Asynchronous: synchronise the stream before reading."""
    sp = StepParams()
    keep = []
    for name, blk in (("attn", attn), ("prune", prune), ("accept", accept)):
        if blk is not None:
            setattr(sp, name, blk)
            setattr(sp, "run_" + name, 1)
            keep.append(blk)
    for d in (host_in, host_out):
        for k, t in (d or {}).items():
            if t is not None:
                assert not t.is_cuda and t.is_contiguous()
                setattr(sp, k, C.c_void_p(t.data_ptr()))
                keep.append(t)
    if overlap is not None:
        cs, ea, eb = overlap
        sp.copy_stream, sp.event_a, sp.event_b = cs.cuda_stream, ea.cuda_event, eb.cuda_event
        keep.append(overlap)
    dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
    st = lib().pvlm_verify_step(C.byref(sp), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_verify_step")
    sp._keep = keep
    return sp


def verify_step_again(sp: StepParams, device=None) -> None:
    """Queue the step of a parameter block that verify_step returned once more (same buffers, same stages): the
    marshalling is done once, a repeated step costs the C call alone."""
    dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
    st = lib().pvlm_verify_step(C.byref(sp), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_verify_step")


def uvprune_select_static(mass_cur, mass_ref, vis_start: int, m: int, k: int, kept_idx, score=None):
    """Top-K selection through pvlm_uvprune_select_static, the entry point for callers that
    cannot allocate device memory: the library's built-in key buffer is the only scratch and
    the call itself allocates nothing, so the caller passes the output tensors
    (kept_idx int32 [k], optionally score fp32 [m]).  m is limited to SELECT_STATIC_MAX_M;
    calls that may overlap on the GPU share the buffer and must be ordered."""
    _need_cuda(mass_cur, mass_ref, kept_idx, score)
    st = lib().pvlm_uvprune_select_static(_ptr(mass_cur), _ptr(mass_ref), vis_start, m, k, _ptr(kept_idx),
                                          _ptr(score), _stream(mass_cur.device))
    if st != 0:
        raise PvlmError(st, "pvlm_uvprune_select_static")
    return kept_idx


def select_from_scores(score, k: int, *, workspace=None):
    """Top-K over given fp32 scores (see pvlm_select_from_scores).  Returns kept_idx int32 [k], ascending."""
    _need_cuda(score)
    assert score.dtype == torch.float32 and score.dim() == 1 and score.is_contiguous()
    dev, m = score.device, score.numel()
    kept = torch.empty(k, dtype=torch.int32, device=dev)
    pp = PruneParams()
    pp.m = m
    need = lib().pvlm_uvprune_workspace_bytes(C.byref(pp))
    ws = workspace if workspace is not None else _workspace(dev, "prune", need)
    st = lib().pvlm_select_from_scores(_ptr(score), m, k, _ptr(kept), _ptr(ws), ws.numel(), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_select_from_scores")
    return kept


def accept_from_probs(p_tok, q_tok, uniforms):
    """First rejection from given token probabilities (see pvlm_accept_from_probs).
    p_tok, q_tok fp32 [batch, gamma] (or [gamma]); uniforms fp32 [batch, >= gamma].  Returns n_accept int32 [batch]."""
    _need_cuda(p_tok, q_tok, uniforms)
    if p_tok.dim() == 1:
        p_tok, q_tok, uniforms = p_tok[None], q_tok[None], uniforms[None]
    B, gamma = p_tok.shape
    assert q_tok.shape == (B, gamma) and uniforms.shape[0] == B and uniforms.shape[1] >= gamma
    assert p_tok.dtype == q_tok.dtype == uniforms.dtype == torch.float32
    assert p_tok.is_contiguous() and q_tok.is_contiguous() and uniforms.stride(1) == 1
    n = torch.empty(B, dtype=torch.int32, device=p_tok.device)
    st = lib().pvlm_accept_from_probs(_ptr(p_tok), _ptr(q_tok), _ptr(uniforms), uniforms.stride(0) if B > 1 else uniforms.shape[1],
                                      gamma, B, _ptr(n), _stream(p_tok.device))
    if st != 0:
        raise PvlmError(st, "pvlm_accept_from_probs")
    return n


def uvprune_similarity(hidden, vis_start: int, m: int, text_start: int, n: int, *, out=None, workspace=None):
    """sum_j cos(V_i, X_j) for the m visual rows of a layer's token representations
    (see pvlm_uvprune_similarity).  hidden: bf16 [rows, d] -> fp32 [m], or several layers at once,
    bf16 [L, rows, d] -> fp32 [L, m] (one launch of each kernel for all of them)."""
    _need_cuda(hidden)
    assert hidden.dtype == torch.bfloat16 and hidden.dim() in (2, 3) and hidden.stride(-1) == 1
    layered = hidden.dim() == 3
    L = hidden.shape[0] if layered else 1
    shape = (L, m) if layered else (m,)
    sim = out if out is not None else torch.empty(shape, dtype=torch.float32, device=hidden.device)
    assert tuple(sim.shape) == shape and sim.stride(-1) == 1
    p = SimilarityParams()
    p.hidden, p.hidden_row_stride = _ptr(hidden), hidden.stride(-2)
    p.vis_start, p.m, p.text_start, p.n, p.d = vis_start, m, text_start, n, hidden.shape[-1]
    p.sim = _ptr(sim)
    if layered:
        p.n_layers, p.hidden_layer_stride, p.sim_layer_stride = L, hidden.stride(0), sim.stride(0)
    need = lib().pvlm_uvprune_similarity_workspace_bytes(C.byref(p))
    ws = workspace if workspace is not None else _workspace(hidden.device, "sim", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    st = lib().pvlm_uvprune_similarity(C.byref(p), _stream(hidden.device))
    if st != 0:
        raise PvlmError(st, "pvlm_uvprune_similarity")
    return sim


def sample(logits, uniforms, temperature: float = 1.0, *, workspace=None):
    """Draw one token per row from softmax(logits / temperature) by inverse CDF: pvlm_spec_accept with
    gamma = 0 (nothing to verify), the form the draft model's own decoding step uses.
    logits fp32 [B, V] (or [V]), uniforms fp32 [B] (or scalar tensor).  Returns int32 tokens [B]."""
    _need_cuda(logits, uniforms)
    lg = logits if logits.dim() == 2 else logits[None]
    B, V = lg.shape
    assert lg.dtype == torch.float32 and lg.stride(1) == 1 and uniforms.dtype == torch.float32
    dev = lg.device
    n_accept = torch.empty(B, dtype=torch.int32, device=dev)
    out = torch.empty((B, 1), dtype=torch.int32, device=dev)
    p = AcceptParams()
    p.target_logits = _ptr(lg)
    p.target_row_stride, p.target_batch_stride = V, lg.stride(0)
    p.uniforms = _ptr(uniforms.contiguous())
    p.batch, p.gamma, p.V, p.temperature = B, 0, V, float(temperature)
    p.n_accept, p.out_tokens = _ptr(n_accept), _ptr(out)
    need = lib().pvlm_spec_accept_workspace_bytes(C.byref(p))
    ws = workspace if workspace is not None else _workspace(dev, "accept", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    st = lib().pvlm_spec_accept(C.byref(p), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_spec_accept")
    return out[:, 0]


def window_size(t_target: float, t_draft: float, mode: str = "nearest") -> int:
    """Draft window from measured forward times (see pvlm_window_size); mode nearest / down / up."""
    f = lib().pvlm_window_size
    f.restype = C.c_int
    f.argtypes = [C.c_double, C.c_double, C.c_int]
    return int(f(float(t_target), float(t_draft), {"nearest": 0, "down": 1, "up": 2}[mode]))


def parallel_decode(target_logits, draft_logits, gamma: int, K: int, u_draft, u_accept, u_resample, *,
                    temperature: float = 1.0, target_attn=None, draft_attn=None, serial: bool = False,
                    draft_stream=None, want_ms: bool = False):
    """The Pre-/Post-verify round loop on two streams (see pvlm_parallel_decode).
    target_logits / draft_logits fp32 [P, V] on the device (row i = distribution of generated position i),
    u_draft / u_accept fp32 [rounds, gamma], u_resample fp32 [rounds] on the device.  target_attn / draft_attn:
    optional AttnParams blocks whose attention runs every round over the two caches as they stand (their n_ctx = context
    before the first generated token; k / v and workspace must cover n_ctx + K + 2 * gamma + 1 rows).  The target side
    uses the current stream.  Returns dict(tokens int32 [K], rounds, log int32 [rounds, DECODE_LOG_COLS], round_ms or None)."""
    _need_cuda(target_logits, draft_logits, u_draft, u_accept, u_resample)
    P, V = target_logits.shape
    assert draft_logits.shape == (P, V) and target_logits.stride(1) == 1 and draft_logits.stride(0) == target_logits.stride(0)
    assert target_logits.dtype == torch.float32 and draft_logits.dtype == torch.float32
    dev = target_logits.device
    max_rounds = u_resample.numel()
    assert u_draft.shape == (max_rounds, gamma) and u_accept.shape == (max_rounds, gamma)
    ud, ua, ur = u_draft.contiguous(), u_accept.contiguous(), u_resample.contiguous()
    tokens = torch.empty(K, dtype=torch.int32)
    log = torch.zeros((max_rounds, DECODE_LOG_COLS), dtype=torch.int32)
    n_rounds = torch.zeros(1, dtype=torch.int32)
    ms = torch.zeros(max_rounds, dtype=torch.float32) if want_ms else None
    p = DecodeParams()
    p.target_logits, p.draft_logits, p.row_stride = _ptr(target_logits), _ptr(draft_logits), target_logits.stride(0)
    p.P, p.V, p.gamma, p.K, p.temperature = P, V, gamma, K, float(temperature)
    p.u_draft, p.u_accept, p.u_resample, p.max_rounds = _ptr(ud), _ptr(ua), _ptr(ur), max_rounds
    p.tokens, p.round_log, p.n_rounds = _ptr(tokens), _ptr(log), _ptr(n_rounds)
    p.round_ms = _ptr(ms)
    if target_attn is not None:
        p.target_attn = C.pointer(target_attn)
    if draft_attn is not None:
        p.draft_attn = C.pointer(draft_attn)
    p.serial = 1 if serial else 0
    need = lib().pvlm_parallel_decode_workspace_bytes(C.byref(p))
    ws = _workspace(dev, "decode", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    if draft_stream is None and not serial:
        draft_stream = _side_stream(dev)
    st = lib().pvlm_parallel_decode(C.byref(p), _stream(dev), None if serial else C.c_void_p(draft_stream.cuda_stream))
    if st != 0:
        raise PvlmError(st, "pvlm_parallel_decode")
    n = int(n_rounds[0])
    return dict(tokens=tokens, rounds=n, log=log[:n], round_ms=None if ms is None else ms[:n])


_SIDE: dict = {}


def _side_stream(dev):
    s = _SIDE.get(dev.index)
    if s is None:
        s = _SIDE[dev.index] = torch.cuda.Stream(device=dev)
    return s


def acceptance_rate(target_logits, draft_logits, tokens, uniforms, temperature: float = 1.0, *, want_probs: bool = True):
    """Token-wise acceptance of a given text (see pvlm_acceptance_rate).  target_logits / draft_logits fp32 [N, V],
    tokens int32 [N], uniforms fp32 [N].  Returns dict(accepted int32 [N], n_accepted int32 [1], p_tok, q_tok)."""
    _need_cuda(target_logits, draft_logits, tokens, uniforms)
    N, V = target_logits.shape
    assert draft_logits.shape == (N, V) and target_logits.dtype == torch.float32 and draft_logits.dtype == torch.float32
    assert (N == 0 or (target_logits.stride(1) == 1 and draft_logits.stride(1) == 1)) and tokens.dtype == torch.int32
    dev = target_logits.device
    accepted = torch.empty(N, dtype=torch.int32, device=dev)
    cnt = torch.empty(1, dtype=torch.int32, device=dev)
    p_tok = torch.empty(N, dtype=torch.float32, device=dev) if want_probs else None
    q_tok = torch.empty(N, dtype=torch.float32, device=dev) if want_probs else None
    p = RateParams()
    p.target_logits, p.draft_logits = _ptr(target_logits), _ptr(draft_logits)
    p.target_row_stride = target_logits.stride(0) if N else V
    p.draft_row_stride = draft_logits.stride(0) if N else V
    p.tokens, p.uniforms = _ptr(tokens.contiguous()), _ptr(uniforms.contiguous())
    p.N, p.V, p.temperature = N, V, float(temperature)
    p.accepted, p.p_tok, p.q_tok, p.n_accepted = _ptr(accepted), _ptr(p_tok), _ptr(q_tok), _ptr(cnt)
    need = lib().pvlm_acceptance_rate_workspace_bytes(C.byref(p))
    ws = _workspace(dev, "rate", need)
    p.workspace, p.workspace_bytes = _ptr(ws), ws.numel()
    st = lib().pvlm_acceptance_rate(C.byref(p), _stream(dev))
    if st != 0:
        raise PvlmError(st, "pvlm_acceptance_rate")
    return dict(accepted=accepted, n_accepted=cnt, p_tok=p_tok, q_tok=q_tok)
