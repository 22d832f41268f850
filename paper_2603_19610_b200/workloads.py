"""Seeded synthetic inputs shaped like the paper's Video-LLM workloads.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic (no attention, no softmax, no selection).  Both the CUDA
path's tests/bench and the CPU oracle's tests take their inputs from here so
that the two sides see identical bytes.

Shapes follow the paper's setting: a multimodal prefix of m visual tokens
(frames x tokens per frame) followed by n text tokens (Sec. 2.1), a draft
window of gamma tokens verified in one target pass (Sec. 2.2), pruning ratio
alpha with keep ratio 1 - alpha (Eq. 3 / Eq. 5), vocabulary 152,064 for the
Qwen2-family targets the paper evaluates (Sec. 5).

bf16 tensors are carried as uint16 bit patterns (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
from numpy.random import Generator, Philox

BASE_SEED = 260319000

# random streams (one Philox key per (config, stream, layer))
S_Q, S_K, S_V, S_REF, S_TLOGIT, S_DNOISE, S_DTOK, S_STEPU, S_STRUCT, S_HIDDEN = range(10)


@dataclass(frozen=True)
class Config:
    """One workload: attention geometry, context split, window, vocab, pruning."""

    cid: int
    name: str
    Hq: int
    Hkv: int
    D: int
    frames: int
    tok_per_frame: int
    n_text: int
    gamma: int
    V: int
    keep_percent: int       # keep ratio r = 1 - alpha, as an integer percent
    n_layers: int
    sink: bool              # +6 logit spike on token 0
    draft_sigma: float
    repeat_frac: float = 0.0  # share of frames drawn from one repeated pattern
    ref_layer: int = 0      # layer pair for the variation score (multi-layer)
    cur_layer: int = 0
    d_model: int = 256      # width of the target's token representations (hidden-state criterion)

    @property
    def m(self) -> int:
        return self.frames * self.tok_per_frame

    @property
    def n_ctx(self) -> int:
        return self.m + self.n_text

    @property
    def R(self) -> int:
        return self.gamma + 1

    @property
    def T(self) -> int:
        return self.n_ctx + self.R

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def k_keep(self) -> int:
        return (self.m * self.keep_percent) // 100

    @property
    def kv_bytes_per_layer(self) -> int:
        return 2 * self.T * self.Hkv * self.D * 2


CONFIGS = (
    Config(0, "tiny", 4, 1, 64, 14, 64, 128, 4, 1024, 25, 1, False, 0.5, d_model=256),
    Config(1, "qwen2.5-vl-7b-layer", 28, 4, 128, 64, 240, 1024, 8, 152064, 10, 1, True, 0.5, d_model=3584),
    Config(2, "qwen2.5-vl-32b-64L", 40, 8, 128, 128, 240, 2048, 12, 152064, 10, 64, True, 0.5,
           ref_layer=0, cur_layer=19, d_model=5120),
    Config(3, "llava-ov-72b-80L", 64, 8, 128, 64, 196, 512, 10, 152064, 15, 80, True, 0.8,
           ref_layer=0, cur_layer=19, d_model=8192),
    Config(4, "long-video-stress", 40, 8, 128, 512, 256, 2048, 16, 152064, 5, 1, True, 0.5,
           repeat_frac=0.3, d_model=5120),
)


def rng_for(cfg_id: int, stream: int, layer: int = 0) -> Generator:
    return Generator(Philox(key=[BASE_SEED + 100 * cfg_id + stream, layer]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit pattern (finite inputs)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def position_bias(T: int, sink: bool) -> np.ndarray:
    """Additive logit bias per key position: a recency ramp 0 -> 2, plus an
    attention-sink spike of +6 on token 0 (the two ends Fig. 2 of the paper
    shows attention-guided picks piling onto)."""
    j = np.arange(T, dtype=np.float64)
    b = 2.0 * j / max(T - 1, 1)
    if sink:
        b[0] += 6.0
    return b.astype(np.float32)


def make_qkv_f32(Hq: int, Hkv: int, D: int, R: int, T: int, sink: bool, rng_q: Generator,
                 rng_k: Generator, rng_v: Generator, bias: bool = True):
    """Q [R,Hq,D], K,V [T,Hkv,D] in fp32 before bf16 rounding, N(0,1) content.  The positional
    bias is carried in the data so that the kernel stays a plain attention:
    channel D-1 of every query is sqrt(D) and channel D-1 of key j is b(j), so
    the scaled dot product gains b(j) (up to bf16 rounding of sqrt(D))."""
    q = rng_q.standard_normal((R, Hq, D), dtype=np.float32)
    k = rng_k.standard_normal((T, Hkv, D), dtype=np.float32)
    v = rng_v.standard_normal((T, Hkv, D), dtype=np.float32)
    if bias:
        q[:, :, D - 1] = np.float32(np.sqrt(D))
        k[:, :, D - 1] = position_bias(T, sink)[:, None]
    return q, k, v


def make_qkv(Hq: int, Hkv: int, D: int, R: int, T: int, sink: bool, seed: int, bias: bool = True):
    """Free-shape variant for tests: bf16 bit patterns of (Q, K, V) from one seed."""
    rq, rk, rv = (Generator(Philox(key=[seed, i])) for i in range(3))
    q, k, v = make_qkv_f32(Hq, Hkv, D, R, T, sink, rq, rk, rv, bias)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def attn_layer(cfg: Config, layer: int = 0, role: str = "cur"):
    """One layer's verify-attention inputs for a config: (q, k, v) bf16 bits.

    role="ref" draws the synthetic reference layer used by single-layer
    configs for the variation score: independent content, same bias channel
    (positional bias is layer-invariant, which is the paper's argument for
    taking layer-to-layer differences, Appendix E)."""
    if role == "ref":
        rq = rng_for(cfg.cid, S_REF, 3 * layer)
        rk = rng_for(cfg.cid, S_REF, 3 * layer + 1)
        rv = rng_for(cfg.cid, S_REF, 3 * layer + 2)
    else:
        rq, rk, rv = (rng_for(cfg.cid, s, layer) for s in (S_Q, S_K, S_V))
    q, k, v = make_qkv_f32(cfg.Hq, cfg.Hkv, cfg.D, cfg.R, cfg.T, cfg.sink, rq, rk, rv)
    if cfg.repeat_frac > 0.0:
        _apply_repeated_frames(cfg, k, v, layer, role)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def _apply_repeated_frames(cfg: Config, k: np.ndarray, v: np.ndarray, layer: int, role: str) -> None:
    """Long-video stress: a seeded 30 % of the frames hold one shared pattern
    frame plus N(0, 0.1^2) noise, so attention masses have near-ties."""
    rs = rng_for(cfg.cid, S_STRUCT, 2 * layer + (1 if role == "ref" else 0))
    n_rep = int(cfg.repeat_frac * cfg.frames)
    frames = np.sort(rs.choice(cfg.frames, size=n_rep, replace=False))
    tpf, D = cfg.tok_per_frame, cfg.D
    pat_k = rs.standard_normal((tpf, cfg.Hkv, D), dtype=np.float32)
    pat_v = rs.standard_normal((tpf, cfg.Hkv, D), dtype=np.float32)
    for f in frames:
        lo = f * tpf
        bias_col = k[lo:lo + tpf, :, D - 1].copy()
        k[lo:lo + tpf] = pat_k + np.float32(0.1) * rs.standard_normal((tpf, cfg.Hkv, D), dtype=np.float32)
        k[lo:lo + tpf, :, D - 1] = bias_col
        v[lo:lo + tpf] = pat_v + np.float32(0.1) * rs.standard_normal((tpf, cfg.Hkv, D), dtype=np.float32)


def make_logits(V: int, gamma: int, sigma: float, rng_t: Generator, rng_d: Generator,
                target_std: float = 3.0):
    """target fp32 [gamma+1, V] ~ N(0, target_std^2); draft[t] = target[t] + N(0, sigma^2)."""
    target = (np.float32(target_std) * rng_t.standard_normal((gamma + 1, V), dtype=np.float32))
    draft = target[:gamma] + np.float32(sigma) * rng_d.standard_normal((gamma, V), dtype=np.float32)
    return np.ascontiguousarray(target, dtype=np.float32), np.ascontiguousarray(draft, dtype=np.float32)


def unit_uniforms(rng: Generator, shape) -> np.ndarray:
    """fp32 uniforms in [0, 1): integer multiples of 2^-24."""
    return (rng.integers(0, 1 << 24, size=shape).astype(np.float32) * np.float32(2.0 ** -24))


def gumbel_draft_tokens(draft_logits: np.ndarray, rng: Generator, temperature: float = 1.0) -> np.ndarray:
    """Drafted tokens x_t distributed as the draft model's distribution at the
    given temperature, drawn by the Gumbel-max trick (argmax of logits/temp
    plus Gumbel noise) so that no softmax is evaluated here."""
    u = rng.random(draft_logits.shape)
    u = np.clip(u, 1e-300, 1.0 - 1e-16)
    g = -np.log(-np.log(u))
    return np.argmax(draft_logits.astype(np.float64) / temperature + g, axis=1).astype(np.int32)


def accept_inputs(cfg: Config, step: int = 0):
    """(target_logits, draft_logits, draft_tokens, uniforms[gamma+1]) for one step."""
    t, d = make_logits(cfg.V, cfg.gamma, cfg.draft_sigma, rng_for(cfg.cid, S_TLOGIT, step),
                       rng_for(cfg.cid, S_DNOISE, step))
    tok = gumbel_draft_tokens(d, rng_for(cfg.cid, S_DTOK, step))
    u = unit_uniforms(rng_for(cfg.cid, S_STEPU, step), cfg.gamma + 1)
    return t, d, tok, u


def kv_cache_layers(cfg: Config, n_layers: int, layer0: int = 0):
    """Stacked K, V [n_layers, T, Hkv, D] bf16 bits (for gather tests)."""
    ks, vs = [], []
    for l in range(layer0, layer0 + n_layers):
        _, k, v = attn_layer(cfg, l)
        ks.append(k)
        vs.append(v)
    return np.stack(ks), np.stack(vs)


def hidden_layer(cfg: Config, layer: int, d_model: int | None = None, m: int | None = None, n: int | None = None):
    """Token representations of one early target layer, bf16 bits [m + n, d]: visual rows then text
    rows (the prefix order of Sec. 2.1).  Content is N(0,1) per layer; on top of it every row carries
    a layer-invariant positional component beta(i) * p along a fixed direction p that the text rows
    share (ramp towards the text boundary, spike on token 0), so that raw similarity favours the two
    ends of the video and the layer-to-layer variation does not (Appendix E's argument)."""
    d = d_model or cfg.d_model
    m = cfg.m if m is None else m
    n = cfg.n_text if n is None else n
    rc = rng_for(cfg.cid, S_HIDDEN, layer + 1)
    rp = rng_for(cfg.cid, S_HIDDEN, 0)                    # positional direction: the same in every layer
    h = rc.standard_normal((m + n, d), dtype=np.float32)
    p = rp.standard_normal(d, dtype=np.float32)
    p *= np.float32(np.sqrt(d) / np.linalg.norm(p))
    beta = np.zeros(m + n, dtype=np.float32)
    beta[:m] = 0.6 * np.arange(m, dtype=np.float32) / max(m - 1, 1)
    beta[0] += 1.0
    beta[m:] = 0.8
    h += beta[:, None] * p[None, :]
    # a layer-dependent "semantic" gain for a seeded subset of visual tokens: these gain alignment with the text
    sem = rng_for(cfg.cid, S_HIDDEN, 0).choice(m, size=max(1, m // 10), replace=False)
    t_dir = h[m:].mean(axis=0)
    h[sem] += np.float32(0.03 * layer) * t_dir[None, :]
    return f32_to_bf16_bits(h)
