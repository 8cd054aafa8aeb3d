"""Seeded synthetic inputs shaped like the paper's LLaVA-Video streaming workloads.

This module only *draws inputs*: bf16 weight matrices, prompt/question/answer hidden
states and per-frame visual-token hidden states.  It contains none of the method's
arithmetic (no pooling, projection, attention, eviction), so both the CPU oracle's
tests and the CUDA path's tests may feed from it without sharing any method code.

Generator: counter based.  The 64-bit word for element ``index`` of tensor ``tag`` under
``seed`` is ``splitmix64(seed * GOLDEN + tag * 2**40 + index)``; its two 32-bit halves
give two uniforms, which Box-Muller turns into one standard normal in fp64.  Values are
scaled in fp64 and rounded to bf16 (fp64 -> fp32 -> bf16, both round-to-nearest-even;
this is the generator's definition of the input, not a precision claim).  All tensors
are returned as ``numpy.uint16`` arrays of bf16 bit patterns so that every consumer
sees the same bits.

Workloads (the paper's evaluation streams are 1 fps videos, 169-210 visual tokens per
frame after pooling, a Qwen2-7B-shaped backbone and a bank of 64 or 128 carriers --
Section 4.1 and Table 1; the videos themselves are not available, these stand in):

* ``tiny``      d=256, 4 query / 1 KV head, head_dim 64, 8-token prefix, 8 frames x 16
                tokens iid N(0,1), bank 4, 4 decode tokens.
* ``layer``     one Qwen2-7B-shaped layer: d=3584, 28/4 heads, head_dim 128, 64-token
                prefix, 64 frames x 169 tokens (frame-shared N(0,1) vector + per-token
                N(0,0.5) noise), bank 64, 32 decode tokens.
* ``long``      same layer, 1024 frames; the frame-level vector is AR(1) with rho=0.9
                and is redrawn with probability 0.5 at every 100th frame (scene cut);
                bank 256; 64-token question then 64 decode tokens.
* ``deep``      28 independent layers with a residual stream (no MLP), 512 frames,
                bank 512, 32-token question, 128 decode tokens.
* ``batched``   16 independent streams of up to 256 frames x 196 tokens, ragged lengths
                uniform in [64, 256], bank capacity 1024, 64 decode tokens per stream.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# tensor tags (one per logical tensor family; the layer / stream / frame index is mixed in)
TAG_WEIGHT = 1
TAG_PREFIX = 2
TAG_FRAME_SHARED = 3
TAG_FRAME_NOISE = 4
TAG_QUESTION = 5
TAG_DECODE = 6
TAG_SCENE_CUT = 7
TAG_LENGTHS = 8
TAG_BIAS = 9
TAG_NORM_W = 10
TAG_W_O = 11
TAG_W_GATE = 12
TAG_W_UP = 13
TAG_W_DOWN = 14
TAG_NORM2_W = 15
TAG_W_LM = 16
TAG_NORM_F_W = 17


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 finaliser on uint64 counters (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = x + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _counter_base(seed: int, tag: int) -> np.uint64:
    return np.uint64((seed * 0x9E3779B97F4A7C15 + (tag << 40)) & 0xFFFFFFFFFFFFFFFF)


def uniform_words(seed: int, tag: int, n: int, offset: int = 0) -> np.ndarray:
    idx = np.arange(offset, offset + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return splitmix64(_counter_base(seed, tag) + idx)


def standard_normal(seed: int, tag: int, n: int, offset: int = 0) -> np.ndarray:
    """``n`` fp64 standard normals, element i depending only on (seed, tag, offset+i)."""
    w = uniform_words(seed, tag, n, offset)
    hi = (w >> np.uint64(32)).astype(np.float64)
    lo = (w & np.uint64(0xFFFFFFFF)).astype(np.float64)
    u1 = (hi + 1.0) / 4294967296.0          # (0, 1]
    u2 = lo / 4294967296.0                  # [0, 1)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 (RNE) -> bf16 (RNE) bit patterns as uint16."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(seed: int, tag: int, shape, std: float = 1.0, offset: int = 0) -> np.ndarray:
    n = int(np.prod(shape))
    return to_bf16_bits(standard_normal(seed, tag, n, offset) * std).reshape(shape)


@dataclasses.dataclass
class Workload:
    """Shape and recipe of one synthetic streaming workload."""
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prefix_len: int
    n_frames: int
    tokens_per_frame: int
    bank_capacity: int
    question_len: int
    decode_tokens: int
    n_streams: int = 1
    frame_model: str = "iid"          # "iid" | "shared" | "ar1"
    token_noise_std: float = 0.5
    ar_rho: float = 0.9
    cut_period: int = 100
    cut_prob: float = 0.5
    min_frames: int = 0               # ragged stream lengths in [min_frames, n_frames] when > 0
    use_rmsnorm: int = 0
    residual: int = 0
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6
    weight_std: float = 0.02
    seed: int = 0

    @property
    def e_out(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    # ---- weights ---------------------------------------------------------------------
    def weight(self, layer: int) -> np.ndarray:
        """W_qkv of one layer, bf16 bits, shape [E_out, d_model] ("out x in", row-major).
        Rows are ordered Q heads, then K heads, then V heads."""
        n = self.e_out * self.d_model
        return normal_bf16(self.seed, TAG_WEIGHT, (self.e_out, self.d_model),
                           self.weight_std, offset=layer * n)

    def block_weights(self, layer: int, d_ff: int) -> dict:
        """The rest of decoder layer `layer` (output projection and SwiGLU MLP of width d_ff), bf16 bits,
        all "out x in"; drawn like the projection weights, N(0, weight_std^2)."""
        d = self.d_model
        draw = lambda tag, shape: normal_bf16(self.seed, tag, shape, self.weight_std, offset=layer * shape[0] * shape[1])
        return {"w_o": draw(TAG_W_O, (d, d)), "w_gate": draw(TAG_W_GATE, (d_ff, d)),
                "w_up": draw(TAG_W_UP, (d_ff, d)), "w_down": draw(TAG_W_DOWN, (d, d_ff))}

    def lm_weights(self, vocab: int) -> np.ndarray:
        """Vocabulary projection [vocab, d_model] of the language-model head, bf16 bits, N(0, weight_std^2)."""
        return normal_bf16(self.seed, TAG_W_LM, (vocab, self.d_model), self.weight_std)

    # ---- text-side hidden states -----------------------------------------------------
    def prefix_hidden(self, stream: int = 0) -> np.ndarray:
        n = self.prefix_len * self.d_model
        return normal_bf16(self.seed, TAG_PREFIX, (self.prefix_len, self.d_model), 1.0,
                           offset=stream * n)

    def question_hidden(self, stream: int = 0) -> np.ndarray:
        n = self.question_len * self.d_model
        return normal_bf16(self.seed, TAG_QUESTION, (self.question_len, self.d_model), 1.0,
                           offset=stream * n)

    def decode_hidden(self, step: int, stream: int = 0) -> np.ndarray:
        """Hidden state of one answer token (there is no LM head to feed back): [1, d]."""
        off = (stream * max(self.decode_tokens, 1) + step) * self.d_model
        return normal_bf16(self.seed, TAG_DECODE, (1, self.d_model), 1.0, offset=off)

    # ---- frames ----------------------------------------------------------------------
    def stream_lengths(self) -> List[int]:
        if self.min_frames <= 0:
            return [self.n_frames] * self.n_streams
        w = uniform_words(self.seed, TAG_LENGTHS, self.n_streams)
        span = self.n_frames - self.min_frames + 1
        return [int(self.min_frames + int(v % np.uint64(span))) for v in w]

    def frame_shared(self, stream: int = 0, n_frames: Optional[int] = None) -> np.ndarray:
        """Frame-level component f_t for t < n_frames, fp64 [n_frames, d]."""
        T = self.n_frames if n_frames is None else n_frames
        d = self.d_model
        base = stream * self.n_frames * d
        g = standard_normal(self.seed, TAG_FRAME_SHARED, T * d, offset=base).reshape(T, d)
        if self.frame_model != "ar1":
            return g
        cuts = uniform_words(self.seed, TAG_SCENE_CUT, T, offset=stream * self.n_frames)
        cut_u = (cuts >> np.uint64(11)).astype(np.float64) / float(1 << 53)
        f = np.empty_like(g)
        f[0] = g[0]
        c = math.sqrt(1.0 - self.ar_rho * self.ar_rho)
        for t in range(1, T):
            if t % self.cut_period == 0 and cut_u[t] < self.cut_prob:
                f[t] = g[t]                      # scene cut: redraw
            else:
                f[t] = self.ar_rho * f[t - 1] + c * g[t]
        return f

    def frame_hidden(self, t: int, stream: int = 0, shared: Optional[np.ndarray] = None) -> np.ndarray:
        """Visual-token hidden states of frame t: bf16 bits [N, d]."""
        N, d = self.tokens_per_frame, self.d_model
        off = (stream * self.n_frames + t) * N * d
        if self.frame_model == "iid":
            return normal_bf16(self.seed, TAG_FRAME_NOISE, (N, d), 1.0, offset=off)
        if shared is None:
            shared = self.frame_shared(stream, t + 1)
        noise = standard_normal(self.seed, TAG_FRAME_NOISE, N * d, offset=off).reshape(N, d)
        return to_bf16_bits(shared[t][None, :] + self.token_noise_std * noise)


def workload(name: str, **overrides) -> Workload:
    """The five named workloads; keyword overrides shrink them for tests."""
    q7 = dict(d_model=3584, n_q_heads=28, n_kv_heads=4, head_dim=128)
    table: Dict[str, dict] = {
        "tiny": dict(n_layers=1, d_model=256, n_q_heads=4, n_kv_heads=1, head_dim=64,
                     prefix_len=8, n_frames=8, tokens_per_frame=16, bank_capacity=4,
                     question_len=0, decode_tokens=4, frame_model="iid"),
        "layer": dict(n_layers=1, **q7, prefix_len=64, n_frames=64, tokens_per_frame=169,
                      bank_capacity=64, question_len=0, decode_tokens=32, frame_model="shared"),
        "long": dict(n_layers=1, **q7, prefix_len=64, n_frames=1024, tokens_per_frame=169,
                     bank_capacity=256, question_len=64, decode_tokens=64, frame_model="ar1"),
        "deep": dict(n_layers=28, **q7, prefix_len=64, n_frames=512, tokens_per_frame=169,
                     bank_capacity=512, question_len=32, decode_tokens=128, frame_model="ar1",
                     use_rmsnorm=1, residual=1),
        "batched": dict(n_layers=1, **q7, prefix_len=64, n_frames=256, tokens_per_frame=196,
                        bank_capacity=1024, question_len=0, decode_tokens=64, n_streams=16,
                        frame_model="ar1", min_frames=64),
    }
    if name not in table:
        raise KeyError(f"unknown workload {name!r}; choose from {sorted(table)}")
    kw = dict(table[name])
    kw.update(overrides)
    return Workload(name=name, **kw)
