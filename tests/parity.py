"""Shared machinery of the GPU parity tests: runs the same seeded inputs through the CUDA
library (via the C ABI binding) and through the CPU oracle, and compares.

Tolerances (bf16 inputs, fp32 accumulation on the GPU, fp64 oracle): attention outputs
max |err| <= 2e-2 and relative RMS <= 1e-2; bank bookkeeping, eviction trace and carrier
embeddings bit-exact; bank K/V within one bf16 unit in the last place of the oracle's.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from oracle import videoscan_oracle as vo
from paper_2503_09387_b200 import binding, synth

MAX_ABS = 2e-2
REL_RMS = 1e-2


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def errors(got: np.ndarray, want: np.ndarray):
    diff = got - want
    max_abs = float(np.max(np.abs(diff))) if diff.size else 0.0
    rel_rms = float(np.sqrt(np.mean(diff ** 2)) / max(np.sqrt(np.mean(want ** 2)), 1e-30)) if diff.size else 0.0
    return max_abs, rel_rms


def assert_close(got: np.ndarray, want: np.ndarray, what: str):
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite GPU output"
    max_abs, rel_rms = errors(got, want)
    assert max_abs <= MAX_ABS and rel_rms <= REL_RMS, f"{what}: max_abs={max_abs:.3e} rel_rms={rel_rms:.3e}"
    return max_abs, rel_rms


def assert_close_stored(got: np.ndarray, want: np.ndarray, what: str, widen: float = 1.0):
    """For outputs that are bf16 storage points on both sides (the hidden state a full decoder block returns): the
    two values are roundings of unrounded values that meet an absolute bound, and each rounding moves its value by
    at most half a bf16 unit, so |got - want| <= bound + one unit in the last place of the value (2^-8 .. 2^-7 of
    it: 3.1e-2 at |h| in [4, 8)).  The bound is the stated 2e-2 times `widen`: the stated figure covers one
    contraction over d_model of bf16-rounded operands; the block adds one over d_ff of the bf16-stored activation,
    and rounding noise grows with the square root of the contraction length, widen = sqrt(1 + d_ff / d_model).
    Relative RMS as stated."""
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite GPU output"
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 2.0 ** -126))) - 7)
    bad = np.abs(got - want) > MAX_ABS * widen + ulp
    max_abs, rel_rms = errors(got, want)
    assert not bad.any() and rel_rms <= REL_RMS, f"{what}: {int(bad.sum())} elements beyond {MAX_ABS * widen:.1e} + 1 ulp, max_abs={max_abs:.3e} rel_rms={rel_rms:.3e}"
    return max_abs, rel_rms


def assert_within_one_ulp(got_bits: np.ndarray, want_vals: np.ndarray, what: str):
    got = synth.bf16_bits_to_f64(got_bits)
    want = np.asarray(want_vals, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    # one bf16 ulp is at most 2^-7 relative; values that cancel to ~0 in the rotation carry the
    # fp32 accumulation error of O(1) operands, hence the absolute floor
    tol = np.maximum(np.abs(want) * 2.0 ** -7, 1e-5)
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{what}: {int(bad.sum())} elements differ by more than one bf16 ulp"
    frac = float(np.mean(got != want))
    assert frac < 0.05, f"{what}: {frac:.3%} of elements differ from the oracle's rounding"


_WEIGHTS = {}


def layer_weight(w: synth.Workload, layer: int) -> np.ndarray:
    """w.weight(layer), kept for the session: the 28-layer workloads regenerate ~1 GB of weights per test otherwise."""
    key = (w.seed, w.e_out, w.d_model, w.weight_std, layer)
    if key not in _WEIGHTS:
        _WEIGHTS[key] = w.weight(layer)
    return _WEIGHTS[key]


class Pair:
    """One workload run side by side: ``gpu`` (StreamBatch) and ``ora`` (one OracleStream per stream)."""

    def __init__(self, w: synth.Workload, n_streams: Optional[int] = None, max_step_tokens: int = 64,
                 evict_policy: int = 0, agg_mode: int = 0, with_bias: bool = False, with_gain: bool = False,
                 max_tokens_per_frame: Optional[int] = None, max_prefix: Optional[int] = None,
                 max_text: Optional[int] = None, out_dtype: int = 1, max_chunk_frames: int = 1, d_ff: int = 0):
        self.w = w
        S = n_streams or w.n_streams
        self.S = S
        wbits = [layer_weight(w, l) for l in range(w.n_layers)]
        bbits = [synth.normal_bf16(w.seed, synth.TAG_BIAS, (w.e_out,), 0.1, offset=l * w.e_out)
                 for l in range(w.n_layers)] if with_bias else None
        gbits = [synth.to_bf16_bits(1.0 + 0.1 * synth.standard_normal(w.seed, synth.TAG_NORM_W, w.d_model,
                                                                      offset=l * w.d_model))
                 for l in range(w.n_layers)] if with_gain else None
        self.cfg = binding.make_config(
            w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim,
            max_tokens_per_frame or w.tokens_per_frame,
            max_prefix if max_prefix is not None else max(w.prefix_len, 1),
            max_text if max_text is not None else max(w.question_len + w.decode_tokens, 1),
            w.bank_capacity, n_streams=S, max_step_tokens=max_step_tokens, agg_mode=agg_mode,
            evict_policy=evict_policy, use_rmsnorm=w.use_rmsnorm, residual=w.residual,
            rope_theta=w.rope_theta, rms_eps=w.rms_eps, out_dtype=out_dtype, max_chunk_frames=max_chunk_frames, d_ff=d_ff)
        # the rest of the decoder block (output projection, SwiGLU MLP), with a gain for its norm when gains are on
        blk = [w.block_weights(l, d_ff) for l in range(w.n_layers)] if d_ff else None
        g2 = [synth.to_bf16_bits(1.0 + 0.1 * synth.standard_normal(w.seed, synth.TAG_NORM2_W, w.d_model, offset=l * w.d_model))
              for l in range(w.n_layers)] if (d_ff and with_gain) else None
        dev_block = None
        if blk:
            dev_block = {k: [to_dev(b[k]) for b in blk] for k in ("w_o", "w_gate", "w_up", "w_down")}
            dev_block["norm2_w"] = [to_dev(g) for g in g2] if g2 else None
        self.gpu = binding.StreamBatch(self.cfg, [to_dev(b) for b in wbits],
                                       [to_dev(b) for b in bbits] if bbits else None,
                                       [to_dev(b) for b in gbits] if gbits else None, dev_block)
        ocfg = vo.OracleConfig(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity,
                               agg_mode=agg_mode, evict_policy=evict_policy, use_rmsnorm=w.use_rmsnorm,
                               residual=w.residual, rope_theta=w.rope_theta, rms_eps=w.rms_eps)
        f64 = synth.bf16_bits_to_f64
        oblk = [vo.BlockWeights(f64(b["w_o"]), f64(b["w_gate"]), f64(b["w_up"]), f64(b["w_down"]),
                                f64(g2[l]) if g2 else None) for l, b in enumerate(blk)] if blk else None
        self.ora: List[vo.OracleStream] = [
            vo.OracleStream(ocfg, [f64(b) for b in wbits],
                            [f64(b) for b in bbits] if bbits else None,
                            [f64(b) for b in gbits] if gbits else None, oblk) for _ in range(S)]
        self.worst = [0.0, 0.0]
        widen = float(np.sqrt(1.0 + d_ff / w.d_model))
        self.close_fn = (lambda g, t, what: assert_close_stored(g, t, what, widen)) if d_ff else assert_close

    def _note(self, e):
        self.worst[0] = max(self.worst[0], e[0])
        self.worst[1] = max(self.worst[1], e[1])

    def text(self, ids: List[int], bits: List[np.ndarray], what: str = "text", compare: bool = True):
        """bits[i]: [T, d] for stream ids[i]."""
        x = to_dev(np.stack(bits))
        out = self.gpu.decode_step(ids, x)
        got = to_f64(out)
        for i, sid in enumerate(ids):
            want = self.ora[sid].text_step(synth.bf16_bits_to_f64(bits[i]))
            if compare:
                self._note(self.close_fn(got[i], want, f"{what} stream {sid}"))
        return got

    def frame(self, ids: List[int], bits: List[np.ndarray], what: str = "frame", mode="full",
              override: Optional[List[np.ndarray]] = None):
        """bits[i]: [N, d].  mode: 'full' compares outputs; 'carrier' / 'meta' only advance the oracle.
        A list gives every listed stream its own mode."""
        modes = [mode] * len(ids) if isinstance(mode, str) else list(mode)
        x = to_dev(np.stack(bits))
        ov = to_dev(np.stack(override)) if override is not None else None
        out = self.gpu.frame_prefill(ids, x, carrier_override=ov, want_out=("full" in modes))
        got = to_f64(out) if out is not None else None
        for i, sid in enumerate(ids):
            o = synth.bf16_bits_to_f64(override[i]) if override is not None else None
            want = self.ora[sid].frame_step(synth.bf16_bits_to_f64(bits[i]), carrier_override=o, mode=modes[i])
            if modes[i] == "full":
                self._note(self.close_fn(got[i], want, f"{what} stream {sid}"))
        return got

    def frame_chunk(self, sid: int, bits: List[np.ndarray], what: str = "chunk"):
        """bits[j]: [N, d], consecutive frames of stream sid in one vs_frame_prefill_chunk call; the
        oracle takes them as streaming steps, one at a time."""
        out = self.gpu.frame_prefill_chunk(sid, to_dev(np.stack(bits)))
        got = to_f64(out)
        for j, b in enumerate(bits):
            want = self.ora[sid].frame_step(synth.bf16_bits_to_f64(b), mode="full")
            self._note(assert_close(got[j], want, f"{what} frame {j} of the chunk"))
        return got

    def bank_forward(self, sid: int = 0, what: str = "carriers-only forward"):
        """vs_bank_forward against the oracle's carriers_only_forward; neither may change the stream."""
        want = self.ora[sid].carriers_only_forward()
        got = to_f64(self.gpu.bank_forward(sid, want.shape[0]))
        if want.shape[0]:
            self._note(assert_close(got, want, what))
        return got

    def check_bank(self, sid: int = 0, layer: Optional[int] = 0, kv: bool = True):
        ora = self.ora[sid]
        st = self.gpu.bank_state(sid, layer=layer if kv else None, want_emb=True)
        assert st["device_status"] == 0
        M = self.w.bank_capacity
        assert st["count"] == len(ora.bank) == min(ora.frames_seen, M)
        assert st["frames_seen"] == ora.frames_seen and st["evictions"] == ora.evictions
        assert st["next_pos"] == ora.next_pos and st["prefix_len"] == ora.prefix_len
        assert st["text_len"] == ora.text_len
        assert st["last_victim_frame"] == ora.last_victim_frame
        assert list(st["frame_ids"]) == ora.bank_frame_ids()
        assert list(st["positions"]) == ora.bank_positions()
        assert len(set(st["slots"].tolist())) == st["count"]
        n_log = len(st["evict_log"])
        assert [tuple(r) for r in st["evict_log"].tolist()] == ora.evict_log[len(ora.evict_log) - n_log:]
        if st["count"]:
            want_emb = np.stack([vo.bf16_bits_of(e.emb) for e in ora.bank])
            assert np.array_equal(st["emb"], want_emb), "carrier embeddings are not bit-exact"
        if kv and st["count"] and ora.bank[0].K is not None:
            wk = np.stack([e.K[layer] for e in ora.bank])
            wv = np.stack([e.V[layer] for e in ora.bank])
            if layer == 0 and not self.w.use_rmsnorm:
                assert_within_one_ulp(st["k"], wk, "bank K")
                assert_within_one_ulp(st["v"], wv, "bank V")
            else:   # the bf16 normalised input and, deeper down, the bf16 residual stream are
                    # GPU-internal roundings the oracle does not mirror
                assert_close(synth.bf16_bits_to_f64(st["k"]), wk, f"bank K layer {layer}")
                assert_close(synth.bf16_bits_to_f64(st["v"]), wv, f"bank V layer {layer}")
        return st

    def close(self):
        self.gpu.close()
