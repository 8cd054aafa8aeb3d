"""CPU oracle for the VideoScan streaming attention path -- TEST INFRASTRUCTURE ONLY.

Plain, slow, fp64 numpy restatement of what the paper's inference procedure computes
for one attention sub-block per layer.  It is not part of the product: only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import it, and it shares
no code with the CUDA path.

What it follows (VideoScan, arXiv 2503.09387):

* Section 3.1, Eq. (1): ``Y = Softmax(Q K^T / sqrt(d_k)) V`` with ``Q = X W_Q`` etc.
* Section 3.2: the semantic carrier's input embedding is the average of the frame's
  token embeddings; the carrier sits at the END of its frame's visual tokens; its K/V is
  kept in the cache.
* Section 3.3, prefilling: ``C^t = (1/N) sum_i E^t_i``; up to M historical carriers are
  retrieved; order of the context is system prompt, visual, text.
* Section 3.3, decoding: visual tokens are processed once and discarded; decoding reads
  carriers only.
* Section 3.3, memory mechanism: the bank holds at most M carriers (embedding + K/V);
  when full, the older carrier with the largest cosine similarity to the incoming one
  is discarded.
* Section 3.4 / Fig. 3: later tokens may only see earlier frames through their carriers.

Readings taken where the paper is silent (all restated in the project's design notes):
multi-head GQA with rotary position embedding as in the Qwen2 backbone the paper uses
(Section 4.1); positions are those of the un-pruned sequence; keys are cached rotated;
attention of frame t sees the bank as left by frame t-1, then evict-if-full, then
append; eviction ties go to the oldest carrier; a zero-norm embedding has cosine 0.

Rounding points: inputs and weights are bf16 values held in fp64.  All arithmetic is
fp64.  Values are rounded to bf16 only where the method stores them: the carrier
embedding, K/V entering bank / prefix / text tail, and the residual stream between
layers.

Optional rest of the decoder block (the backbone of Section 4.1 is a Qwen2 decoder): with
``BlockWeights`` a layer is  h1 = h + A W_o^T,  h2 = h1 + (SiLU(n W_gate^T) * (n W_up^T)) W_down^T
with A the attention rows and n = RMSNorm(h1); storage points (bf16) are A, h1, the gated
activation and h2, and a step then returns the last layer's h2 instead of its attention rows.

Optional language-model head (``lm_head``): the final RMSNorm of the backbone, the vocabulary
projection and the greedy choice of the next token -- what turns the hidden state of the last
position into the first answer token of Section 3.3's decoding phase.

Parity pins (tests/test_oracle_*.py): closed forms for the pooling, softmax row sums,
GQA == MHA with repeated heads, brute-force dense masked attention over the un-pruned
sequence, textbook causal attention for M = 0 and one-frame streams, RoPE identities,
hand-built eviction sequences.  Beyond those identities the numerical values of the
attention output have no printed example in the paper: parity unpinned by the paper
itself, pinned by the definitions above.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------------------
# bf16 storage rounding (fp64 -> nearest bf16 value, ties to even, no intermediate fp32)
# --------------------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16-representable value of each fp64 element, ties to even.

    bf16 keeps 8 significant bits and has fp32's exponent range, so the spacing of
    representable values around x = m * 2^e (0.5 <= |m| < 1) is 2^(e-8), but never
    finer than the subnormal spacing 2^-133.  Rounding = nearest multiple of that
    spacing; ``np.rint`` rounds halves to even.
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    q = np.maximum(e - 8, -133)
    scaled = np.ldexp(x, -q)               # exact: power-of-two scaling
    return np.ldexp(np.rint(scaled), q)


def bf16_bits_of(x: np.ndarray) -> np.ndarray:
    """Bit patterns (uint16) of fp64 values that are already bf16-representable."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    if not np.array_equal(f.astype(np.float64), np.asarray(x, dtype=np.float64)):
        raise ValueError("value is not bf16-representable")
    u = np.ascontiguousarray(f).view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("value is not bf16-representable")
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------------------
# Section 3.3 (prefilling): semantic carrier = average pool of the frame's tokens
# --------------------------------------------------------------------------------------
def carrier_embedding(E: np.ndarray, agg_mode: int = 0) -> np.ndarray:
    """C = (1/N) sum_i E_i, shape [d] (Section 3.3).  ``agg_mode=1`` is the ablation of
    Section 4.3 / Table 4 ("w/o emb"): the last visual token stands in for the mean.
    The result is an input token of the bf16 model, hence rounded once to bf16."""
    E = np.asarray(E, dtype=np.float64)
    if agg_mode == 1:
        return E[-1].copy()
    N = E.shape[0]
    return round_to_bf16(E.sum(axis=0) / float(N))


# --------------------------------------------------------------------------------------
# Rotary position embedding (Qwen2-style rotate-half pairing)
# --------------------------------------------------------------------------------------
def rope_angles(positions: Sequence[int], head_dim: int, theta: float) -> np.ndarray:
    """angle[p, k] = pos_p * theta^(-2k/D), k < D/2, fp64."""
    k = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = theta ** (-2.0 * k / float(head_dim))
    return np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]


def apply_rope(x: np.ndarray, angles: np.ndarray) -> np.ndarray:
    """x: [rows, heads, D]; pairs (k, k + D/2) are rotated by angle[row, k]."""
    half = x.shape[-1] // 2
    c = np.cos(angles)[:, None, :]
    s = np.sin(angles)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


# --------------------------------------------------------------------------------------
# Eq. (1): softmax attention of some query rows over a key/value set with a mask
# --------------------------------------------------------------------------------------
def attention_rows(Q: np.ndarray, K: np.ndarray, V: np.ndarray, visible: np.ndarray) -> np.ndarray:
    """Q: [rows, Hq, D]; K, V: [keys, Hkv, D]; visible: bool [rows, keys].
    Query head q reads KV head q // (Hq / Hkv).  Returns [rows, Hq, D]."""
    rows, Hq, D = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    out = np.empty((rows, Hq, D), dtype=np.float64)
    scale = 1.0 / math.sqrt(float(D))
    for q in range(Hq):
        kv = q // G
        s = (Q[:, q, :] @ K[:, kv, :].T) * scale
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, q, :] = p @ V[:, kv, :]
    return out


# --------------------------------------------------------------------------------------
# Section 3.3 (memory mechanism): duplication-based eviction
# --------------------------------------------------------------------------------------
def _canonical_sum(prod: np.ndarray) -> np.ndarray:
    """Sum over the last axis in the fixed order both implementations agree on, so that
    the fp64 result is reproducible bit for bit: 32 interleaved running sums (element k
    goes to sum k mod 32, ascending k), then a pairwise tree 16, 8, 4, 2, 1."""
    d = prod.shape[-1]
    pad = (-d) % 32
    if pad:
        prod = np.concatenate([prod, np.zeros(prod.shape[:-1] + (pad,))], axis=-1)
    blocks = prod.reshape(prod.shape[:-1] + (-1, 32))
    acc = np.zeros(prod.shape[:-1] + (32,), dtype=np.float64)
    for r in range(blocks.shape[-2]):
        acc = acc + blocks[..., r, :]
    width = 16
    while width >= 1:
        acc = acc[..., :width] + acc[..., width:2 * width]
        width //= 2
    return acc[..., 0]


def canonical_dot(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Dot product over the last axis; the products of two bf16 values are exact in fp64."""
    with np.errstate(invalid="ignore", over="ignore"):
        return _canonical_sum(np.asarray(a, dtype=np.float64) * np.asarray(b, dtype=np.float64))


def cosine_similarity(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    dot = canonical_dot(a, b)
    na = canonical_dot(a, a)
    nb = canonical_dot(b, b)
    den = np.sqrt(na) * np.sqrt(nb)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        s = dot / den
    # the cosine is undefined for a zero vector and for a vector holding Inf or NaN: both count as 0
    # (the paper does not say; with 0 such a carrier is never preferred over a real duplicate, and
    # the argmax below always names a stored carrier)
    return np.where((na == 0.0) | (nb == 0.0) | ~np.isfinite(s), 0.0, s)


def choose_victim(bank_emb: np.ndarray, incoming: np.ndarray, policy: int = 0) -> int:
    """Index (temporal order, 0 = oldest) of the carrier to discard when the bank is full.

    Section 3.3 (memory mechanism) states the rule in one sentence that can be read two ways:
    policy 0: the stored carrier most similar (cosine) to the incoming carrier leaves -- every
              stored carrier is older than the incoming one, which is never the victim.
    policy 1: over the temporal sequence e_0 .. e_{M-1}, e_in, the older member of the most
              similar pair of NEIGHBOURS leaves (the reading that takes the comparison to be
              between carriers adjacent in time).
    policy 2: FIFO (oldest leaves); a test aid, not in the paper.
    Ties go to the oldest carrier; an undefined cosine (zero or non-finite vector) counts as 0."""
    if policy == 2:
        return 0
    if policy == 0:
        s = cosine_similarity(bank_emb, incoming[None, :])
    elif policy == 1:
        seq = np.concatenate([bank_emb, incoming[None, :]], axis=0)
        s = cosine_similarity(seq[:-1], seq[1:])
    else:
        raise ValueError("unknown eviction policy")
    return int(np.argmax(s))           # np.argmax returns the first (oldest) maximum


# --------------------------------------------------------------------------------------
# Stream state and the per-step procedure (Section 3.3)
# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class OracleConfig:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    bank_capacity: int
    agg_mode: int = 0
    evict_policy: int = 0
    use_rmsnorm: int = 0
    residual: int = 0
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6


@dataclasses.dataclass
class BlockWeights:
    """The rest of one decoder layer (Qwen2 block, Section 4.1 names the backbone): output
    projection and SwiGLU MLP.  All "out x in", bf16-valued fp64."""
    w_o: np.ndarray                 # [d, Hq*D]
    w_gate: np.ndarray              # [I, d]
    w_up: np.ndarray                # [I, d]
    w_down: np.ndarray              # [d, I]
    norm2_w: Optional[np.ndarray] = None   # [d] gain of the post-attention RMSNorm, or None (unit gain)


def silu(x: np.ndarray) -> np.ndarray:
    """SiLU(x) = x * sigmoid(x) = x / (1 + exp(-x))."""
    return x / (1.0 + np.exp(-x))


def lm_head(h: np.ndarray, w_lm: np.ndarray, gain: Optional[np.ndarray] = None, use_rmsnorm: bool = True,
            rms_eps: float = 1e-6):
    """Hidden states of the positions to be continued -> (logits, greedy next tokens).

    Section 3.3 (decoding phase): the answer is generated token by token from the model's output at the
    last position; the backbone of Section 4.1 (a Qwen2 decoder) ends in an RMSNorm and a vocabulary
    projection.  h: [rows][d] (rounded to bf16 on entry: a hidden state is a stored tensor);
    w_lm: [vocab][d] ("out x in"); gain: [d] of the final norm or None (unit gain).
    logits[r][v] = sum_k n[r][k] * w_lm[v][k] with n = RMSNorm(h) * gain (n = h without the norm), kept in
    fp64; token[r] = the index of the largest logit, the lowest index among equals."""
    h = round_to_bf16(np.asarray(h, dtype=np.float64))
    n = h
    if use_rmsnorm:
        ms = np.mean(h * h, axis=1, keepdims=True)
        n = h / np.sqrt(ms + rms_eps)
        if gain is not None:
            n = n * np.asarray(gain, dtype=np.float64)[None, :]
    logits = n @ np.asarray(w_lm, dtype=np.float64).T
    tokens = np.array([greedy_token(row) for row in logits], dtype=np.int64)
    return logits, tokens


def greedy_token(logits_row: np.ndarray) -> int:
    """Index of the largest value; the lowest index among equal largest values.  A NaN counts as
    smaller than every number (a row of NaNs gives token 0)."""
    best, best_v = 0, -math.inf
    for i, v in enumerate(np.asarray(logits_row, dtype=np.float64)):
        if v > best_v:                       # false for NaN
            best, best_v = i, float(v)
    return best


@dataclasses.dataclass
class BankEntry:
    frame_id: int
    pos: int
    emb: np.ndarray                 # [d] bf16-valued
    K: Optional[np.ndarray]         # [L, Hkv, D] bf16-valued (None in metadata-only runs)
    V: Optional[np.ndarray]


class OracleStream:
    """One video stream: prompt prefix, bounded carrier bank, per-turn text tail."""

    def __init__(self, cfg: OracleConfig, w_qkv: List[np.ndarray],
                 b_qkv: Optional[List[Optional[np.ndarray]]] = None,
                 norm_w: Optional[List[Optional[np.ndarray]]] = None,
                 blocks: Optional[List[BlockWeights]] = None):
        self.cfg = cfg
        self.blocks = blocks            # None: attention sub-block only (the five workloads)
        if blocks is not None and not cfg.residual:
            raise ValueError("the full decoder block needs the residual stream")
        L = cfg.n_layers
        self.w = [np.asarray(w, dtype=np.float64) for w in w_qkv]       # [E_out, d]
        self.b = b_qkv if b_qkv is not None else [None] * L
        self.g = norm_w if norm_w is not None else [None] * L
        Hkv, D = cfg.n_kv_heads, cfg.head_dim
        self.prefix_K = [np.zeros((0, Hkv, D)) for _ in range(L)]
        self.prefix_V = [np.zeros((0, Hkv, D)) for _ in range(L)]
        self.tail_K = [np.zeros((0, Hkv, D)) for _ in range(L)]
        self.tail_V = [np.zeros((0, Hkv, D)) for _ in range(L)]
        self.bank: List[BankEntry] = []
        self.frames_seen = 0
        self.next_pos = 0
        self.text_len = 0
        self.evictions = 0
        self.evict_log: List[tuple] = []        # (frame step, victim frame id)
        self.last_victim_frame = -1
        # test aid: when set to a list, every step appends {"kind", "h": [layer inputs], "O": [layer outputs]}
        self.record: Optional[list] = None

    # -- pieces -------------------------------------------------------------------------
    def _layer_input(self, h: np.ndarray, layer: int) -> np.ndarray:
        if not self.cfg.use_rmsnorm:
            return h
        ms = np.mean(h * h, axis=1, keepdims=True)
        y = h / np.sqrt(ms + self.cfg.rms_eps)
        if self.g[layer] is not None:
            y = y * np.asarray(self.g[layer], dtype=np.float64)[None, :]
        return y

    def _project(self, x: np.ndarray, layer: int):
        cfg = self.cfg
        y = x @ self.w[layer].T
        if self.b[layer] is not None:
            y = y + np.asarray(self.b[layer], dtype=np.float64)[None, :]
        nq, nk = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
        rows = x.shape[0]
        Q = y[:, :nq].reshape(rows, cfg.n_q_heads, cfg.head_dim)
        K = y[:, nq:nq + nk].reshape(rows, cfg.n_kv_heads, cfg.head_dim)
        V = y[:, nq + nk:].reshape(rows, cfg.n_kv_heads, cfg.head_dim)
        return Q, K, V

    def _rest_of_block(self, h: np.ndarray, O: np.ndarray, layer: int) -> np.ndarray:
        """h (layer input, bf16-valued) and the layer's attention rows O -> the layer's output h2."""
        blk = self.blocks[layer]
        A = round_to_bf16(O)                                   # the attention rows are a stored tensor
        h1 = round_to_bf16(h + A @ np.asarray(blk.w_o, dtype=np.float64).T)
        self.last_h1 = h1                                      # kept for inspection (the other stored tensor of the residual path)
        n = h1
        if self.cfg.use_rmsnorm:
            ms = np.mean(h1 * h1, axis=1, keepdims=True)
            n = h1 / np.sqrt(ms + self.cfg.rms_eps)
            if blk.norm2_w is not None:
                n = n * np.asarray(blk.norm2_w, dtype=np.float64)[None, :]
        g = n @ np.asarray(blk.w_gate, dtype=np.float64).T
        u = n @ np.asarray(blk.w_up, dtype=np.float64).T
        act = round_to_bf16(silu(g) * u)
        return round_to_bf16(h1 + act @ np.asarray(blk.w_down, dtype=np.float64).T)

    def _bank_kv(self, layer: int):
        Hkv, D = self.cfg.n_kv_heads, self.cfg.head_dim
        if not self.bank:
            return np.zeros((0, Hkv, D)), np.zeros((0, Hkv, D))
        return (np.stack([e.K[layer] for e in self.bank]),
                np.stack([e.V[layer] for e in self.bank]))

    # -- Section 3.3, prefilling phase: one frame ------------------------------------------
    def frame_step(self, E: np.ndarray, carrier_override: Optional[np.ndarray] = None,
                   mode: str = "full"):
        """Process frame t.  ``E``: [N, d] bf16-valued hidden states of the visual tokens.

        mode "full":    everything; returns the last layer's attention output [N+1, Hq*D].
        mode "carrier": single-layer streams only -- the carrier row's K/V needs no
                        attention, so only that row is projected (for long streams);
                        returns None.
        mode "meta":    pooling, eviction and bookkeeping only (bank K/V left as None).
        """
        cfg = self.cfg
        if self.text_len != 0:
            raise RuntimeError("a frame arrived while a text turn is open")
        E = np.asarray(E, dtype=np.float64)
        N = E.shape[0]
        c = carrier_embedding(E, cfg.agg_mode) if carrier_override is None \
            else np.asarray(carrier_override, dtype=np.float64)
        positions = [self.next_pos + i for i in range(N + 1)]
        L, Hkv, D = cfg.n_layers, cfg.n_kv_heads, cfg.head_dim
        out = None
        cK = cV = None
        if mode == "full":
            X = np.concatenate([E, c[None, :]], axis=0)          # carrier is the last token
            ang = rope_angles(positions, D, cfg.rope_theta)
            cK = np.zeros((L, Hkv, D))
            cV = np.zeros((L, Hkv, D))
            h = X
            rec = {"kind": "frame", "h": [], "O": []}
            for l in range(L):
                rec["h"].append(h)
                Q, K, V = self._project(self._layer_input(h, l), l)
                Q = apply_rope(Q, ang)
                K = apply_rope(K, ang)
                bK, bV = self._bank_kv(l)
                P, nb = self.prefix_K[l].shape[0], bK.shape[0]
                Kall = np.concatenate([self.prefix_K[l], bK, K], axis=0)
                Vall = np.concatenate([self.prefix_V[l], bV, V], axis=0)
                vis = np.ones((N + 1, P + nb + N + 1), dtype=bool)
                vis[:, P + nb:] = np.tril(np.ones((N + 1, N + 1), dtype=bool))
                O = attention_rows(Q, Kall, Vall, vis).reshape(N + 1, -1)
                cK[l] = round_to_bf16(K[N])
                cV[l] = round_to_bf16(V[N])
                out = O
                rec["O"].append(O)
                if self.blocks is not None:
                    h = self._rest_of_block(h, O, l)
                    out = h
                elif cfg.residual:
                    h = round_to_bf16(h + O)
                rec.setdefault("h_out", []).append(h)
                rec.setdefault("h1", []).append(getattr(self, "last_h1", None))
            if self.record is not None:
                self.record.append(rec)
        elif mode == "carrier":
            if L != 1 or cfg.use_rmsnorm:
                raise ValueError("carrier-only mode needs a single layer without norm")
            ang = rope_angles(positions[N:], D, cfg.rope_theta)
            _, K, V = self._project(c[None, :], 0)
            K = apply_rope(K, ang)
            cK = round_to_bf16(K[0])[None]
            cV = round_to_bf16(V[0])[None]
        elif mode != "meta":
            raise ValueError(mode)

        # memory mechanism: evict if full, then append
        self.last_victim_frame = -1
        M = cfg.bank_capacity
        if M > 0:
            if len(self.bank) == M:
                emb = np.stack([e.emb for e in self.bank])
                j = choose_victim(emb, c, cfg.evict_policy)
                victim = self.bank.pop(j)
                self.evictions += 1
                self.last_victim_frame = victim.frame_id
                self.evict_log.append((self.frames_seen, victim.frame_id))
            self.bank.append(BankEntry(self.frames_seen, positions[N], c, cK, cV))
        self.next_pos += N + 1
        self.frames_seen += 1
        return out

    # -- Section 3.3, decoding phase (and the text part of prefilling) ---------------------
    def text_step(self, X: np.ndarray) -> np.ndarray:
        """T text tokens (prompt prefix before the first frame, otherwise question /
        answer tokens).  Each sees prefix, bank, and text tokens up to itself."""
        cfg = self.cfg
        X = np.asarray(X, dtype=np.float64)
        T = X.shape[0]
        L, D = cfg.n_layers, cfg.head_dim
        to_prefix = self.frames_seen == 0
        base = self.next_pos if to_prefix else self.next_pos + self.text_len
        ang = rope_angles([base + i for i in range(T)], D, cfg.rope_theta)
        h = X
        out = None
        rec = {"kind": "text", "h": [], "O": []}
        for l in range(L):
            rec["h"].append(h)
            Q, K, V = self._project(self._layer_input(h, l), l)
            Q = apply_rope(Q, ang)
            K = round_to_bf16(apply_rope(K, ang))
            V = round_to_bf16(V)
            bK, bV = self._bank_kv(l)
            # before the first frame the bank and the tail are empty, so this is the prefix alone
            ctxK = [self.prefix_K[l], bK, self.tail_K[l]]
            ctxV = [self.prefix_V[l], bV, self.tail_V[l]]
            nctx = sum(a.shape[0] for a in ctxK)
            Kall = np.concatenate(ctxK + [K], axis=0)
            Vall = np.concatenate(ctxV + [V], axis=0)
            vis = np.ones((T, nctx + T), dtype=bool)
            vis[:, nctx:] = np.tril(np.ones((T, T), dtype=bool))
            O = attention_rows(Q, Kall, Vall, vis).reshape(T, -1)
            if to_prefix:
                self.prefix_K[l] = np.concatenate([self.prefix_K[l], K], axis=0)
                self.prefix_V[l] = np.concatenate([self.prefix_V[l], V], axis=0)
            else:
                self.tail_K[l] = np.concatenate([self.tail_K[l], K], axis=0)
                self.tail_V[l] = np.concatenate([self.tail_V[l], V], axis=0)
            out = O
            rec["O"].append(O)
            if self.blocks is not None:
                h = self._rest_of_block(h, O, l)
                out = h
            elif cfg.residual:
                h = round_to_bf16(h + O)
            rec.setdefault("h_out", []).append(h)
            rec.setdefault("h1", []).append(getattr(self, "last_h1", None))
        if self.record is not None:
            self.record.append(rec)
        if to_prefix:
            self.next_pos += T
        else:
            self.text_len += T
        return out

    def carriers_only_forward(self) -> np.ndarray:
        """The bank's carriers as ordinary tokens, one per frame (Section 3.4, stage 1: the visual
        input is the semantic carrier tokens only; Section 4.3, inference without KV reuse): the
        stored carrier *embeddings*, in temporal order, go through the layers after the prompt
        prefix, each seeing the prefix and the carriers up to itself.  The stored K/V are not
        used and nothing changes.  Carrier i of this compact sequence sits at position
        prefix_len + i.  Returns the last layer's outputs [count, Hq*D]."""
        cfg = self.cfg
        T = len(self.bank)
        if T == 0:
            return np.zeros((0, cfg.n_q_heads * cfg.head_dim))
        h = np.stack([np.asarray(e.emb, dtype=np.float64) for e in self.bank])
        ang = rope_angles([self.prefix_len + i for i in range(T)], cfg.head_dim, cfg.rope_theta)
        out = None
        for l in range(cfg.n_layers):
            Q, K, V = self._project(self._layer_input(h, l), l)
            Q = apply_rope(Q, ang)
            K = round_to_bf16(apply_rope(K, ang))
            V = round_to_bf16(V)
            P = self.prefix_K[l].shape[0]
            Kall = np.concatenate([self.prefix_K[l], K], axis=0)
            Vall = np.concatenate([self.prefix_V[l], V], axis=0)
            vis = np.ones((T, P + T), dtype=bool)
            vis[:, P:] = np.tril(np.ones((T, T), dtype=bool))
            out = attention_rows(Q, Kall, Vall, vis).reshape(T, -1)
            if self.blocks is not None:
                h = self._rest_of_block(h, out, l)          # full decoder layer: the result is its hidden state
                out = h
            elif cfg.residual:
                h = round_to_bf16(h + out)
        return out

    def end_turn(self) -> None:
        """Drop the question/answer tail; prefix and bank stay, frame positions do not move."""
        Hkv, D = self.cfg.n_kv_heads, self.cfg.head_dim
        for l in range(self.cfg.n_layers):
            self.tail_K[l] = np.zeros((0, Hkv, D))
            self.tail_V[l] = np.zeros((0, Hkv, D))
        self.text_len = 0

    # -- inspection ------------------------------------------------------------------------
    @property
    def prefix_len(self) -> int:
        return self.prefix_K[0].shape[0]

    def bank_frame_ids(self) -> List[int]:
        return [e.frame_id for e in self.bank]

    def bank_positions(self) -> List[int]:
        return [e.pos for e in self.bank]
