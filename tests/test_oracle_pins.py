"""Pins for the CPU oracle: closed forms, invariants, library routines and brute force.

None of these tests touches the CUDA path.  Each one is chosen so that a plausible
mistake in the oracle (dropped term, wrong sign or index, transposed operand, wrong
visibility) makes it fail.
"""
import math

import numpy as np
import pytest
import torch

from oracle import videoscan_oracle as vo
from paper_2503_09387_b200 import synth


def _rng(seed):
    return np.random.default_rng(seed)


def _bf16_vals(rng, shape, std=1.0):
    """bf16-representable fp64 values via torch's own conversion (independent of the oracle)."""
    x = torch.from_numpy(rng.standard_normal(shape) * std).to(torch.float32).to(torch.bfloat16)
    return x.to(torch.float64).numpy()


# ------------------------------------------------------------------ bf16 storage rounding
def test_round_to_bf16_matches_torch_on_fp32_inputs():
    rng = _rng(1)
    x32 = (rng.standard_normal(200000) * np.exp(rng.uniform(-30, 30, 200000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = vo.round_to_bf16(x32.astype(np.float64))
    assert np.array_equal(got, want)


def test_round_to_bf16_no_double_rounding_and_ties_to_even():
    # just above a tie: fp32 would first round down to the tie, then to even (1.0): wrong
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert vo.round_to_bf16(np.array([x]))[0] == 1.0 + 2.0 ** -7
    # exact ties go to the even mantissa
    assert vo.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert vo.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    # carry into the next binade
    assert vo.round_to_bf16(np.array([1.998046875 + 2.0 ** -9]))[0] == 2.0
    # sign symmetry, zero, subnormal spacing 2^-133
    assert vo.round_to_bf16(np.array([-x]))[0] == -(1.0 + 2.0 ** -7)
    assert vo.round_to_bf16(np.array([0.0]))[0] == 0.0
    assert vo.round_to_bf16(np.array([2.0 ** -133 * 2.6]))[0] == 2.0 ** -133 * 3


def test_bf16_bits_roundtrip():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    vals = vo.bf16_bits_to_f64(bits)
    assert np.array_equal(vo.bf16_bits_of(vals), bits)
    assert np.array_equal(vo.round_to_bf16(vals), vals)
    assert np.array_equal(synth.bf16_bits_to_f64(bits), vals)


# ------------------------------------------------------------------ Section 3.3: pooling
def test_carrier_constant_frame_is_the_constant():
    v = _bf16_vals(_rng(2), (64,))
    E = np.tile(v, (13, 1))
    assert np.array_equal(vo.carrier_embedding(E), v)


def test_carrier_one_hot_rows_give_counts_over_n():
    N, d = 16, 8
    cols = [0, 0, 0, 0, 1, 1, 2, 2, 2, 2, 2, 2, 2, 2, 5, 7]
    E = np.zeros((N, d))
    E[np.arange(N), cols] = 1.0
    want = np.bincount(cols, minlength=d) / N          # all exactly representable in bf16
    assert np.array_equal(vo.carrier_embedding(E), want)


def test_carrier_linear_ramp_and_rounding():
    N = 169
    E = np.arange(N, dtype=np.float64)[:, None] * np.array([[1.0, -2.0, 0.5]])
    mean = (N - 1) / 2.0 * np.array([1.0, -2.0, 0.5])
    want = torch.tensor(mean, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(vo.carrier_embedding(E), want)


def test_carrier_sum_is_exact_in_any_order_and_linear_under_projection():
    rng = _rng(3)
    E = _bf16_vals(rng, (169, 96))
    fwd = np.zeros(96)
    bwd = np.zeros(96)
    for i in range(169):
        fwd += E[i]
        bwd += E[168 - i]
    assert np.array_equal(fwd, bwd)
    assert np.array_equal(fwd, E.sum(axis=0))
    W = rng.standard_normal((96, 40))
    assert np.allclose((E.sum(axis=0) / 169) @ W, (E @ W).mean(axis=0), rtol=0, atol=1e-12)


def test_carrier_last_token_mode():
    E = _bf16_vals(_rng(4), (5, 7))
    assert np.array_equal(vo.carrier_embedding(E, agg_mode=1), E[-1])


# ------------------------------------------------------------------ RoPE
def test_rope_identity_at_position_zero_and_norm_preserved():
    rng = _rng(5)
    x = rng.standard_normal((3, 2, 16))
    a0 = vo.rope_angles([0, 0, 0], 16, 1e6)
    assert np.array_equal(vo.apply_rope(x, a0), x)
    a = vo.rope_angles([7, 1234, 170000], 16, 1e6)
    y = vo.apply_rope(x, a)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), atol=1e-12)


def test_rope_pairing_and_direction_closed_form():
    # D = 4: pairs are (0, 2) with frequency 1 and (1, 3) with frequency theta^(-1/2)
    theta = 100.0
    x = np.array([[[1.0, 0.0, 0.0, 0.0]], [[0.0, 1.0, 0.0, 0.0]]])
    y = vo.apply_rope(x, vo.rope_angles([2, 3], 4, theta))
    assert np.allclose(y[0, 0], [math.cos(2.0), 0.0, math.sin(2.0), 0.0], atol=1e-15)
    assert np.allclose(y[1, 0], [0.0, math.cos(0.3), 0.0, math.sin(0.3)], atol=1e-15)


def test_rope_scores_depend_on_relative_position_only():
    rng = _rng(6)
    q = rng.standard_normal((1, 1, 32))
    k = rng.standard_normal((1, 1, 32))
    def score(pq, pk):
        return float(np.sum(vo.apply_rope(q, vo.rope_angles([pq], 32, 1e4)) *
                            vo.apply_rope(k, vo.rope_angles([pk], 32, 1e4))))
    assert abs(score(10, 3) - score(1010, 1003)) < 1e-9
    assert abs(score(10, 3) - score(3, 10)) > 1e-3       # direction matters


def test_rope_matches_complex_rotation():
    rng = _rng(7)
    D = 64
    x = rng.standard_normal((4, 3, D))
    pos = [0, 5, 99, 4321]
    got = vo.apply_rope(x, vo.rope_angles(pos, D, 1e6))
    z = x[..., :D // 2] + 1j * x[..., D // 2:]
    for r, p in enumerate(pos):
        for k in range(D // 2):
            w = z[r, :, k] * np.exp(1j * p * (1e6 ** (-2.0 * k / D)))
            assert np.allclose(got[r, :, k], w.real, atol=1e-12)
            assert np.allclose(got[r, :, k + D // 2], w.imag, atol=1e-12)


# ------------------------------------------------------------------ Eq. (1)
def test_attention_rows_are_a_softmax():
    rng = _rng(8)
    Q = rng.standard_normal((5, 4, 8))
    K = rng.standard_normal((9, 2, 8))
    vis = rng.random((5, 9)) < 0.6
    vis[:, 0] = True
    ones = np.ones((9, 2, 8))
    assert np.allclose(vo.attention_rows(Q, K, ones, vis), 1.0, atol=1e-12)
    # one visible key -> that key's value; equal scores -> plain average of visible values
    V = rng.standard_normal((9, 2, 8))
    only = np.zeros((5, 9), dtype=bool)
    only[:, 3] = True
    out = vo.attention_rows(Q, K, V, only)
    assert np.allclose(out[:, 0], V[3, 0]) and np.allclose(out[:, 3], V[3, 1])
    out = vo.attention_rows(np.zeros_like(Q), K, V, vis)
    for r in range(5):
        assert np.allclose(out[r, 1], V[vis[r], 0].mean(axis=0), atol=1e-12)


def test_attention_matches_torch_sdpa_and_gqa_equals_repeated_mha():
    rng = _rng(9)
    rows, keys, Hq, Hkv, D = 7, 11, 6, 2, 16
    Q = rng.standard_normal((rows, Hq, D))
    K = rng.standard_normal((keys, Hkv, D))
    V = rng.standard_normal((keys, Hkv, D))
    vis = rng.random((rows, keys)) < 0.7
    vis[:, 0] = True
    got = vo.attention_rows(Q, K, V, vis)
    Kr = np.repeat(K, Hq // Hkv, axis=1)
    Vr = np.repeat(V, Hq // Hkv, axis=1)
    assert np.allclose(vo.attention_rows(Q, Kr, Vr, vis), got, atol=1e-13)
    t = lambda a: torch.from_numpy(a).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(
        t(Q), t(Kr), t(Vr), attn_mask=torch.from_numpy(vis)[None, None])
    assert np.allclose(ref[0].permute(1, 0, 2).numpy(), got, atol=1e-12)


# ------------------------------------------------------------------ streaming == dense masked attention
def _dense_reference(cfg, Ws, prefix_X, frames, texts, evict_after, norm=False, residual=False,
                     theta=1e6, eps=1e-6, gains=None, biases=None, carriers=None):
    """Textbook masked attention over the full un-pruned sequence
    [prefix | f0 tokens, c0 | f1 tokens, c1 | ... | text] with positions 0..S-1 and the
    semantic-aware mask of Section 3.4 / Fig. 3: a token sees the prefix, the carriers of
    earlier frames that are still in the bank when its own segment is processed, and the
    tokens of its own segment up to itself.  Written with explicit loops and complex
    rotations, independently of the oracle's vectorised code.  Optional per-layer RMSNorm gain
    (a multiply AFTER the division by the root mean square), per-layer bias (added to the
    projected row BEFORE the rotation, Eq. 1 with an affine term) and caller-supplied carrier
    tokens (they replace the mean as the frame's last token)."""
    Hq, Hkv, D = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    G = Hq // Hkv
    toks, seg, is_carrier = [], [], []
    for x in prefix_X:
        toks.append(x); seg.append(-1); is_carrier.append(False)
    for t, E in enumerate(frames):
        for x in E:
            toks.append(x); seg.append(t); is_carrier.append(False)
        toks.append(E.mean(axis=0) if carriers is None else carriers[t]); seg.append(t); is_carrier.append(True)
    TEXT = len(frames)
    for x in texts:
        toks.append(x); seg.append(TEXT); is_carrier.append(False)
    S = len(toks)
    h = np.stack(toks)
    # evict_after[j] = step s at whose end carrier j left the bank (or None)
    def sees(i, j):
        if j > i:
            return False
        if seg[j] == -1:
            return True
        if seg[j] == seg[i]:
            return True
        if not is_carrier[j]:
            return False
        if seg[i] == -1:
            return False
        gone = evict_after.get(seg[j])
        return gone is None or gone >= seg[i]
    freqs = np.array([theta ** (-2.0 * k / D) for k in range(D // 2)])
    outs = []
    for li, W in enumerate(Ws):
        x = h
        if norm:
            x = h / np.sqrt((h * h).mean(axis=1, keepdims=True) + eps)
            if gains is not None:
                x = np.stack([row * gains[li] for row in x])
        y = x @ W.T
        if biases is not None:
            y = np.stack([row + biases[li] for row in y])
        Qm = y[:, :Hq * D].reshape(S, Hq, D)
        Km = y[:, Hq * D:(Hq + Hkv) * D].reshape(S, Hkv, D)
        Vm = y[:, (Hq + Hkv) * D:].reshape(S, Hkv, D)
        rot = np.exp(1j * np.arange(S)[:, None] * freqs[None, :])[:, None, :]
        Qc = (Qm[..., :D // 2] + 1j * Qm[..., D // 2:]) * rot
        Kc = (Km[..., :D // 2] + 1j * Km[..., D // 2:]) * rot
        O = np.zeros((S, Hq, D))
        for i in range(S):
            js = [j for j in range(S) if sees(i, j)]
            for q in range(Hq):
                kv = q // G
                sc = np.array([np.real(np.sum(Qc[i, q] * np.conj(Kc[j, kv]))) for j in js]) / math.sqrt(D)
                p = np.exp(sc - sc.max())
                p /= p.sum()
                O[i, q] = sum(p[n] * Vm[j, kv] for n, j in enumerate(js))
        O = O.reshape(S, Hq * D)
        outs.append(O)
        if residual:
            h = h + O
    return outs[-1], seg


@pytest.mark.parametrize("layers,norm,policy,affine,override",
                         [(1, False, 0, False, False), (2, True, 0, False, False), (1, False, 1, False, False),
                          (2, True, 0, True, False), (1, False, 0, True, True), (2, True, 1, True, True)])
def test_streaming_equals_dense_masked_attention(monkeypatch, layers, norm, policy, affine, override):
    # storage rounding is pinned on its own above; switch it off so the comparison with
    # the textbook computation is exact to fp64 rounding
    monkeypatch.setattr(vo, "round_to_bf16", lambda x: np.asarray(x, dtype=np.float64))
    rng = _rng(10 + layers)
    d, Hq, Hkv, D, M, N, P, F, T = 32, 4, 2, 8, 2, 3, 2, 5, 3
    cfg = vo.OracleConfig(layers, d, Hq, Hkv, D, M, use_rmsnorm=int(norm), residual=int(layers > 1),
                          evict_policy=policy)
    Ws = [rng.standard_normal(((Hq + 2 * Hkv) * D, d)) * 0.3 for _ in range(layers)]
    prefix = rng.standard_normal((P, d))
    frames = [rng.standard_normal((N, d)) for _ in range(F)]
    texts = rng.standard_normal((T, d))
    E_out = (Hq + 2 * Hkv) * D
    # affine: RMSNorm gain far from 1 and a bias as large as the projected values, so that a gain
    # applied inside the root, or a bias added after the rotation, moves the result visibly
    gains = [1.0 + 0.5 * rng.standard_normal(d) for _ in range(layers)] if (affine and norm) else None
    biases = [rng.standard_normal(E_out) for _ in range(layers)] if affine else None
    # override: the caller's carrier token replaces the mean everywhere -- as the frame's last
    # token, as the bank's embedding (so eviction follows it) and as the source of the kept K/V
    carriers = [rng.standard_normal(d) for _ in range(F)] if override else None
    st = vo.OracleStream(cfg, Ws, biases, gains)
    got = [st.text_step(prefix)]
    for t, E in enumerate(frames):
        got.append(st.frame_step(E, carrier_override=None if carriers is None else carriers[t]))
    got.append(st.text_step(texts[:2]))
    got.append(st.text_step(texts[2:]))
    got = np.concatenate(got, axis=0)
    # eviction trace recomputed naively from the carrier embeddings
    embs = [E.mean(axis=0) for E in frames] if carriers is None else carriers
    bank, gone = [], {}
    cos = lambda a, b: float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))
    for t in range(F):
        if len(bank) == M:
            if policy == 0:
                s = [cos(embs[j], embs[t]) for j in bank]
            else:
                seq = bank + [t]
                s = [cos(embs[seq[n]], embs[seq[n + 1]]) for n in range(M)]
            gone[bank.pop(int(np.argmax(s)))] = t
        bank.append(t)
    assert [(s, v) for v, s in sorted(gone.items(), key=lambda kv: kv[1])] == st.evict_log
    want, _ = _dense_reference(cfg, Ws, prefix, frames, texts, gone, norm=norm, residual=layers > 1,
                               gains=gains, biases=biases, carriers=carriers)
    assert got.shape == want.shape
    assert np.max(np.abs(got - want)) < 1e-10
    if override:
        assert all(np.array_equal(e.emb, carriers[e.frame_id]) for e in st.bank)


def test_zero_capacity_is_plain_causal_attention_per_frame(monkeypatch):
    monkeypatch.setattr(vo, "round_to_bf16", lambda x: np.asarray(x, dtype=np.float64))
    rng = _rng(20)
    d, Hq, Hkv, D, N, P = 24, 2, 2, 12, 5, 3
    cfg = vo.OracleConfig(1, d, Hq, Hkv, D, 0, rope_theta=1e4)
    W = rng.standard_normal(((Hq + 2 * Hkv) * D, d)) * 0.3
    st = vo.OracleStream(cfg, [W])
    prefix = rng.standard_normal((P, d))
    st.text_step(prefix)
    for t in range(3):
        E = rng.standard_normal((N, d))
        got = st.frame_step(E)
        assert len(st.bank) == 0
        # textbook: causal attention over [prefix | frame tokens | mean], the frame sitting at
        # its place in the un-pruned sequence (earlier frames' tokens are simply absent)
        X = np.concatenate([prefix, E, E.mean(axis=0, keepdims=True)])
        y = X @ W.T
        S = X.shape[0]
        ang = vo.rope_angles(list(range(P)) + [P + t * (N + 1) + i for i in range(N + 1)], D, 1e4)
        Q = vo.apply_rope(y[:, :Hq * D].reshape(S, Hq, D), ang)
        K = vo.apply_rope(y[:, Hq * D:(Hq + Hkv) * D].reshape(S, Hkv, D), ang)
        V = y[:, (Hq + Hkv) * D:].reshape(S, Hkv, D)
        tt = lambda a: torch.from_numpy(a).permute(1, 0, 2)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(tt(Q), tt(K), tt(V), is_causal=True)
        ref = ref[0].permute(1, 0, 2).reshape(S, Hq * D).numpy()[P:]
        assert np.max(np.abs(got - ref)) < 1e-9


# ------------------------------------------------------------------ causal layout of a frame
def test_carrier_is_last_and_causal():
    rng = _rng(21)
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, 4)
    W = synth.bf16_bits_to_f64(w.weight(0))
    E = synth.bf16_bits_to_f64(w.frame_hidden(0))
    base = vo.OracleStream(cfg, [W]).frame_step(E)
    E2 = E.copy()
    E2[9] += 1.0
    out2 = vo.OracleStream(cfg, [W]).frame_step(E2)
    assert np.array_equal(out2[:9], base[:9])                 # rows before the change are untouched
    assert np.max(np.abs(out2[9:-1] - base[9:-1])) > 1e-6     # later visual rows change
    assert np.max(np.abs(out2[-1] - base[-1])) > 1e-6         # the carrier sees every visual token
    assert base.shape == (E.shape[0] + 1, w.n_q_heads * w.head_dim)


def test_later_frames_see_earlier_frames_only_through_the_carrier():
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, 4)
    W = synth.bf16_bits_to_f64(w.weight(0))
    E0 = synth.bf16_bits_to_f64(w.frame_hidden(0))
    E1 = synth.bf16_bits_to_f64(w.frame_hidden(1))
    a = vo.OracleStream(cfg, [W]); a.frame_step(E0); out_a = a.frame_step(E1)
    # permuting frame 0's visual tokens keeps its mean, hence (one layer) its carrier K/V
    b = vo.OracleStream(cfg, [W]); b.frame_step(E0[::-1].copy()); out_b = b.frame_step(E1)
    assert np.array_equal(out_a, out_b)
    # a different mean does change what frame 1 computes
    c = vo.OracleStream(cfg, [W]); c.frame_step(E0 * 0.5); out_c = c.frame_step(E1)
    assert np.max(np.abs(out_a - out_c)) > 1e-6


# ------------------------------------------------------------------ memory mechanism
def test_eviction_hand_built_sequences():
    d = 64
    eye = np.eye(d)
    bank = np.stack([eye[0], eye[1], eye[2], eye[3]])
    assert vo.choose_victim(bank, 2.0 * eye[2], 0) == 2          # scale invariance of the cosine
    assert vo.choose_victim(bank, -eye[1] + 0.01 * eye[3], 0) == 3
    dup = np.stack([eye[0], eye[5], eye[5], eye[3]])
    assert vo.choose_victim(dup, eye[5], 0) == 1                 # identical entries: the older leaves
    assert vo.choose_victim(dup, eye[9], 0) == 0                 # all cosines 0: oldest leaves
    a, b, c = eye[0], eye[1], eye[2]
    assert vo.choose_victim(np.stack([a, a, b, c]), eye[7], 1) == 0   # adjacent pair (a, a)
    assert vo.choose_victim(np.stack([a, b, c, eye[7]]), eye[7], 1) == 3  # pair (last, incoming)
    assert vo.choose_victim(np.stack([a, b, c, eye[7]]), eye[7], 0) == 3
    assert vo.choose_victim(np.stack([a, b]), c, 2) == 0
    z = np.zeros(d)
    assert vo.choose_victim(np.stack([z, b]), b, 0) == 1         # zero norm counts as cosine 0
    assert vo.choose_victim(np.stack([z, a]), b, 0) == 0
    # a non-finite embedding has no cosine either: it counts as 0, so a real duplicate still wins,
    # and with nothing else to prefer the oldest leaves (the index always names a stored carrier)
    bad = a.copy(); bad[3] = np.nan
    inf = a.copy(); inf[0] = np.inf
    assert vo.choose_victim(np.stack([bad, b, c]), b, 0) == 1
    assert vo.choose_victim(np.stack([a, inf, c]), c, 0) == 2
    assert vo.choose_victim(np.stack([a, b, c]), bad, 0) == 0    # every cosine undefined
    assert vo.choose_victim(np.stack([a, b, c]), inf, 1) == 0    # only the pair with the incoming is undefined; rest orthogonal
    assert vo.choose_victim(np.stack([a, a, bad]), c, 1) == 0    # pair (a, a) = 1 beats the undefined pairs


def test_canonical_cosine_agrees_with_naive():
    rng = _rng(22)
    A = _bf16_vals(rng, (50, 3584))
    v = _bf16_vals(rng, (3584,))
    got = vo.cosine_similarity(A, v[None, :])
    want = (A @ v) / (np.linalg.norm(A, axis=1) * np.linalg.norm(v))
    assert np.allclose(got, want, rtol=0, atol=1e-13)
    # the canonical order is an order of the same exact products: the dot of bf16 vectors
    # must equal the exact rational sum whenever that sum is representable
    ints = rng.integers(-8, 9, size=(4, 100)).astype(np.float64)
    assert np.array_equal(vo.canonical_dot(ints, ints[::-1]), np.sum(ints * ints[::-1], axis=1))


def test_bank_count_and_order_tiny_workload():
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity)
    st = vo.OracleStream(cfg, [synth.bf16_bits_to_f64(w.weight(0))])
    st.text_step(synth.bf16_bits_to_f64(w.prefix_hidden()))
    for t in range(w.n_frames):
        st.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(t)))
        ids = st.bank_frame_ids()
        assert len(ids) == min(t + 1, w.bank_capacity)
        assert ids == sorted(ids) and ids[-1] == t
        assert st.bank_positions() == [w.prefix_len + i * 17 + 16 for i in ids]
        for e in st.bank:
            assert e.K.shape == (1, w.n_kv_heads, w.head_dim)
    assert st.evictions == 4 and [s for s, _ in st.evict_log] == [4, 5, 6, 7]
    assert st.next_pos == 8 + 8 * 17


def test_bank_never_evicts_when_capacity_equals_frames():
    w = synth.workload("layer", d_model=128, n_q_heads=2, n_kv_heads=1, head_dim=64,
                       tokens_per_frame=9, n_frames=64)
    cfg = vo.OracleConfig(1, w.d_model, 2, 1, 64, 64)
    st = vo.OracleStream(cfg, [synth.bf16_bits_to_f64(w.weight(0))])
    shared = w.frame_shared()
    for t in range(64):
        st.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(t, shared=shared)), mode="meta")
    assert st.evictions == 0 and st.bank_frame_ids() == list(range(64))


def test_carrier_only_mode_reproduces_full_bank():
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity)
    W = synth.bf16_bits_to_f64(w.weight(0))
    a, b = vo.OracleStream(cfg, [W]), vo.OracleStream(cfg, [W])
    for t in range(w.n_frames):
        E = synth.bf16_bits_to_f64(w.frame_hidden(t))
        a.frame_step(E)
        b.frame_step(E, mode="carrier")
    assert a.bank_frame_ids() == b.bank_frame_ids()
    for x, y in zip(a.bank, b.bank):
        assert np.allclose(x.K, y.K, atol=1e-12) and np.allclose(x.V, y.V, atol=1e-12)
        assert np.array_equal(x.emb, y.emb)


# ------------------------------------------------------------------ decoding
def test_question_prefill_equals_token_by_token_decode():
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity)
    W = synth.bf16_bits_to_f64(w.weight(0))
    X = _bf16_vals(_rng(23), (5, w.d_model))
    def fresh():
        st = vo.OracleStream(cfg, [W])
        st.text_step(synth.bf16_bits_to_f64(w.prefix_hidden()))
        for t in range(3):
            st.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(t)))
        return st
    a = fresh(); whole = a.text_step(X)
    b = fresh(); steps = np.concatenate([b.text_step(X[i:i + 1]) for i in range(5)])
    assert np.max(np.abs(whole - steps)) < 1e-12
    assert a.text_len == b.text_len == 5
    # the tail is per turn: after end_turn the next question starts from prefix + bank again
    a.end_turn(); again = a.text_step(X)
    assert np.max(np.abs(again - whole)) < 1e-12
    with pytest.raises(RuntimeError):
        a.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(3)))


def test_decode_sees_only_prefix_bank_and_text():
    # poisoning what a frame step leaves behind (other than the bank) cannot matter: the
    # oracle keeps nothing else, so decode over a stream equals decode over a hand-built
    # context made of prefix K/V and carrier K/V alone
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity)
    W = synth.bf16_bits_to_f64(w.weight(0))
    st = vo.OracleStream(cfg, [W])
    st.text_step(synth.bf16_bits_to_f64(w.prefix_hidden()))
    for t in range(6):
        st.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(t)))
    x = synth.bf16_bits_to_f64(w.decode_hidden(0))
    got = st.text_step(x)
    y = x @ W.T
    Hq, Hkv, D = w.n_q_heads, w.n_kv_heads, w.head_dim
    pos = st.next_pos
    ang = vo.rope_angles([pos], D, 1e6)
    Q = vo.apply_rope(y[:, :Hq * D].reshape(1, Hq, D), ang)
    K = vo.round_to_bf16(vo.apply_rope(y[:, Hq * D:(Hq + Hkv) * D].reshape(1, Hkv, D), ang))
    V = vo.round_to_bf16(y[:, (Hq + Hkv) * D:].reshape(1, Hkv, D))
    Kall = np.concatenate([st.prefix_K[0]] + [e.K[0][None] for e in st.bank] + [K])
    Vall = np.concatenate([st.prefix_V[0]] + [e.V[0][None] for e in st.bank] + [V])
    assert Kall.shape[0] == 8 + 4 + 1
    want = vo.attention_rows(Q, Kall, Vall, np.ones((1, 13), dtype=bool)).reshape(1, -1)
    assert np.max(np.abs(got - want)) < 1e-12


# ------------------------------------------------------------- carriers as ordinary tokens
def test_carriers_only_forward_is_a_text_prefill_of_the_stored_embeddings():
    # special case that reduces to a routine pinned above: on a stream that has seen no frame,
    # feeding the bank's embeddings as text right after the same prompt is the same computation
    # (same positions prefix_len + i, same causal context), whatever the bank's K/V hold
    w = synth.workload("tiny", n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64,
                       use_rmsnorm=1, residual=1)
    cfg = vo.OracleConfig(2, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity,
                          use_rmsnorm=1, residual=1)
    Ws = [synth.bf16_bits_to_f64(w.weight(l)) for l in range(2)]
    st = vo.OracleStream(cfg, Ws)
    st.text_step(synth.bf16_bits_to_f64(w.prefix_hidden()))
    for t in range(7):                                   # capacity 4: evictions reorder the bank
        st.frame_step(synth.bf16_bits_to_f64(w.frame_hidden(t)))
    before = (st.next_pos, st.frames_seen, st.evictions, [e.frame_id for e in st.bank])
    got = st.carriers_only_forward()
    assert (st.next_pos, st.frames_seen, st.evictions, [e.frame_id for e in st.bank]) == before
    assert got.shape == (4, w.n_q_heads * w.head_dim)
    ref = vo.OracleStream(cfg, Ws)
    ref.text_step(synth.bf16_bits_to_f64(w.prefix_hidden()))
    want = ref.text_step(np.stack([e.emb for e in st.bank]))
    assert np.max(np.abs(got - want)) < 1e-12
    assert vo.OracleStream(cfg, Ws).carriers_only_forward().shape == (0, w.n_q_heads * w.head_dim)


def test_carriers_only_forward_brute_force_one_layer():
    # written out independently: complex rotation for RoPE, explicit loops for the softmax
    rng = _rng(77)
    d, Hq, Hkv, D, P, theta = 64, 2, 1, 32, 3, 1e4
    cfg = vo.OracleConfig(1, d, Hq, Hkv, D, 5, rope_theta=theta)
    W = _bf16_vals(rng, ((Hq + 2 * Hkv) * D, d), 0.1)
    st = vo.OracleStream(cfg, [W])
    Xp = _bf16_vals(rng, (P, d))
    st.text_step(Xp)
    for t in range(4):
        st.frame_step(_bf16_vals(rng, (6, d)))
    got = st.carriers_only_forward()
    C = np.stack([e.emb for e in st.bank])               # [4, d]
    X = np.concatenate([Xp, C])                          # the compact sequence: prompt, then one token per frame
    T = X.shape[0]
    Y = X @ W.T
    def rot(v, pos):                                     # v: [D]; pairs (i, i + D/2) as complex numbers
        z = v[:D // 2] + 1j * v[D // 2:]
        z = z * np.exp(1j * pos * theta ** (-2.0 * np.arange(D // 2) / D))
        return np.concatenate([z.real, z.imag])
    out = np.zeros((4, Hq * D))
    for hq in range(Hq):
        hk = hq // (Hq // Hkv)
        Kr = np.stack([vo.round_to_bf16(rot(Y[t, (Hq + hk) * D:(Hq + hk + 1) * D], t)) for t in range(T)])
        Vr = np.stack([vo.round_to_bf16(Y[t, (Hq + Hkv + hk) * D:(Hq + Hkv + hk + 1) * D]) for t in range(T)])
        for i in range(4):
            t = P + i
            q = rot(Y[t, hq * D:(hq + 1) * D], t)
            s = np.array([q @ Kr[u] / math.sqrt(D) for u in range(t + 1)])
            p = np.exp(s - s.max()); p /= p.sum()
            out[i, hq * D:(hq + 1) * D] = sum(p[u] * Vr[u] for u in range(t + 1))
    assert np.max(np.abs(got - out)) < 1e-12
