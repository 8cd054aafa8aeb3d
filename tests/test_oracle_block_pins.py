"""CPU pins of the oracle's optional rest of the decoder block (output projection + SwiGLU MLP; the
backbone of Section 4.1 is a Qwen2 decoder).  The paper prints no numbers for it; the pins are closed
forms, special cases that reduce to the attention-only oracle, and a library restatement in torch
(fp64 F.linear / F.silu) -- chosen so that a transposed weight, SiLU on the wrong branch, a missing
residual or a norm taken of the wrong tensor fails one of them."""
import math

import numpy as np
import pytest
import torch

from oracle import videoscan_oracle as vo


def _bf(x):
    return vo.round_to_bf16(np.asarray(x, dtype=np.float64))


def _setup(seed=0, L=2, d=32, Hq=4, Hkv=2, D=8, inter=48, norm=True, gain=True):
    rng = np.random.default_rng(seed)
    cfg = vo.OracleConfig(L, d, Hq, Hkv, D, bank_capacity=2, use_rmsnorm=1 if norm else 0, residual=1)
    Ws = [_bf(rng.normal(0, 0.2, ((Hq + 2 * Hkv) * D, d))) for _ in range(L)]
    gains = [_bf(1 + 0.1 * rng.normal(size=d)) for _ in range(L)] if gain else None
    blocks = [vo.BlockWeights(_bf(rng.normal(0, 0.2, (d, Hq * D))), _bf(rng.normal(0, 0.2, (inter, d))),
                              _bf(rng.normal(0, 0.2, (inter, d))), _bf(rng.normal(0, 0.2, (d, inter))),
                              _bf(1 + 0.1 * rng.normal(size=d)) if gain else None) for _ in range(L)]
    return rng, cfg, Ws, gains, blocks


def _run(cfg, Ws, gains, blocks, rng_seed=1, frames=4, N=5):
    rng = np.random.default_rng(rng_seed)
    st = vo.OracleStream(cfg, Ws, None, gains, blocks)
    st.record = []
    outs = [st.text_step(_bf(rng.normal(size=(3, cfg.d_model))))]
    for _ in range(frames):
        outs.append(st.frame_step(_bf(rng.normal(size=(N, cfg.d_model)))))
    outs.append(st.text_step(_bf(rng.normal(size=(2, cfg.d_model)))))
    outs.append(st.text_step(_bf(rng.normal(size=(1, cfg.d_model)))))
    return st, outs


def test_silu_closed_forms():
    assert vo.silu(np.array([0.0]))[0] == 0.0
    assert abs(vo.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(vo.silu(np.array([-1.0]))[0] + 1.0 / (1.0 + math.e)) < 1e-15
    x = np.linspace(-6, 6, 101)
    assert np.allclose(vo.silu(x) - vo.silu(-x), x, atol=1e-14)            # x sigma(x) - (-x) sigma(-x) = x
    assert np.allclose(vo.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)


def test_identity_output_projection_and_silent_mlp_reduce_to_the_attention_residual():
    """W_o = I and W_down = 0: the layer's output is bf16(h + bf16(O)), O being the attention rows the
    attention-only procedure computes on the same layer input."""
    _, cfg, Ws, gains, blocks = _setup(L=1)
    blocks[0].w_o = np.eye(cfg.d_model)
    blocks[0].w_down = np.zeros_like(blocks[0].w_down)
    st, outs = _run(cfg, Ws, gains, blocks)
    for rec, out in zip(st.record, outs):
        want = _bf(rec["h"][0] + _bf(rec["O"][0]))
        assert np.array_equal(out, want)


def test_zero_gate_makes_the_mlp_add_nothing():
    _, cfg, Ws, gains, blocks = _setup(L=2)
    for b in blocks:
        b.w_gate = np.zeros_like(b.w_gate)                                     # SiLU(0) = 0
    st, outs = _run(cfg, Ws, gains, blocks)
    for rec in st.record:
        for l in range(cfg.n_layers):
            h1 = _bf(rec["h"][l] + _bf(rec["O"][l]) @ blocks[l].w_o.T)
            assert np.array_equal(rec["h_out"][l], h1)
            if l + 1 < cfg.n_layers:
                assert np.array_equal(rec["h"][l + 1], h1)                      # and it is the next layer's input


@pytest.mark.parametrize("norm,gain", [(True, True), (True, False), (False, False)])
def test_block_matches_a_torch_restatement(norm, gain):
    """Every recorded layer: torch fp64 linear / silu on the recorded layer input and attention rows."""
    _, cfg, Ws, gains, blocks = _setup(seed=3, L=2, norm=norm, gain=gain)
    st, outs = _run(cfg, Ws, gains, blocks, rng_seed=5)
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.ascontiguousarray(np.asarray(a, dtype=np.float64)))
    for rec, out in zip(st.record, outs):
        for l in range(cfg.n_layers):
            b = blocks[l]
            h = t(rec["h"][l])
            a = t(_bf(rec["O"][l]))
            h1 = t(_bf((h + F.linear(a, t(b.w_o))).numpy()))
            n = h1
            if norm:
                n = h1 * torch.rsqrt((h1 * h1).mean(dim=1, keepdim=True) + cfg.rms_eps)
                if gain:
                    n = n * t(b.norm2_w)
            act = t(_bf((F.silu(F.linear(n, t(b.w_gate))) * F.linear(n, t(b.w_up))).numpy()))
            h2 = _bf((h1 + F.linear(act, t(b.w_down))).numpy())
            assert np.allclose(rec["h_out"][l], h2, atol=1e-12, rtol=0)
            # bf16 roundings of nearly equal fp64 values agree except on exact ties: demand equality on 99.9 %
            assert np.mean(rec["h_out"][l] == h2) > 0.999
        assert np.array_equal(out, rec["h_out"][-1])                           # a step returns the last layer's output


def test_attention_only_streams_are_untouched_by_the_option():
    _, cfg, Ws, gains, blocks = _setup(seed=4, L=2)
    st_a, outs_a = _run(cfg, Ws, gains, None)
    st_b = vo.OracleStream(cfg, Ws, None, gains)                               # blocks defaulted
    rng = np.random.default_rng(1)
    out0 = st_b.text_step(_bf(rng.normal(size=(3, cfg.d_model))))
    assert np.array_equal(out0, outs_a[0]) and out0.shape[1] == cfg.n_q_heads * cfg.head_dim


def test_bank_keeps_attention_keys_of_the_block_stream():
    """The bank's K/V of a deeper layer come from that layer's input, which now carries the MLP: a stream with
    blocks and one without differ in layer 1's bank K/V but not in layer 0's (same frames, same layer-0 input)."""
    _, cfg, Ws, gains, blocks = _setup(seed=6, L=2)
    st_a, _ = _run(cfg, Ws, gains, blocks)
    st_b, _ = _run(cfg, Ws, gains, None)
    assert len(st_a.bank) == len(st_b.bank) == 2
    for ea, eb in zip(st_a.bank, st_b.bank):
        assert ea.frame_id == eb.frame_id and np.array_equal(ea.emb, eb.emb)
        assert np.array_equal(ea.K[0], eb.K[0]) and not np.array_equal(ea.K[1], eb.K[1])


# ------------------------------------------------------------------ language-model head
def test_lm_head_matches_a_library_restatement_and_scaling_laws():
    """logits against torch (fp64 F.linear of a hand-normalised input); RMSNorm makes the logits
    invariant to a power-of-two scaling of the hidden state (exact in bf16) up to the epsilon term;
    without the norm they scale linearly."""
    rng = np.random.default_rng(3)
    d, V, R = 48, 37, 5
    h = _bf(rng.normal(size=(R, d))); W = _bf(rng.normal(0, 0.3, (V, d))); g = _bf(1 + 0.2 * rng.normal(size=d))
    logits, tok = vo.lm_head(h, W, g, True, 1e-6)
    ht = torch.from_numpy(h)
    nt = ht * torch.rsqrt((ht * ht).mean(dim=1, keepdim=True) + 1e-6) * torch.from_numpy(g)
    want = torch.nn.functional.linear(nt, torch.from_numpy(W)).numpy()
    np.testing.assert_allclose(logits, want, rtol=1e-12, atol=1e-12)
    assert list(tok) == list(want.argmax(axis=1))
    l4, _ = vo.lm_head(4.0 * h, W, g, True, 0.0)
    l1, _ = vo.lm_head(h, W, g, True, 0.0)
    np.testing.assert_allclose(l4, l1, rtol=1e-12, atol=1e-12)
    p4, _ = vo.lm_head(4.0 * h, W, None, False)
    p1, _ = vo.lm_head(h, W, None, False)
    np.testing.assert_allclose(p4, 4.0 * p1, rtol=1e-12, atol=1e-12)


def test_lm_head_closed_forms():
    """One-hot vocabulary rows read single channels of the normalised state; a constant hidden row
    normalises to +-1 per channel; the gain multiplies after the normalisation (a gain inside the
    mean of squares, or a transposed weight, fails here)."""
    d = 16
    W = np.eye(d)                                   # vocab = d, row v reads channel v
    h = np.full((1, d), 3.0)
    logits, tok = vo.lm_head(h, W, None, True, 0.0)
    np.testing.assert_allclose(logits, np.ones((1, d)), atol=1e-12)
    assert tok[0] == 0                              # all equal: lowest index
    g = np.arange(1, d + 1, dtype=np.float64)
    logits, tok = vo.lm_head(-h, W, g, True, 0.0)
    np.testing.assert_allclose(logits, -g[None, :], atol=1e-12)
    assert tok[0] == 0                              # -1 is the largest of -1 .. -16
    h2 = np.zeros((1, d)); h2[0, 5] = 2.0           # one live channel: rms = 2 / sqrt(d)
    logits, tok = vo.lm_head(h2, W, g, True, 0.0)
    assert tok[0] == 5 and abs(logits[0, 5] - math.sqrt(d) * 6.0) < 1e-12
    Wr = np.zeros((3, d)); Wr[0, 1] = 1.0; Wr[1, 2] = 1.0; Wr[2, 1] = 1.0       # non-square: [vocab][d]
    h3 = np.zeros((1, d)); h3[0, 2] = 1.0
    assert vo.lm_head(h3, Wr, None, False)[1][0] == 1


def test_greedy_token_ties_and_non_finite_values():
    assert vo.greedy_token(np.array([1.0, 3.0, 3.0, 2.0])) == 1
    assert vo.greedy_token(np.array([-math.inf, -math.inf])) == 0
    assert vo.greedy_token(np.array([math.nan, -5.0, math.nan])) == 1
    assert vo.greedy_token(np.array([math.nan, math.nan])) == 0
    assert vo.greedy_token(np.array([0.0, math.inf, math.inf])) == 1
    rng = np.random.default_rng(0)
    for _ in range(20):
        x = rng.integers(-3, 4, size=50).astype(np.float64)
        assert vo.greedy_token(x) == int(np.argmax(x))          # numpy's argmax also takes the first maximum


def test_lm_head_rounds_the_hidden_state_on_entry():
    """The hidden state is a stored (bf16) tensor: values that differ below bf16 resolution give the
    same logits."""
    rng = np.random.default_rng(5)
    h = _bf(rng.normal(size=(2, 32))); W = _bf(rng.normal(size=(9, 32)))
    a, _ = vo.lm_head(h, W, None, True)
    b, _ = vo.lm_head(h * (1 + 2.0 ** -12), W, None, True)
    np.testing.assert_array_equal(a, b)


def test_carriers_only_forward_with_the_block_is_a_text_prefill_of_the_stored_embeddings():
    """With the full decoder block too, feeding the bank's embeddings as text right after the same prompt on a
    stream that has seen no frame is the same computation (positions prefix_len + i, causal context), and the
    call changes nothing of the stream."""
    rng, cfg, Ws, gains, blocks = _setup(seed=8, L=2)
    st, _ = _run(cfg, Ws, gains, blocks, frames=5)
    st.end_turn()
    before = (st.next_pos, st.frames_seen, st.evictions, [e.frame_id for e in st.bank])
    got = st.carriers_only_forward()
    assert (st.next_pos, st.frames_seen, st.evictions, [e.frame_id for e in st.bank]) == before
    assert got.shape == (2, cfg.d_model)
    ref = vo.OracleStream(cfg, Ws, None, gains, blocks)
    r2 = np.random.default_rng(1)
    ref.text_step(_bf(r2.normal(size=(3, cfg.d_model))))          # the same prompt _run feeds (seed 1, 3 rows)
    want = ref.text_step(np.stack([e.emb for e in st.bank]))
    assert np.max(np.abs(got - want)) < 1e-12
    # and it is not the attention-only result: the block is really applied
    plain = vo.OracleStream(cfg, Ws, None, gains, None)
    r3 = np.random.default_rng(1)
    plain.text_step(_bf(r3.normal(size=(3, cfg.d_model))))
    assert np.max(np.abs(plain.text_step(np.stack([e.emb for e in st.bank])) - got)) > 1e-3
