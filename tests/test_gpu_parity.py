"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle on the same
seeded inputs.  Sizes span several tiles and ragged tails; tolerances are in tests/parity.py."""
import numpy as np
import pytest
import torch

from paper_2503_09387_b200 import binding, synth
from tests.parity import Pair, assert_close, bits_of, to_dev, to_f64

pytestmark = pytest.mark.gpu


def run_stream(p: Pair, w: synth.Workload, n_frames=None, check_every=1, question=True):
    """Prefix, frames, optional question, decode tokens -- everything compared."""
    if w.prefix_len:
        p.text([0], [w.prefix_hidden()], "prefix")
    shared = w.frame_shared() if w.frame_model != "iid" else None
    F = n_frames if n_frames is not None else w.n_frames
    for t in range(F):
        p.frame([0], [w.frame_hidden(t, shared=shared)], f"frame {t}")
        if t % check_every == 0 or t == F - 1:
            st = p.check_bank(0, layer=w.n_layers - 1)
            k, v = p.gpu.last_step_kv(w.tokens_per_frame + 1)
            if st["count"]:      # the append is a pure copy of the carrier row of this step
                assert np.array_equal(k[-1].reshape(w.n_kv_heads, w.head_dim), st["k"][-1])
                assert np.array_equal(v[-1].reshape(w.n_kv_heads, w.head_dim), st["v"][-1])
    if question and w.question_len:
        p.text([0], [w.question_hidden()], "question")
    for i in range(w.decode_tokens):
        p.text([0], [w.decode_hidden(i)], f"decode {i}")
    p.check_bank(0)


def test_tiny_workload_end_to_end():
    w = synth.workload("tiny")
    p = Pair(w)
    run_stream(p, w)
    assert p.ora[0].evictions == 4
    p.close()


@pytest.mark.parametrize("N,P,M,policy", [(1, 0, 0, 0), (7, 1, 1, 0), (17, 3, 2, 1), (33, 5, 3, 2), (16, 8, 4, 1)])
def test_odd_shapes_and_policies(N, P, M, policy):
    w = synth.workload("tiny", tokens_per_frame=N, prefix_len=P, bank_capacity=M, n_frames=7,
                       question_len=5, decode_tokens=3, seed=11 + N)
    p = Pair(w, evict_policy=policy)
    run_stream(p, w)
    p.close()


def test_bias_last_token_aggregation_and_carrier_override():
    w = synth.workload("tiny", seed=5, n_frames=6)
    p = Pair(w, with_bias=True, agg_mode=1)
    run_stream(p, w)
    p.close()
    p = Pair(w)
    p.text([0], [w.prefix_hidden()])
    for t in range(6):
        ov = synth.normal_bf16(77, synth.TAG_PREFIX, (w.d_model,), 1.0, offset=t * w.d_model)
        p.frame([0], [w.frame_hidden(t)], f"override frame {t}", override=[ov])
        p.check_bank(0)
    p.close()


def test_bf16_output_mode_adds_only_storage_rounding():
    w = synth.workload("tiny", seed=3)
    a, b = Pair(w, out_dtype=1), Pair(w, out_dtype=0)
    xs = [w.prefix_hidden()] + [w.frame_hidden(t) for t in range(4)] + [w.decode_hidden(0)]
    for i, x in enumerate(xs):
        fn = (lambda p: p.frame([0], [x])) if 1 <= i <= 4 else (lambda p: p.text([0], [x], compare=False))
        if not (1 <= i <= 4):
            full = a.text([0], [x])
            half = to_f64(b.gpu.decode_step([0], to_dev(x[None])))
            b.ora[0].text_step(synth.bf16_bits_to_f64(x))
        else:
            full = a.frame([0], [x])
            half = to_f64(b.gpu.frame_prefill([0], to_dev(x[None])))
            b.ora[0].frame_step(synth.bf16_bits_to_f64(x))
        want = torch.from_numpy(full).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
        assert np.array_equal(half, want)          # bf16 mode == fp32 mode rounded once
    a.close(); b.close()


def test_multi_layer_residual_rmsnorm_small():
    w = synth.workload("deep", n_layers=4, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64,
                       tokens_per_frame=21, n_frames=9, bank_capacity=4, prefix_len=6, question_len=7,
                       decode_tokens=3)
    p = Pair(w, with_gain=True)
    run_stream(p, w, check_every=100)
    for layer in range(4):
        p.check_bank(0, layer=layer)
    p.close()


def test_scratch_holds_no_state_between_steps():
    """Section 3.3: visual tokens are discarded after prefill.  Overwriting every per-step
    scratch region with NaN between steps must not change any later output."""
    w = synth.workload("tiny")
    a, b = Pair(w), Pair(w)
    outs = []
    for p, poison in ((a, False), (b, True)):
        o = [p.text([0], [w.prefix_hidden()])]
        for t in range(w.n_frames):
            o.append(p.frame([0], [w.frame_hidden(t)]))
            if poison:
                p.gpu.poison_scratch()
        for i in range(w.decode_tokens):
            o.append(p.text([0], [w.decode_hidden(i)]))
            if poison:
                p.gpu.poison_scratch()
        outs.append(o)
    for x, y in zip(*outs):
        assert np.array_equal(x, y)
    a.close(); b.close()


def test_question_prefill_decode_and_end_turn():
    w = synth.workload("tiny", question_len=13, decode_tokens=6, n_frames=5)
    p = Pair(w, max_text=19)
    p.text([0], [w.prefix_hidden()])
    for t in range(5):
        p.frame([0], [w.frame_hidden(t)])
    q = w.question_hidden()
    whole = p.text([0], [q], "question")
    for i in range(6):
        p.text([0], [w.decode_hidden(i)], f"decode {i}")
    # tail full: one more token must be refused without touching the stream
    with pytest.raises(binding.VsError) as e:
        p.gpu.decode_step([0], to_dev(w.decode_hidden(0)[None]))
    assert e.value.code == binding.VS_ERR_CAPACITY
    with pytest.raises(binding.VsError) as e:
        p.gpu.frame_prefill([0], to_dev(w.frame_hidden(5)[None]))
    assert e.value.code == binding.VS_ERR_STATE
    p.gpu.end_turn([0]); p.ora[0].end_turn()
    # token by token gives the same rows as the multi-token prefill
    rows = [p.text([0], [q[i:i + 1]], f"question token {i}")[0] for i in range(13)]
    assert_close(np.concatenate(rows), whole[0], "token-by-token vs prefill")
    p.gpu.end_turn([0]); p.ora[0].end_turn()
    p.frame([0], [w.frame_hidden(5)], "frame after the turn")
    p.check_bank(0)
    p.close()


def test_batched_ragged_streams_small():
    w = synth.workload("batched", d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=19,
                       n_frames=12, min_frames=4, bank_capacity=6, n_streams=5, prefix_len=4, decode_tokens=3)
    lengths = w.stream_lengths()
    assert len(set(lengths)) > 1
    p = Pair(w)
    ids = list(range(5))
    p.text(ids, [w.prefix_hidden(s) for s in ids], "prefix")
    shared = [w.frame_shared(s) for s in ids]
    for t in range(max(lengths)):
        act = [s for s in ids if lengths[s] > t]
        p.frame(act, [w.frame_hidden(t, s, shared=shared[s]) for s in act], f"frame {t}")
    for i in range(3):
        p.text(ids, [w.decode_hidden(i, s) for s in ids], f"decode {i}")
    for s in ids:
        st = p.check_bank(s)
        assert st["frames_seen"] == lengths[s]
    p.close()


def test_one_layer_qwen_shape_full_stream():
    """The single-layer Qwen2-7B-shaped workload in full: 64-token prefix, 64 frames x 169
    tokens, bank 64 (never evicts), 32 decode tokens."""
    w = synth.workload("layer")
    p = Pair(w)
    run_stream(p, w, check_every=16)
    assert p.ora[0].evictions == 0
    st = p.gpu.bank_state(0)
    assert st["count"] == 64 and st["persistent_bytes"] < st["workspace_bytes"]
    print("worst errors (max_abs, rel_rms):", p.worst)
    p.close()
