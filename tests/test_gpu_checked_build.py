"""The checked build (-DVS_DEBUG_BOUNDS) of the same CUDA sources, standing in for a memory checker:
every kernel store into the workspace is tested against the region it names (a store outside is
skipped and recorded, nothing traps), and 256 guard bytes lie behind every workspace region;
vs_bank_state reports either finding as VS_ERR_BOUNDS.  The small odd-shaped cases run through it
against the oracle: parity must hold and no finding may be reported."""
import numpy as np
import pytest

from paper_2503_09387_b200 import binding, build, synth
from tests.parity import Pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked_library():
    lib = binding.load_library(build.build_library(checked=True))
    saved = binding._lib
    binding._lib = lib
    try:
        yield lib
    finally:
        binding._lib = saved


def _stream(p, w, n_frames, chunk=0):
    if w.prefix_len:
        p.text([0], [w.prefix_hidden()], "prefix")
    t = 0
    while t < n_frames:
        if chunk and t + chunk <= n_frames and t % 2 == 1:
            p.frame_chunk(0, [w.frame_hidden(t + j) for j in range(chunk)], f"chunk at {t}")
            t += chunk
        else:
            p.frame([0], [w.frame_hidden(t)], f"frame {t}")
            t += 1
        st = p.check_bank(0, layer=w.n_layers - 1)          # asserts device_status == 0: no refused store, guards intact
        assert st["device_status"] == 0
    if w.question_len:
        p.text([0], [w.question_hidden()], "question")
    for i in range(w.decode_tokens):
        p.text([0], [w.decode_hidden(i)], f"decode {i}")
    assert p.check_bank(0)["device_status"] == 0


@pytest.mark.parametrize("N,P,M,policy", [(1, 0, 0, 0), (7, 1, 1, 0), (17, 3, 2, 1), (33, 5, 3, 2), (16, 8, 4, 0)])
def test_odd_shapes_through_the_checked_build(checked_library, N, P, M, policy):
    w = synth.workload("tiny", tokens_per_frame=N, prefix_len=P, bank_capacity=M, n_frames=7, question_len=5,
                       decode_tokens=2, seed=40 + N)
    p = Pair(w, evict_policy=policy, max_text=8, max_chunk_frames=3)
    _stream(p, w, 7, chunk=3)
    p.close()


def test_layers_norm_and_scratch_poison_through_the_checked_build(checked_library):
    w = synth.workload("deep", n_layers=3, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=21,
                       n_frames=6, bank_capacity=3, prefix_len=6, question_len=7, decode_tokens=3)
    p = Pair(w, with_gain=True, with_bias=True)
    p.text([0], [w.prefix_hidden()], "prefix")
    for t in range(w.n_frames):
        p.frame([0], [w.frame_hidden(t)], f"frame {t}")
        p.gpu.poison_scratch()                               # the guards behind the scratch regions are put back
        for layer in range(w.n_layers):
            assert p.check_bank(0, layer=layer)["device_status"] == 0
    p.text([0], [w.question_hidden()], "question")
    for i in range(w.decode_tokens):
        p.text([0], [w.decode_hidden(i)], f"decode {i}")
    assert p.check_bank(0)["device_status"] == 0
    p.close()


def test_two_streams_at_a_wider_shape_through_the_checked_build(checked_library):
    w = synth.workload("batched", d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, tokens_per_frame=30, n_frames=5,
                       min_frames=0, bank_capacity=2, prefix_len=4, decode_tokens=2, n_streams=2)
    p = Pair(w)
    ids = [0, 1]
    p.text(ids, [w.prefix_hidden(s) for s in ids], "prefix")
    for t in range(w.n_frames):
        p.frame(ids, [w.frame_hidden(t, s) for s in ids], f"frame {t}")
    for i in range(w.decode_tokens):
        p.text(ids, [w.decode_hidden(i, s) for s in ids], f"decode {i}")
    for s in ids:
        assert p.check_bank(s)["device_status"] == 0
    p.close()


def test_the_guard_check_is_alive(checked_library):
    """The caller (this test) overwrites the guard bytes behind the workspace's last region -- its own memory,
    written with a plain torch assignment -- and vs_bank_state must report VS_ERR_BOUNDS."""
    w = synth.workload("tiny", n_frames=2)
    p = Pair(w)
    p.text([0], [w.prefix_hidden()], "prefix")
    p.frame([0], [w.frame_hidden(0)], "frame 0")
    assert p.check_bank(0)["device_status"] == 0
    off = p.gpu._ws_ptr - p.gpu.workspace.data_ptr()
    p.gpu.workspace[off + p.gpu.workspace_bytes - 256: off + p.gpu.workspace_bytes] = 0
    with pytest.raises(binding.VsError) as err:
        p.gpu.bank_state(0)
    assert err.value.code == binding.VS_ERR_BOUNDS
    p.close()


def test_lm_head_through_the_checked_build(checked_library):
    """The language-model head writes only its own scratch (normalised rows, row statistics) and the caller's
    logits: parity holds and no guard byte behind a region changes."""
    from tests.test_gpu_parity import _lm_case, _check_lm
    for (d, vocab, rows, norm, gain, od) in [(256, 384, 3, True, True, 1), (320, 1152, 16, False, False, 0)]:
        got, gt, want, wt = _lm_case(d, vocab, rows, norm, gain, od)      # asserts device_status == 0 after the call
        _check_lm(got, gt, want, wt, f"checked build, lm head d={d} vocab={vocab}")


def test_block_in_chunks_and_carriers_only_forward_through_the_checked_build(checked_library):
    """The full decoder block inside a chunk of frames and inside the carriers-only forward: the GEMMs of the block
    run on F * (N + 1) rows (several token tiles) and write the activation, both residual buffers and the gained
    copies; no store may leave its region and no guard byte may change."""
    w = synth.workload("deep", n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=33,
                       n_frames=7, bank_capacity=3, prefix_len=6, question_len=5, decode_tokens=2)
    p = Pair(w, with_gain=True, d_ff=320, max_chunk_frames=3)
    p.text([0], [w.prefix_hidden()], "prefix")
    p.frame([0], [w.frame_hidden(0)], "frame 0")
    p.frame_chunk(0, [w.frame_hidden(1 + j) for j in range(3)], "chunk of 3")
    assert p.check_bank(0, layer=1)["device_status"] == 0
    p.bank_forward(0)
    p.frame_chunk(0, [w.frame_hidden(4 + j) for j in range(3)], "second chunk of 3")
    p.bank_forward(0)
    p.text([0], [w.question_hidden()], "question")
    for i in range(w.decode_tokens):
        p.text([0], [w.decode_hidden(i)], f"decode {i}")
    assert p.check_bank(0)["device_status"] == 0
    p.close()


def test_qwen_shape_through_the_checked_build(checked_library):
    """The kernels' full-size launch shapes (K split over four CTAs, 176-column token tiles, clusters of two in the
    attention, the matrix-vector projection and the split decode attention) with every workspace store checked:
    one Qwen2-7B-shaped attention layer, bank of 4 so that frames evict; then one layer with RMSNorm, the decoder
    block (d_ff 1024) and the language-model head."""
    w = synth.workload("layer", n_frames=7, bank_capacity=4, question_len=9, decode_tokens=3)
    p = Pair(w, max_text=12, max_chunk_frames=2)
    _stream(p, w, 7, chunk=2)
    p.close()
    w = synth.workload("deep", n_layers=1, n_frames=3, bank_capacity=2, prefix_len=16, question_len=5, decode_tokens=2)
    p = Pair(w, d_ff=1024, vocab=1024, max_text=8)
    _stream(p, w, 3)
    logits, tok = p.gpu.lm_head(p.last_out[0][-1:].contiguous())
    assert p.check_bank(0)["device_status"] == 0
    p.close()
