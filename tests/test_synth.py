"""The seeded input generator: determinism, distribution, recipe structure."""
import numpy as np

from paper_2503_09387_b200 import synth


def test_counter_based_draws_are_chunk_independent():
    a = synth.standard_normal(3, synth.TAG_WEIGHT, 1000)
    b = np.concatenate([synth.standard_normal(3, synth.TAG_WEIGHT, 400),
                        synth.standard_normal(3, synth.TAG_WEIGHT, 600, offset=400)])
    assert np.array_equal(a, b)
    assert not np.array_equal(a, synth.standard_normal(4, synth.TAG_WEIGHT, 1000))
    assert not np.array_equal(a, synth.standard_normal(3, synth.TAG_PREFIX, 1000))


def test_normals_have_the_stated_moments():
    z = synth.standard_normal(0, synth.TAG_FRAME_NOISE, 400000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    assert abs(np.mean(z ** 3)) < 0.03 and abs(np.mean(z ** 4) - 3.0) < 0.1
    w = synth.workload("tiny")
    W = synth.bf16_bits_to_f64(w.weight(0))
    assert W.shape == (384, 256) and abs(W.std() - 0.02) < 0.001


def test_bf16_bits_are_round_to_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0])
    got = synth.bf16_bits_to_f64(synth.to_bf16_bits(x))
    assert np.array_equal(got, [1.0, 1.0, 1.0 + 2.0 ** -6, -2.5, 0.0])


def test_workload_shapes():
    w = synth.workload("layer")
    assert (w.e_out, w.d_model, w.tokens_per_frame, w.bank_capacity) == (4608, 3584, 169, 64)
    assert synth.workload("deep").n_layers == 28 and synth.workload("deep").use_rmsnorm == 1
    b = synth.workload("batched")
    L = b.stream_lengths()
    assert len(L) == 16 and min(L) >= 64 and max(L) <= 256 and len(set(L)) > 4
    assert synth.workload("long").stream_lengths() == [1024]


def test_frame_recipes():
    w = synth.workload("layer", d_model=512, tokens_per_frame=64, n_frames=4)
    shared = w.frame_shared()
    E = synth.bf16_bits_to_f64(w.frame_hidden(2, shared=shared))
    assert E.shape == (64, 512)
    resid = E - shared[2][None, :]
    assert abs(resid.std() - 0.5) < 0.02                      # per-token noise N(0, 0.5)
    assert np.array_equal(w.frame_hidden(2), w.frame_hidden(2, shared=shared))
    a = synth.workload("long", d_model=2048, n_frames=401)
    f = a.frame_shared()
    rho = np.array([np.corrcoef(f[t], f[t + 1])[0, 1] for t in range(400)])
    cuts = [t + 1 for t in range(400) if rho[t] < 0.5]
    assert all(c % 100 == 0 for c in cuts)                    # only scene cuts decorrelate
    smooth = [rho[t] for t in range(400) if (t + 1) % 100 != 0]
    assert abs(np.mean(smooth) - 0.9) < 0.02
    assert abs(f.std() - 1.0) < 0.05                          # AR(1) is variance preserving
