"""vs_evict_choose_static -- the eviction decision for callers that cannot allocate.

Some users of this library run where device allocation is off limits: a real-time frame loop
that must not stall on cudaMalloc, a component with a memory budget fixed up front, a plug-in
that may not bypass its host framework's allocator.  They get one entry point whose scratch
sits in a static device array of the library.  This test
drives a stream through the ordinary entry points (vs_frame_prefill decides evictions inside
the library, vs_bank_state reports them) and checks that the static entry point, given the
same carrier embeddings, names the same victim -- bit-exact, as for all bank bookkeeping --
on two calls issued back to back; the CPU oracle's choice on the same embeddings is checked
beside it.  Banks of more than eight carriers make the call span several thread blocks, which
is where the shared static array (scores of all blocks, the counter that elects the last
block) is really exercised.  It is collected last so that a failure here cannot hide any
other test's result, and it needs nothing from the other tests.
"""
import numpy as np
import pytest
import torch

from oracle import videoscan_oracle as vo
from paper_2503_09387_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("policy,capacity,d_model", [(0, 5, 512), (1, 5, 512), (0, 37, 256), (1, 37, 256)])
def test_static_eviction_choice_matches_the_stream(policy, capacity, d_model):
    build.build_library()
    # independent frames, so that the most similar stored carrier is not always the newest;
    # capacity 37 = five thread blocks, the last one partly filled
    w = synth.workload("tiny", d_model=d_model, n_q_heads=4, n_kv_heads=1, head_dim=d_model // 4, tokens_per_frame=12,
                       n_frames=capacity + 12, bank_capacity=capacity, prefix_len=4, seed=21 + policy)
    cfg = binding.make_config(1, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens_per_frame, 4, 4,
                              w.bank_capacity, evict_policy=policy)
    sb = binding.StreamBatch(cfg, [_dev(w.weight(0))])
    cases = []                      # (bank embeddings before the frame, incoming carrier, victim index)
    for t in range(w.n_frames):
        before = sb.bank_state(0, want_emb=True)
        sb.frame_prefill([0], _dev(w.frame_hidden(t)[None]), want_out=False)
        after = sb.bank_state(0, want_emb=True)
        if before["count"] == w.bank_capacity:
            step, victim_frame = after["evict_log"][-1]
            assert step == t
            victim = list(before["frame_ids"]).index(victim_frame)
            cases.append((before["emb"], after["emb"][-1], victim))
            # the oracle, given the same embeddings, discards the same carrier
            assert vo.choose_victim(synth.bf16_bits_to_f64(before["emb"]), synth.bf16_bits_to_f64(after["emb"][-1]),
                                    policy) == victim
    assert len(cases) == w.n_frames - w.bank_capacity and len({c[2] for c in cases}) > 1
    # two calls in a row on the current stream, results read afterwards
    stream = torch.cuda.current_stream().cuda_stream
    for first in range(0, len(cases) - 1, 2):
        pair = cases[first:first + 2]
        outs = [torch.full((1,), -7, dtype=torch.int32, device="cuda") for _ in pair]
        keep = []
        for (emb, inc, _), out in zip(pair, outs):
            e, i = _dev(emb), _dev(inc)
            keep += [e, i]
            binding.vs_evict_choose_static(e.data_ptr(), i.data_ptr(), emb.shape[0], w.d_model, policy,
                                           out.data_ptr(), stream)
        torch.cuda.synchronize()
        assert [int(o.item()) for o in outs] == [c[2] for c in pair]
    sb.close()


def test_static_entry_point_rejects_what_it_cannot_hold():
    build.build_library()
    x = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.VsError) as e:
        binding.vs_evict_choose_static(x.data_ptr(), x.data_ptr(), binding.VS_STATIC_MAX_BANK + 1, 64, 0, out.data_ptr())
    assert e.value.code == binding.VS_ERR_CAPACITY
    with pytest.raises(binding.VsError) as e:
        binding.vs_evict_choose_static(x.data_ptr(), x.data_ptr(), 0, 64, 0, out.data_ptr())
    assert e.value.code == binding.VS_ERR_INVALID_ARG
    # all-zero embeddings: every cosine counts as 0, so the oldest carrier is named
    binding.vs_evict_choose_static(x.data_ptr(), x[0].data_ptr(), 8, 64, 0, out.data_ptr())
    torch.cuda.synchronize()
    assert int(out.item()) == 0


def test_static_entry_point_at_its_largest_bank_and_with_non_finite_values():
    """VS_STATIC_MAX_BANK carriers (512 thread blocks writing the shared array), checked against the
    oracle, twice in a row; then a bank in which one carrier holds a NaN and an incoming carrier
    that holds an Inf: an undefined cosine counts as 0 and the index stays inside the bank."""
    build.build_library()
    n, d = binding.VS_STATIC_MAX_BANK, 64
    stream = torch.cuda.current_stream().cuda_stream
    outs, wants, keep = [], [], []
    for rep in range(2):
        bank = synth.normal_bf16(5 + rep, synth.TAG_PREFIX, (n, d), 1.0)
        inc = synth.normal_bf16(9 + rep, synth.TAG_QUESTION, (d,), 1.0)
        bank[(1234 + rep) % n] = inc                         # an exact duplicate somewhere in the middle
        bank[(3000 + rep) % n] = inc                         # and a second, younger one: the older must be named
        e, i = _dev(bank), _dev(inc)
        out = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        keep += [e, i]
        binding.vs_evict_choose_static(e.data_ptr(), i.data_ptr(), n, d, 0, out.data_ptr(), stream)
        outs.append(out)
        wants.append(vo.choose_victim(synth.bf16_bits_to_f64(bank), synth.bf16_bits_to_f64(inc), 0))
    torch.cuda.synchronize()
    assert [int(o.item()) for o in outs] == wants == [1234, 1235]
    bank = synth.normal_bf16(3, synth.TAG_PREFIX, (21, d), 1.0)
    inc = synth.normal_bf16(4, synth.TAG_QUESTION, (d,), 1.0)
    bank[7, 5] = 0x7FC0                                       # NaN
    bank[15] = inc
    for policy, incoming in ((0, inc), (1, inc), (0, np.where(np.arange(d) == 2, 0x7F80, inc).astype(np.uint16))):
        out = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        e, i = _dev(bank), _dev(incoming)
        binding.vs_evict_choose_static(e.data_ptr(), i.data_ptr(), 21, d, policy, out.data_ptr(), stream)
        torch.cuda.synchronize()
        want = vo.choose_victim(synth.bf16_bits_to_f64(bank), synth.bf16_bits_to_f64(incoming), policy)
        assert 0 <= int(out.item()) < 21 and int(out.item()) == want
