#!/usr/bin/env python
"""Benchmark of the streaming attention path on B200.

A step = one whole stream of the one-layer Qwen2-7B-shaped workload through the C ABI:
reset, 64-token prompt prefix, 64 frames x 169 visual tokens (one vs_frame_prefill call per
frame, bank capacity 64), 32 single-token decode steps.  Inputs are seeded synthetic tensors
(paper_2503_09387_b200.synth) already resident in HBM; L2 is flushed between steps.  Device
time is taken with CUDA events around the three phases; `value` = frames / frame-phase time.

Extra legs (same process, same workload):
  e2e          -- the same step with HOST (pinned) inputs: per-call H2D copy of the hidden
                  states and D2H copy of the output inside the timed region (copies on their
                  own streams, double-buffered, so they overlap the kernels).
  roofline     -- the dominant kernel's average launch duration from CUDA events recorded
                  around every launch (vs_profile_enable) in one extra pass of the step.
  cpu_baseline -- the CPU oracle, as it stands, on a bounded sample of the same workload.
`--impl reference` times the oracle alone (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_09387_b200 import synth  # noqa: E402


CHUNK_FRAMES = 8                            # frames per vs_frame_prefill_chunk call in the `chunked_prefill` leg
ORACLE_KIND = "oracle (numpy, BLAS threads)"
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel at the bench's
# shape, from the ncu capture summarised under profiles/ (cold cache: the weights come from DRAM,
# whereas inside the timed one-layer loop they are L2-resident).  None = not captured since the
# kernel last changed.
DOMINANT_KERNEL_TRAFFIC = {"bytes": 34.38e6 + 0.02e6,
                           "source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of one cold-cache frame launch "
                                     "(profiles/qkv_gemm_frame_170rows.md); in the timed loop the weights are L2-resident"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ algorithmic work
def frame_flops(w, n_bank):
    rows = w.tokens_per_frame + 1
    proj = 2.0 * rows * w.d_model * w.e_out
    keys_ctx = w.prefix_len + n_bank
    attn = 4.0 * w.n_q_heads * w.head_dim * (rows * keys_ctx + rows * (rows + 1) / 2.0)
    return proj, attn


def frame_bytes(w, n_bank, out_bytes_per_el, weights_from_hbm):
    rows = w.tokens_per_frame + 1
    b = w.tokens_per_frame * w.d_model * 2                       # hidden in
    b += rows * w.n_q_heads * w.head_dim * out_bytes_per_el      # attention out
    b += (w.prefix_len + n_bank) * 2 * w.n_kv_heads * w.head_dim * 2   # prefix + bank K/V
    b += 2 * w.n_kv_heads * w.head_dim * 2 + w.d_model * 2       # carrier K/V + embedding append
    if weights_from_hbm:
        b += w.e_out * w.d_model * 2
    return float(b)


def decode_bytes(w, n_keys, out_bytes_per_el):
    b = w.e_out * w.d_model * 2                                  # weights
    b += n_keys * 2 * w.n_kv_heads * w.head_dim * 2              # K/V read
    b += 2 * w.n_kv_heads * w.head_dim * 2                       # tail append
    b += w.d_model * 2 + w.n_q_heads * w.head_dim * out_bytes_per_el
    return float(b)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ------------------------------------------------------------------ the oracle legs
def oracle_stream(w):
    from oracle import videoscan_oracle as vo
    cfg = vo.OracleConfig(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity,
                          use_rmsnorm=w.use_rmsnorm, residual=w.residual, rope_theta=w.rope_theta, rms_eps=w.rms_eps)
    return vo.OracleStream(cfg, [synth.bf16_bits_to_f64(w.weight(l)) for l in range(w.n_layers)])


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle_sample(w, n_frames, n_decode):
    """Times the oracle on prefix + n_frames frames + n_decode tokens; returns (frames/s, tok/s, seconds)."""
    f64 = synth.bf16_bits_to_f64
    st = oracle_stream(w)
    shared = w.frame_shared(0, n_frames) if w.frame_model != "iid" else None
    frames = [f64(w.frame_hidden(t, shared=shared)) for t in range(n_frames)]
    prefix = f64(w.prefix_hidden())
    dec = [f64(w.decode_hidden(i)) for i in range(n_decode)]
    t0 = time.perf_counter()
    st.text_step(prefix)
    t1 = time.perf_counter()
    for E in frames:
        st.frame_step(E)
    t2 = time.perf_counter()
    for x in dec:
        st.text_step(x)
    t3 = time.perf_counter()
    return n_frames / (t2 - t1), (n_decode / (t3 - t2) if n_decode else 0.0), t3 - t0


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_frames, n_decode = 4, 4
    for _ in range(args.warmup):
        time_oracle_sample(w, 1, 1)
    t_frames = t_total = 0.0
    fps_list, tps_list = [], []
    for _ in range(args.steps):
        fps, tps, secs = time_oracle_sample(w, n_frames, n_decode)
        fps_list.append(fps); tps_list.append(tps); t_total += secs
    fps = len(fps_list) / sum(1.0 / f for f in fps_list)
    tps = len(tps_list) / sum(1.0 / f for f in tps_list)
    cores = blas_threads()
    sample = f"per step: {w.prefix_len}-token prefix, first {n_frames} frames, {n_decode} decode tokens of the workload"
    print(json.dumps({
        "impl": "reference", "metric": "streamed_frames_per_s", "value": fps, "unit": "frames/s",
        "decode_tokens_per_s": tps, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": cores, "kind": ORACLE_KIND, "sample": sample},
        "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_config(w):
    return {"workload": f"{w.name}: {w.n_layers} Qwen2-7B-shaped attention layer(s), d={w.d_model}, "
                        f"{w.n_q_heads}/{w.n_kv_heads} heads x {w.head_dim}, {w.prefix_len}-token prefix, "
                        f"{w.n_frames} frames x {w.tokens_per_frame} tokens, bank {w.bank_capacity}, "
                        f"{w.decode_tokens} decode tokens; one vs_frame_prefill call per frame",
            "l2": "flushed between steps (256 MiB write); inside a step the 33 MB weight matrix stays L2-resident",
            "out_dtype": "fp32"}


# ------------------------------------------------------------------ replicas
def max_over_ranks(t, world):
    """Slowest rank's value of every element of tensor `t` (in place): the job ends when it does."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t


def replica_throughput(world, units_per_rank, ms):
    """Whole-job rate of `world` independent replicas that each did `units_per_rank` in `ms`
    (the slowest rank's time): no rank shares work with another, so the units add up."""
    return world * units_per_rank / (ms * 1e-3)


# ------------------------------------------------------------------ our arm
REPEATS = 5                                 # the --steps block is timed this many times; the median block is reported
DEEP_TIMED_FRAMES = 16                      # deep leg: the last frames of the 512-frame stream are the timed ones
DEEP_TIMED_DECODE = 32


def draw_parallel(fn, n):
    """fn(i) for i < n on a thread pool (numpy releases the GIL inside the generator's array
    operations); the draws are counter based, so the order of evaluation does not matter."""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=max(1, min(16, (os.cpu_count() or 2) - 1))) as ex:
        return list(ex.map(fn, range(n)))


class Streamer:
    """One handle of the library fed from device-resident synthetic inputs of workload `w`."""

    def __init__(self, w, dev, local, lib, binding, torch, chunk_frames=1, out_dtype=1, share=None):
        import ctypes as C
        self.w, self.dev, self.lib, self.C, self.torch = w, dev, lib, C, torch
        to_dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)
        if share is not None:       # a second handle over the same device-resident inputs and weights
            self.weights, self.frames_host, self.frames = share.weights, share.frames_host, share.frames
            self.prefix, self.question, self.dec = share.prefix, share.question, share.dec
        else:
            self.weights = [to_dev(b) for b in draw_parallel(w.weight, w.n_layers)]
            shared = w.frame_shared() if w.frame_model != "iid" else None
            self.frames_host = np.stack(draw_parallel(lambda t: w.frame_hidden(t, shared=shared), w.n_frames))
            self.frames = to_dev(self.frames_host)                          # [F, N, d]
            self.prefix = to_dev(w.prefix_hidden())
            self.question = to_dev(w.question_hidden()) if w.question_len else None
            self.dec = to_dev(np.concatenate([w.decode_hidden(i) for i in range(w.decode_tokens)]))   # [n_dec, d]
        cfg = binding.make_config(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens_per_frame,
                                  max(w.prefix_len, 1), max(w.question_len + w.decode_tokens, 1), w.bank_capacity,
                                  n_streams=1, max_step_tokens=max(64, w.prefix_len), use_rmsnorm=w.use_rmsnorm,
                                  residual=w.residual, rope_theta=w.rope_theta, rms_eps=w.rms_eps, device=local,
                                  max_chunk_frames=chunk_frames, out_dtype=out_dtype)
        self.sb = binding.StreamBatch(cfg, self.weights)
        odt = torch.float32 if out_dtype == 1 else torch.bfloat16
        N, HD = w.tokens_per_frame, w.n_q_heads * w.head_dim
        self.N, self.HD = N, HD
        self.out_frame = torch.empty((N + 1, HD), dtype=odt, device=dev)
        self.out_text = torch.empty((max(w.prefix_len, w.question_len, 1), HD), dtype=odt, device=dev)
        self.out_dec = torch.empty((1, HD), dtype=odt, device=dev)
        self.stream = torch.cuda.current_stream(dev)
        self.sptr = C.c_void_p(self.stream.cuda_stream)
        self.ids = (C.c_int32 * 1)(0)
        self.h = C.c_void_p(self.sb.handle)
        self.frame_ptrs = [C.c_void_p(self.frames[t].data_ptr()) for t in range(w.n_frames)]
        self.dec_ptrs = [C.c_void_p(self.dec[i:i + 1].data_ptr()) for i in range(w.decode_tokens)]
        self.p_out_frame, self.p_out_dec = C.c_void_p(self.out_frame.data_ptr()), C.c_void_p(self.out_dec.data_ptr())
        self.p_out_text = C.c_void_p(self.out_text.data_ptr())
        self.binding = binding

    def ck(self, code):
        if code != 0:
            raise RuntimeError("library call failed: %s" % self.binding.status_string(code))

    def reset(self):
        self.ck(self.lib.vs_reset_stream(self.h, self.ids, 1, self.sptr))

    def text(self, x, T):
        self.ck(self.lib.vs_decode_step(self.h, self.ids, 1, self.C.c_void_p(x.data_ptr()), T, self.p_out_text, self.sptr))

    def frames_range(self, t0, t1):
        for t in range(t0, t1):
            self.ck(self.lib.vs_frame_prefill(self.h, self.ids, 1, self.frame_ptrs[t], self.N, None, self.p_out_frame, self.sptr))

    def decode_range(self, i0, i1):
        for i in range(i0, i1):
            self.ck(self.lib.vs_decode_step(self.h, self.ids, 1, self.dec_ptrs[i], 1, self.p_out_dec, self.sptr))

    def end_turn(self):
        self.ck(self.lib.vs_end_turn(self.h, self.ids, 1))


def kernel_table(phase):
    k = {n: {"launches": v[1], "total_ms": round(v[0], 4), "avg_us": round(1e3 * v[0] / v[1], 3)}
         for n, v in phase.items() if v[1]}
    tot = sum(v["total_ms"] for v in k.values())
    for v in k.values():
        v["share"] = round(v["total_ms"] / tot, 4) if tot else 0.0
    return k


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2503_09387_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()
    lib = binding.load_library()
    C = __import__("ctypes")

    # ---- inputs (replicas only: every rank streams its own copy of the workload) ----------
    S = Streamer(w, dev, local, lib, binding, torch, chunk_frames=CHUNK_FRAMES)
    sb, N, d, HD = S.sb, S.N, w.d_model, S.HD
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = S.stream

    def one_step(events=None, on_phase=None):
        S.reset()
        if events: events[0].record(stream)
        if w.prefix_len:
            S.text(S.prefix, w.prefix_len)
        if events: events[1].record(stream)
        if on_phase: on_phase("prefix")
        S.frames_range(0, w.n_frames)
        if events: events[2].record(stream)
        if on_phase: on_phase("frames")
        S.decode_range(0, w.decode_tokens)
        if events: events[3].record(stream)
        if on_phase: on_phase("decode")

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        flush.zero_()
        one_step()
    sb.profile_read()                                   # clear launch counters
    sampler = ClockSampler(local)
    sampler.start()
    # ---- the timed region: REPEATS blocks of exactly --steps steps, each block bracketed by a
    # barrier + synchronize; per phase the device time of a block is the sum over its steps of the
    # CUDA-event intervals, the slowest rank's block counts, and the median block is reported
    blocks = []
    wall0 = time.perf_counter()
    for _ in range(REPEATS):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
        barrier()
        for k in range(args.steps):
            flush.zero_()
            one_step(ev[k])
        barrier()
        t = torch.tensor([sum(e[0].elapsed_time(e[1]) for e in ev), sum(e[1].elapsed_time(e[2]) for e in ev),
                          sum(e[2].elapsed_time(e[3]) for e in ev)], dtype=torch.float64, device=dev)
        blocks.append(max_over_ranks(t, world).tolist())
    wall = time.perf_counter() - wall0
    counts = sb.profile_read()
    gpu_launches = sum(v[2] for v in counts.values()) // REPEATS      # of one block of --steps steps
    blocks.sort(key=lambda b: b[1])
    ms_prefix, ms_frames, ms_decode = blocks[len(blocks) // 2]
    fps = replica_throughput(world, args.steps * w.n_frames, ms_frames)
    tps = replica_throughput(world, args.steps * w.decode_tokens, ms_decode) if w.decode_tokens else 0.0

    # ---- the same frames, CHUNK_FRAMES per call (offline form; informative, not the headline) ----
    chunk_fps = None
    if w.n_frames % CHUNK_FRAMES == 0:
        out_chunk = torch.empty((CHUNK_FRAMES, N + 1, HD), dtype=torch.float32, device=dev)
        p_out_chunk = C.c_void_p(out_chunk.data_ptr())
        chunk_ptrs = [C.c_void_p(S.frames[t].data_ptr()) for t in range(0, w.n_frames, CHUNK_FRAMES)]

        def chunk_step(e0=None, e1=None):
            S.reset()
            if w.prefix_len:
                S.text(S.prefix, w.prefix_len)
            if e0: e0.record(stream)
            for cp in chunk_ptrs:
                S.ck(lib.vs_frame_prefill_chunk(S.h, 0, cp, CHUNK_FRAMES, N, p_out_chunk, S.sptr))
            if e1: e1.record(stream)

        for _ in range(3):
            flush.zero_(); chunk_step()
        c_steps = max(1, min(args.steps, 20))
        cev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(c_steps)]
        barrier()
        for k in range(c_steps):
            flush.zero_(); chunk_step(*cev[k])
        barrier()
        ms_chunk = torch.tensor([sum(a_.elapsed_time(b_) for a_, b_ in cev)], dtype=torch.float64, device=dev)
        chunk_fps = replica_throughput(world, c_steps * w.n_frames, max_over_ranks(ms_chunk, world).item())
        sb.profile_read()

    # ---- per-kernel pass: events around every launch, one extra step ------------------------
    per_phase = {}
    launches_per_step = gpu_launches // max(args.steps, 1) + 16
    sb.profile_enable(True, launches_per_step)
    flush.zero_()
    one_step(on_phase=lambda name: per_phase.__setitem__(name, sb.profile_read()))
    sb.profile_enable(False)

    # ---- deep leg: the 28-layer stack, where the weights (925 MB per pass) come from HBM -------
    deep = None
    if not args.no_deep and w.name == "layer":
        deep = run_deep_leg(args, dev, local, lib, binding, torch, flush, barrier, world)
    batched = None
    if not args.no_batched and w.name == "layer":
        batched = run_batched_leg(dev, local, binding, torch, flush, barrier, world)
    block = None
    if not args.no_block and w.name == "layer":
        block = run_block_leg(dev, local, binding, torch, flush, barrier, world)
    clocks = sampler.stop()

    result = None
    if rank == 0:
        peaks = load_peaks()
        kernels = kernel_table(per_phase["frames"])
        kernels_dec = kernel_table(per_phase["decode"])
        dom = max(kernels, key=lambda k: kernels[k]["total_ms"])
        proj_flops, _ = frame_flops(w, 0)
        avg_bank = (min(w.n_frames, w.bank_capacity) - 1) / 2.0 if w.bank_capacity else 0.0
        _, attn_flops = frame_flops(w, avg_bank)
        if dom == "qkv_gemm":
            ach = proj_flops / (kernels[dom]["avg_us"] * 1e-6) / 1e12
            roof = {"kernel": dom, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                    "peak_burst": peaks["bf16_tflops"], "frac_of_burst": ach / peaks["bf16_tflops"],
                    "traffic": DOMINANT_KERNEL_TRAFFIC.get("bytes") if (N, d, w.e_out) == (169, 3584, 4608) else None,
                    "traffic_source": DOMINANT_KERNEL_TRAFFIC.get("source"),
                    "peak_source": peaks["source"] + ": sustained bf16 figure (the kernel is timed inside a long step, "
                                   "tens of thousands of launches back to back); the burst figure is quoted beside it",
                    "flops_per_launch": proj_flops, "avg_launch_us": kernels[dom]["avg_us"]}
        else:
            # every other kernel of the frame step moves bytes: report against HBM
            rows = N + 1
            alg = {"prefill_attention": rows * (HD * 2 * 2 + 2 * w.n_kv_heads * w.head_dim * 2) + rows * HD * 4
                   + (w.prefix_len + avg_bank) * 2 * w.n_kv_heads * w.head_dim * 2,
                   "pool": 2 * N * d * 2 + d * 4}.get(dom, 0.0)
            ach = alg / (kernels[dom]["avg_us"] * 1e-6) / 1e9
            roof = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                    "bytes_per_launch": alg, "avg_launch_us": kernels[dom]["avg_us"]}
        us_frame = 1e3 * ms_frames / (args.steps * w.n_frames)
        flops_frame = (proj_flops + attn_flops) * w.n_layers
        bytes_frame = frame_bytes(w, avg_bank, 4, weights_from_hbm=w.n_layers > 1)
        ideal_c = flops_frame / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6
        ideal_h = bytes_frame / (peaks["hbm_gbs"] * 1e9) * 1e6
        ideal = max(ideal_c, ideal_h)
        n_keys = w.prefix_len + min(w.n_frames, w.bank_capacity) + w.decode_tokens / 2.0
        us_tok = 1e3 * ms_decode / (args.steps * max(w.decode_tokens, 1))
        bytes_tok = decode_bytes(w, n_keys, 4)
        dec_ideal = bytes_tok / (peaks["hbm_gbs"] * 1e9) * 1e6
        result = {
            "metric": "streamed_frames_per_s", "value": fps, "unit": "frames/s",
            "decode_tokens_per_s": tps, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "repeats": REPEATS,
            "ms_per_step": ms_prefix / args.steps + ms_frames / args.steps + ms_decode / args.steps,
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(w),
            "phase_ms_per_step": {"prefix": ms_prefix / args.steps, "frames": ms_frames / args.steps,
                                  "decode": ms_decode / args.steps},
            "timing": f"median of {REPEATS} blocks of {args.steps} steps; frames-phase ms of every block: "
                      + ", ".join("%.3f" % b[1] for b in blocks),
            "wall_s": wall, "clocks": clocks, "gpu_launches": gpu_launches,
            "roofline": roof, "kernels_frame_phase": kernels, "kernels_decode_phase": kernels_dec,
            "kernels_note": "per-launch CUDA events (one extra pass): each pair adds a few microseconds and "
                            "serialises launches that otherwise overlap, so the shares overstate the small kernels",
            "chunked_prefill": {"frames_per_call": CHUNK_FRAMES, "value": chunk_fps, "unit": "frames/s",
                                "note": "same frames through vs_frame_prefill_chunk (offline form); not the headline"},
            "step_roofline": {
                "frame": {"us_per_frame": us_frame, "ideal_us": ideal, "frac": ideal / us_frame,
                          "flops_per_frame": flops_frame, "hbm_bytes_per_frame": bytes_frame,
                          "ideal_compute_us": ideal_c, "ideal_hbm_us": ideal_h,
                          "peak_tflops": peaks["bf16_tflops_sustained"], "peak_gbs": peaks["hbm_gbs"],
                          "note": "ideal = max(flops / sustained bf16 peak, bytes / HBM peak); single-layer "
                                  "weights are L2-resident so they are not counted as HBM bytes"},
                "decode": {"us_per_token": us_tok, "ideal_hbm_us": dec_ideal, "frac": dec_ideal / us_tok,
                           "bytes_per_token": bytes_tok, "peak_gbs": peaks["hbm_gbs"],
                           "note": "bytes = weights + K/V + append; the weights are L2-resident in the "
                                   "one-layer workload, so this fraction is NOT a DRAM fraction: "
                                   "step_roofline_deep.decode is"}},
        }
        if deep is not None:
            result["step_roofline_deep"] = deep_rooflines(deep, peaks)
        if block is not None:
            result["full_block_leg"] = block_rooflines(block, peaks)
        if batched is not None:
            result["batched_leg"] = batched_rooflines(batched, peaks)

    # ---- end to end: host inputs, H2D + D2H inside the timed region ---------------------------
    # Three streams, two buffers each way: the copy of frame t+1 to the device and the copy of
    # frame t-1's output back overlap the kernels of frame t, as a caller that streams video would
    # arrange it (the library only sees the stream it is given).
    pin_frames = torch.from_numpy(S.frames_host.view(np.int16)).pin_memory()
    dev_in = [torch.empty((N, d), dtype=torch.int16, device=dev) for _ in range(2)]
    p_dev_in = [C.c_void_p(t_.data_ptr()) for t_ in dev_in]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]      # frame landed in dev_in[k]
    ev_done = [torch.cuda.Event() for _ in range(2)]    # kernels of the frame using buffers k finished
    ev_out = [torch.cuda.Event() for _ in range(2)]     # dev_out[k] copied back

    def e2e_step(S, pin_out, dev_out, p_dev_out):
        S.reset()
        if w.prefix_len:
            S.text(S.prefix, w.prefix_len)
        for t in range(w.n_frames):
            k = t & 1
            with torch.cuda.stream(s_in):
                if t >= 2:
                    s_in.wait_event(ev_done[k])          # dev_in[k] is free again
                dev_in[k].copy_(pin_frames[t], non_blocking=True)
                ev_in[k].record(s_in)
            stream.wait_event(ev_in[k])
            if t >= 2:
                stream.wait_event(ev_out[k])             # dev_out[k] is free again
            S.ck(lib.vs_frame_prefill(S.h, S.ids, 1, p_dev_in[k], N, None, p_dev_out[k], S.sptr))
            ev_done[k].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[k])
                pin_out[k].copy_(dev_out[k], non_blocking=True)
                ev_out[k].record(s_out)
        stream.synchronize(); s_in.synchronize(); s_out.synchronize()

    e_steps = max(1, min(args.steps, 3))

    def e2e_run(S_, odt):
        pin_out = [torch.empty((N + 1, HD), dtype=odt).pin_memory() for _ in range(2)]
        dev_out = [torch.empty((N + 1, HD), dtype=odt, device=dev) for _ in range(2)]
        p_dev_out = [C.c_void_p(t_.data_ptr()) for t_ in dev_out]
        e2e_step(S_, pin_out, dev_out, p_dev_out)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e_steps):
            e2e_step(S_, pin_out, dev_out, p_dev_out)
        barrier()
        secs = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device=dev)
        max_over_ranks(secs, world)
        return secs

    e2e_s = e2e_run(S, torch.float32)
    # the same with the rows returned as bf16 (out_dtype = 0): half the bytes on the way back
    S16 = Streamer(w, dev, local, lib, binding, torch, out_dtype=0, share=S)
    e2e_s16 = e2e_run(S16, torch.bfloat16)
    S16.sb.close()
    if rank == 0:
        result["e2e"] = {"value": replica_throughput(world, e_steps * w.n_frames, 1e3 * e2e_s.item()), "unit": "frames/s",
                         "h2d_bytes_per_step": int(w.n_frames * N * d * 2),
                         "d2h_bytes_per_step": int(w.n_frames * (N + 1) * HD * 4),
                         "note": "frames phase only; per frame: pinned H2D of the hidden states, "
                                 "vs_frame_prefill, D2H of the fp32 output, the copies on streams of their own "
                                 "(two buffers each way); wall clock incl. launch cost",
                         "bf16_output": {"value": replica_throughput(world, e_steps * w.n_frames, 1e3 * e2e_s16.item()),
                                         "unit": "frames/s", "d2h_bytes_per_step": int(w.n_frames * (N + 1) * HD * 2),
                                         "note": "the same loop on a handle with out_dtype = 0 (rows returned as "
                                                 "bf16, the fp32 result rounded once)"}}
        if not args.no_cpu_baseline and world == 1:
            # the whole stream, repeated until about ten seconds of CPU work have been timed
            n_frames, n_decode = w.n_frames, w.decode_tokens
            inv_f, inv_t, secs, reps = 0.0, 0.0, 0.0, 0
            while secs < 10.0 and reps < 64:
                f_, t_, s_ = time_oracle_sample(w, n_frames, n_decode)
                inv_f += 1.0 / f_; inv_t += (1.0 / t_ if t_ else 0.0); secs += s_; reps += 1
            fps_cpu = reps / inv_f
            tps_cpu = reps / inv_t if inv_t else 0.0
            result["cpu_baseline"] = {"value": fps_cpu, "unit": "frames/s", "decode_tokens_per_s": tps_cpu,
                                      "cores": blas_threads(), "kind": ORACLE_KIND, "seconds": secs,
                                      "sample": f"{reps} x ({w.prefix_len}-token prefix, {n_frames} frames and "
                                                f"{n_decode} decode tokens): the same workload, whole"}
        print(json.dumps(result))
    sb.close()
    if world > 1:
        dist.destroy_process_group()


def run_deep_leg(args, dev, local, lib, binding, torch, flush, barrier, world):
    """The 28-layer workload at its stated size, end of the stream: the bank is filled by the first
    512 - DEEP_TIMED_FRAMES frames outside the timed region, then the last DEEP_TIMED_FRAMES frames
    are timed (bank 496 .. 511 carriers), the 32-token question is prefilled (untimed) and
    DEEP_TIMED_DECODE single-token steps are timed over [64-token prefix | 512 carriers | text]."""
    wd = synth.workload("deep")
    D = Streamer(wd, dev, local, lib, binding, torch)
    F0 = wd.n_frames - DEEP_TIMED_FRAMES
    n_dec = min(DEEP_TIMED_DECODE, wd.decode_tokens)

    def pass_(ev=None):
        D.reset()
        D.text(D.prefix, wd.prefix_len)
        D.frames_range(0, F0)
        flush.zero_()
        if ev: ev[0].record(D.stream)
        D.frames_range(F0, wd.n_frames)
        if ev: ev[1].record(D.stream)
        D.text(D.question, wd.question_len)
        flush.zero_()
        if ev: ev[2].record(D.stream)
        D.decode_range(0, n_dec)
        if ev: ev[3].record(D.stream)
        D.end_turn()

    pass_()                                                    # warm-up (every kernel has run before)
    D.sb.profile_read()
    reps = []
    for _ in range(REPEATS):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        barrier()
        pass_(ev)
        barrier()
        t = torch.tensor([ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3])], dtype=torch.float64, device=dev)
        reps.append(max_over_ranks(t, world).tolist())
    counts = D.sb.profile_read()
    # per-kernel times of the timed parts, one extra pass with events around every launch
    D.reset(); D.text(D.prefix, wd.prefix_len); D.frames_range(0, F0)
    D.sb.profile_read()
    D.sb.profile_enable(True, wd.n_layers * 4 * (DEEP_TIMED_FRAMES + n_dec + 2) + 64)
    D.frames_range(F0, wd.n_frames)
    k_frames = D.sb.profile_read()
    D.text(D.question, wd.question_len)
    D.sb.profile_read()
    D.decode_range(0, n_dec)
    k_dec = D.sb.profile_read()
    D.sb.profile_enable(False)
    D.end_turn()
    ms_f = sorted(r[0] for r in reps)[len(reps) // 2]
    ms_d = sorted(r[1] for r in reps)[len(reps) // 2]
    out = dict(w=wd, ms_frames=ms_f, ms_decode=ms_d, n_frames=DEEP_TIMED_FRAMES, n_decode=n_dec, F0=F0,
               all_ms_frames=[r[0] for r in reps], all_ms_decode=[r[1] for r in reps],
               kernels_frames=kernel_table(k_frames), kernels_decode=kernel_table(k_dec),
               launches=sum(v[2] for v in counts.values()) // REPEATS, world=world)
    D.sb.close()
    return out


BLOCK_LAYERS, BLOCK_D_FF, BLOCK_VOCAB, BLOCK_FRAMES, BLOCK_DECODE = 2, 18944, 152064, 8, 16
BATCHED_WARM, BATCHED_FRAMES, BATCHED_DECODE = 24, 8, 16


def run_batched_leg(dev, local, binding, torch, flush, barrier, world):
    """Sixteen streams per call (the 16-stream workload's shape: 196 tokens per frame, one Qwen2-7B-shaped
    attention layer, bank capacity 1024): BATCHED_WARM untimed frame steps of all streams, then BATCHED_FRAMES timed
    ones, then BATCHED_DECODE timed single-token steps of all streams.  Frames are seeded iid N(0, 1) rows drawn
    on the device; weights from the workload's generator."""
    wq = synth.workload("batched")
    S_, N, d, HD = wq.n_streams, wq.tokens_per_frame, wq.d_model, wq.n_q_heads * wq.head_dim
    to_dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)
    g = torch.Generator(device=dev); g.manual_seed(4321 + local)
    n_fr = BATCHED_WARM + BATCHED_FRAMES
    frames = torch.randn((n_fr, S_, N, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    prefix = torch.randn((S_, wq.prefix_len, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    dec = torch.randn((BATCHED_DECODE, S_, 1, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    cfg = binding.make_config(1, d, wq.n_q_heads, wq.n_kv_heads, wq.head_dim, N, wq.prefix_len, BATCHED_DECODE,
                              wq.bank_capacity, n_streams=S_, max_step_tokens=max(64, wq.prefix_len),
                              rope_theta=wq.rope_theta, rms_eps=wq.rms_eps, device=local)
    sb = binding.StreamBatch(cfg, [to_dev(wq.weight(0))])
    ids = list(range(S_))
    out_f = torch.empty((S_, N + 1, HD), dtype=torch.float32, device=dev)
    out_d = torch.empty((S_, 1, HD), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def pass_(ev=None):
        sb.reset(ids)
        sb.decode_step(ids, prefix)
        for t in range(BATCHED_WARM):
            sb.frame_prefill(ids, frames[t], out=out_f)
        flush.zero_()
        if ev: ev[0].record(stream)
        for t in range(BATCHED_WARM, n_fr):
            sb.frame_prefill(ids, frames[t], out=out_f)
        if ev: ev[1].record(stream)
        flush.zero_()
        if ev: ev[2].record(stream)
        for i in range(BATCHED_DECODE):
            sb.decode_step(ids, dec[i], out=out_d)
        if ev: ev[3].record(stream)
        sb.end_turn(ids)

    pass_()
    reps = []
    for _ in range(3):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        barrier()
        pass_(ev)
        barrier()
        t = torch.tensor([ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3])], dtype=torch.float64, device=dev)
        reps.append(max_over_ranks(t, world).tolist())
    assert sb.bank_state(0)["device_status"] == 0
    sb.close()
    med = lambda k: sorted(r[k] for r in reps)[len(reps) // 2]
    return dict(w=wq, ms_frames=med(0), ms_decode=med(1), world=world)


def batched_rooflines(bt, peaks):
    wq = bt["w"]
    S_, rows = wq.n_streams, wq.tokens_per_frame + 1
    n_bank = BATCHED_WARM + (BATCHED_FRAMES - 1) / 2.0
    proj, attn = frame_flops(wq, n_bank)                      # per stream (its own rows and keys)
    flops = S_ * (proj + attn)
    us_step = 1e3 * bt["ms_frames"] / BATCHED_FRAMES
    ideal = flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6
    us_dec = 1e3 * bt["ms_decode"] / BATCHED_DECODE
    return {
        "workload": f"{S_} streams per call, {wq.tokens_per_frame} tokens per frame, one Qwen2-7B-shaped attention layer, "
                    f"{wq.prefix_len}-token prefix, bank capacity {wq.bank_capacity}; {BATCHED_WARM} untimed frame steps, "
                    f"{BATCHED_FRAMES} timed, then {BATCHED_DECODE} timed batched decode steps; median of 3 passes",
        "frame": {"us_per_batched_step": us_step, "frames_per_s": bt["world"] * S_ * 1e6 / us_step, "ideal_us": ideal,
                  "frac": ideal / us_step, "flops_per_step": flops, "peak_tflops": peaks["bf16_tflops_sustained"],
                  "note": "ideal = flops / sustained bf16 peak (weights L2-resident: one layer)"},
        "decode": {"us_per_batched_step": us_dec, "tokens_per_s": bt["world"] * S_ * 1e6 / us_dec},
    }


def run_block_leg(dev, local, binding, torch, flush, barrier, world):
    """Full Qwen2-7B decoder layers (attention, output projection, SwiGLU MLP of width 18944, RMSNorm before each
    half) and the language-model head (vocabulary 152064): BLOCK_LAYERS layers, a 64-token prefix and 8 untimed
    frames, then 8 timed frames; then BLOCK_DECODE timed token steps, each one vs_decode_step + vs_lm_head of its
    output row; then the head alone.  Weights are seeded N(0, 0.02^2) drawn on the device (2.1 GB)."""
    wb = synth.workload("layer", n_layers=BLOCK_LAYERS, use_rmsnorm=1, residual=1, n_frames=2 * BLOCK_FRAMES,
                        decode_tokens=BLOCK_DECODE)
    g = torch.Generator(device=dev); g.manual_seed(1234 + local)
    draw = lambda *shape: (torch.randn(shape, generator=g, device=dev, dtype=torch.float32) * wb.weight_std).to(torch.bfloat16)
    d, L = wb.d_model, wb.n_layers
    weights = [draw(wb.e_out, d) for _ in range(L)]
    blockw = {"w_o": [draw(d, d) for _ in range(L)], "w_gate": [draw(BLOCK_D_FF, d) for _ in range(L)],
              "w_up": [draw(BLOCK_D_FF, d) for _ in range(L)], "w_down": [draw(d, BLOCK_D_FF) for _ in range(L)], "norm2_w": None}
    w_lm = draw(BLOCK_VOCAB, d)
    cfg = binding.make_config(L, d, wb.n_q_heads, wb.n_kv_heads, wb.head_dim, wb.tokens_per_frame, wb.prefix_len,
                              wb.decode_tokens, wb.bank_capacity, use_rmsnorm=1, residual=1, rope_theta=wb.rope_theta,
                              rms_eps=wb.rms_eps, device=local, d_ff=BLOCK_D_FF, vocab=BLOCK_VOCAB)
    sb = binding.StreamBatch(cfg, weights, block=blockw, lm=(w_lm, None))
    to_dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)
    shared = wb.frame_shared() if wb.frame_model != "iid" else None
    frames = to_dev(np.stack(draw_parallel(lambda t: wb.frame_hidden(t, shared=shared), wb.n_frames)))
    prefix = to_dev(wb.prefix_hidden())
    dec = to_dev(np.concatenate([wb.decode_hidden(i) for i in range(wb.decode_tokens)]))
    out_f = torch.empty((1, wb.tokens_per_frame + 1, d), dtype=torch.float32, device=dev)
    out_d = torch.empty((1, 1, d), dtype=torch.float32, device=dev)
    logits = torch.empty((1, BLOCK_VOCAB), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def pass_(ev=None):
        sb.reset([0])
        sb.decode_step([0], prefix[None])
        for t in range(BLOCK_FRAMES):
            sb.frame_prefill([0], frames[t][None], out=out_f)
        flush.zero_()
        if ev: ev[0].record(stream)
        for t in range(BLOCK_FRAMES, 2 * BLOCK_FRAMES):
            sb.frame_prefill([0], frames[t][None], out=out_f)
        if ev: ev[1].record(stream)
        flush.zero_()
        if ev: ev[2].record(stream)
        for i in range(BLOCK_DECODE):
            sb.decode_step([0], dec[i:i + 1][None], out=out_d)
            sb.lm_head(out_d[0], logits=logits)
        if ev: ev[3].record(stream)
        flush.zero_()
        if ev: ev[4].record(stream)
        for i in range(4):
            sb.lm_head(out_d[0], logits=logits)
        if ev: ev[5].record(stream)
        sb.end_turn([0])

    pass_()
    reps = []
    for _ in range(3):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        barrier()
        pass_(ev)
        barrier()
        t = torch.tensor([ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3]), ev[4].elapsed_time(ev[5])], dtype=torch.float64, device=dev)
        reps.append(max_over_ranks(t, world).tolist())
    assert sb.bank_state(0)["device_status"] == 0
    sb.close()
    med = lambda k: sorted(r[k] for r in reps)[len(reps) // 2]
    return dict(w=wb, ms_frames=med(0), ms_tokens=med(1), ms_head=med(2), world=world)


def block_rooflines(blk, peaks):
    wb = blk["w"]
    L, d, E, I, V, rows = wb.n_layers, wb.d_model, wb.e_out, BLOCK_D_FF, BLOCK_VOCAB, wb.tokens_per_frame + 1
    w_layer = (E * d + d * d + 3 * I * d) * 2                                  # bytes of one layer's matrices
    flops_frame = L * 2 * rows * (E * d + d * d + 3 * I * d)                   # attention's own flops left out (< 1 %)
    us_frame = 1e3 * blk["ms_frames"] / BLOCK_FRAMES
    us_tok = 1e3 * blk["ms_tokens"] / BLOCK_DECODE
    us_head = 1e3 * blk["ms_head"] / 4
    ideal_frame = max(flops_frame / (peaks["bf16_tflops_sustained"] * 1e12), L * w_layer / (peaks["hbm_gbs"] * 1e9)) * 1e6
    b_tok = L * w_layer + V * d * 2 + V * 4
    return {
        "workload": f"{L} full Qwen2-7B decoder layers (d={d}, d_ff={I}) + language-model head (vocabulary {V}); "
                    f"{BLOCK_FRAMES} timed frames of {wb.tokens_per_frame} tokens, then {BLOCK_DECODE} token steps "
                    f"(vs_decode_step + vs_lm_head), then the head alone; median of 3 passes; L2 flushed before each part",
        "frame": {"us_per_frame": us_frame, "us_per_layer": us_frame / L, "ideal_us": ideal_frame, "frac": ideal_frame / us_frame,
                  "flops_per_frame": flops_frame, "weight_bytes_per_layer": w_layer,
                  "note": "ideal = max(flops / sustained bf16 peak, weight bytes / HBM peak)"},
        "token": {"us_per_token": us_tok, "tokens_per_s": blk["world"] * 1e6 / us_tok, "bytes_per_token": b_tok,
                  "ideal_hbm_us": b_tok / (peaks["hbm_gbs"] * 1e9) * 1e6, "frac": b_tok / (peaks["hbm_gbs"] * 1e9) * 1e6 / us_tok,
                  "achieved_gbs": b_tok / us_tok * 1e-3,
                  "note": "a DRAM fraction: bytes = every layer's matrices + the vocabulary projection + the logits"},
        "lm_head": {"us_per_call": us_head, "bytes_per_call": V * d * 2 + V * 4,
                    "achieved_gbs": (V * d * 2 + V * 4) / us_head * 1e-3,
                    "frac": (V * d * 2 + V * 4) / (peaks["hbm_gbs"] * 1e9) * 1e6 / us_head},
    }


def deep_rooflines(deep, peaks):
    wd = deep["w"]
    L = wd.n_layers
    n_bank = deep["F0"] + (deep["n_frames"] - 1) / 2.0                     # carriers on the key axis of a timed frame
    proj, attn = frame_flops(wd, n_bank)
    flops = (proj + attn) * L
    rows = wd.tokens_per_frame + 1
    kv_row = 2 * wd.n_kv_heads * wd.head_dim * 2                           # K + V bytes of one key, one layer
    b_frame = (L * wd.e_out * wd.d_model * 2                               # every layer's weights
               + L * (wd.prefix_len + n_bank) * kv_row                     # prefix + bank K/V read per layer
               + L * kv_row + wd.d_model * 2                               # carrier K/V per layer + embedding
               + wd.tokens_per_frame * wd.d_model * 2                      # hidden in
               + rows * wd.n_q_heads * wd.head_dim * 4)                    # last layer's output (fp32)
    us_frame = 1e3 * deep["ms_frames"] / deep["n_frames"]
    ideal_c = flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6
    ideal_h = b_frame / (peaks["hbm_gbs"] * 1e9) * 1e6
    n_keys = wd.prefix_len + wd.bank_capacity + wd.question_len + (deep["n_decode"] + 1) / 2.0
    b_tok = (L * wd.e_out * wd.d_model * 2 + L * n_keys * kv_row + L * kv_row
             + wd.d_model * 2 + wd.n_q_heads * wd.head_dim * 4)
    us_tok = 1e3 * deep["ms_decode"] / deep["n_decode"]
    ideal_t = b_tok / (peaks["hbm_gbs"] * 1e9) * 1e6
    return {
        "workload": f"deep: {L} layers (RMSNorm, residual, no MLP), d={wd.d_model}, {wd.n_q_heads}/{wd.n_kv_heads} heads x "
                    f"{wd.head_dim}, {wd.prefix_len}-token prefix, bank {wd.bank_capacity}; frames 0..{deep['F0'] - 1} "
                    f"of the {wd.n_frames}-frame stream fill the bank outside the timed region; timed: frames "
                    f"{deep['F0']}..{wd.n_frames - 1}, then (after the untimed {wd.question_len}-token question) "
                    f"{deep['n_decode']} single-token decode steps; median of {REPEATS} passes; L2 flushed before "
                    f"each timed part (925 MB of weights per pass do not fit in L2 anyway)",
        "frame": {"us_per_frame": us_frame, "frames_per_s": deep["world"] * 1e6 / us_frame,
                  "us_per_layer": us_frame / L, "ideal_us": max(ideal_c, ideal_h),
                  "frac": max(ideal_c, ideal_h) / us_frame, "ideal_compute_us": ideal_c, "ideal_hbm_us": ideal_h,
                  "flops_per_frame": flops, "hbm_bytes_per_frame": b_frame,
                  "peak_tflops": peaks["bf16_tflops_sustained"], "peak_gbs": peaks["hbm_gbs"],
                  "ms_all_passes": deep["all_ms_frames"]},
        "decode": {"us_per_token": us_tok, "tokens_per_s": deep["world"] * 1e6 / us_tok, "us_per_layer": us_tok / L,
                   "ideal_hbm_us": ideal_t, "frac": ideal_t / us_tok,
                   "achieved_gbs": b_tok / (us_tok * 1e-6) / 1e9, "bytes_per_token": b_tok, "peak_gbs": peaks["hbm_gbs"],
                   "ms_all_passes": deep["all_ms_decode"],
                   "note": "a DRAM fraction: bytes = every layer's weights + K/V of all keys + append + hidden"},
        "kernels_frame_phase": deep["kernels_frames"], "kernels_decode_phase": deep["kernels_decode"],
        "gpu_launches": deep["launches"],
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="layer")
    ap.add_argument("--frames", type=int, default=None, help="override the number of frames (exploration only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-deep", action="store_true", help="skip the 28-layer leg")
    ap.add_argument("--no-batched", action="store_true", help="skip the 16-streams-per-call leg")
    ap.add_argument("--no-block", action="store_true", help="skip the full-decoder-block + language-model-head leg")
    args = ap.parse_args()
    kw = {}
    if args.frames:
        kw["n_frames"] = args.frames
    w = synth.workload(args.workload, **kw)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
