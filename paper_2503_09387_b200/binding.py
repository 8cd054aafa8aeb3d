"""ctypes binding of ``libvideoscan.so`` -- argument marshalling only.

The functions keep the C names (``vs_create_stream``, ``vs_frame_prefill``,
``vs_decode_step``, ``vs_bank_state`` ...).  :class:`StreamBatch` is a convenience
wrapper that owns the torch tensors the library borrows (weights, workspace) and turns
tensors into pointers; every step of the method runs inside the library's CUDA kernels.
There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libvideoscan.so")

VS_OK = 0
VS_ERR_INVALID_ARG = -1
VS_ERR_STATE = -2
VS_ERR_CAPACITY = -3
VS_ERR_CUDA = -4
VS_ERR_DEVICE_TIMEOUT = -5
VS_ERR_UNSUPPORTED = -6
VS_ERR_BOUNDS = -7
VS_MAX_BATCH = 64

EXPORTS = ["vs_workspace_bytes", "vs_create_stream", "vs_frame_prefill", "vs_frame_prefill_chunk", "vs_bank_forward", "vs_decode_step",
           "vs_lm_head", "vs_end_turn", "vs_bank_state", "vs_last_step_kv", "vs_poison_scratch",
           "vs_destroy_stream", "vs_status_string", "vs_reset_stream", "vs_profile_enable",
           "vs_profile_read", "vs_kernel_class_name", "vs_evict_choose_static"]
VS_STATIC_MAX_BANK = 4096
VS_N_KERNEL_CLASSES = 10


class VsConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "max_tokens_per_frame",
        "max_prefix", "max_text", "max_step_tokens", "bank_capacity", "n_streams", "agg_mode",
        "evict_policy", "use_rmsnorm", "residual")] + [
        ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("device", C.c_int32),
        ("evict_log_capacity", C.c_int32), ("out_dtype", C.c_int32),
        ("max_chunk_frames", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32)]


class VsWeights(C.Structure):
    _fields_ = [("w_qkv", C.POINTER(C.c_void_p)), ("b_qkv", C.POINTER(C.c_void_p)),
                ("norm_w", C.POINTER(C.c_void_p)), ("w_o", C.POINTER(C.c_void_p)), ("w_gate", C.POINTER(C.c_void_p)),
                ("w_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)), ("norm2_w", C.POINTER(C.c_void_p)),
                ("w_lm", C.c_void_p), ("norm_f_w", C.c_void_p)]


class VsBankInfo(C.Structure):
    _fields_ = [("count", C.c_int32), ("capacity", C.c_int32), ("frames_seen", C.c_int64),
                ("evictions", C.c_int64), ("next_pos", C.c_int64), ("prefix_len", C.c_int64),
                ("text_len", C.c_int64), ("last_victim_frame", C.c_int32),
                ("device_status", C.c_int32), ("persistent_bytes", C.c_uint64),
                ("workspace_bytes", C.c_uint64)]


class VsError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no other path)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} is missing: build it with `python -m paper_2503_09387_b200.build` "
            "(the library is the only implementation; nothing falls back to the CPU)")
    lib = C.CDLL(p)
    vp, i32, i32p = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
    lib.vs_workspace_bytes.argtypes = [C.POINTER(VsConfig), C.POINTER(C.c_size_t)]
    lib.vs_create_stream.argtypes = [C.POINTER(VsConfig), C.POINTER(VsWeights), vp, C.c_size_t, C.POINTER(vp)]
    lib.vs_frame_prefill.argtypes = [vp, i32p, i32, vp, i32, vp, vp, vp]
    lib.vs_frame_prefill_chunk.argtypes = [vp, i32, vp, i32, i32, vp, vp]
    lib.vs_bank_forward.argtypes = [vp, i32, vp, vp]
    lib.vs_decode_step.argtypes = [vp, i32p, i32, vp, i32, vp, vp]
    lib.vs_end_turn.argtypes = [vp, i32p, i32]
    lib.vs_lm_head.argtypes = [vp, vp, i32, vp, vp, vp]
    lib.vs_bank_state.argtypes = [vp, i32, C.POINTER(VsBankInfo), i32p, C.POINTER(C.c_int64), i32p,
                                  i32p, i32, i32p, vp, i32, vp, vp]
    lib.vs_last_step_kv.argtypes = [vp, vp, vp, i32]
    lib.vs_poison_scratch.argtypes = [vp, vp]
    lib.vs_destroy_stream.argtypes = [vp]
    lib.vs_status_string.argtypes = [C.c_int]
    lib.vs_status_string.restype = C.c_char_p
    lib.vs_reset_stream.argtypes = [vp, i32p, i32, vp]
    lib.vs_profile_enable.argtypes = [vp, i32, i32]
    lib.vs_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.vs_evict_choose_static.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    lib.vs_kernel_class_name.argtypes = [i32]
    lib.vs_kernel_class_name.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("vs_status_string", "vs_kernel_class_name"):
            getattr(lib, name).restype = C.c_int
    if path is None:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().vs_status_string(code).decode()


def _check(code: int, what: str) -> None:
    if code != VS_OK:
        raise VsError(code, what)


def _ids(stream_ids: Sequence[int]):
    arr = (C.c_int32 * len(stream_ids))(*stream_ids)
    return arr, len(stream_ids)


# ---- C-named entry points (thin) ----------------------------------------------------------
def vs_workspace_bytes(cfg: VsConfig) -> int:
    out = C.c_size_t(0)
    _check(load_library().vs_workspace_bytes(C.byref(cfg), C.byref(out)), "vs_workspace_bytes")
    return int(out.value)


def vs_create_stream(cfg: VsConfig, w_ptrs: List[int], b_ptrs: Optional[List[Optional[int]]],
                     g_ptrs: Optional[List[Optional[int]]], workspace_ptr: int, workspace_bytes: int,
                     block_ptrs: Optional[dict] = None, lm_ptrs: Optional[Sequence[Optional[int]]] = None) -> int:
    """block_ptrs (full decoder block, cfg.d_ff > 0): {"w_o", "w_gate", "w_up", "w_down": [L pointers], "norm2_w": [L] or None}.
    lm_ptrs (language-model head, cfg.vocab > 0): (w_lm pointer, final-norm gain pointer or None)."""
    L = cfg.n_layers
    arr = lambda ptrs: C.cast((C.c_void_p * L)(*[p or None for p in ptrs]), C.POINTER(C.c_void_p)) if ptrs is not None else None
    keep = [arr(w_ptrs), arr(b_ptrs), arr(g_ptrs)]
    for name in ("w_o", "w_gate", "w_up", "w_down", "norm2_w"):
        keep.append(arr(block_ptrs.get(name)) if block_ptrs else None)
    ws = VsWeights(*keep, (lm_ptrs[0] if lm_ptrs else None), (lm_ptrs[1] if lm_ptrs else None) or None)
    handle = C.c_void_p(None)
    _check(load_library().vs_create_stream(C.byref(cfg), C.byref(ws), workspace_ptr, workspace_bytes,
                                           C.byref(handle)), "vs_create_stream")
    return handle.value


def vs_frame_prefill(handle: int, stream_ids: Sequence[int], hidden_ptr: int, N: int,
                     carrier_override_ptr: Optional[int], out_ptr: Optional[int], cuda_stream: int = 0) -> None:
    ids, n = _ids(stream_ids)
    _check(load_library().vs_frame_prefill(handle, ids, n, hidden_ptr, N, carrier_override_ptr or None,
                                           out_ptr or None, cuda_stream or None), "vs_frame_prefill")


def vs_lm_head(handle: int, hidden_ptr: int, rows: int, logits_ptr: int, next_token_ptr: Optional[int],
               cuda_stream: Optional[int] = None) -> None:
    _check(load_library().vs_lm_head(handle, hidden_ptr, rows, logits_ptr, next_token_ptr or None, cuda_stream or None),
           "vs_lm_head")


def vs_bank_forward(handle: int, stream_id: int, out_ptr: int, cuda_stream: Optional[int] = None) -> None:
    _check(load_library().vs_bank_forward(handle, stream_id, out_ptr, cuda_stream or None), "vs_bank_forward")


def vs_frame_prefill_chunk(handle: int, stream_id: int, hidden_ptr: int, F: int, N: int,
                           out_ptr: Optional[int] = None, cuda_stream: Optional[int] = None) -> None:
    _check(load_library().vs_frame_prefill_chunk(handle, stream_id, hidden_ptr, F, N, out_ptr or None,
                                                 cuda_stream or None), "vs_frame_prefill_chunk")


def vs_decode_step(handle: int, stream_ids: Sequence[int], hidden_ptr: int, T: int, out_ptr: int,
                   cuda_stream: int = 0) -> None:
    ids, n = _ids(stream_ids)
    _check(load_library().vs_decode_step(handle, ids, n, hidden_ptr, T, out_ptr, cuda_stream or None),
           "vs_decode_step")


def vs_end_turn(handle: int, stream_ids: Sequence[int]) -> None:
    ids, n = _ids(stream_ids)
    _check(load_library().vs_end_turn(handle, ids, n), "vs_end_turn")


def vs_reset_stream(handle: int, stream_ids: Sequence[int], cuda_stream: int = 0) -> None:
    ids, n = _ids(stream_ids)
    _check(load_library().vs_reset_stream(handle, ids, n, cuda_stream or None), "vs_reset_stream")


def vs_profile_enable(handle: int, on: bool, max_launches: int = 0) -> None:
    _check(load_library().vs_profile_enable(handle, 1 if on else 0, max_launches), "vs_profile_enable")


def vs_profile_read(handle: int) -> dict:
    """{class name: (summed ms of timed launches, timed launches, all launches)} since the last read."""
    lib = load_library()
    ms = (C.c_double * VS_N_KERNEL_CLASSES)()
    timed = (C.c_int64 * VS_N_KERNEL_CLASSES)()
    launches = (C.c_int64 * VS_N_KERNEL_CLASSES)()
    _check(lib.vs_profile_read(handle, ms, timed, launches), "vs_profile_read")
    return {lib.vs_kernel_class_name(k).decode(): (ms[k], int(timed[k]), int(launches[k]))
            for k in range(VS_N_KERNEL_CLASSES)}


def vs_evict_choose_static(bank_emb_ptr: int, incoming_ptr: int, count: int, d_model: int, policy: int,
                           victim_out_ptr: int, cuda_stream: int = 0) -> None:
    """Enqueues the allocation-free eviction decision; the result lands in the int32 at victim_out_ptr."""
    _check(load_library().vs_evict_choose_static(bank_emb_ptr, incoming_ptr, count, d_model, policy,
                                                 victim_out_ptr, cuda_stream or None), "vs_evict_choose_static")


def vs_destroy_stream(handle: int) -> None:
    _check(load_library().vs_destroy_stream(handle), "vs_destroy_stream")


def vs_poison_scratch(handle: int, cuda_stream: int = 0) -> None:
    _check(load_library().vs_poison_scratch(handle, cuda_stream or None), "vs_poison_scratch")


def vs_bank_state(handle: int, stream_id: int, cfg: VsConfig, layer: Optional[int] = None,
                  want_emb: bool = False) -> dict:
    """Synchronises and returns the bank of one stream in temporal order (numpy arrays;
    bf16 tensors as uint16 bit patterns)."""
    lib = load_library()
    M = max(cfg.bank_capacity, 1)
    info = VsBankInfo()
    frame_ids = np.zeros(M, dtype=np.int32)
    positions = np.zeros(M, dtype=np.int64)
    slots = np.zeros(M, dtype=np.int32)
    cap = max(cfg.evict_log_capacity, 1)
    log = np.zeros((cap, 2), dtype=np.int32)
    log_n = C.c_int32(0)
    emb = np.zeros((M, cfg.d_model), dtype=np.uint16) if want_emb else None
    k = v = None
    if layer is not None:
        k = np.zeros((M, cfg.n_kv_heads, cfg.head_dim), dtype=np.uint16)
        v = np.zeros_like(k)
    p = lambda a: a.ctypes.data_as(C.c_void_p) if a is not None else None
    code = lib.vs_bank_state(handle, stream_id, C.byref(info),
                             frame_ids.ctypes.data_as(C.POINTER(C.c_int32)),
                             positions.ctypes.data_as(C.POINTER(C.c_int64)),
                             slots.ctypes.data_as(C.POINTER(C.c_int32)),
                             log.ctypes.data_as(C.POINTER(C.c_int32)), cap, C.byref(log_n),
                             p(emb), layer if layer is not None else 0, p(k), p(v))
    _check(code, "vs_bank_state")
    n = info.count
    res = dict(count=n, capacity=info.capacity, frames_seen=info.frames_seen, evictions=info.evictions,
               next_pos=info.next_pos, prefix_len=info.prefix_len, text_len=info.text_len,
               last_victim_frame=info.last_victim_frame, device_status=info.device_status,
               persistent_bytes=info.persistent_bytes, workspace_bytes=info.workspace_bytes,
               frame_ids=frame_ids[:n].copy(), positions=positions[:n].copy(), slots=slots[:n].copy(),
               evict_log=log[:log_n.value].copy())
    if emb is not None:
        res["emb"] = emb[:n].copy()
    if k is not None:
        res["k"] = k[:n].copy()
        res["v"] = v[:n].copy()
    return res


def vs_last_step_kv(handle: int, rows: int, n_kv_heads: int, head_dim: int):
    k = np.zeros((rows, n_kv_heads * head_dim), dtype=np.uint16)
    v = np.zeros_like(k)
    _check(load_library().vs_last_step_kv(handle, k.ctypes.data_as(C.c_void_p), v.ctypes.data_as(C.c_void_p), rows),
           "vs_last_step_kv")
    return k, v


# ---- convenience wrapper: owns the borrowed tensors -------------------------------------------
class StreamBatch:
    """A handle plus the device tensors it borrows.  ``weights`` are torch bf16 CUDA tensors
    [E_out, d_model] per layer.  All methods take / return torch CUDA tensors and only enqueue
    work on the current torch stream."""

    def __init__(self, cfg: VsConfig, weights, biases=None, norm_weights=None, block=None, lm=None):
        # block (cfg.d_ff > 0): {"w_o", "w_gate", "w_up", "w_down": [L device tensors], "norm2_w": [L] or None}
        # lm (cfg.vocab > 0): (w_lm [vocab, d_model] device tensor, final-norm gain [d_model] or None)
        import torch
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        self.weights = [w.contiguous() for w in weights]
        self.biases = biases
        self.norm_weights = norm_weights
        self.block = block
        self.lm = lm
        nbytes = vs_workspace_bytes(cfg)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.workspace_bytes = nbytes
        self.handle = vs_create_stream(
            cfg, [w.data_ptr() for w in self.weights],
            [b.data_ptr() if b is not None else None for b in biases] if biases is not None else None,
            [g.data_ptr() if g is not None else None for g in norm_weights] if norm_weights is not None else None,
            self._ws_ptr, nbytes,
            {k: ([t.data_ptr() if t is not None else None for t in v] if v is not None else None) for k, v in block.items()}
            if block else None,
            (lm[0].data_ptr(), lm[1].data_ptr() if lm[1] is not None else None) if lm else None)
        self.out_width = cfg.n_q_heads * cfg.head_dim
        self.out_torch_dtype = torch.float32 if cfg.out_dtype == 1 else torch.bfloat16

    def _stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def lm_head(self, hidden, logits=None, want_token=True):
        """hidden: [rows, d_model] of the handle's output dtype -> (logits fp32 [rows, vocab], next tokens int32 [rows] or None)."""
        rows = hidden.shape[0]
        assert hidden.is_contiguous() and hidden.dtype == self.out_torch_dtype and hidden.numel() == rows * self.cfg.d_model
        if logits is None:
            logits = self.torch.empty((rows, self.cfg.vocab), dtype=self.torch.float32, device=self.device)
        token = self.torch.empty((rows,), dtype=self.torch.int32, device=self.device) if want_token else None
        vs_lm_head(self.handle, hidden.data_ptr(), rows, logits.data_ptr(), token.data_ptr() if want_token else None, self._stream())
        return logits, token

    def frame_prefill(self, stream_ids, hidden, carrier_override=None, out=None, want_out=True):
        n = len(stream_ids)
        N = hidden.shape[-2]
        assert hidden.is_contiguous() and hidden.numel() == n * N * self.cfg.d_model
        if out is None and want_out:
            out = self.torch.empty((n, N + 1, self.out_width), dtype=self.out_torch_dtype, device=self.device)
        vs_frame_prefill(self.handle, stream_ids, hidden.data_ptr(), N,
                         carrier_override.data_ptr() if carrier_override is not None else None,
                         out.data_ptr() if out is not None else None, self._stream())
        return out

    def frame_prefill_chunk(self, stream_id, hidden, out=None, want_out=True):
        """hidden: [F][N][d] of one stream."""
        F, N = hidden.shape[0], hidden.shape[1]
        assert hidden.is_contiguous() and hidden.numel() == F * N * self.cfg.d_model
        if out is None and want_out:
            out = self.torch.empty((F, N + 1, self.out_width), dtype=self.out_torch_dtype, device=self.device)
        vs_frame_prefill_chunk(self.handle, stream_id, hidden.data_ptr(), F, N,
                               out.data_ptr() if out is not None else None, self._stream())
        return out

    def bank_forward(self, stream_id, count):
        """Carriers-only forward of one stream's bank; `count` = carriers in it."""
        out = self.torch.empty((count, self.out_width), dtype=self.out_torch_dtype, device=self.device)
        vs_bank_forward(self.handle, stream_id, out.data_ptr(), self._stream())
        return out

    def decode_step(self, stream_ids, hidden, out=None):
        n = len(stream_ids)
        T = hidden.shape[-2]
        assert hidden.is_contiguous() and hidden.numel() == n * T * self.cfg.d_model
        if out is None:
            out = self.torch.empty((n, T, self.out_width), dtype=self.out_torch_dtype, device=self.device)
        vs_decode_step(self.handle, stream_ids, hidden.data_ptr(), T, out.data_ptr(), self._stream())
        return out

    def end_turn(self, stream_ids):
        vs_end_turn(self.handle, stream_ids)

    def bank_state(self, stream_id=0, layer=None, want_emb=False):
        return vs_bank_state(self.handle, stream_id, self.cfg, layer, want_emb)

    def last_step_kv(self, rows):
        return vs_last_step_kv(self.handle, rows, self.cfg.n_kv_heads, self.cfg.head_dim)

    def reset(self, stream_ids):
        vs_reset_stream(self.handle, stream_ids, self._stream())

    def profile_enable(self, on, max_launches=0):
        vs_profile_enable(self.handle, on, max_launches)

    def profile_read(self):
        return vs_profile_read(self.handle)

    def poison_scratch(self):
        vs_poison_scratch(self.handle, self._stream())

    def close(self):
        if self.handle:
            vs_destroy_stream(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_config(n_layers, d_model, n_q_heads, n_kv_heads, head_dim, max_tokens_per_frame, max_prefix,
                max_text, bank_capacity, n_streams=1, max_step_tokens=64, agg_mode=0, evict_policy=0,
                use_rmsnorm=0, residual=0, rope_theta=1.0e6, rms_eps=1.0e-6, device=0,
                evict_log_capacity=4096, out_dtype=1, max_chunk_frames=1, d_ff=0, vocab=0) -> VsConfig:
    return VsConfig(n_layers, d_model, n_q_heads, n_kv_heads, head_dim, max_tokens_per_frame, max_prefix,
                    max_text, max_step_tokens, bank_capacity, n_streams, agg_mode, evict_policy, use_rmsnorm,
                    residual, rope_theta, rms_eps, device, evict_log_capacity, out_dtype, max_chunk_frames, d_ff, vocab)
