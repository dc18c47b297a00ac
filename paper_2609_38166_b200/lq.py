"""Thin Python binding of the C-ABI library (``include/lq.h``): argument marshalling only.

Every entry point has the name of its C symbol without the ``lq_`` prefix and takes torch tensors
(device memory and streams are PyTorch's; every step of the computation runs in the library's kernels).
There is no fallback of any kind: if ``liblq.so`` is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

GATE_SCALAR = 0
GATE_DIAG = 1

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblq.so")
_lib = None

EXPORTS = ["lq_decode_step", "lq_decode_step_profiled", "lq_decode_step_host", "lq_decode_step_host_pipelined", "lq_decode_step_host_static", "lq_decode_stage_bytes", "lq_head_bytes", "lq_record_floats",
           "lq_window_flush",
           "lq_quantize_state", "lq_dequantize_state", "lq_ref_decode_step_f32", "lq_ref_decode_step_bf16",
           "lq_decode_launches", "lq_check_device", "lq_clear_device_flags", "lq_selftest_bounded_wait",
           "lq_static_stage_bytes", "lq_import_state", "lq_export_state", "lq_status_string", "lq_version"]


class LqError(RuntimeError):
    pass


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("batch", "heads_v", "heads_qk", "d_k", "d_v", "W", "r", "n_iter", "gate", "smooth", "delta", "rec16", "state_bf16")]


class _State(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("heads", "records", "decays", "win_pos", "work")]


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built (``python -m paper_2609_38166_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise LqError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_38166_b200.build`")
        L = C.CDLL(_LIB_PATH)
        L.lq_status_string.restype = C.c_char_p
        L.lq_status_string.argtypes = [C.c_int]
        L.lq_version.restype = C.c_int
        L.lq_decode_stage_bytes.restype = C.c_uint64
        L.lq_decode_stage_bytes.argtypes = [C.c_void_p]
        for name in ("lq_head_bytes", "lq_record_floats"):
            getattr(L, name).restype = C.c_uint64
            getattr(L, name).argtypes = [C.c_void_p]
        L.lq_decode_launches.restype = C.c_int
        L.lq_decode_launches.argtypes = [C.c_void_p]
        L.lq_static_stage_bytes.restype = C.c_uint64
        L.lq_static_stage_bytes.argtypes = []
        L.lq_clear_device_flags.restype = C.c_int
        L.lq_clear_device_flags.argtypes = []
        L.lq_selftest_bounded_wait.restype = C.c_int
        L.lq_selftest_bounded_wait.argtypes = [C.c_void_p]
        for name in ("lq_import_state", "lq_export_state"):
            getattr(L, name).restype = C.c_int
        for name in ("lq_decode_step", "lq_decode_step_profiled", "lq_decode_step_host", "lq_decode_step_host_pipelined",
                     "lq_decode_step_host_static", "lq_check_device", "lq_window_flush", "lq_quantize_state",
                     "lq_dequantize_state", "lq_ref_decode_step_f32", "lq_ref_decode_step_bf16"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


@dataclass
class Shape:
    batch: int
    heads_v: int
    heads_qk: int
    d_k: int = 128
    d_v: int = 128
    W: int = 16
    r: int = 4
    n_iter: int = 1
    gate: int = GATE_SCALAR
    smooth: int = 1
    delta: int = 1
    rec16: int = 0
    state_bf16: int = 0

    def c(self) -> _Shape:
        return _Shape(self.batch, self.heads_v, self.heads_qk, self.d_k, self.d_v, self.W, self.r, self.n_iter,
                      self.gate, self.smooth, self.delta, self.rec16, self.state_bf16)


def head_bytes(sh: Shape) -> int:
    s = sh.c()
    return int(lib().lq_head_bytes(C.byref(s)))


def record_floats(sh: Shape) -> int:
    s = sh.c()
    return int(lib().lq_record_floats(C.byref(s)))


class State:
    """Device tensors of the window representation of B x Hv heads, in the layout of ``lq_state``:
    ``heads`` (one contiguous byte block per head), ``records`` (one fp32 row per buffered record),
    ``decays`` (scalar gate) and ``win_pos``.  The named pieces (codes, col_scale, row_smooth, comp_k,
    comp_u, buf_k, buf_u, buf_a) are strided views into those tensors."""

    def __init__(self, sh: Shape, device="cuda", storage=None, work=True):
        """``storage``: optionally the four tensors (heads, records, decays, win_pos) to use instead of fresh
        ones - contiguous, of the shapes and dtypes below (callers that place the state in memory of their own).
        ``work``: give the state the ``work`` words (LQ_WORK_WORDS) with which the decode kernel hands out the heads
        of its last round to the CTAs that get there first; without them every CTA takes the same number."""
        B, H, K, V, W, r = sh.batch, sh.heads_v, sh.d_k, sh.d_v, sh.W, sh.r
        self.shape = sh
        self.work = torch.zeros((8,), dtype=torch.int32, device=device) if work else None
        hb, rf = head_bytes(sh), record_floats(sh)
        assert hb > 0 and rf > 0, "shape not supported by the library"
        rec_dtype = torch.float16 if sh.rec16 else torch.float32
        if storage is None:
            self.heads = torch.zeros((B, H, hb), dtype=torch.uint8, device=device)
            self.records = torch.zeros((B, H, W, rf), dtype=rec_dtype, device=device)
            self.decays = torch.zeros((B, H, W), dtype=torch.float32, device=device)
            self.win_pos = torch.zeros((B,), dtype=torch.int32, device=device)
        else:
            self.heads, self.records, self.decays, self.win_pos = storage
            for t, shape, dt in ((self.heads, (B, H, hb), torch.uint8), (self.records, (B, H, W, rf), rec_dtype),
                                 (self.decays, (B, H, W), torch.float32), (self.win_pos, (B,), torch.int32)):
                assert tuple(t.shape) == shape and t.dtype == dt and t.is_contiguous(), (tuple(t.shape), shape, t.dtype, dt)
        if sh.state_bf16:                    # per-window BF16: the head block is S^T in bfloat16, nothing else
            assert hb == 2 * K * V
            self.state16 = self.heads.view(torch.bfloat16).unflatten(-1, (V, K))
            self.codes = self.col_scale = self.row_smooth = self.comp_k = self.comp_u = None
            self._record_views(sh)
            return
        o = 0
        self.codes = self.heads[..., o:o + K * V].view(torch.int8).unflatten(-1, (V, K)); o += K * V   # Z^T
        self.col_scale = self.heads[..., o:o + 4 * V].view(torch.float32); o += 4 * V
        self.row_smooth = self.heads[..., o:o + 4 * K].view(torch.float32); o += 4 * K
        self.comp_k = self.heads[..., o:o + 2 * r * K].view(torch.float16).unflatten(-1, (r, K)); o += 2 * r * K
        self.comp_u = self.heads[..., o:o + 2 * r * V].view(torch.float16).unflatten(-1, (r, V)); o += 2 * r * V
        assert o == hb
        if storage is None:
            self.row_smooth.fill_(1.0)
        self._record_views(sh)

    def _record_views(self, sh: Shape) -> None:
        K, V = sh.d_k, sh.d_v
        self.buf_k = self.records[..., 0:K]
        self.buf_u = self.records[..., K:K + V]
        self.buf_a = self.records[..., K + V:K + V + K] if sh.gate == GATE_DIAG else self.decays

    def tensors(self):
        return (self.heads, self.records, self.decays, self.win_pos)

    def c(self, b0: int = 0) -> _State:
        """ctypes view; ``b0`` offsets every array to sequence b0 (sub-batches are addressed by pointer)."""
        return _State(*[t.data_ptr() + b0 * t.stride(0) * t.element_size() for t in self.tensors()],
                      self.work.data_ptr() if self.work is not None else None)

    def nbytes_quantized(self) -> int:
        return self.heads.numel()


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise LqError(f"{what}: {lib().lq_status_string(rc).decode()} (status {rc})")


def _ptr(t: Optional[torch.Tensor], b0: int = 0) -> C.c_void_p:
    if t is None:
        return C.c_void_p(None)
    assert t.is_contiguous()
    return C.c_void_p(t.data_ptr() + b0 * t.stride(0) * t.element_size())


def _sub(sh: Shape, b0: int, nb: Optional[int]) -> Shape:
    nb = sh.batch - b0 if nb is None else nb
    return Shape(nb, sh.heads_v, sh.heads_qk, sh.d_k, sh.d_v, sh.W, sh.r, sh.n_iter, sh.gate, sh.smooth, sh.delta, sh.rec16, sh.state_bf16)


def decode_step(sh: Shape, st: State, q, k, v, beta, alpha, o, stream=None, b0: int = 0, nb: Optional[int] = None):
    """lq_decode_step on sequences [b0, b0+nb) of the tensors (all of them by default)."""
    s = _sub(sh, b0, nb).c()
    cs = st.c(b0)
    _check(lib().lq_decode_step(C.byref(s), C.byref(cs), _ptr(q, b0), _ptr(k, b0), _ptr(v, b0), _ptr(beta, b0),
                                _ptr(alpha, b0), _ptr(o, b0), _stream(stream)), "lq_decode_step")


def decode_step_profiled(sh: Shape, st: State, q, k, v, beta, alpha, o, event_between, stream=None):
    """lq_decode_step_profiled: ``event_between`` is a torch.cuda.Event that has been recorded once before
    (so that its CUDA handle exists); it is re-recorded between the two kernels of the step."""
    s = sh.c()
    cs = st.c()
    _check(lib().lq_decode_step_profiled(C.byref(s), C.byref(cs), _ptr(q), _ptr(k), _ptr(v), _ptr(beta),
                                         _ptr(alpha), _ptr(o), _stream(stream), C.c_void_p(event_between.cuda_event)),
           "lq_decode_step_profiled")


def decode_stage_bytes(sh: Shape) -> int:
    s = sh.c()
    return int(lib().lq_decode_stage_bytes(C.byref(s)))


def decode_launches(sh: Shape) -> int:
    s = sh.c()
    return int(lib().lq_decode_launches(C.byref(s)))


def decode_step_host(sh: Shape, st: State, q_h, k_h, v_h, beta_h, alpha_h, o_h, stage, stream=None):
    """lq_decode_step_host: the token's tensors are (pinned) CPU tensors, ``stage`` a device byte buffer."""
    for t in (q_h, k_h, v_h, beta_h, alpha_h, o_h):
        assert t.device.type == "cpu" and t.is_contiguous()
    s = sh.c()
    cs = st.c()
    _check(lib().lq_decode_step_host(C.byref(s), C.byref(cs), _ptr(q_h), _ptr(k_h), _ptr(v_h), _ptr(beta_h),
                                     _ptr(alpha_h), _ptr(o_h), _ptr(stage), _stream(stream)), "lq_decode_step_host")


def decode_step_host_pipelined(sh: Shape, st: State, q_h, k_h, v_h, beta_h, alpha_h, o_h, stage, stream=None):
    """lq_decode_step_host_pipelined: same arguments as decode_step_host; copies and kernels overlap."""
    for t in (q_h, k_h, v_h, beta_h, alpha_h, o_h):
        assert t.device.type == "cpu" and t.is_contiguous()
    s = sh.c()
    cs = st.c()
    _check(lib().lq_decode_step_host_pipelined(C.byref(s), C.byref(cs), _ptr(q_h), _ptr(k_h), _ptr(v_h), _ptr(beta_h),
                                               _ptr(alpha_h), _ptr(o_h), _ptr(stage), _stream(stream)),
           "lq_decode_step_host_pipelined")


STATIC_STAGE_BYTES = 16 << 20


def decode_step_host_static(sh: Shape, st: State, q_h, k_h, v_h, beta_h, alpha_h, o_h, stream=None):
    """lq_decode_step_host_static: like decode_step_host, for callers that cannot allocate the staging
    buffer; the staging is a fixed array inside the library (requests above STATIC_STAGE_BYTES are refused)."""
    for t in (q_h, k_h, v_h, beta_h, alpha_h, o_h):
        assert t.device.type == "cpu" and t.is_contiguous()
    s = sh.c()
    cs = st.c()
    _check(lib().lq_decode_step_host_static(C.byref(s), C.byref(cs), _ptr(q_h), _ptr(k_h), _ptr(v_h), _ptr(beta_h),
                                            _ptr(alpha_h), _ptr(o_h), _stream(stream)), "lq_decode_step_host_static")


def window_flush(sh: Shape, st: State, force: bool = False, stream=None):
    s = sh.c()
    cs = st.c()
    _check(lib().lq_window_flush(C.byref(s), C.byref(cs), C.c_int(1 if force else 0), _stream(stream)),
           "lq_window_flush")


def quantize_state(sh: Shape, S, st: State, stream=None, b0: int = 0, nb: Optional[int] = None):
    s = _sub(sh, b0, nb).c()
    cs = st.c(b0)
    _check(lib().lq_quantize_state(C.byref(s), _ptr(S, b0), C.byref(cs), _stream(stream)), "lq_quantize_state")


def dequantize_state(sh: Shape, st: State, S, stream=None, b0: int = 0, nb: Optional[int] = None):
    """lq_dequantize_state on sequences [b0, b0+nb) of the state; ``S`` receives exactly those sequences."""
    s = _sub(sh, b0, nb).c()
    cs = st.c(b0)
    _check(lib().lq_dequantize_state(C.byref(s), C.byref(cs), _ptr(S), _stream(stream)), "lq_dequantize_state")


def ref_decode_step_f32(sh: Shape, S, q, k, v, beta, alpha, o, stream=None, b0: int = 0, nb: Optional[int] = None):
    s = _sub(sh, b0, nb).c()
    _check(lib().lq_ref_decode_step_f32(C.byref(s), _ptr(S, b0), _ptr(q, b0), _ptr(k, b0), _ptr(v, b0),
                                        _ptr(beta, b0), _ptr(alpha, b0), _ptr(o, b0), _stream(stream)),
           "lq_ref_decode_step_f32")


def ref_decode_step_bf16(sh: Shape, S16, q, k, v, beta, alpha, o, stream=None):
    s = sh.c()
    _check(lib().lq_ref_decode_step_bf16(C.byref(s), _ptr(S16), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(alpha),
                                         _ptr(o), _stream(stream)), "lq_ref_decode_step_bf16")


def check_device() -> int:
    """lq_check_device: synchronises the device and returns the kernels' error flags (0 = none)."""
    flags = C.c_int(0)
    _check(lib().lq_check_device(C.byref(flags)), "lq_check_device")
    return int(flags.value)


class _StateArrays(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos")]


class StateArrays:
    """The window representation as separate device tensors in the paper's orientation (``lq_state_arrays``):
    codes int8 [B,Hv,d_k,d_v], col_scale / row_smooth fp32, comp_k / comp_u fp16, buf_k / buf_u / buf_a fp32,
    win_pos int32 [B]."""

    def __init__(self, sh: Shape, device="cuda"):
        B, H, K, V, W, r = sh.batch, sh.heads_v, sh.d_k, sh.d_v, sh.W, sh.r
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
        self.codes = z((B, H, K, V), torch.int8)
        self.col_scale = z((B, H, V), torch.float32)
        self.row_smooth = z((B, H, K), torch.float32)
        self.comp_k = z((B, H, r, K), torch.float16)
        self.comp_u = z((B, H, r, V), torch.float16)
        self.buf_k = z((B, H, W, K), torch.float32)
        self.buf_u = z((B, H, W, V), torch.float32)
        self.buf_a = z((B, H, W, K) if sh.gate == GATE_DIAG else (B, H, W), torch.float32)
        self.win_pos = z((B,), torch.int32)

    def c(self) -> _StateArrays:
        ptr = lambda t: t.data_ptr() if t.numel() else None
        return _StateArrays(ptr(self.codes), ptr(self.col_scale), ptr(self.row_smooth), ptr(self.comp_k), ptr(self.comp_u),
                            ptr(self.buf_k), ptr(self.buf_u), ptr(self.buf_a), ptr(self.win_pos))


def import_state(sh: Shape, arrays: StateArrays, st: State, stream=None) -> None:
    """lq_import_state: fill the packed state from the separate arrays."""
    s, a, cs = sh.c(), arrays.c(), st.c()
    _check(lib().lq_import_state(C.byref(s), C.byref(a), C.byref(cs), _stream(stream)), "lq_import_state")


def export_state(sh: Shape, st: State, arrays: StateArrays, stream=None) -> None:
    """lq_export_state: write the packed state out as separate arrays."""
    s, a, cs = sh.c(), arrays.c(), st.c()
    _check(lib().lq_export_state(C.byref(s), C.byref(cs), C.byref(a), _stream(stream)), "lq_export_state")


def clear_device_flags() -> None:
    """lq_clear_device_flags: the error flags stay set until this is called."""
    _check(lib().lq_clear_device_flags(), "lq_clear_device_flags")


def selftest_bounded_wait(stream=None) -> None:
    """lq_selftest_bounded_wait: one warp lets a bounded wait run out; sets bit 3 of the error flags."""
    _check(lib().lq_selftest_bounded_wait(_stream(stream)), "lq_selftest_bounded_wait")


def static_stage_bytes() -> int:
    """LQ_STATIC_STAGE_BYTES as the loaded library was built with."""
    return int(lib().lq_static_stage_bytes())


def version() -> int:
    return int(lib().lq_version())
