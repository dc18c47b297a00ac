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

EXPORTS = ["lq_decode_step", "lq_decode_step_host", "lq_decode_stage_bytes", "lq_window_flush",
           "lq_quantize_state", "lq_dequantize_state", "lq_ref_decode_step_f32", "lq_ref_decode_step_bf16",
           "lq_decode_launches", "lq_check_device", "lq_status_string", "lq_version"]


class LqError(RuntimeError):
    pass


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("batch", "heads_v", "heads_qk", "d_k", "d_v", "W", "r", "n_iter", "gate", "smooth")]


class _State(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos")]


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
        L.lq_decode_launches.restype = C.c_int
        L.lq_decode_launches.argtypes = [C.c_void_p]
        for name in ("lq_decode_step", "lq_decode_step_host", "lq_check_device", "lq_window_flush", "lq_quantize_state",
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
    n_iter: int = 4
    gate: int = GATE_SCALAR
    smooth: int = 1

    def c(self) -> _Shape:
        return _Shape(self.batch, self.heads_v, self.heads_qk, self.d_k, self.d_v, self.W, self.r, self.n_iter,
                      self.gate, self.smooth)


class State:
    """Device tensors of the window representation of B x Hv heads (layouts as in ``lq_state``)."""

    def __init__(self, sh: Shape, device="cuda"):
        B, H, K, V, W, r = sh.batch, sh.heads_v, sh.d_k, sh.d_v, sh.W, sh.r
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
        self.shape = sh
        self.codes = z((B, H, K, V), torch.int8)
        self.col_scale = z((B, H, V), torch.float32)
        self.row_smooth = torch.ones((B, H, K), dtype=torch.float32, device=device)
        self.comp_k = z((B, H, max(r, 1), K), torch.float16)
        self.comp_u = z((B, H, max(r, 1), V), torch.float16)
        self.buf_k = z((B, H, W, K), torch.float32)
        self.buf_u = z((B, H, W, V), torch.float32)
        self.buf_a = z((B, H, W, K) if sh.gate == GATE_DIAG else (B, H, W), torch.float32)
        self.win_pos = z((B,), torch.int32)

    def tensors(self):
        return (self.codes, self.col_scale, self.row_smooth, self.comp_k, self.comp_u, self.buf_k, self.buf_u,
                self.buf_a, self.win_pos)

    def c(self, b0: int = 0) -> _State:
        """ctypes view; ``b0`` offsets every array to sequence b0 (sub-batches are addressed by pointer)."""
        return _State(*[t.data_ptr() + b0 * (t.stride(0) * t.element_size() if t.dim() > 0 else 0)
                        for t in self.tensors()])

    def nbytes_quantized(self) -> int:
        r = self.shape.r
        per_head = (self.shape.d_k * self.shape.d_v + 4 * self.shape.d_v + 4 * self.shape.d_k
                    + 2 * r * (self.shape.d_k + self.shape.d_v))
        return per_head * self.shape.batch * self.shape.heads_v


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
    return Shape(nb, sh.heads_v, sh.heads_qk, sh.d_k, sh.d_v, sh.W, sh.r, sh.n_iter, sh.gate, sh.smooth)


def decode_step(sh: Shape, st: State, q, k, v, beta, alpha, o, stream=None, b0: int = 0, nb: Optional[int] = None):
    """lq_decode_step on sequences [b0, b0+nb) of the tensors (all of them by default)."""
    s = _sub(sh, b0, nb).c()
    cs = st.c(b0)
    _check(lib().lq_decode_step(C.byref(s), C.byref(cs), _ptr(q, b0), _ptr(k, b0), _ptr(v, b0), _ptr(beta, b0),
                                _ptr(alpha, b0), _ptr(o, b0), _stream(stream)), "lq_decode_step")


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


def window_flush(sh: Shape, st: State, force: bool = False, stream=None):
    s = sh.c()
    cs = st.c()
    _check(lib().lq_window_flush(C.byref(s), C.byref(cs), C.c_int(1 if force else 0), _stream(stream)),
           "lq_window_flush")


def quantize_state(sh: Shape, S, st: State, stream=None, b0: int = 0, nb: Optional[int] = None):
    s = _sub(sh, b0, nb).c()
    cs = st.c(b0)
    _check(lib().lq_quantize_state(C.byref(s), _ptr(S, b0), C.byref(cs), _stream(stream)), "lq_quantize_state")


def dequantize_state(sh: Shape, st: State, S, stream=None):
    s = sh.c()
    cs = st.c()
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


def version() -> int:
    return int(lib().lq_version())
