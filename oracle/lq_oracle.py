"""numpy front end of the CPU oracle (``lq_oracle.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU
baseline leg use it; the product path never imports it.  It compiles the C file
with gcc on first use (``-O2 -ffp-contract=off -fopenmp``) and passes numpy
arrays through ctypes.  Three builds exist: the defining one (fp32, fixed
summation tree, fixed-point readout), a "wide" one whose sums run left to right
in binary64, and a "plain" one that in addition takes the readout as the plain
definition (no fixed-point grid); the last two measure what is attributable to
fp32 summation order and to the grid.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lq_oracle.c")

GATE_SCALAR = 0  # Gated DeltaNet
GATE_DIAG = 1    # Kimi Delta Attention


def build(force: bool = False) -> None:
    """Compile both oracle builds next to the source (no-op when up to date)."""
    for name, extra in (("liblq_oracle.so", []), ("liblq_oracle_wide.so", ["-DLQO_WIDE"]),
                        ("liblq_oracle_plain.so", ["-DLQO_PLAIN"])):
        out = os.path.join(_HERE, name)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
               *extra, _SRC, "-o", out + ".tmp", "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(out + ".tmp", out)


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("batch", "heads_v", "heads_qk", "d_k", "d_v", "W", "r", "n_iter", "gate", "smooth", "delta", "rec16", "state_bf16")]


class _State(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos", "S0")]


@dataclass
class Shape:
    batch: int
    heads_v: int
    heads_qk: int
    d_k: int
    d_v: int
    W: int
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


class State:
    """Window representation of B x Hv heads, held in numpy arrays.

    ``quant=False`` keeps the boundary state in fp32 (``S0``) and uses no
    compensators: the windowed algebra with the quantizer replaced by the
    identity.  With ``sh.state_bf16`` (per-window BF16) the boundary state
    lives in ``S0`` as well, as bfloat16 values held in fp32.
    """

    def __init__(self, sh: Shape, quant: bool = True):
        B, H, K, V, W, r = sh.batch, sh.heads_v, sh.d_k, sh.d_v, sh.W, sh.r
        quant = quant and not sh.state_bf16
        self.shape = sh
        self.quant = quant
        self.codes = np.zeros((B, H, K, V), np.int8)
        self.col_scale = np.zeros((B, H, V), np.float32)
        self.row_smooth = np.ones((B, H, K), np.float32)
        self.comp_k = np.zeros((B, H, r, K), np.uint16)
        self.comp_u = np.zeros((B, H, r, V), np.uint16)
        self.buf_k = np.zeros((B, H, W, K), np.float32)
        self.buf_u = np.zeros((B, H, W, V), np.float32)
        self.buf_a = np.zeros((B, H, W, K) if sh.gate == GATE_DIAG else (B, H, W), np.float32)
        self.win_pos = np.zeros((B,), np.int32)
        self.S0 = None if quant else np.zeros((B, H, K, V), np.float32)

    def c(self) -> _State:
        p = lambda a: None if a is None else a.ctypes.data
        if self.quant:
            return _State(p(self.codes), p(self.col_scale), p(self.row_smooth), p(self.comp_k), p(self.comp_u),
                          p(self.buf_k), p(self.buf_u), p(self.buf_a), p(self.win_pos), None)
        return _State(None, None, None, None, None, p(self.buf_k), p(self.buf_u), p(self.buf_a), p(self.win_pos),
                      p(self.S0))

    def comp_k_f32(self) -> np.ndarray:
        return self.comp_k.view(np.float16).astype(np.float32)

    def comp_u_f32(self) -> np.ndarray:
        return self.comp_u.view(np.float16).astype(np.float32)


def _chk(a: np.ndarray, dtype, shape=None) -> np.ndarray:
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


class Oracle:
    def __init__(self, wide: bool = False, plain: bool = False):
        build()
        name = "liblq_oracle_plain.so" if plain else "liblq_oracle_wide.so" if wide else "liblq_oracle.so"
        self.lib = C.CDLL(os.path.join(_HERE, name))
        L = self.lib
        L.lqo_csum_dot.restype = C.c_float
        L.lqo_csum_dot.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.lqo_csum_abs.restype = C.c_float
        L.lqo_csum_abs.argtypes = [C.c_void_p, C.c_int]
        L.lqo_f32_to_f16.restype = C.c_uint16
        L.lqo_f32_to_f16.argtypes = [C.c_float]
        L.lqo_f16_to_f32.restype = C.c_float
        L.lqo_f16_to_f32.argtypes = [C.c_uint16]
        L.lqo_f32_to_bf16.restype = C.c_uint16
        L.lqo_f32_to_bf16.argtypes = [C.c_float]
        L.lqo_threads.restype = C.c_int
        for f in ("lqo_ref_step_f32", "lqo_ref_step_bf16", "lqo_quantize_state", "lqo_dequantize_state",
                  "lqo_window_flush", "lqo_decode_step"):
            getattr(L, f).restype = C.c_int

    # --- scalar helpers (exposed so that the tests can pin them) ---
    def csum_dot(self, a, b) -> float:
        a = np.ascontiguousarray(a, np.float32); b = np.ascontiguousarray(b, np.float32)
        return float(self.lib.lqo_csum_dot(a.ctypes.data, b.ctypes.data, a.size))

    def csum_abs(self, x) -> float:
        x = np.ascontiguousarray(x, np.float32)
        return float(self.lib.lqo_csum_abs(x.ctypes.data, x.size))

    def f32_to_f16(self, x: float) -> int:
        return int(self.lib.lqo_f32_to_f16(C.c_float(x)))

    def f16_to_f32(self, h: int) -> float:
        return float(self.lib.lqo_f16_to_f32(C.c_uint16(h)))

    def f32_to_bf16(self, x: float) -> int:
        return int(self.lib.lqo_f32_to_bf16(C.c_float(x)))

    def threads(self) -> int:
        return int(self.lib.lqo_threads())

    # --- the operations ---
    def _tok(self, sh: Shape, q, k, v, beta, alpha):
        B, H, G, K, V = sh.batch, sh.heads_v, sh.heads_qk, sh.d_k, sh.d_v
        _chk(q, np.uint16, (B, G, K)); _chk(k, np.uint16, (B, G, K)); _chk(v, np.uint16, (B, H, V))
        _chk(beta, np.uint16, (B, H))
        _chk(alpha, np.uint16, (B, H, K) if sh.gate == GATE_DIAG else (B, H))
        return [C.c_void_p(x.ctypes.data) for x in (q, k, v, beta, alpha)]

    def ref_step_f32(self, sh: Shape, S, q, k, v, beta, alpha) -> np.ndarray:
        """Eq. 1 on a dense fp32 state ``S`` [B,Hv,d_k,d_v] (updated in place); returns o [B,Hv,d_v]."""
        _chk(S, np.float32, (sh.batch, sh.heads_v, sh.d_k, sh.d_v))
        o = np.zeros((sh.batch, sh.heads_v, sh.d_v), np.float32)
        rc = self.lib.lqo_ref_step_f32(C.byref(sh.c()), C.c_void_p(S.ctypes.data), *self._tok(sh, q, k, v, beta, alpha),
                                       C.c_void_p(o.ctypes.data))
        assert rc == 0, rc
        return o

    def ref_step_bf16(self, sh: Shape, S16, q, k, v, beta, alpha) -> np.ndarray:
        _chk(S16, np.uint16, (sh.batch, sh.heads_v, sh.d_k, sh.d_v))
        o = np.zeros((sh.batch, sh.heads_v, sh.d_v), np.float32)
        rc = self.lib.lqo_ref_step_bf16(C.byref(sh.c()), C.c_void_p(S16.ctypes.data),
                                        *self._tok(sh, q, k, v, beta, alpha), C.c_void_p(o.ctypes.data))
        assert rc == 0, rc
        return o

    def quantize_state(self, sh: Shape, S, st: State) -> None:
        _chk(S, np.float32, (sh.batch, sh.heads_v, sh.d_k, sh.d_v))
        cs = st.c()
        rc = self.lib.lqo_quantize_state(C.byref(sh.c()), C.c_void_p(S.ctypes.data), C.byref(cs))
        assert rc == 0, rc

    def dequantize_state(self, sh: Shape, st: State) -> np.ndarray:
        S = np.zeros((sh.batch, sh.heads_v, sh.d_k, sh.d_v), np.float32)
        cs = st.c()
        rc = self.lib.lqo_dequantize_state(C.byref(sh.c()), C.byref(cs), C.c_void_p(S.ctypes.data))
        assert rc == 0, rc
        return S

    def window_flush(self, sh: Shape, st: State, force: bool = False) -> None:
        cs = st.c()
        rc = self.lib.lqo_window_flush(C.byref(sh.c()), C.byref(cs), C.c_int(1 if force else 0))
        assert rc == 0, rc

    def decode_step(self, sh: Shape, st: State, q, k, v, beta, alpha) -> np.ndarray:
        o = np.zeros((sh.batch, sh.heads_v, sh.d_v), np.float32)
        cs = st.c()
        rc = self.lib.lqo_decode_step(C.byref(sh.c()), C.byref(cs), *self._tok(sh, q, k, v, beta, alpha),
                                      C.c_void_p(o.ctypes.data))
        assert rc == 0, rc
        return o
