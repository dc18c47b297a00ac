"""Seeded synthetic decode inputs for GDN / KDA heads.

This module holds no arithmetic of the method: it only draws the per-token
inputs (q, k, v, beta, alpha) that a linear-attention layer would hand to the
decode step, rounds them to bf16, and returns them as numpy arrays of bf16 bit
patterns.  The CPU oracle and the CUDA library are both fed from here, so the
two see the same bits.

Every tensor is drawn from a Philox stream keyed by (seed, step, tensor), so a
given token's inputs do not depend on which other tokens were generated.

Distributions (the kernel benchmark of the paper is itself shape-only: one
layer, 32 heads, d_k = d_v = 128):
  q, k  ~ N(0,1), L2-normalised over d_k per q/k head
  v     ~ N(0,1), or Student-t(3) for the heavy-tailed drift workload
  beta  = sigmoid(N(0,1))                          one per value head
  alpha = exp(-softplus(N(0,1)))                   one per value head (scalar
          gate) or one per key channel of each value head (diagonal gate)
Outlier workload: per head a fixed seeded set of ceil(frac*d) key channels and
value channels is scaled by ``outlier_mag`` (keys before the normalisation, so
that the key keeps unit length), which grows persistent outlier rows and
columns in the state.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

GATE_SCALAR = 0
GATE_DIAG = 1

_TENSOR_ID = {"q": 1, "k": 2, "v": 3, "beta": 4, "alpha": 5, "out_k": 6, "out_v": 7, "dense": 8}


@dataclass(frozen=True)
class Workload:
    name: str
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
    delta: int = 1                  # 1: delta rule (GDN, KDA); 0: no read-back, u = v (Mamba2, GLA, ...)
    rec16: int = 0                  # 1: fp16 record buffer (the paper's storage), 0: fp32
    state_bf16: int = 0             # 1: per-window BF16 boundary state (the -w baseline; r = 0), 0: the 8-bit method
    v_dist: str = "normal"          # "normal" | "student3"
    outlier_frac: float = 0.0
    outlier_mag: float = 1.0
    seed: int = 0

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _rng(seed: int, step: int, tensor: str) -> np.random.Generator:
    key = (np.uint64(seed) << np.uint64(32)) ^ np.uint64(step & 0xFFFFFFFF)
    return np.random.Generator(np.random.Philox(key=[int(key), _TENSOR_ID[tensor]]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 values to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return u.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _outlier_sets(wl: Workload):
    """Fixed per-head channel sets that carry the outliers (empty when the workload has none)."""
    if wl.outlier_frac <= 0.0:
        return None, None
    nk = int(np.ceil(wl.outlier_frac * wl.d_k))
    nv = int(np.ceil(wl.outlier_frac * wl.d_v))
    gk = _rng(wl.seed, 0, "out_k")
    gv = _rng(wl.seed, 0, "out_v")
    mk = np.ones((wl.batch, wl.heads_qk, wl.d_k), np.float64)
    mv = np.ones((wl.batch, wl.heads_v, wl.d_v), np.float64)
    for b in range(wl.batch):
        for h in range(wl.heads_qk):
            mk[b, h, gk.choice(wl.d_k, nk, replace=False)] = wl.outlier_mag
        for h in range(wl.heads_v):
            mv[b, h, gv.choice(wl.d_v, nv, replace=False)] = wl.outlier_mag
    return mk, mv


_OUTLIER_CACHE: dict = {}


def token_inputs(wl: Workload, step: int) -> dict:
    """Inputs of decode token ``step`` for the whole batch, as bf16 bit patterns (uint16).

    q, k: [B, Hqk, d_k]; v: [B, Hv, d_v]; beta: [B, Hv]; alpha: [B, Hv] or [B, Hv, d_k].
    """
    B, H, G, K, V = wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v
    q = _rng(wl.seed, step, "q").standard_normal((B, G, K))
    k = _rng(wl.seed, step, "k").standard_normal((B, G, K))
    gv = _rng(wl.seed, step, "v")
    v = gv.standard_t(3.0, (B, H, V)) if wl.v_dist == "student3" else gv.standard_normal((B, H, V))
    if wl.outlier_frac > 0.0:
        if wl not in _OUTLIER_CACHE:
            _OUTLIER_CACHE[wl] = _outlier_sets(wl)
        mk, mv = _OUTLIER_CACHE[wl]
        k = k * mk
        v = v * mv
    q = q / np.linalg.norm(q, axis=-1, keepdims=True)
    k = k / np.linalg.norm(k, axis=-1, keepdims=True)
    beta = 1.0 / (1.0 + np.exp(-_rng(wl.seed, step, "beta").standard_normal((B, H))))
    ashape = (B, H, K) if wl.gate == GATE_DIAG else (B, H)
    alpha = np.exp(-np.logaddexp(0.0, _rng(wl.seed, step, "alpha").standard_normal(ashape)))
    cast = lambda x: f32_to_bf16_bits(x.astype(np.float32))
    return {"q": cast(q), "k": cast(k), "v": cast(v), "beta": cast(beta), "alpha": cast(alpha)}


def dense_states(wl: Workload, tag: int = 0, rank: int = 6, noise: float = 0.05) -> np.ndarray:
    """Random dense fp32 states [B, Hv, d_k, d_v] with a few dominant singular directions plus noise,
    and, for an outlier workload, a few rows and columns scaled up.  Used as inputs of the quantizer."""
    B, H, K, V = wl.batch, wl.heads_v, wl.d_k, wl.d_v
    g = _rng(wl.seed, tag, "dense")
    rank = min(rank, K, V)
    L = g.standard_normal((B, H, K, rank)) / np.sqrt(K)
    R = g.standard_normal((B, H, rank, V))
    sv = 2.0 ** (-np.arange(rank, dtype=np.float64))
    S = np.einsum("bhkr,r,bhrv->bhkv", L, sv, R) + noise * g.standard_normal((B, H, K, V)) / np.sqrt(K)
    if wl.outlier_frac > 0.0:
        nk = int(np.ceil(wl.outlier_frac * K)); nv = int(np.ceil(wl.outlier_frac * V))
        for b in range(B):
            for h in range(H):
                S[b, h, g.choice(K, nk, replace=False), :] *= wl.outlier_mag
                S[b, h, :, g.choice(V, nv, replace=False)] *= wl.outlier_mag
    return np.ascontiguousarray(S, np.float32)


# ---------------------------------------------------------------------------
# The benchmark configurations, by name.
# ---------------------------------------------------------------------------

def config(name: str) -> Workload:
    if name == "single_gdn":        # one head, 64 tokens, W = 16, zero initial state
        return Workload(name, 1, 1, 1, 128, 128, 16, 4, gate=GATE_SCALAR, seed=0)
    if name == "gdn_b256":          # headline: 256 x 32 value heads (16 q/k heads), W in {8,16,32}
        return Workload(name, 256, 32, 16, 128, 128, 16, 4, gate=GATE_SCALAR, seed=2)
    if name == "kda_b128_outlier":  # KDA, outliers of 8x on 2 % of the channels
        return Workload(name, 128, 32, 32, 128, 128, 16, 4, gate=GATE_DIAG, outlier_frac=0.02, outlier_mag=8.0,
                        seed=3)
    if name == "gdn_drift":         # long chain, heavy-tailed values
        return Workload(name, 64, 16, 16, 128, 128, 16, 4, gate=GATE_SCALAR, v_dist="student3", seed=4)
    raise KeyError(name)
