"""Textbook binary64 statements of the recurrences, used to pin the oracle.

Nothing here comes from the oracle or from the CUDA path: these are the native
GDN / KDA updates as the models define them (Appendix A), dense and in float64.
"""
import numpy as np

from paper_2609_38166_b200 import synth


def widen(tok, wl, b=0, h=0):
    """float64 views of one value head's inputs for a token drawn by synth.token_inputs."""
    g = wl.heads_v // wl.heads_qk
    f = lambda a: synth.bf16_bits_to_f32(a).astype(np.float64)
    q = f(tok["q"])[b, h // g]
    k = f(tok["k"])[b, h // g]
    v = f(tok["v"])[b, h]
    beta = float(f(tok["beta"])[b, h])
    alpha = f(tok["alpha"])[b, h]
    return q, k, v, beta, alpha


def native_step(S, q, k, v, beta, alpha, gate):
    """One token of the model's own update on a dense d_k x d_v state; returns (S_new, o).

    GDN: S <- alpha (I - beta k k^T) S + beta k v^T          (alpha a scalar)
    KDA: S <- (I - beta k k^T) Diag(alpha) S + beta k v^T    (alpha a d_k vector)
    """
    K = S.shape[0]
    P = np.eye(K) - beta * np.outer(k, k)
    if gate == synth.GATE_SCALAR:
        Sn = float(alpha) * (P @ S) + beta * np.outer(k, v)
    else:
        Sn = P @ (alpha[:, None] * S) + beta * np.outer(k, v)
    return Sn, Sn.T @ q


def general_step(S, q, k, v, beta, alpha, gate):
    """Eq. 1 with the coefficients of Table 4: D = Diag(alpha), write key beta*k, read vector alpha (.) k."""
    K = S.shape[0]
    a = np.full(K, float(alpha)) if gate == synth.GATE_SCALAR else alpha
    u = v - S.T @ (a * k)
    Sn = a[:, None] * S + np.outer(beta * k, u)
    return Sn, Sn.T @ q


def dequant_plain(codes, col_scale, row_smooth, comp_k16, comp_u16):
    """C (Z/127) B + Kc Uc^T for one head, in float64 (Appendix B.3, Eq. 6); col_scale holds B/127."""
    Z = codes.astype(np.float64)
    S = row_smooth.astype(np.float64)[:, None] * Z * col_scale.astype(np.float64)[None, :]
    kc = comp_k16.view(np.float16).astype(np.float64)
    uc = comp_u16.view(np.float16).astype(np.float64)
    return S + kc.T @ uc
