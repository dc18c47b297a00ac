"""Pins for the window-boundary quantizer of the oracle: the 8-bit code, the smoothing scales and the
Compensator-Token fit, against brute force, closed forms, numpy's SVD (Eckart-Young) and the paper's
stated format size."""
import os

import numpy as np
import pytest

from oracle.lq_oracle import Shape, State
from paper_2609_38166_b200 import synth
from tests import refmath as rm


def _quant(oracle, S, r=4, n_iter=4, smooth=1, gate=synth.GATE_SCALAR, W=4):
    B, H, K, V = S.shape
    sh = Shape(B, H, H, K, V, W, r, n_iter, gate, smooth)
    st = State(sh)
    oracle.quantize_state(sh, S, st)
    return sh, st


def test_plain_code_is_the_nearest_of_255_levels(oracle):
    # no compensators, no smoothing: per-value-channel symmetric INT8 with dequant = (Z/127) B (Appendix B.3)
    rng = np.random.default_rng(0)
    S = (rng.standard_normal((1, 3, 24, 40)) * rng.uniform(0.1, 5, (1, 3, 1, 40))).astype(np.float32)
    sh, st = _quant(oracle, S, r=0, smooth=0)
    assert np.array_equal(st.row_smooth, np.ones_like(st.row_smooth))
    S64 = S.astype(np.float64)
    assert np.array_equal(st.col_scale, np.abs(S).max(axis=2) / np.float32(127.0))   # step = column absmax / 127
    levels = np.arange(-127, 128, dtype=np.float64)
    for h in range(3):
        grid = levels[None, None, :] * st.col_scale[0, h].astype(np.float64)[None, :, None]
        best = levels[np.argmin(np.abs(S64[0, h][:, :, None] - grid), axis=2)]
        assert np.array_equal(st.codes[0, h].astype(np.float64), best)
        err = np.abs(rm.dequant_plain(st.codes[0, h], st.col_scale[0, h], st.row_smooth[0, h],
                                      st.comp_k[0, h], st.comp_u[0, h]) - S64[0, h])
        assert np.all(err <= st.col_scale[0, h][None, :] / 2.0 * (1 + 1e-6))
    # the column's largest entry maps to +-127 and the code range is symmetric
    assert np.all(np.abs(st.codes).max(axis=2) == 127) and st.codes.min() >= -127
    # dequantize is the same formula
    assert np.allclose(oracle.dequantize_state(sh, st)[0, 0],
                       rm.dequant_plain(st.codes[0, 0], st.col_scale[0, 0], st.row_smooth[0, 0],
                                        st.comp_k[0, 0], st.comp_u[0, 0]), rtol=1e-6, atol=0)


def test_plain_code_is_idempotent_and_handles_zero_columns(oracle):
    rng = np.random.default_rng(1)
    S = rng.standard_normal((1, 1, 16, 16)).astype(np.float32)
    S[0, 0, :, 3] = 0.0
    sh, st = _quant(oracle, S, r=0, smooth=0)
    assert st.col_scale[0, 0, 3] == 0.0 and np.all(st.codes[0, 0, :, 3] == 0)
    S1 = oracle.dequantize_state(sh, st)
    st2 = State(sh)
    oracle.quantize_state(sh, S1, st2)
    assert np.array_equal(st2.codes, st.codes)
    assert np.allclose(st2.col_scale, st.col_scale, rtol=1e-6)
    # the all-zero state (the initial state of a fresh sequence) quantizes to zeros with a positive floor on c
    sh, st = _quant(oracle, np.zeros((1, 1, 16, 16), np.float32), r=2, smooth=1)
    assert not st.codes.any() and not st.comp_k.any() and not st.comp_u.any() and not st.col_scale.any()
    assert np.all(st.row_smooth > 0)
    assert not oracle.dequantize_state(sh, st).any()


def test_smoothing_scale_is_sqrt_of_row_mean_abs_and_is_invertible(oracle):
    # Sec. 3.4: c_i = sqrt(mean_j |R_ij|); quantize C^-1 R; multiplying back by C restores the coordinates
    rng = np.random.default_rng(2)
    S = (rng.standard_normal((1, 2, 32, 48)) * rng.uniform(0.01, 30, (1, 2, 32, 1))).astype(np.float32)
    sh, st = _quant(oracle, S, r=0, smooth=1)
    want_c = np.sqrt(np.abs(S.astype(np.float64)).mean(axis=3))
    assert np.allclose(st.row_smooth, want_c, rtol=1e-6)
    X = S.astype(np.float64) / want_c[..., None]
    # after smoothing every row's mean magnitude is the square root of what it was
    assert np.allclose(np.abs(X).mean(axis=3), want_c, rtol=1e-12)
    # the value-channel scale is taken on the smoothed residual
    assert np.allclose(st.col_scale, np.abs(X).max(axis=2) / 127.0, rtol=1e-6)
    # elementwise error bound of the whole chain: half a code step in the original coordinates
    D = oracle.dequantize_state(sh, st).astype(np.float64)
    bound = st.row_smooth[..., None].astype(np.float64) * st.col_scale[:, :, None, :] / 2.0
    assert np.all(np.abs(D - S) <= bound * (1 + 1e-5) + 1e-12)
    # smoothing must help on rows of very different magnitude: compare with the unsmoothed code
    sh0, st0 = _quant(oracle, S, r=0, smooth=0)
    e1 = np.linalg.norm(D - S)
    e0 = np.linalg.norm(oracle.dequantize_state(sh0, st0).astype(np.float64) - S)
    assert e1 < e0
    # a row of zeros hits the floor instead of dividing by zero
    S[0, 0, 5, :] = 0
    sh, st = _quant(oracle, S, r=0, smooth=1)
    assert st.row_smooth[0, 0, 5] == np.float32(1e-6) and np.all(st.codes[0, 0, 5] == 0)


def _gapped(rng, K, V, sv):
    U, _ = np.linalg.qr(rng.standard_normal((K, K)))
    Vt, _ = np.linalg.qr(rng.standard_normal((V, V)))
    n = min(K, V)
    s = np.zeros(n); s[:len(sv)] = sv
    s[len(sv):] = 0.01 * rng.uniform(0.5, 1.0, n - len(sv))
    return (U[:, :n] * s) @ Vt[:, :n].T


@pytest.mark.parametrize("r", [1, 2, 4])
def test_compensators_are_the_best_rank_r_fit(oracle, r):
    """Eq. 5 / Eq. 6 define the compensators as the Frobenius minimiser, whose value Eckart-Young gives from
    the singular values.  With enough power-iteration steps the oracle's fit must reach it up to the fp16
    storage of the factors."""
    rng = np.random.default_rng(3)
    K, V = 48, 64
    M = _gapped(rng, K, V, [8.0, 4.0, 2.0, 1.0, 0.5])
    S = M[None, None].astype(np.float32)
    sh, st = _quant(oracle, S, r=r, n_iter=60, smooth=0)
    kc = st.comp_k_f32()[0, 0].astype(np.float64)
    uc = st.comp_u_f32()[0, 0].astype(np.float64)
    resid = M - kc.T @ uc
    sv = np.linalg.svd(M, compute_uv=False)
    best = np.sqrt((sv[r:] ** 2).sum())
    fp16_slack = 2.0 ** -11 * np.sqrt((sv[:r] ** 2).sum()) * 2
    assert np.linalg.norm(resid) <= best + fp16_slack
    assert np.linalg.norm(resid) >= best * (1 - 1e-6)      # nothing beats the optimum
    # each compensator key is a unit left singular vector, the value side carries the singular value
    Usvd, s, Vt = np.linalg.svd(M)
    for h in range(r):
        assert abs(abs(kc[h] @ Usvd[:, h]) - 1) < 2e-3
        assert abs(np.linalg.norm(uc[h]) - s[h]) < 2e-3 * s[h]
    # Eq. 6: dequant(R_hat) + K U^T differs from S only by the quantization of the residual
    # (plus the fp32 roundings of the r + 1 terms that the residual and its reconstruction go through)
    D = oracle.dequantize_state(sh, st)[0, 0].astype(np.float64)
    fp32_slack = (r + 2) * 2.0 ** -24 * np.abs(M).max()
    assert np.all(np.abs(D - M) <= st.col_scale[0, 0][None, :] / 2.0 * (1 + 1e-5) + fp32_slack)
    assert np.allclose(st.col_scale[0, 0], np.abs(resid).max(axis=0) / 127.0, rtol=1e-5)


def test_default_iteration_count_already_captures_the_energy(oracle):
    # few steps from the data-independent start vectors: residual norm must fall with every added compensator
    # and be close to the optimum on a state with the fast-decaying spectrum decode states have
    wl = synth.Workload("t", 1, 4, 4, 128, 128, seed=21)
    S = synth.dense_states(wl, 3)
    norms = []
    for r in range(0, 6):
        sh, st = _quant(oracle, S, r=r, n_iter=4, smooth=0)
        kc = st.comp_k_f32().astype(np.float64); uc = st.comp_u_f32().astype(np.float64)
        R = S.astype(np.float64) - np.einsum("bhrk,bhrv->bhkv", kc, uc)
        norms.append(np.linalg.norm(R, axis=(2, 3)))
    norms = np.array(norms)
    assert np.all(np.diff(norms, axis=0) < 0)
    sv = np.linalg.svd(S.astype(np.float64), compute_uv=False)
    best4 = np.sqrt((sv[..., 4:] ** 2).sum(-1))
    assert np.all(norms[4] <= 1.25 * best4)


def test_planted_rank_one_outlier_is_removed_exactly(oracle):
    # a state that is one fp16-representable row: the compensator reproduces it and the residual is zero
    K, V = 32, 32
    S = np.zeros((1, 1, K, V), np.float32)
    row = (np.arange(V) - 11.0) / 4.0
    S[0, 0, 7, :] = row
    sh, st = _quant(oracle, S, r=1, n_iter=2, smooth=1)
    assert not st.codes.any() and not st.col_scale.any()
    assert np.array_equal(oracle.dequantize_state(sh, st), S)
    kc = st.comp_k_f32()[0, 0, 0]
    assert abs(kc[7]) == 1.0 and np.count_nonzero(kc) == 1
    # rank-one outlier spanning a row AND a column pattern: x y^T with fp16-exact factors of unit-norm x
    x = np.zeros(K); x[[3, 9, 20, 31]] = 0.5
    y = (np.arange(V) % 7 - 3.0) * 0.25
    S2 = np.outer(x, y)[None, None].astype(np.float32)
    sh, st = _quant(oracle, S2, r=1, n_iter=3, smooth=1)
    assert np.abs(oracle.dequantize_state(sh, st) - S2).max() <= 1e-6 and np.abs(st.codes).max() <= 127
    assert st.col_scale.max() < 1e-3          # what is left to quantize is rounding dust


def test_outlier_rows_and_columns_are_absorbed(oracle):
    # the paper's motivation (Sec. 3.3-3.4): compensators + smoothing reduce the error of one quantization
    wl = synth.Workload("t", 2, 4, 4, 128, 128, outlier_frac=0.02, outlier_mag=8.0, seed=22)
    S = synth.dense_states(wl, 4)
    errs = {}
    for name, (r, smooth) in {"int8": (0, 0), "comp": (4, 0), "full": (4, 1)}.items():
        sh, st = _quant(oracle, S, r=r, smooth=smooth)
        errs[name] = np.linalg.norm(oracle.dequantize_state(sh, st).astype(np.float64) - S) / np.linalg.norm(S)
    assert errs["full"] < errs["comp"] < errs["int8"]


def test_format_size_matches_the_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "format_sizes.txt")
    gold = {}
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 2:
            gold[line[0]] = float(line[1])
    sh = Shape(1, 1, 1, 128, 128, 16, 4)
    st = State(sh)
    nbytes = st.codes.nbytes + st.col_scale.nbytes + st.row_smooth.nbytes + st.comp_k.nbytes + st.comp_u.nbytes
    assert round(nbytes / (128 * 128), 2) == gold["bytes_per_element_128x128_r4"]
    assert round(4.0 / (nbytes / (128 * 128)), 1) == gold["traffic_reduction_vs_fp32"]
    # this build buffers records in fp32; the paper's fp16 figure is half of ours
    rec = st.buf_k.nbytes + st.buf_u.nbytes + st.buf_a.nbytes
    assert rec // 2 == gold["fp16_buffer_bytes_p16_gdn"]


@pytest.mark.parametrize("gate", [synth.GATE_SCALAR, synth.GATE_DIAG])
def test_flush_fit_from_record_start_vectors_reaches_the_optimum(oracle, gate):
    """At a window boundary column h of the power iteration starts from the (h+1)-th newest record's u
    instead of a data-independent vector.  Whatever the start, with enough steps the fit of Eqs. 5-6 must end at
    the Eckart-Young optimum of the state that the window representation holds (Eq. 7), here computed by a
    library SVD of the dequantized pre-flush state."""
    rng = np.random.default_rng(17)
    B, H, K, V, W, r = 1, 2, 128, 128, 6, 3
    sh = Shape(B, H, H, K, V, W, r, 80, gate, 0)
    st = State(sh)
    oracle.quantize_state(sh, np.zeros((B, H, K, V), np.float32), st)
    # six records with well separated weights: the state is their decayed sum, rank 6 with a gapped spectrum
    wts = np.array([0.6, 4.0, 0.3, 9.0, 1.5, 0.1])[None, None, :, None]
    qk, _ = np.linalg.qr(rng.standard_normal((H, K, W)))
    qu, _ = np.linalg.qr(rng.standard_normal((H, V, W)))
    st.buf_k[...] = (qk.transpose(0, 2, 1)[None] * wts).astype(np.float32)
    st.buf_u[...] = qu.transpose(0, 2, 1)[None].astype(np.float32)
    st.buf_a[...] = rng.uniform(0.8, 1.0, st.buf_a.shape).astype(np.float32)
    st.win_pos[...] = W
    Sp = oracle.dequantize_state(sh, st).astype(np.float64)
    oracle.window_flush(sh, st)
    assert st.win_pos[0] == 0
    for h in range(H):
        kc = st.comp_k_f32()[0, h].astype(np.float64)
        uc = st.comp_u_f32()[0, h].astype(np.float64)
        sv = np.linalg.svd(Sp[0, h], compute_uv=False)
        best = np.sqrt((sv[r:] ** 2).sum())
        resid = np.linalg.norm(Sp[0, h] - kc.T @ uc)
        assert resid <= best * (1 + 2e-3) + 2.0 ** -10 * np.sqrt((sv[:r] ** 2).sum())
        assert resid >= best * (1 - 1e-6)


def test_record_start_vector_is_what_the_first_step_multiplies(oracle):
    """One power-iteration step from start vector w gives k = S w / |S w|.  With a single record whose u is
    orthogonal to everything else in the state, S u_newest is along that record's key: the first compensator
    key after one step must be that (decayed) key direction, which a data-independent start would not give."""
    rng = np.random.default_rng(5)
    B, H, K, V, W = 1, 1, 128, 128, 4
    sh = Shape(B, H, H, K, V, W, 1, 1, synth.GATE_SCALAR, 0)
    st = State(sh)
    oracle.quantize_state(sh, np.zeros((B, H, K, V), np.float32), st)
    q, _ = np.linalg.qr(rng.standard_normal((V, W)))
    keys = rng.standard_normal((W, K)); keys /= np.linalg.norm(keys, axis=1, keepdims=True)
    st.buf_k[0, 0] = keys.astype(np.float32)
    st.buf_u[0, 0] = (q.T * np.array([5.0, 3.0, 2.0, 0.05])[:, None]).astype(np.float32)   # newest one is small
    st.buf_a[...] = 1.0
    st.win_pos[...] = W
    oracle.window_flush(sh, st)
    k1 = st.comp_k_f32()[0, 0, 0].astype(np.float64)
    # S u_3 = sum_j k_j (u_j . u_3) = k_3 |u_3|^2 : the newest record's key, although it is the weakest one
    assert abs(abs(k1 @ keys[3]) - 1.0) < 2e-3
    assert abs(k1 @ keys[0]) < 0.5


@pytest.mark.parametrize("r", [2, 3, 5])
def test_fitted_keys_are_orthonormal_for_any_count(oracle, r):
    """The keys come out of an orthonormalisation.  The stored keys must then be unit vectors, mutually
    orthogonal up to the fp16 rounding of their entries, and R + K U^T must give back the state (Eq. 6) with a
    residual norm smaller than after r - 1 tokens."""
    rng = np.random.default_rng(40 + r)
    M = _gapped(rng, 128, 128, [9.0, 5.0, 3.0, 2.0, 1.2, 0.7])
    S = M[None, None].astype(np.float32)
    sh, st = _quant(oracle, S, r=r, n_iter=3, smooth=0)
    kc = st.comp_k_f32()[0, 0].astype(np.float64)
    uc = st.comp_u_f32()[0, 0].astype(np.float64)
    G = kc @ kc.T
    assert np.allclose(np.diag(G), 1.0, atol=2e-3)
    assert np.max(np.abs(G - np.diag(np.diag(G)))) < 5e-3
    resid = M - kc.T @ uc
    sh2, st2 = _quant(oracle, S, r=r - 1, n_iter=3, smooth=0)
    resid_fewer = M - st2.comp_k_f32()[0, 0].astype(np.float64).T @ st2.comp_u_f32()[0, 0].astype(np.float64)
    assert np.linalg.norm(resid) < np.linalg.norm(resid_fewer)
    # the residual is what the codes hold: dequantized state = Z*step + K U^T, within half a code step of M
    D = oracle.dequantize_state(sh, st)[0, 0].astype(np.float64)
    fp32_slack = (r + 2) * 2.0 ** -24 * np.abs(M).max()
    assert np.all(np.abs(D - M) <= st.col_scale[0, 0][None, :] / 2.0 * (1 + 1e-5) + fp32_slack)


def test_state_without_a_second_direction_stops_after_the_first_token(oracle):
    """A state that is exactly a multiple of one outer product has no second direction.  With fp16-exact
    factors the first token removes it exactly, so every later token and every code must be zero."""
    k = np.zeros(128, np.float32); k[5] = 1.0
    u = (np.arange(128) % 7 - 3).astype(np.float32) / 8.0
    S = np.outer(k, u)[None, None].astype(np.float32)
    sh, st = _quant(oracle, S, r=4, n_iter=2, smooth=1)
    k0, u0 = st.comp_k_f32()[0, 0, 0], st.comp_u_f32()[0, 0, 0]
    sign = 1.0 if k0[5] > 0 else -1.0                         # the pair is fixed up to a common sign
    assert np.array_equal(sign * k0, k) and np.array_equal(sign * u0, u)
    assert not st.comp_k[0, 0, 1:].any() and not st.comp_u[0, 0, 1:].any()
    assert not st.codes.any()


def _fit_inputs(seed=50, r=4):
    rng = np.random.default_rng(seed)
    M = _gapped(rng, 128, 128, [9.0, 5.0, 3.0, 2.0, 1.2, 0.7])
    return M, M[None, None].astype(np.float32)


def _walsh(h, n):
    return np.array([-1.0 if bin(h & j).count("1") % 2 else 1.0 for j in range(n)])


@pytest.mark.parametrize("n_iter", [1, 2])
def test_value_sides_are_least_squares_for_what_the_earlier_tokens_left(oracle, n_iter):
    """Eq. 5 applied in turn: token h is fitted to R_h = S - sum_{a<h} k_a u_a^T, and for a given key the
    Frobenius minimiser over u is u_h = R_h^T k_h (|k_h| = 1).  Recomputed here in float64 from the STORED keys
    and values; the oracle gets there without forming R_h (through k_a^T k_h), so a wrong sign or index in
    that shortcut shows up as a value side that is off by far more than its fp16 rounding."""
    M, S = _fit_inputs()
    sh, st = _quant(oracle, S, r=4, n_iter=n_iter, smooth=0)
    kc = st.comp_k_f32()[0, 0].astype(np.float64)
    uc = st.comp_u_f32()[0, 0].astype(np.float64)
    R = M.copy()
    for h in range(4):
        want = R.T @ kc[h]
        assert np.all(np.abs(uc[h] - want) <= 2.0 ** -11 * np.abs(want) + 2.0 ** -24 * 16), h
        R = R - np.outer(kc[h], uc[h])
    # and the keys of a single step are Gram-Schmidt on S W0, W0 = the Walsh start vectors (a dense state has
    # no buffered record to start from): the Q factor of a library QR, column signs fixed by a positive diagonal
    if n_iter == 1:
        W0 = np.stack([_walsh(h, 128) for h in range(4)], axis=1)
        Q, Rq = np.linalg.qr(M @ W0)
        Q = Q * np.sign(np.diag(Rq))[None, :]
        assert np.all(np.abs(kc.T - Q) <= 2.0 ** -11 * np.abs(Q) + 1e-5)


def test_start_vectors_without_records_are_walsh_functions(oracle):
    """One step from start vector w gives k = S w / |S w|.  A diagonal state with fp16-exact entries makes S w
    readable: its first key must be the all-equal pattern (Walsh 0), and what the second key keeps after the
    first is taken out must follow the alternating pattern of Walsh 1."""
    d = np.array([2.0 ** -(i % 4) for i in range(128)])
    S = np.diag(d)[None, None].astype(np.float32)
    sh, st = _quant(oracle, S, r=2, n_iter=1, smooth=0)
    kc = st.comp_k_f32()[0, 0].astype(np.float64)
    t0 = d * _walsh(0, 128)
    assert np.allclose(kc[0], t0 / np.linalg.norm(t0), rtol=2.0 ** -10, atol=0)
    t1 = d * _walsh(1, 128)
    t1 = t1 - kc[0] * (kc[0] @ t1)
    assert np.allclose(kc[1], t1 / np.linalg.norm(t1), rtol=0, atol=2e-4)


def test_directions_already_spanned_are_dropped(oracle):
    """A state of rank two has nothing for a third and a fourth token: what the orthonormalisation has left of
    their start directions is rounding noise, which must not be blown up into a key.  Those tokens are all-zero
    bits, and the two that exist reproduce the state to fp16 accuracy."""
    for seed in (7, 9, 11):        # (on 7 and 11 the noise left of the third direction has a positive squared length)
        rng = np.random.default_rng(seed)
        A = rng.standard_normal((128, 2)); B = rng.standard_normal((128, 2))
        M = A @ B.T
        sh, st = _quant(oracle, M[None, None].astype(np.float32), r=4, n_iter=2, smooth=0)
        assert st.comp_k[0, 0, :2].any(axis=1).all() and st.comp_u[0, 0, :2].any(axis=1).all()
        assert not st.comp_k[0, 0, 2:].any() and not st.comp_u[0, 0, 2:].any()
        kc = st.comp_k_f32()[0, 0].astype(np.float64); uc = st.comp_u_f32()[0, 0].astype(np.float64)
        assert np.linalg.norm(M - kc.T @ uc) <= 2.0 ** -9 * np.linalg.norm(M)
