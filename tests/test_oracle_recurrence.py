"""Pins for the oracle's recurrences: the dense reference step, the windowed decode step and the
reconstruction, against the models' native updates written densely in float64, against closed-form
special cases, and against brute force on tiny states."""
import numpy as np
import pytest

from oracle.lq_oracle import Shape, State
from paper_2609_38166_b200 import synth
from tests import refmath as rm

GATES = [synth.GATE_SCALAR, synth.GATE_DIAG]


def _shape(wl):
    return Shape(wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth, wl.delta, wl.rec16, wl.state_bf16)


def _rel(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / (np.linalg.norm(b) + 1e-30))


@pytest.mark.parametrize("gate", GATES)
def test_native_update_equals_general_form(gate):
    # the identity of Appendix A that lets GDN and KDA use Eq. 1; pure float64 mathematics
    wl = synth.Workload("t", 1, 1, 1, 32, 24, gate=gate, seed=11)
    S = np.random.default_rng(0).standard_normal((32, 24))
    for step in range(5):
        q, k, v, beta, alpha = rm.widen(synth.token_inputs(wl, step), wl)
        S1, o1 = rm.native_step(S, q, k, v, beta, alpha, gate)
        S2, o2 = rm.general_step(S, q, k, v, beta, alpha, gate)
        assert np.allclose(S1, S2, rtol=0, atol=1e-12) and np.allclose(o1, o2, rtol=0, atol=1e-12)
        S = S1


@pytest.mark.parametrize("gate", GATES)
def test_reference_step_follows_native_update(oracle, gate):
    wl = synth.Workload("t", 2, 4, 2, 128, 128, gate=gate, seed=12)
    sh = _shape(wl)
    S = np.zeros((2, 4, 128, 128), np.float32)
    S64 = np.zeros((2, 4, 128, 128))
    for step in range(40):
        tok = synth.token_inputs(wl, step)
        o = oracle.ref_step_f32(sh, S, **tok)
        for b in range(2):
            for h in range(4):
                S64[b, h], o64 = rm.native_step(S64[b, h], *rm.widen(tok, wl, b, h), gate)
                assert np.allclose(o[b, h], o64, rtol=1e-5, atol=1e-5)
    assert _rel(S, S64) < 1e-6


def test_delta_rule_write_is_exact_recall(oracle):
    # alpha = beta = 1 and |k| = 1: the update stores v under k, so reading with q = k returns v.
    # Keys are +-1/8 on 64 channels, exactly representable and of unit length.
    K = V = 64
    sh = Shape(1, 1, 1, K, V, 4, 0, 1, synth.GATE_SCALAR, 1)
    rng = np.random.default_rng(5)
    S = rng.standard_normal((1, 1, K, V)).astype(np.float32)
    one = synth.f32_to_bf16_bits(np.ones((1, 1), np.float32))
    for _ in range(6):
        k = (rng.integers(0, 2, (1, 1, K)) * 2 - 1).astype(np.float32) / 8.0
        v = synth.f32_to_bf16_bits(rng.standard_normal((1, 1, V)).astype(np.float32))
        kb = synth.f32_to_bf16_bits(k)
        o = oracle.ref_step_f32(sh, S, kb, kb, v, one, one)
        assert np.allclose(o, synth.bf16_bits_to_f32(v), rtol=0, atol=2e-5)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("W", [1, 3, 16])
def test_windowed_decode_without_quantizer_equals_dense_recurrence(oracle, gate, W):
    # Eq. 4 / Eq. 9: with quant_b the identity the windowed form is the recurrence itself
    wl = synth.Workload("t", 2, 2, 1, 128, 128, W=W, r=0, gate=gate, seed=13)
    sh = _shape(wl)
    st = State(sh, quant=False)
    S64 = np.zeros((2, 2, 128, 128))
    for step in range(2 * W + 5):
        tok = synth.token_inputs(wl, step)
        o = oracle.decode_step(sh, st, **tok)
        for b in range(2):
            for h in range(2):
                S64[b, h], o64 = rm.native_step(S64[b, h], *rm.widen(tok, wl, b, h), gate)
                assert np.allclose(o[b, h], o64, rtol=1e-5, atol=1e-5), (step, b, h)
        assert np.all(st.win_pos == (step + 1) % W)
        assert _rel(oracle.dequantize_state(sh, st), S64) < 1e-6


@pytest.mark.parametrize("gate", GATES)
def test_recall_special_case_holds_with_quantization_on(oracle, gate):
    # With alpha = beta = 1, |k| = 1 and q = k the windowed output is v whatever the quantized state holds,
    # because the same readout enters u and o and cancels.
    K = V = 64
    wl = synth.Workload("t", 1, 2, 2, K, V, W=4, r=2, gate=gate, seed=14)
    sh = _shape(wl)
    st = State(sh)
    oracle.quantize_state(sh, synth.dense_states(wl, 1), st)
    rng = np.random.default_rng(6)
    one = synth.f32_to_bf16_bits(np.ones((1, 2), np.float32))
    ones_a = one if gate == synth.GATE_SCALAR else synth.f32_to_bf16_bits(np.ones((1, 2, K), np.float32))
    for _ in range(9):
        kb = synth.f32_to_bf16_bits((rng.integers(0, 2, (1, 2, K)) * 2 - 1).astype(np.float32) / 8.0)
        v = synth.f32_to_bf16_bits(rng.standard_normal((1, 2, V)).astype(np.float32))
        o = oracle.decode_step(sh, st, kb, kb, v, one, ones_a)
        assert np.allclose(o, synth.bf16_bits_to_f32(v), rtol=0, atol=1e-5)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("dims", [(4, 4, 3, 1), (4, 4, 2, 2), (8, 16, 3, 2), (5, 3, 4, 1)])
@pytest.mark.parametrize("build", ["defining", "plain"])
def test_brute_force_on_tiny_states(oracle, oracle_plain, build, gate, dims):
    """Materialise the state densely before every token (Eq. 7 written out in float64 from the stored arrays),
    apply the native update, and compare the token's output and the record it appends.  Both the defining build
    (fixed summation tree, fixed-point readout) and the plain one (binary64 sums, no grid) must pass."""
    oracle = oracle_plain if build == "plain" else oracle
    K, V, W, r = dims
    wl = synth.Workload("t", 2, 2, 2, K, V, W=W, r=r, gate=gate, seed=15)
    sh = _shape(wl)
    st = State(sh)
    oracle.quantize_state(sh, synth.dense_states(wl, 2, rank=2), st)
    for step in range(3 * W + 1):
        tok = synth.token_inputs(wl, step)
        dense = np.zeros((2, 2, K, V))
        for b in range(2):
            n = int(st.win_pos[b])
            for h in range(2):
                S = rm.dequant_plain(st.codes[b, h], st.col_scale[b, h], st.row_smooth[b, h], st.comp_k[b, h],
                                     st.comp_u[b, h])
                for j in range(n):     # apply the buffered records in order (Eq. 3)
                    a = st.buf_a[b, h, j].astype(np.float64)
                    a = np.full(K, float(a)) if gate == synth.GATE_SCALAR else a
                    S = a[:, None] * S + np.outer(st.buf_k[b, h, j].astype(np.float64),
                                                  st.buf_u[b, h, j].astype(np.float64))
                dense[b, h] = S
        assert np.allclose(oracle.dequantize_state(sh, st), dense, rtol=1e-5, atol=1e-6)
        n_before = st.win_pos.copy()
        o = oracle.decode_step(sh, st, **tok)
        for b in range(2):
            for h in range(2):
                q, k, v, beta, alpha = rm.widen(tok, wl, b, h)
                Sn, o64 = rm.native_step(dense[b, h], q, k, v, beta, alpha, gate)
                assert np.allclose(o[b, h], o64, rtol=1e-5, atol=1e-5), (step, b, h)
                if n_before[b] + 1 < W:   # the record is still in the buffer: u = v - S^T (alpha (.) k)
                    a = np.full(K, float(alpha)) if gate == synth.GATE_SCALAR else alpha
                    u64 = v - dense[b, h].T @ (a * k)
                    assert np.allclose(st.buf_u[b, h, n_before[b]], u64, rtol=1e-5, atol=1e-5)
                    assert np.allclose(st.buf_k[b, h, n_before[b]], beta * k, rtol=1e-6, atol=0)
        assert np.all(st.win_pos == (n_before + 1) % W)


def test_grouped_heads_read_the_right_query_head(oracle):
    # value head h uses q/k head h // (Hv/Hqk): make q/k heads wildly different and compare per head
    wl = synth.Workload("t", 1, 4, 2, 16, 8, W=4, r=1, seed=16)
    sh = _shape(wl)
    S = np.zeros((1, 4, 16, 8), np.float32)
    S64 = np.zeros((4, 16, 8))
    for step in range(6):
        tok = synth.token_inputs(wl, step)
        o = oracle.ref_step_f32(sh, S, **tok)
        for h in range(4):
            S64[h], o64 = rm.native_step(S64[h], *rm.widen(tok, wl, 0, h), wl.gate)
            assert np.allclose(o[0, h], o64, rtol=1e-5, atol=1e-6)


def test_bf16_state_baseline_rounds_state_each_token(oracle):
    wl = synth.Workload("t", 1, 2, 2, 32, 32, seed=17)
    sh = _shape(wl)
    S16 = np.zeros((1, 2, 32, 32), np.uint16)
    S64 = np.zeros((2, 32, 32))
    for step in range(10):
        tok = synth.token_inputs(wl, step)
        o = oracle.ref_step_bf16(sh, S16, **tok)
        for h in range(2):
            Sn, o64 = rm.native_step(S64[h], *rm.widen(tok, wl, 0, h), wl.gate)
            assert np.allclose(o[0, h], o64, rtol=1e-5, atol=1e-6)
            S64[h] = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(Sn.astype(np.float32))).astype(np.float64)
            got = synth.bf16_bits_to_f32(S16[0, h]).astype(np.float64)
            # equal up to an occasional one-ulp difference where the fp32 and fp64 values straddle a tie
            assert np.mean(got != S64[h]) < 0.01 and np.allclose(got, S64[h], rtol=2.0 ** -7, atol=1e-8)
            S64[h] = got


def test_boundary_term_is_exact_up_to_the_fixed_point_grid(oracle):
    """(B/127) Z^T (C Gamma x) with the vector on a 30-bit block fixed-point grid and exact integer sums:
    against float64 the error is the grid's (2^-29 of the largest entry per term) plus two fp32 roundings,
    far below what an fp32 accumulation of 128 terms leaves."""
    wl = synth.Workload("t", 2, 2, 2, 128, 128, W=4, r=0, seed=18)
    sh = _shape(wl)
    st = State(sh)
    oracle.quantize_state(sh, synth.dense_states(wl, 3), st)
    tok = synth.token_inputs(wl, 0)
    oracle.decode_step(sh, st, **tok)          # n = 0, r = 0: u = v - (B/127) Z^T (c . alpha k)
    for b in range(2):
        for h in range(2):
            q, k, v, beta, alpha = rm.widen(tok, wl, b, h)
            c = st.row_smooth[b, h].astype(np.float64)
            x = (c.astype(np.float32) * (np.float32(alpha) * k.astype(np.float32))).astype(np.float64)
            s = st.col_scale[b, h].astype(np.float64)
            Z = st.codes[b, h].astype(np.float64)
            exact = s * (Z.T @ x)
            got = v - st.buf_u[b, h, 0].astype(np.float64)
            grid = 2.0 ** -29 * 2 * np.abs(x).max() * np.abs(Z).sum(axis=0) * s
            assert np.all(np.abs(got - exact) <= grid + 3 * 2.0 ** -24 * (np.abs(exact) + np.abs(v)))


def _grid_probe(oracle, tail):
    """u of one token against a hand-made state: codes Z[1][j] = j - 64 (else 0), step 1, c = 1, alpha = beta = 1,
    v = 0 and key (1, tail, 0, ...): u_j = -(j - 64) * tail-as-the-readout-sees-it."""
    sh = Shape(1, 1, 1, 128, 128, 4, 0, 1, synth.GATE_SCALAR, 0)
    st = State(sh)
    st.codes[0, 0, 1, :] = np.arange(128) - 64
    st.col_scale[...] = 1.0
    k = np.zeros((1, 1, 128), np.float32); k[0, 0, 0] = 1.0; k[0, 0, 1] = tail
    kb = synth.f32_to_bf16_bits(k)
    assert np.array_equal(synth.bf16_bits_to_f32(kb), k)          # the probe values are bfloat16 numbers
    one = synth.f32_to_bf16_bits(np.ones((1, 1), np.float32))
    zero_v = synth.f32_to_bf16_bits(np.zeros((1, 1, 128), np.float32))
    oracle.decode_step(sh, st, kb, kb, zero_v, one, one)
    return -st.buf_u[0, 0, 0].astype(np.float64) / (np.arange(128) - 64 + 1e-300)


def test_fixed_point_grid_is_thirty_bits_below_the_bound(oracle, oracle_plain):
    """The readout vector is rounded to multiples of 2^(e-29), 2^e <= max|x| < 2^(e+1), ties to even.  With
    max|x| = 1 a second entry of 2^-29 must pass through exactly (a 28-bit grid would lose it), 2^-30 is a tie
    that goes to zero and 3 * 2^-30 a tie that goes to 2^-28 (a finer grid would keep both).  The plain build
    has no grid and returns all three as they are."""
    for tail, on_grid in ((2.0 ** -29, 2.0 ** -29), (2.0 ** -30, 0.0), (3 * 2.0 ** -30, 2.0 ** -28)):
        seen = _grid_probe(oracle, tail)
        seen_plain = _grid_probe(oracle_plain, tail)
        keep = np.arange(128) != 64
        assert np.all(seen[keep] == on_grid), (tail, seen[:3])
        assert np.all(seen_plain[keep] == tail), (tail, seen_plain[:3])


@pytest.mark.parametrize("gate", GATES)
def test_defining_build_agrees_with_the_plain_definition_along_a_chain(oracle, oracle_plain, gate):
    """What the fixed summation tree and the fixed-point readout cost against the plain definition, measured
    on the CPU with both builds started from the same state at every token (so that differences do not
    compound): outputs and records within 1e-3 relative / 1e-5 absolute; after a boundary, heads whose fp16
    compensators came out identical differ by at most one code step on at most 0.01 % of the entries."""
    wl = synth.Workload("t", 2, 4, 2, 128, 128, W=8, r=4, gate=gate, seed=71)
    sh = _shape(wl)
    st = State(sh)
    oracle.quantize_state(sh, synth.dense_states(wl, 3), st)
    same_heads = diff_entries = entries = 0
    for step in range(3 * wl.W):
        tok = synth.token_inputs(wl, step)
        st_p = State(sh)
        for name in ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos"):
            getattr(st_p, name)[...] = getattr(st, name)
        o = oracle.decode_step(sh, st, **tok)
        o_p = oracle_plain.decode_step(sh, st_p, **tok)
        assert np.allclose(o, o_p, rtol=1e-3, atol=1e-5), step
        assert np.array_equal(st.win_pos, st_p.win_pos)
        if st.win_pos[0] != 0:
            n = st.win_pos[0] - 1
            assert np.allclose(st.buf_u[:, :, n], st_p.buf_u[:, :, n], rtol=1e-3, atol=1e-5)
            continue
        for b in range(wl.batch):
            for h in range(wl.heads_v):
                if not (np.array_equal(st.comp_k[b, h], st_p.comp_k[b, h]) and
                        np.array_equal(st.comp_u[b, h], st_p.comp_u[b, h])):
                    continue
                same_heads += 1
                d = np.abs(st.codes[b, h].astype(int) - st_p.codes[b, h].astype(int))
                assert d.max() <= 1
                diff_entries += int((d > 0).sum()); entries += d.size
                assert np.allclose(st.col_scale[b, h], st_p.col_scale[b, h], rtol=1e-3, atol=1e-5)
                assert np.allclose(st.row_smooth[b, h], st_p.row_smooth[b, h], rtol=1e-3, atol=1e-5)
    assert same_heads > 0 and diff_entries <= 1e-4 * entries, (same_heads, diff_entries, entries)


@pytest.mark.parametrize("gate", GATES)
def test_without_the_delta_rule_the_state_is_a_decayed_sum_of_outer_products(oracle, gate):
    """b_t = 0 (Table 4: linear attention, RetNet, Mamba2 with the scalar gate; GLA, RWKV6, HGRN2 with the diagonal
    one): nothing is read back, so S_t = sum_i (prod_{i<j<=t} D_j) k~_i v_i^T in closed form and
    o_t = sum_i <prod D_j k~_i, q_t> v_i.  Checked for the dense reference step and, with a quantized state, for
    the windowed decode (error at the 8-bit level) and with the quantizer off (equal up to fp32 rounding)."""
    wl = synth.Workload("t", 2, 4, 2, 128, 128, W=4, r=2, gate=gate, seed=61, delta=0)
    sh = _shape(wl)
    B, H, T = 2, 4, 11
    toks = [synth.token_inputs(wl, t) for t in range(T)]
    # closed form in float64
    o_want = np.zeros((T, B, H, 128))
    for b in range(B):
        for h in range(H):
            w = [rm.widen(tok, wl, b, h) for tok in toks]             # (q, k, v, beta, alpha) in float64
            for t in range(T):
                acc = np.zeros(128)
                for i in range(t + 1):
                    q_t = w[t][0]
                    kt = w[i][3] * w[i][1]
                    for j in range(i + 1, t + 1):
                        kt = kt * w[j][4]                             # scalar or per-channel decay
                    acc += (kt @ q_t) * w[i][2]
                o_want[t, b, h] = acc
    S = np.zeros((B, H, 128, 128), np.float32)
    st_off = State(sh, quant=False)
    st_q = State(sh)
    oracle.quantize_state(sh, S, st_q)
    for t in range(T):
        o_ref = oracle.ref_step_f32(sh, S, **toks[t])
        o_off = oracle.decode_step(sh, st_off, **toks[t])
        o_q = oracle.decode_step(sh, st_q, **toks[t])
        assert np.allclose(o_ref, o_want[t], rtol=1e-5, atol=1e-5)
        assert np.allclose(o_off, o_want[t], rtol=1e-5, atol=1e-5)
        assert _rel(o_q, o_want[t]) < 2e-3
    # and the delta rule really is off: with it on, the same tokens give a different output
    wl_on = wl.with_(delta=1)
    S2 = np.zeros((B, H, 128, 128), np.float32)
    for t in range(T):
        o_on = oracle.ref_step_f32(_shape(wl_on), S2, **toks[t])
    assert _rel(o_on, o_want[T - 1]) > 1e-2
