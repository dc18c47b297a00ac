"""GPU parity: every entry point of the library against the CPU oracle on the same seeded inputs.

Bar (written out in gpu_util.assert_state_parity): 8-bit codes bit-exact except <= 1 code step on <= 0.01 %
of the entries; outputs and dequantized states within 1e-3 relative / 1e-5 absolute.  Because the library
and the oracle take every sum in the same fixed order, the tests also demand bit-for-bit equality."""
import numpy as np
import pytest
import torch

from oracle.lq_oracle import State as OState
from paper_2609_38166_b200 import lq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

GATES = [synth.GATE_SCALAR, synth.GATE_DIAG]


def _close(got, want, what=""):
    assert np.allclose(got, want, rtol=1e-3, atol=1e-5), (what, float(np.abs(got - want).max()))
    assert np.array_equal(got, want), (what, "not bit-exact", float(np.abs(got - want).max()))


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("r,smooth,n_iter", [(4, 1, 4), (0, 1, 1), (8, 1, 2), (4, 0, 3), (1, 1, 1), (16, 1, 4)])
def test_quantize_state(oracle, gate, r, smooth, n_iter):
    wl = synth.Workload("q", 3, 5, 5, r=r, n_iter=n_iter, smooth=smooth, gate=gate, seed=100 + r,
                        outlier_frac=0.02, outlier_mag=8.0)
    osh, lsh = gu.shapes(wl)
    S = synth.dense_states(wl, 1)
    S[0, 0] = 0.0                 # an all-zero state: compensators vanish, scales hit their floors
    S[0, 1, :, 5] = 0.0           # a zero value channel
    S[0, 2, 9, :] = 0.0           # a zero key row
    ost = OState(osh)
    oracle.quantize_state(osh, S, ost)
    st = lq.State(lsh)
    st.win_pos.fill_(3)
    lq.quantize_state(lsh, gu.dev(S), st)
    gu.assert_state_parity(st, ost, r, "quantize")


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("W,r", [(16, 4), (1, 0), (7, 2), (64, 8)])
def test_dequantize_state_mid_window(oracle, gate, W, r):
    wl = synth.Workload("d", 4, 3, 3, W=W, r=r, gate=gate, seed=200 + W)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    oracle.quantize_state(osh, synth.dense_states(wl, 2), ost)
    # different fill levels per sequence, records drawn at random (the reconstruction does not care where
    # they came from)
    rng = np.random.default_rng(W)
    ost.win_pos[:] = [0, min(1, W - 1), W // 2, W - 1]
    ost.buf_k[...] = rng.standard_normal(ost.buf_k.shape).astype(np.float32) * 0.1
    ost.buf_u[...] = rng.standard_normal(ost.buf_u.shape).astype(np.float32)
    ost.buf_a[...] = rng.uniform(0.2, 1.0, ost.buf_a.shape).astype(np.float32)
    want = oracle.dequantize_state(osh, ost)
    st = gu.state_to_dev(ost, lsh)
    S = torch.empty((4, 3, 128, 128), dtype=torch.float32, device="cuda")
    lq.dequantize_state(lsh, st, S)
    _close(gu.host(S), want, "dequantize")
    gu.assert_state_parity(st, ost, r, "dequantize leaves the state alone")


@pytest.mark.parametrize("gate", GATES)
def test_reference_kernels(oracle, gate):
    wl = synth.Workload("ref", 3, 4, 2, gate=gate, seed=300)
    osh, lsh = gu.shapes(wl)
    S = np.zeros((3, 4, 128, 128), np.float32)
    S16 = np.zeros((3, 4, 128, 128), np.uint16)
    Sd = gu.dev(S); S16d = gu.dev(S16)
    o = torch.empty((3, 4, 128), dtype=torch.float32, device="cuda")
    for step in range(24):
        tok = synth.token_inputs(wl, step)
        td = gu.tok_dev(tok)
        want = oracle.ref_step_f32(osh, S, **tok)
        lq.ref_decode_step_f32(lsh, Sd, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        _close(gu.host(o), want, f"f32 o step {step}")
        want16 = oracle.ref_step_bf16(osh, S16, **tok)
        lq.ref_decode_step_bf16(lsh, S16d, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        _close(gu.host(o), want16, f"bf16 o step {step}")
    _close(gu.host(Sd), S, "f32 state")
    assert np.array_equal(gu.host(S16d), S16)


def _run_chain(oracle, wl, steps, init="zero", stagger=False, check_every=1, work=True):
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = np.zeros((wl.batch, wl.heads_v, 128, 128), np.float32) if init == "zero" else synth.dense_states(wl, 9)
    oracle.quantize_state(osh, S0, ost)
    st = lq.State(lsh, work=work)
    lq.quantize_state(lsh, gu.dev(S0), st)
    if stagger:       # window positions spread over [0, W): pre-fill with harmless records of zero update
        pos = (np.arange(wl.batch) * wl.W // max(wl.batch, 1)).astype(np.int32) % wl.W
        ost.win_pos[:] = pos
        ost.buf_a[...] = 1.0
        st = gu.state_to_dev(ost, lsh, work=work)
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    for step in range(steps):
        tok = synth.token_inputs(wl, step)
        td = gu.tok_dev(tok)
        want = oracle.decode_step(osh, ost, **tok)
        lq.decode_step(lsh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        _close(gu.host(o), want, f"o at step {step}")
        if step % check_every == 0 or step == steps - 1:
            gu.assert_state_parity(st, ost, wl.r, f"state after step {step}")
    return ost, st


def test_config1_single_head_64_tokens(oracle):
    # one GDN head, zero initial state, 64 tokens, W = 16: four boundaries, every step compared
    _run_chain(oracle, synth.config("single_gdn"), 64)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("W,r", [(8, 4), (16, 4), (32, 4), (16, 8), (1, 0), (3, 2), (64, 4)])
def test_staggered_batch_chain(oracle, gate, W, r):
    # the shape of the headline workload at a batch the oracle finishes in seconds: grouped heads,
    # window offsets spread uniformly, two full windows
    wl = synth.Workload("c2", 6, 4, 2, W=W, r=r, gate=gate, seed=400 + W + r)
    _run_chain(oracle, wl, 2 * W + 3 if W <= 16 else W + 5, init="dense", stagger=True, check_every=4)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("r,n_iter", [(4, 2), (8, 3), (16, 2), (3, 4)])
def test_chain_with_several_rounds_of_power_iteration(oracle, gate, r, n_iter):
    # more than one round: the boundary kernel then also runs W = S^T T and its orthonormalisation between the passes;
    # r = 8 and 16 take the instances of the kernel whose Cholesky factor is computed by a warp
    wl = synth.Workload("iters", 5, 4, 2, W=8, r=r, n_iter=n_iter, gate=gate, seed=470 + r + n_iter)
    _run_chain(oracle, wl, 2 * wl.W + 3, init="dense", stagger=True, check_every=4)


@pytest.mark.parametrize("gate", GATES)
def test_chain_without_the_delta_rule(oracle, gate):
    """b_t = 0 (Mamba2 / GLA style instances): u = v; decode, boundaries and both baseline kernels against the oracle."""
    wl = synth.Workload("nd", 5, 4, 2, W=4, r=2, gate=gate, seed=470, delta=0)
    _run_chain(oracle, wl, 14, init="dense", stagger=True, check_every=3)
    osh, lsh = gu.shapes(wl)
    S_o = synth.dense_states(wl, 2)
    S_d = gu.dev(S_o.copy())
    S16_o = synth.f32_to_bf16_bits(S_o)
    S16_d = gu.dev(S16_o.copy())
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    for step in range(3):
        tok = synth.token_inputs(wl, step)
        td = gu.tok_dev(tok)
        args = (td["q"], td["k"], td["v"], td["beta"], td["alpha"])
        want = oracle.ref_step_f32(osh, S_o, **tok)
        lq.ref_decode_step_f32(lsh, S_d, *args, o)
        _close(o.cpu().numpy(), want, f"fp32 baseline without the delta rule, step {step}")
        want16 = oracle.ref_step_bf16(osh, S16_o, **tok)
        lq.ref_decode_step_bf16(lsh, S16_d, *args, o)
        _close(o.cpu().numpy(), want16, f"bf16 baseline without the delta rule, step {step}")
    assert np.array_equal(S_d.cpu().numpy(), S_o)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("W,r", [(16, 4), (5, 2), (32, 0)])
def test_chain_with_fp16_records(oracle, gate, W, r):
    """The record buffer in fp16 (the paper's storage): append rounds kt, u (and the diagonal gate's alpha) with
    saturation; decode, boundaries, forced flush and dequantization against the oracle, bit for bit."""
    wl = synth.Workload("r16", 6, 4, 2, W=W, r=r, gate=gate, seed=480 + W, rec16=1)
    ost, st = _run_chain(oracle, wl, 2 * W + 3 if W <= 16 else W + 5, init="dense", stagger=True, check_every=4)
    osh, lsh = gu.shapes(wl)
    S = torch.empty((wl.batch, wl.heads_v, 128, 128), dtype=torch.float32, device="cuda")
    lq.dequantize_state(lsh, st, S)
    assert np.array_equal(S.cpu().numpy(), oracle.dequantize_state(osh, ost))
    oracle.window_flush(osh, ost, force=True)
    lq.window_flush(lsh, st, force=True)
    gu.assert_state_parity(st, ost, wl.r, "forced flush, fp16 records")


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("rec16", [0, 1])
def test_largest_supported_shape(oracle, gate, rec16):
    """W = 64 and r = 16 together (the largest shared-memory plans of both kernels), windows nearly full so that
    the step crosses a boundary with 64 records; without the delta rule for one of the combinations."""
    wl = synth.Workload("max", 2, 2, 1, W=64, r=16, gate=gate, seed=490 + rec16, rec16=rec16,
                        delta=0 if (gate == synth.GATE_DIAG and rec16) else 1)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = synth.dense_states(wl, 3)
    oracle.quantize_state(osh, S0, ost)
    rng = np.random.default_rng(5)
    n0 = 62                                                    # two tokens later the window is full
    ost.buf_k[:, :, :n0] = (rng.standard_normal(ost.buf_k[:, :, :n0].shape) / 16).astype(np.float16).astype(np.float32)
    ost.buf_u[:, :, :n0] = (rng.standard_normal(ost.buf_u[:, :, :n0].shape) / 4).astype(np.float16).astype(np.float32)
    ost.buf_a[:, :, :n0] = rng.uniform(0.9, 1.0, ost.buf_a[:, :, :n0].shape).astype(np.float16).astype(np.float32)
    ost.win_pos[:] = n0
    st = gu.state_to_dev(ost, lsh)
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    for step in range(4):
        tok = synth.token_inputs(wl, step)
        want = oracle.decode_step(osh, ost, **tok)
        td = gu.tok_dev(tok)
        lq.decode_step(lsh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        _close(o.cpu().numpy(), want, f"largest shape, step {step}")
        gu.assert_state_parity(st, ost, wl.r, f"largest shape, step {step}")
    assert int(ost.win_pos[0]) == 2 and lq.check_device() == 0


@pytest.mark.parametrize("gate", GATES)
def test_fused_step_kernel_gives_the_same_bits(oracle, gate, monkeypatch):
    """The step as one cooperative kernel (decode slots and boundary CTAs side by side; off by default because it
    is slower on this GPU): same chain, same oracle, bit for bit, with boundaries in every call."""
    monkeypatch.setenv("LQ_FUSED_STEP", "1")
    wl = synth.Workload("fu", 40, 4, 2, W=4, r=2, gate=gate, seed=495)
    _run_chain(oracle, wl, 11, init="dense", stagger=True, check_every=2)
    assert lq.check_device() == 0


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("work", [False, True])
def test_heads_of_the_last_round_are_drawn(oracle, gate, work):
    """More than three heads per resident CTA: with the scratch words in the state (lq_state.work) the decode kernel
    hands the heads of its last rounds to the CTAs that get there first (here every CTA takes two heads in turn and
    the other third of the heads is drawn; the full-size tests have seven in turn and two rounds drawn), without them
    every CTA takes the heads that fall to it in turn.  Same chain, same oracle, bit for bit; the words are zero
    after every call."""
    wl = synth.Workload("pool", 90, 32, 16, W=4, r=2, gate=gate, seed=496)
    _, st = _run_chain(oracle, wl, 6, init="dense", stagger=True, check_every=2, work=work)
    assert (st.work is not None) == work
    if work:
        assert int(st.work.abs().sum().item()) == 0
    assert lq.check_device() == 0


def test_steps_captured_in_a_cuda_graph_replay_identically():
    """W steps captured once (the two kernels of a step are programmatic dependents of each other) and replayed
    must leave the same state and outputs as the same steps issued directly."""
    wl = synth.Workload("cg", 24, 4, 2, W=4, r=2, seed=497)
    _, lsh = gu.shapes(wl)
    S0 = gu.dev(synth.dense_states(wl, 4))
    toks = [gu.tok_dev(synth.token_inputs(wl, t)) for t in range(4)]
    outs = {}
    for mode in ("direct", "graph"):
        st = lq.State(lsh)
        lq.quantize_state(lsh, S0, st)
        o = torch.zeros((4, wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            def steps():
                for t in range(4):
                    d = toks[t]
                    lq.decode_step(lsh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o[t], stream)
            if mode == "direct":
                for _ in range(3):
                    steps()
            else:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    steps()
                for _ in range(3):                  # (the capture itself runs nothing)
                    g.replay()
        stream.synchronize()
        outs[mode] = (o.cpu().numpy(), [t.cpu().numpy() for t in st.tensors()])
    assert np.array_equal(outs["direct"][0], outs["graph"][0])
    for a, b in zip(outs["direct"][1], outs["graph"][1]):
        assert np.array_equal(a, b)
    assert lq.check_device() == 0


def test_kda_outlier_chain(oracle):
    wl = synth.config("kda_b128_outlier").with_(batch=3, heads_v=4, heads_qk=4)
    _run_chain(oracle, wl, 40, stagger=True, check_every=5)


def test_heavy_tailed_chain_and_drift(oracle):
    # long-chain workload at reduced batch: Student-t(3) values, W = 16; codes match the oracle along the
    # chain, and the drift against the unquantized fp32 recurrence stays small
    wl = synth.config("gdn_drift").with_(batch=2, heads_v=2, heads_qk=2)
    osh, lsh = gu.shapes(wl)
    ost, st = _run_chain(oracle, wl, 96, check_every=16)
    # drift: replay on the GPU against the fp32-state baseline kernel
    st = lq.State(lsh)
    S = torch.zeros((2, 2, 128, 128), dtype=torch.float32, device="cuda")
    lq.quantize_state(lsh, S, st)
    o = torch.empty((2, 2, 128), dtype=torch.float32, device="cuda"); oref = torch.empty_like(o)
    rel = []
    for step in range(160):
        td = gu.tok_dev(synth.token_inputs(wl, step))
        args = (td["q"], td["k"], td["v"], td["beta"], td["alpha"])
        lq.decode_step(lsh, st, *args, o)
        lq.ref_decode_step_f32(lsh, S, *args, oref)
        if step >= 32:
            rel.append(float((o - oref).norm() / oref.norm()))
    assert np.mean(rel) < 5e-3, np.mean(rel)


def test_forced_flush_and_skip_of_full_windows(oracle):
    wl = synth.Workload("f", 4, 2, 1, W=8, r=4, seed=500)
    osh, lsh = gu.shapes(wl)
    ost, st = _run_chain(oracle, wl, 5, init="dense")
    lq.window_flush(lsh, st, force=False)           # nothing is full
    gu.assert_state_parity(st, ost, wl.r, "unforced flush is a no-op")
    oracle.window_flush(osh, ost, force=True)
    lq.window_flush(lsh, st, force=True)
    gu.assert_state_parity(st, ost, wl.r, "forced flush")
    # a sequence that enters with a full window gets no token (its output rows stay as they were); the
    # boundary pass of the same call flushes it, exactly like lq_window_flush
    st.win_pos[1] = wl.W
    ost.win_pos[1] = wl.W
    o = torch.full((4, 2, 128), 7.0, dtype=torch.float32, device="cuda")
    tok = synth.token_inputs(wl, 99)
    td = gu.tok_dev(tok)
    lq.decode_step(lsh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
    torch.cuda.synchronize()
    assert torch.all(o[1] == 7.0) and not torch.any(o[0] == 7.0)
    assert st.win_pos.tolist() == [1, 0, 1, 1]
    oracle.window_flush(osh, ost, force=False)
    assert np.array_equal(gu.gpu_codes(st)[1], ost.codes[1])
    for name in ("col_scale", "row_smooth"):
        assert np.array_equal(gu.host(getattr(st, name))[1], getattr(ost, name)[1]), name
    assert np.array_equal(gu.host(st.comp_u)[1], ost.comp_u[1])


def test_sub_batches_by_pointer_offset(oracle):
    # stepping sequences [2, 5) only must leave the others alone and equal the oracle on the slice
    wl = synth.Workload("s", 6, 2, 2, W=4, r=2, seed=600)
    osh, lsh = gu.shapes(wl)
    ost, st = _run_chain(oracle, wl, 3, init="dense")
    before = [t.clone() for t in st.tensors()]
    tok = synth.token_inputs(wl, 50)
    td = gu.tok_dev(tok)
    o = torch.zeros((6, 2, 128), dtype=torch.float32, device="cuda")
    lq.decode_step(lsh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o, b0=2, nb=3)
    torch.cuda.synchronize()
    for t0, t1 in zip(before, st.tensors()):
        assert torch.equal(t0[:2], t1[:2]) and torch.equal(t0[5:], t1[5:])
    sub = wl.with_(batch=3)
    osub, _ = gu.shapes(sub)
    ost_sub = OState(osub)
    for name in ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos"):
        getattr(ost_sub, name)[...] = getattr(ost, name)[2:5]
    want = oracle.decode_step(osub, ost_sub, **{k: np.ascontiguousarray(v[2:5]) for k, v in tok.items()})
    _close(gu.host(o)[2:5], want, "sub-batch o")
    assert np.array_equal(gu.gpu_codes(st)[2:5], ost_sub.codes)
    assert st.win_pos.tolist() == [3, 3, 0, 0, 0, 3]


def test_empty_batch_is_a_no_op():
    sh = lq.Shape(0, 4, 2)
    st = lq.State(lq.Shape(1, 4, 2))
    e = torch.empty((16,), dtype=torch.int16, device="cuda")
    o = torch.empty((16,), dtype=torch.float32, device="cuda")
    lq.decode_step(sh, st, e, e, e, e, e, o)
    lq.window_flush(sh, st, True)
    lq.quantize_state(sh, o, st)
    lq.dequantize_state(sh, st, o)
    torch.cuda.synchronize()


@pytest.mark.parametrize("batch", [3, 8])
def test_host_buffer_entry_point(oracle, batch):
    """batch 3: array sizes that are not multiples of 16 bytes (copied with cudaMemcpyAsync); batch 8: the
    path that gathers the pinned inputs with one launch and writes o straight into the pinned host array."""
    wl = synth.Workload("h", batch, 4, 2, W=4, r=2, seed=700)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = synth.dense_states(wl, 9)
    oracle.quantize_state(osh, S0, ost)
    st = lq.State(lsh)
    lq.quantize_state(lsh, gu.dev(S0), st)
    stage = torch.empty((lq.decode_stage_bytes(lsh),), dtype=torch.uint8, device="cuda")
    o_h = torch.empty((batch, 4, 128), dtype=torch.float32).pin_memory()
    for step in range(6):
        tok = synth.token_inputs(wl, step)
        want = oracle.decode_step(osh, ost, **tok)
        pin = {k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in tok.items()}
        lq.decode_step_host(lsh, st, pin["q"], pin["k"], pin["v"], pin["beta"], pin["alpha"], o_h, stage)
        torch.cuda.synchronize()
        _close(o_h.numpy(), want, f"host-buffer step {step}")
    gu.assert_state_parity(st, ost, wl.r, "host-buffer chain")


@pytest.mark.parametrize("gate,batch", [(synth.GATE_SCALAR, 37), (synth.GATE_DIAG, 16), (synth.GATE_SCALAR, 5)])
def test_pipelined_host_entry_point(oracle, gate, batch):
    """Sub-batches with copies on side streams: ragged last sub-batch (37 = 16+16+5+0), an exact split, and a
    batch below the pipelining threshold; seven tokens with W = 4 cross a window boundary on the way."""
    wl = synth.Workload("hp", batch, 4, 2, W=4, r=2, gate=gate, seed=710 + batch)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = synth.dense_states(wl, 11)
    oracle.quantize_state(osh, S0, ost)
    st = lq.State(lsh)
    lq.quantize_state(lsh, gu.dev(S0), st)
    stage = torch.empty((lq.decode_stage_bytes(lsh),), dtype=torch.uint8, device="cuda")
    o_h = torch.full((batch, 4, 128), float("nan"), dtype=torch.float32).pin_memory()
    side = torch.cuda.Stream()
    for step in range(7):
        tok = synth.token_inputs(wl, step)
        want = oracle.decode_step(osh, ost, **tok)
        pin = {k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in tok.items()}
        with torch.cuda.stream(side):
            lq.decode_step_host_pipelined(lsh, st, pin["q"], pin["k"], pin["v"], pin["beta"], pin["alpha"], o_h,
                                          stage, side)
        side.synchronize()
        _close(o_h.numpy(), want, f"pipelined host-buffer step {step}")
    gu.assert_state_parity(st, ost, wl.r, "pipelined host-buffer chain")
    assert lq.check_device() == 0


@pytest.mark.parametrize("gate,state_bf16", [(synth.GATE_SCALAR, 0), (synth.GATE_DIAG, 0), (synth.GATE_SCALAR, 1)])
def test_pipelined_host_steps_back_to_back(oracle, gate, state_bf16):
    """Consecutive pipelined calls without a synchronisation in between chain onto each other (the inputs of a
    call are brought in while the call before it is still computing and copying out): every token has its own
    pinned inputs and its own output array, and everything is compared once at the end."""
    kw = dict(r=0, smooth=0, state_bf16=1) if state_bf16 else dict(r=2)
    wl = synth.Workload("hb", 40, 4, 2, W=4, gate=gate, seed=760, **kw)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = synth.dense_states(wl, 12)
    oracle.quantize_state(osh, S0, ost)
    st = lq.State(lsh)
    lq.quantize_state(lsh, gu.dev(S0), st)
    stage = torch.empty((lq.decode_stage_bytes(lsh),), dtype=torch.uint8, device="cuda")
    steps = 11
    toks = [synth.token_inputs(wl, t) for t in range(steps)]
    pins = [{k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in tok.items()} for tok in toks]
    outs = [torch.full((40, 4, 128), float("nan"), dtype=torch.float32).pin_memory() for _ in range(steps)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for t in range(steps - 1):           # (the last token is the one the unpipelined call below takes)
            d = pins[t]
            lq.decode_step_host_pipelined(lsh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], outs[t], stage, side)
            if t == 5:                       # an unpipelined call in between breaks the chain and must still be ordered
                t2 = steps - 1
                d = pins[t2]
                lq.decode_step_host(lsh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], outs[t2], stage, side)
    side.synchronize()
    order = list(range(6)) + [steps - 1] + list(range(6, steps - 1))
    for t in order:
        want = oracle.decode_step(osh, ost, **toks[t])
        _close(outs[t].numpy(), want, f"back-to-back host step {t}")
    gu.assert_state_parity(st, ost, wl.r, "back-to-back pipelined chain")
    assert lq.check_device() == 0


# ---- per-window BF16 (the -w baseline): bfloat16 boundary state, no scale, smoothing or compensators ----

def _bf16w(name, batch, heads_v, heads_qk, **kw):
    return synth.Workload(name, batch, heads_v, heads_qk, r=0, smooth=0, state_bf16=1, **kw)


@pytest.mark.parametrize("gate", GATES)
@pytest.mark.parametrize("W,rec16,delta", [(16, 0, 1), (1, 0, 1), (5, 1, 1), (64, 0, 1), (40, 1, 0)])
def test_per_window_bf16_chain(oracle, gate, W, rec16, delta):
    """Every output, the bfloat16 boundary state after every boundary and the record buffer, bit for bit."""
    wl = _bf16w("w", 6, 4, 2, W=W, gate=gate, rec16=rec16, delta=delta, seed=600 + W)
    _run_chain(oracle, wl, 2 * W + 3 if W <= 16 else W + 5, init="dense", stagger=True, check_every=4)


@pytest.mark.parametrize("gate", GATES)
def test_per_window_bf16_dequantize_and_forced_flush(oracle, gate):
    wl = _bf16w("wd", 4, 3, 3, W=7, gate=gate, seed=610)
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    oracle.quantize_state(osh, synth.dense_states(wl, 2), ost)
    rng = np.random.default_rng(7)
    ost.win_pos[:] = [0, 1, 3, 6]
    ost.buf_k[...] = rng.standard_normal(ost.buf_k.shape).astype(np.float32) * 0.1
    ost.buf_u[...] = rng.standard_normal(ost.buf_u.shape).astype(np.float32)
    ost.buf_a[...] = rng.uniform(0.2, 1.0, ost.buf_a.shape).astype(np.float32)
    want = oracle.dequantize_state(osh, ost)
    st = gu.state_to_dev(ost, lsh)
    S = torch.empty((4, 3, 128, 128), dtype=torch.float32, device="cuda")
    lq.dequantize_state(lsh, st, S)
    torch.cuda.synchronize()
    assert np.array_equal(gu.host(S), want)
    gu.assert_state_parity(st, ost, 0, "dequantize leaves the state alone")
    lq.window_flush(lsh, st, force=False)
    gu.assert_state_parity(st, ost, 0, "unforced flush is a no-op")
    oracle.window_flush(osh, ost, force=True)
    lq.window_flush(lsh, st, force=True)
    gu.assert_state_parity(st, ost, 0, "forced flush")
    assert st.win_pos.tolist() == [0, 0, 0, 0]


def test_per_window_bf16_refuses_compensators_and_smoothing():
    for kw in ({"r": 2, "smooth": 0}, {"r": 0, "smooth": 1}):
        sh = lq.Shape(1, 1, 1, 128, 128, 16, n_iter=2, state_bf16=1, **kw)
        assert lq.head_bytes(sh) == 0
    assert lq.head_bytes(lq.Shape(1, 1, 1, 128, 128, 16, r=0, smooth=0, state_bf16=1)) == 2 * 128 * 128
