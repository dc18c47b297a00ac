"""Two safety nets for the CUDA path that need no memory checker: guard bands around every buffer a kernel
writes (a stray store shows up as a damaged pattern), and a checkpoint taken in the middle of a window (the
window representation is self-contained: restored into other memory it must continue bit for bit)."""
import numpy as np
import pytest
import torch

from paper_2609_38166_b200 import lq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

GUARD = 256          # bytes of pattern on either side
PATTERN = 0xA5


class Guarded:
    """A tensor of `shape` / `dtype` carved out of a byte buffer with GUARD bytes of pattern before and after."""

    def __init__(self, shape, dtype, fill=0):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 16
        self.raw = torch.full((GUARD + n + pad + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.n = n
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(shape)
        self.t.fill_(fill)

    def intact(self):
        r = self.raw.cpu().numpy()
        return bool((r[:GUARD] == PATTERN).all() and (r[GUARD + self.n:] == PATTERN).all())


def _guarded_state(sh):
    hb, rf = lq.head_bytes(sh), lq.record_floats(sh)
    B, H, W = sh.batch, sh.heads_v, sh.W
    g = {"heads": Guarded((B, H, hb), torch.uint8), "records": Guarded((B, H, W, rf), torch.float16 if sh.rec16 else torch.float32),
         "decays": Guarded((B, H, W), torch.float32), "win_pos": Guarded((B,), torch.int32)}
    st = lq.State(sh, storage=(g["heads"].t, g["records"].t, g["decays"].t, g["win_pos"].t))
    return st, g


@pytest.mark.parametrize("gate", [synth.GATE_SCALAR, synth.GATE_DIAG])
@pytest.mark.parametrize("batch,heads_v,heads_qk,W,r,rec16", [(3, 5, 5, 64, 16, 0),      # the largest window and token count
                                                              (3, 5, 5, 64, 16, 1),
                                                              (41, 23, 23, 4, 2, 0),     # more heads than resident CTAs, odd counts
                                                              (2, 4, 2, 16, 4, 0)])
def test_no_entry_point_writes_outside_its_buffers(gate, batch, heads_v, heads_qk, W, r, rec16):
    wl = synth.Workload("guard", batch, heads_v, heads_qk, W=W, r=r, gate=gate, rec16=rec16, seed=900 + W + r)
    _, sh = gu.shapes(wl)
    st, g = _guarded_state(sh)
    S_in = Guarded((batch, heads_v, 128, 128), torch.float32)
    S_in.t.copy_(gu.dev(synth.dense_states(wl, 2)))
    S_out = Guarded((batch, heads_v, 128, 128), torch.float32)
    o = Guarded((batch, heads_v, 128), torch.float32)
    bufs = dict(g, S_in=S_in, S_out=S_out, o=o)

    def check(after):
        torch.cuda.synchronize()
        for name, b in bufs.items():
            assert b.intact(), (after, name)

    lq.quantize_state(sh, S_in.t, st)
    check("lq_quantize_state")
    steps = min(W + 3, 20)
    for step in range(steps):
        td = gu.tok_dev(synth.token_inputs(wl, step))
        lq.decode_step(sh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o.t)
    check("lq_decode_step")
    lq.dequantize_state(sh, st, S_out.t)
    check("lq_dequantize_state")
    lq.window_flush(sh, st, force=True)
    check("lq_window_flush")
    assert int(st.win_pos.max()) == 0
    assert lq.check_device() == 0


@pytest.mark.parametrize("gate", [synth.GATE_SCALAR, synth.GATE_DIAG])
@pytest.mark.parametrize("rec16", [0, 1])
def test_checkpoint_in_mid_window_resumes_bit_for_bit(gate, rec16):
    """After 5 + 2 W tokens (five records in the buffer) the four arrays of the state are copied to the host; the
    run goes on for W + 7 tokens (through a boundary).  Restored into fresh device memory and fed the same tokens,
    the copy must produce the same outputs and end in the same state, bit for bit."""
    wl = synth.Workload("ckpt", 6, 4, 2, W=8, r=4, gate=gate, rec16=rec16, seed=950 + gate + 2 * rec16)
    _, sh = gu.shapes(wl)
    st = lq.State(sh)
    lq.quantize_state(sh, gu.dev(synth.dense_states(wl, 5)), st)
    # stagger the windows a little: the first three sequences take one token more than the others
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    toks = [gu.tok_dev(synth.token_inputs(wl, t)) for t in range(5 + 2 * wl.W + wl.W + 7 + 1)]

    def step(state, t, out):
        d = toks[t]
        lq.decode_step(sh, state, d["q"], d["k"], d["v"], d["beta"], d["alpha"], out)

    d = toks[-1]
    lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, b0=0, nb=3)
    first = 5 + 2 * wl.W
    for t in range(first):
        step(st, t, o)
    torch.cuda.synchronize()
    assert sorted(set(st.win_pos.tolist())) == [5, 6]
    saved = [t.cpu().clone() for t in st.tensors()]               # the checkpoint
    outs = []
    for t in range(first, first + wl.W + 7):
        step(st, t, o)
        outs.append(o.cpu().clone())
    final = [t.cpu().clone() for t in st.tensors()]
    # restore into other memory (a guard-banded allocation, so the addresses differ from the original ones)
    st2, g = _guarded_state(sh)
    for dst, src in zip(st2.tensors(), saved):
        dst.copy_(src.cuda())
    o2 = torch.empty_like(o)
    for i, t in enumerate(range(first, first + wl.W + 7)):
        step(st2, t, o2)
        assert torch.equal(o2.cpu(), outs[i]), ("output", t)
    torch.cuda.synchronize()
    for name, a, b in zip(("heads", "records", "decays", "win_pos"), st2.tensors(), final):
        assert torch.equal(a.cpu().view(torch.uint8), b.view(torch.uint8)), name
    assert all(b.intact() for b in g.values())
    assert lq.check_device() == 0


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Waits in the kernels are bounded.  The library's self test lets one run out on purpose (a barrier nothing
    completes, 64 polls): the kernel must come back, the give-up must show in the error flags, the flags must stay
    set until cleared, and the device must go on working afterwards."""
    assert lq.check_device() == 0
    lq.selftest_bounded_wait()
    assert lq.check_device() == 8
    assert lq.check_device() == 8                      # sticky
    lq.clear_device_flags()
    assert lq.check_device() == 0
    wl = synth.Workload("after", 2, 2, 2, W=4, r=2, seed=990)
    _, sh = gu.shapes(wl)
    st = lq.State(sh)
    lq.quantize_state(sh, gu.dev(synth.dense_states(wl, 1)), st)
    o = torch.empty((2, 2, 128), dtype=torch.float32, device="cuda")
    td = gu.tok_dev(synth.token_inputs(wl, 0))
    lq.decode_step(sh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
    torch.cuda.synchronize()
    assert lq.check_device() == 0 and bool(torch.isfinite(o).all())


@pytest.mark.parametrize("gate", [synth.GATE_SCALAR, synth.GATE_DIAG])
@pytest.mark.parametrize("rec16", [0, 1])
def test_import_and_export_of_the_separate_array_form(oracle, gate, rec16):
    """A state built by the oracle (the paper's orientation: Z not transposed, one array per piece) is imported into
    the packed layout; decoding from it must give the oracle's outputs bit for bit, and exporting the result must
    give back the oracle's arrays."""
    from oracle.lq_oracle import State as OState
    wl = synth.Workload("imp", 3, 4, 2, W=8, r=4, gate=gate, rec16=rec16, seed=1200 + gate + 2 * rec16)
    osh, sh = gu.shapes(wl)
    ost = OState(osh)
    oracle.quantize_state(osh, synth.dense_states(wl, 4), ost)
    for step in range(5):                                        # five records in the buffer
        oracle.decode_step(osh, ost, **synth.token_inputs(wl, step))
    arr = lq.StateArrays(sh)
    for name in ("codes", "col_scale", "row_smooth", "buf_k", "buf_u", "buf_a", "win_pos"):
        getattr(arr, name).copy_(gu.dev(getattr(ost, name)))
    arr.comp_k.copy_(gu.dev(ost.comp_k).view(torch.float16)); arr.comp_u.copy_(gu.dev(ost.comp_u).view(torch.float16))
    st = lq.State(sh)
    lq.import_state(sh, arr, st)
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    for step in range(5, 5 + wl.W + 2):                          # through a boundary
        tok = synth.token_inputs(wl, step)
        td = gu.tok_dev(tok)
        want = oracle.decode_step(osh, ost, **tok)
        lq.decode_step(sh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        assert np.array_equal(gu.host(o), want), step
    out = lq.StateArrays(sh)
    lq.export_state(sh, st, out)
    torch.cuda.synchronize()
    n = int(ost.win_pos[0])
    assert np.array_equal(gu.host(out.codes), ost.codes) and np.array_equal(gu.host(out.win_pos), ost.win_pos)
    assert np.array_equal(gu.host(out.col_scale), ost.col_scale) and np.array_equal(gu.host(out.row_smooth), ost.row_smooth)
    assert np.array_equal(gu.host(out.comp_k), ost.comp_k) and np.array_equal(gu.host(out.comp_u), ost.comp_u)
    for name in ("buf_k", "buf_u", "buf_a"):                     # the live records
        assert np.array_equal(gu.host(getattr(out, name))[:, :, :n], getattr(ost, name)[:, :, :n]), name
