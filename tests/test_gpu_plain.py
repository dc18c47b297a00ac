"""GPU against the PLAIN definition: the oracle build whose sums run left to right in binary64 and whose
readout is Eq. 10 as written, with no fixed-point grid and no summation tree.

The other GPU tests demand bit equality with the defining oracle build, which fixes a summation order.  These
tests measure instead what the stated tolerance allows: 8-bit codes equal except one code step on at most
0.01 % of the entries, outputs, records, scales and dequantized states within 1e-3 relative / 1e-5 absolute.
Every token starts from the same state on both sides (the state of the defining build, which the GPU is at bit
for bit), so that a difference is the difference of ONE step and does not compound.  A boundary rounds the
compensators to fp16; where the two sides round one of those 1024 values to different neighbours the residual
that is coded differs along a whole row or column, so heads are counted in two groups: compensators identical
(the code bar applies) and compensators flipped (reported; their dequantized state must still agree to within
one code step)."""
import json
import os

import numpy as np
import pytest
import torch

import bench
from oracle.lq_oracle import Shape as OShape, State as OState
from paper_2609_38166_b200 import lq, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-3, 1e-5
FIELDS = ("codes", "col_scale", "row_smooth", "comp_k", "comp_u", "buf_k", "buf_u", "buf_a", "win_pos")


def _copy(ost, osh):
    c = OState(osh)
    for f in FIELDS:
        getattr(c, f)[...] = getattr(ost, f)
    return c


class Tally:
    """Counts over all boundaries seen by one test."""

    def __init__(self):
        self.same = self.flipped = 0
        self.entries = self.diff = self.worst = 0
        self.flipped_entries = self.flipped_diff = 0
        self.flipped_values = 0

    def boundary(self, g_codes, g_scale, g_smooth, g_ck, g_cu, g_dense, p_codes, p_scale, p_smooth, p_ck, p_cu, p_dense, where):
        """One head right after its boundary: g_* from the GPU, p_* from the plain oracle (fp16 as bit patterns)."""
        d = np.abs(g_codes.astype(np.int32) - p_codes.astype(np.int32))
        step = p_smooth.astype(np.float64)[:, None] * p_scale.astype(np.float64)[None, :]     # one code step, per entry
        flips = int((g_ck != p_ck).sum() + (g_cu != p_cu).sum())
        if flips == 0:
            self.same += 1
            self.entries += d.size
            self.diff += int((d > 0).sum())
            self.worst = max(self.worst, int(d.max(initial=0)))
            assert d.max(initial=0) <= 1, (where, int(d.max()))
            assert np.allclose(g_scale, p_scale, rtol=RTOL, atol=ATOL), (where, "col_scale")
            assert np.allclose(g_smooth, p_smooth, rtol=RTOL, atol=ATOL), (where, "row_smooth")
            slack = d * step
        else:
            self.flipped += 1
            self.flipped_values += flips
            self.flipped_entries += d.size
            self.flipped_diff += int((d > 0).sum())
            # the two sets of tokens are still the same fit: a flipped key entry moves its token's value side by
            # about an fp16 rounding of that token's largest entry, not more
            for g, q in ((g_ck, p_ck), (g_cu, p_cu)):
                gf, qf = g.view(np.float16).astype(np.float64), q.view(np.float16).astype(np.float64)
                lim = 2.0 ** -9 * np.abs(qf).max(axis=1, keepdims=True) + 2.0 ** -24
                assert np.all(np.abs(gf - qf) <= lim), (where, "compensator", float(np.abs(gf - qf).max()))
            slack = 1.0 * step                # both states are within half a step of the same dense state
        lim = RTOL * np.abs(p_dense) + ATOL + slack * (1 + 1e-3)
        assert np.all(np.abs(g_dense.astype(np.float64) - p_dense) <= lim), (where, "dequantized state")

    def report(self, name):
        row = {"case": name, "heads_through_a_boundary": self.same + self.flipped, "compensators_identical": self.same,
               "compensators_flipped": self.flipped, "flipped_fp16_values": self.flipped_values,
               "code_entries_compared": self.entries, "code_entries_differing": self.diff,
               "code_mismatch_fraction": self.diff / max(self.entries, 1), "worst_code_difference": self.worst,
               "code_mismatch_fraction_in_flipped_heads": self.flipped_diff / max(self.flipped_entries, 1)}
        print("plain-definition parity:", json.dumps(row))
        report = os.environ.get("LQ_PARITY_REPORT")          # optional: a file to append the rows to
        if report:
            with open(report, "a") as f:
                f.write(json.dumps(row) + "\n")
        assert self.same > 0, "no head with identical compensators: nothing was measured"
        assert self.diff <= 1e-4 * self.entries, row
        assert self.worst <= 1, row


def _dense(oracle_any, osh, ost):
    return oracle_any.dequantize_state(osh, ost)


def _teacher_forced_chain(oracle, oracle_plain, wl, steps, name, init="dense", stagger=True):
    osh, lsh = gu.shapes(wl)
    ost = OState(osh)
    S0 = np.zeros((wl.batch, wl.heads_v, 128, 128), np.float32) if init == "zero" else synth.dense_states(wl, 9)
    oracle.quantize_state(osh, S0, ost)
    if stagger:
        ost.win_pos[:] = (np.arange(wl.batch) * wl.W // max(wl.batch, 1)).astype(np.int32) % wl.W
        ost.buf_a[...] = 1.0
    tally = Tally()
    o = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    for step in range(steps):
        tok = synth.token_inputs(wl, step)
        td = gu.tok_dev(tok)
        st = gu.state_to_dev(ost, lsh)                      # both sides start the token from the same state
        pst = _copy(ost, osh)
        n_before = ost.win_pos.copy()
        lq.decode_step(lsh, st, td["q"], td["k"], td["v"], td["beta"], td["alpha"], o)
        o_plain = oracle_plain.decode_step(osh, pst, **tok)
        want = oracle.decode_step(osh, ost, **tok)          # the defining build moves on (and the GPU is at it)
        got = gu.host(o)
        assert np.array_equal(got, want), ("the GPU left the defining build", step)
        assert np.allclose(got, o_plain, rtol=RTOL, atol=ATOL), ("o", step)
        assert np.array_equal(gu.host(st.win_pos), pst.win_pos)
        bu, bk = gu.host_f32(st.buf_u), gu.host_f32(st.buf_k)
        flushed = [b for b in range(wl.batch) if n_before[b] + 1 == wl.W]
        for b in range(wl.batch):
            if b in flushed:
                continue
            n = int(n_before[b])
            assert np.allclose(bu[b, :, n], pst.buf_u[b, :, n], rtol=RTOL, atol=ATOL), ("record u", step, b)
            assert np.array_equal(bk[b, :, n], pst.buf_k[b, :, n]), ("record key", step, b)
        if flushed:
            S_gpu = torch.empty((wl.batch, wl.heads_v, 128, 128), dtype=torch.float32, device="cuda")
            lq.dequantize_state(lsh, st, S_gpu)
            S_gpu = gu.host(S_gpu)
            S_plain = _dense(oracle_plain, osh, pst).astype(np.float64)
            codes = gu.gpu_codes(st)
            cs, rs = gu.host(st.col_scale), gu.host(st.row_smooth)
            ck, cu = gu.host(st.comp_k), gu.host(st.comp_u)
            for b in flushed:
                for h in range(wl.heads_v):
                    tally.boundary(codes[b, h], cs[b, h], rs[b, h], ck[b, h], cu[b, h], S_gpu[b, h],
                                   pst.codes[b, h], pst.col_scale[b, h], pst.row_smooth[b, h], pst.comp_k[b, h],
                                   pst.comp_u[b, h], S_plain[b, h], (name, step, b, h))
    tally.report(name)


def test_config1_single_head_against_the_plain_definition(oracle, oracle_plain):
    _teacher_forced_chain(oracle, oracle_plain, synth.config("single_gdn"), 64, "single_gdn", init="zero", stagger=False)


@pytest.mark.parametrize("gate,name", [(synth.GATE_SCALAR, "gdn staggered, 12 x 8 heads"),
                                       (synth.GATE_DIAG, "kda outliers staggered, 12 x 8 heads")])
def test_staggered_chain_against_the_plain_definition(oracle, oracle_plain, gate, name):
    if gate == synth.GATE_DIAG:
        wl = synth.config("kda_b128_outlier").with_(batch=12, heads_v=8, heads_qk=8)
    else:
        wl = synth.config("gdn_b256").with_(batch=12, heads_v=8, heads_qk=4)
    _teacher_forced_chain(oracle, oracle_plain, wl, 2 * wl.W + 3, name)


@pytest.mark.parametrize("name,warm,steps", [("gdn_b256", 24, 34), ("kda_b128_outlier", 20, 34)])
def test_full_batch_sampled_sequences_against_the_plain_definition(oracle, oracle_plain, name, warm, steps):
    """The benchmark's batch and launch configuration on the GPU; for sampled sequences the defining build
    retraces the GPU (bit for bit, asserted), and before every token the plain build is started from that state."""
    wl = synth.config(name)
    toks = [synth.token_inputs(wl, t) for t in range(warm + steps)]
    sh, st, o = bench.prepare_state(wl, lq, torch, lambda m: None, warm)
    sample = sorted({0, wl.batch // wl.W + 1, wl.batch // 2 + 3, wl.batch - 1})
    per = max(wl.batch // wl.W, 1)
    groups = (wl.batch + per - 1) // per
    osh = OShape(1, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth, wl.delta,
                 wl.rec16, wl.state_bf16)
    # the defining build up to the first timed token
    states = {}
    for b in sample:
        g = min(b // per, groups - 1)
        cut = lambda tok: {k: np.ascontiguousarray(v[b:b + 1]) for k, v in tok.items()}
        S = np.zeros((1, wl.heads_v, wl.d_k, wl.d_v), np.float32)
        ost = OState(osh)
        for t in range(warm):
            if t == warm - g:
                oracle.quantize_state(osh, S, ost)
            if t < warm - g:
                oracle.ref_step_f32(osh, S, **cut(toks[t]))
            else:
                oracle.decode_step(osh, ost, **cut(toks[t]))
        if g == 0:
            oracle.quantize_state(osh, S, ost)
        states[b] = ost
    tally = Tally()
    S_gpu = torch.empty((len(sample), wl.heads_v, 128, 128), dtype=torch.float32, device="cuda")
    for t in range(steps):
        d = bench.to_dev(toks[warm + t], torch)
        lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o)
        oh = o[sample].cpu().numpy()
        for i, b in enumerate(sample):
            tok = {k: np.ascontiguousarray(v[b:b + 1]) for k, v in toks[warm + t].items()}
            ost = states[b]
            pst = _copy(ost, osh)
            n = int(ost.win_pos[0])
            o_plain = oracle_plain.decode_step(osh, pst, **tok)
            want = oracle.decode_step(osh, ost, **tok)
            assert np.array_equal(oh[i], want[0]), ("the GPU left the defining build", b, t)
            assert np.allclose(oh[i], o_plain[0], rtol=RTOL, atol=ATOL), ("o", b, t)
            if n + 1 < wl.W:
                assert np.allclose(gu.host_f32(st.buf_u[b, :, n]), pst.buf_u[0, :, n], rtol=RTOL, atol=ATOL), ("record u", b, t)
                continue
            lq.dequantize_state(sh, st, S_gpu[i:i + 1], b0=b, nb=1)
            Sg = gu.host(S_gpu[i])
            Sp = oracle_plain.dequantize_state(osh, pst)[0].astype(np.float64)
            codes = np.ascontiguousarray(gu.host(st.codes[b]).transpose(0, 2, 1))
            cs, rs = gu.host(st.col_scale[b]), gu.host(st.row_smooth[b])
            ck, cu = gu.host(st.comp_k[b]), gu.host(st.comp_u[b])
            for h in range(wl.heads_v):
                tally.boundary(codes[h], cs[h], rs[h], ck[h], cu[h], Sg[h], pst.codes[0, h], pst.col_scale[0, h],
                               pst.row_smooth[0, h], pst.comp_k[0, h], pst.comp_u[0, h], Sp[h], (name, t, b, h))
    torch.cuda.synchronize()
    assert lq.check_device() == 0
    tally.report(name + " (full batch, sampled sequences)")
