"""Helpers of the GPU parity tests: move seeded inputs and oracle states to the device and compare."""
import numpy as np
import torch

from oracle.lq_oracle import Shape as OShape, State as OState
from paper_2609_38166_b200 import lq, synth


def shapes(wl):
    """(oracle shape, library shape) of a workload."""
    args = (wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth, wl.delta, wl.rec16, wl.state_bf16)
    return OShape(*args), lq.Shape(*args)


def dev(a: np.ndarray) -> torch.Tensor:
    """numpy -> cuda tensor; 16-bit patterns travel as int16."""
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    a = t.detach().cpu().contiguous()
    if a.dtype == torch.float16:
        return a.view(torch.int16).numpy().view(np.uint16)
    if a.dtype == torch.int16:
        return a.numpy().view(np.uint16)
    return a.numpy()


def host_f32(t: torch.Tensor) -> np.ndarray:
    """values as fp32 (record buffers may be fp16 tensors)"""
    return t.detach().float().cpu().contiguous().numpy()


def tok_dev(tok: dict) -> dict:
    return {k: dev(v) for k, v in tok.items()}


def state_to_dev(ost: OState, lsh, work: bool = True) -> "lq.State":
    st = lq.State(lsh, work=work)
    if lsh.state_bf16:
        st.state16.copy_(dev(np.ascontiguousarray(ost.S0.transpose(0, 1, 3, 2))).to(torch.bfloat16))   # exact: bfloat16 values
        st.buf_k.copy_(dev(ost.buf_k)); st.buf_u.copy_(dev(ost.buf_u)); st.buf_a.copy_(dev(ost.buf_a))
        st.win_pos.copy_(dev(ost.win_pos))
        return st
    st.codes.copy_(dev(np.ascontiguousarray(ost.codes.transpose(0, 1, 3, 2)))); st.col_scale.copy_(dev(ost.col_scale)); st.row_smooth.copy_(dev(ost.row_smooth))
    if lsh.r > 0:
        st.comp_k.copy_(dev(ost.comp_k).view(torch.float16)); st.comp_u.copy_(dev(ost.comp_u).view(torch.float16))
    st.buf_k.copy_(dev(ost.buf_k)); st.buf_u.copy_(dev(ost.buf_u)); st.buf_a.copy_(dev(ost.buf_a))
    st.win_pos.copy_(dev(ost.win_pos))
    return st


def gpu_codes(st) -> np.ndarray:
    """the library keeps Z^T ([B,Hv,d_v,d_k]); returns Z as [B,Hv,d_k,d_v] like the oracle"""
    return np.ascontiguousarray(host(st.codes).transpose(0, 1, 3, 2))


def code_mismatch(gpu_codes: np.ndarray, ref_codes: np.ndarray):
    """(fraction of entries that differ, largest difference in code steps)"""
    d = np.abs(gpu_codes.astype(np.int32) - ref_codes.astype(np.int32))
    return float((d > 0).mean()), int(d.max(initial=0))


def assert_state_parity(st: "lq.State", ost: OState, r: int, what: str = "", exact: bool = True):
    """The bar: 8-bit codes bit-exact except <= 1 code step on <= 0.01 % of the entries; floating-point arrays
    within 1e-3 relative / 1e-5 absolute.  With `exact` (the default) every array must match bit for bit,
    which the fixed summation order makes possible."""
    torch.cuda.synchronize()
    if st.shape.state_bf16:                  # per-window BF16: the boundary state is S0^T in bfloat16
        got = np.ascontiguousarray(st.state16.float().cpu().numpy().transpose(0, 1, 3, 2))
        if exact:
            assert np.array_equal(got, ost.S0), (what, "state16", float(np.abs(got - ost.S0).max()))
        else:
            assert np.allclose(got, ost.S0, rtol=2.0 ** -7, atol=1e-5), (what, "state16")
        for name, g, w in (("buf_k", host_f32(st.buf_k), ost.buf_k), ("buf_u", host_f32(st.buf_u), ost.buf_u),
                           ("buf_a", host_f32(st.buf_a), ost.buf_a)):
            assert np.allclose(g, w, rtol=1e-3, atol=1e-5), (what, name)
            assert not exact or np.array_equal(g, w), (what, name, float(np.abs(g - w).max()))
        assert np.array_equal(host(st.win_pos), ost.win_pos), (what, host(st.win_pos), ost.win_pos)
        return
    frac, worst = code_mismatch(gpu_codes(st), ost.codes)
    assert worst <= 1 and frac <= 1e-4, (what, frac, worst)
    pairs = [("col_scale", host(st.col_scale), ost.col_scale), ("row_smooth", host(st.row_smooth), ost.row_smooth),
             ("buf_k", host_f32(st.buf_k), ost.buf_k), ("buf_u", host_f32(st.buf_u), ost.buf_u),
             ("buf_a", host_f32(st.buf_a), ost.buf_a)]
    if r > 0:
        pairs += [("comp_k", host(st.comp_k).view(np.float16).astype(np.float32), ost.comp_k_f32()),
                  ("comp_u", host(st.comp_u).view(np.float16).astype(np.float32), ost.comp_u_f32())]
    for name, got, want in pairs:
        assert np.allclose(got, want, rtol=1e-3, atol=1e-5), (what, name)
    assert np.array_equal(host(st.win_pos), ost.win_pos), (what, host(st.win_pos), ost.win_pos)
    if exact:
        assert frac == 0.0, (what, "codes", frac)
        for name, got, want in pairs:
            assert np.array_equal(got, want), (what, name, float(np.abs(got - want).max()))
