"""The host-buffer decode step that allocates nothing (lq_decode_step_host_static).

Some users of this library cannot allocate device memory at the time they decode: a serving process that
handed the whole device to its own memory pools at start-up has nothing left for cudaMalloc, and a decode
loop that must not stall cannot call cudaMalloc or cudaFree, which may synchronise the device.  For them the
library keeps the staging area of the host-buffer path in a fixed device array of its own.  The test drives
that entry point through the C boundary next to the ordinary host-buffer entry point (which is given a
torch-allocated staging buffer) on identical states and tokens, two calls in a row, and demands the same
results: the second call proves that what the first call left in the shared array does no harm.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2609_38166_b200 import build, lq, synth

pytestmark = pytest.mark.gpu


def _pinned(tok):
    return {k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in tok.items()}


@pytest.mark.parametrize("gate", [synth.GATE_SCALAR, synth.GATE_DIAG])
def test_static_staging_matches_caller_staging_on_two_calls(gate):
    build.build()
    wl = synth.Workload("noalloc", 5, 4, 2, W=4, r=2, gate=gate, seed=900)
    sh = lq.Shape(wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth)
    S0 = torch.from_numpy(synth.dense_states(wl, 1)).cuda()
    st_a, st_b = lq.State(sh), lq.State(sh)
    lq.quantize_state(sh, S0, st_a)
    lq.quantize_state(sh, S0, st_b)
    # sequence 3 enters with a full window: it gets no token, and its output rows must come back as zeros
    # from the built-in staging (the ordinary entry point leaves whatever its staging buffer held there)
    st_a.win_pos[3] = wl.W
    st_b.win_pos[3] = wl.W
    stage = torch.zeros((lq.decode_stage_bytes(sh),), dtype=torch.uint8, device="cuda")
    o_a = torch.empty((wl.batch, wl.heads_v, wl.d_v), dtype=torch.float32).pin_memory()
    o_b = torch.empty_like(o_a).pin_memory()
    for call in range(2):
        tok = _pinned(synth.token_inputs(wl, call))
        o_a.fill_(-1.0); o_b.fill_(-2.0)
        lq.decode_step_host(sh, st_a, tok["q"], tok["k"], tok["v"], tok["beta"], tok["alpha"], o_a, stage)
        torch.cuda.synchronize()
        free_before, used_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        lq.decode_step_host_static(sh, st_b, tok["q"], tok["k"], tok["v"], tok["beta"], tok["alpha"], o_b)
        torch.cuda.synchronize()
        if call == 1:        # (the first call may load the module and look the array's address up; the second must not
            #                   take or return a byte of device memory, through the driver or through torch)
            assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == used_before
        assert np.allclose(o_b.numpy(), o_a.numpy(), rtol=1e-3, atol=1e-5), call
        assert np.array_equal(o_b.numpy(), o_a.numpy()), call        # same kernels, same bits
        assert call == 1 or not np.any(o_b.numpy()[3])               # cleared rows of the skipped sequence
        for ta, tb in zip(st_a.tensors(), st_b.tensors()):
            assert torch.equal(ta, tb), call
    assert lq.check_device() == 0


def test_requests_beyond_the_built_in_buffer_are_refused():
    build.build()
    L = lq.lib()
    big = lq.Shape(1024, 32, 16)                      # needs about 33 MB of staging
    assert lq.decode_stage_bytes(big) > lq.STATIC_STAGE_BYTES
    s = big.c()
    fake_state = lq._State(0x1000, 0x2000, 0x3000, 0x4000)
    p = C.c_void_p(0x10000)
    rc = L.lq_decode_step_host_static(C.byref(s), C.byref(fake_state), p, p, p, p, p, p, None)
    assert rc == 6 and b"scratch" in L.lq_status_string(rc)
    ok = lq.Shape(256, 32, 16)                        # the benchmark batch fits
    assert lq.decode_stage_bytes(ok) <= lq.STATIC_STAGE_BYTES
