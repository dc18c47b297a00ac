"""CPU checks of the boundary: the shared library builds, loads, exports every symbol the header declares,
and rejects bad arguments before anything is launched (no GPU is touched)."""
import ctypes as C
import os
import re

import pytest

from paper_2609_38166_b200 import build, lq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return lq.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "lq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(lq_[a-z0-9_]+)\s*\(", header)))
    assert declared == sorted(lq.EXPORTS)
    for name in declared:
        assert getattr(L, name) is not None


def test_version_and_status_strings(L):
    assert lq.version() >= 1
    texts = [L.lq_status_string(i).decode() for i in range(7)]
    assert texts[0] == "ok" and len(set(texts)) == 7 and "unknown" not in texts
    assert L.lq_status_string(7).decode() == "unknown status"
    assert lq.static_stage_bytes() == lq.STATIC_STAGE_BYTES      # the binding's constant is the library's


def test_argument_errors_are_reported_before_any_launch(L):
    sh = lq.Shape(2, 4, 2)
    s = sh.c()
    null = C.c_void_p(None)
    st = lq._State(*([None] * 5))
    # null shape / null state / null pointers inside the state
    assert L.lq_decode_step(null, C.byref(st), null, null, null, null, null, null, null) == 1
    assert L.lq_decode_step(C.byref(s), null, null, null, null, null, null, null, null) == 1
    assert L.lq_decode_step(C.byref(s), C.byref(st), null, null, null, null, null, null, null) == 1
    assert L.lq_window_flush(C.byref(s), C.byref(st), 0, null) == 1
    assert L.lq_quantize_state(C.byref(s), null, C.byref(st), null) == 1
    assert L.lq_dequantize_state(C.byref(s), C.byref(st), null, null) == 1
    assert L.lq_ref_decode_step_f32(C.byref(s), null, null, null, null, null, null, null, null) == 1
    # shapes: inconsistent -> SHAPE, valid but outside the fast path -> UNSUPPORTED
    for bad in (lq.Shape(2, 4, 3), lq.Shape(2, 0, 1), lq.Shape(-1, 4, 2), lq.Shape(2, 4, 2, W=0),
                lq.Shape(2, 4, 2, n_iter=0), lq.Shape(2, 4, 2, gate=7)):
        b = bad.c()
        assert L.lq_window_flush(C.byref(b), C.byref(st), 0, null) == 2, bad
    for uns in (lq.Shape(2, 4, 2, d_k=64), lq.Shape(2, 4, 2, d_v=256), lq.Shape(2, 4, 2, W=65),
                lq.Shape(2, 4, 2, r=17)):
        u = uns.c()
        assert L.lq_window_flush(C.byref(u), C.byref(st), 0, null) == 4, uns
        assert L.lq_decode_stage_bytes(C.byref(u)) == 0 and L.lq_head_bytes(C.byref(u)) == 0
    # misaligned pointer (fake non-null addresses: nothing is dereferenced on the host)
    fake = [0x1000 * (i + 1) for i in range(4)]
    st_ok = lq._State(*fake)
    fake[0] += 8
    st_bad = lq._State(*fake)
    assert L.lq_quantize_state(C.byref(s), C.c_void_p(0x100000), C.byref(st_bad), null) == 3
    assert L.lq_quantize_state(C.byref(s), C.c_void_p(0x100004), C.byref(st_ok), null) == 3
    # the optional scratch words: null is fine (checked above), a pointer that is not 4-byte aligned is not
    st_w = lq._State(*[0x1000 * (i + 1) for i in range(4)], 0x5002)
    assert L.lq_quantize_state(C.byref(s), C.c_void_p(0x100000), C.byref(st_w), null) == 3
    # the host-buffer entry points check the state as well before they enqueue anything (fake host / stage pointers)
    hp = C.c_void_p(0x200000)
    assert L.lq_decode_step_host(C.byref(s), null, hp, hp, hp, hp, hp, hp, hp, null) == 1
    assert L.lq_decode_step_host(C.byref(s), C.byref(st), hp, hp, hp, hp, hp, hp, hp, null) == 1
    assert L.lq_decode_step_host(C.byref(s), C.byref(st_bad), hp, hp, hp, hp, hp, hp, hp, null) == 3
    assert L.lq_decode_step_host_static(C.byref(s), C.byref(st), hp, hp, hp, hp, hp, hp, null) == 1
    assert L.lq_decode_step_host_static(C.byref(s), C.byref(st_bad), hp, hp, hp, hp, hp, hp, null) == 3
    # import / export of the separate-array form: null struct, null arrays, a state with a misaligned pointer
    arr = lq._StateArrays(*([None] * 9))
    assert L.lq_import_state(C.byref(s), null, C.byref(st_ok), null) == 1
    assert L.lq_import_state(C.byref(s), C.byref(arr), C.byref(st_ok), null) == 1
    assert L.lq_export_state(C.byref(s), C.byref(st_bad), C.byref(arr), null) == 3
    w16 = lq.Shape(2, 4, 2, r=0, smooth=0, state_bf16=1).c()
    assert L.lq_import_state(C.byref(w16), C.byref(arr), C.byref(st_ok), null) == 4
    big = lq.Shape(64, 32, 16).c()                                # (the pipelined path proper starts at 16 sequences)
    assert L.lq_decode_step_host_pipelined(C.byref(big), C.byref(st_bad), hp, hp, hp, hp, hp, hp, hp, null) == 3
    assert lq.decode_stage_bytes(sh) > 0 and lq.decode_launches(sh) >= 1
    assert lq.head_bytes(sh) == 19456 and lq.record_floats(sh) == 256
    assert lq.record_floats(lq.Shape(2, 4, 2, gate=lq.GATE_DIAG)) == 384


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(lq, "_lib", None)
    monkeypatch.setattr(lq, "_LIB_PATH", "/nonexistent/liblq.so")
    with pytest.raises(lq.LqError):
        lq.lib()
