"""CPU-side checks of the C boundary: the library loads, exports what the header declares,
rejects bad arguments before touching a device, and its host-only gate matches the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as O
from paper_2407_08296_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "qgalore.h")).read()
    return sorted(set(re.findall(r"QG_API[^;(]*?\b(qgalore_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert {"qgalore_quantize_int4", "qgalore_project_step", "qgalore_refresh_subspace",
            "qgalore_subspace_similarity"} <= set(names)
    L = B.lib()
    for n in names:
        assert hasattr(L, n), f"{n} is declared in qgalore.h but not exported"


def test_status_strings_and_workspace_query():
    L = B.lib()
    assert L.qgalore_status_string(0) == b"ok"
    assert L.qgalore_status_string(B.QG_MISALIGNED) == b"misaligned pointer or row pitch"
    ws = B.workspace_bytes(B.QG_OP_PROJECT_STEP, 2048, 5461, 512)
    assert ws >= 512 * 5461 * 2 and ws < (1 << 31)
    assert B.workspace_bytes(B.QG_OP_PROJECT_STEP, 0, 5, 5) == 0
    assert B.workspace_bytes(99, 5, 5, 5) == 0
    assert B.workspace_bytes(B.QG_OP_SIMILARITY, 4096, 0, 1024) >= (4096 // 32) * 1024 * 4


def test_bad_arguments_are_rejected_before_any_device_work():
    L = B.lib()
    q = B._CQTensor(0, 0, 0, 4, 256, 256, 8, 256)
    assert L.qgalore_quantize_int8(None, 4, 256, 256, C.byref(q), None) == B.QG_INVALID_ARGUMENT
    assert L.qgalore_quantize_int8(0x1000, 4, 256, 256, C.byref(q), None) == B.QG_INVALID_ARGUMENT  # null codes
    q = B._CQTensor(0x1000, 0x2000, 0x3000, 4, 256, 256, 8, 256)
    assert L.qgalore_quantize_int8(0x1000, 4, 256, 100, C.byref(q), None) == B.QG_INVALID_ARGUMENT  # ld < cols
    assert L.qgalore_quantize_int8(0x1004, 4, 256, 256, C.byref(q), None) == B.QG_MISALIGNED
    assert L.qgalore_quantize_int4(0x1000, 4, 256, 256, C.byref(q), None) == B.QG_INVALID_ARGUMENT  # bits mismatch
    q8 = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 512, 520, 8, 256)
    assert L.qgalore_dequantize(C.byref(q8), 0x4000, 512, None) == B.QG_MISALIGNED                  # ld % 16
    q128 = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 512, 512, 8, 128)
    assert L.qgalore_dequantize(C.byref(q128), 0x4000, 512, None) == B.QG_INVALID_ARGUMENT          # group != 256
    # project_step: shape and alignment rules
    P = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 32, 64, 4, 256)
    W = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 512, 512, 8, 256)
    h = B._CHyper(0.004, 0.25, 0.9, 0.999, 1e-8, 0.0, 1, 0)
    ws = B.workspace_bytes(B.QG_OP_PROJECT_STEP, 64, 512, 32)
    call = lambda **kw: L.qgalore_project_step(
        kw.get("G", 0x10000), kw.get("ldg", 512), 64, 512, kw.get("r", 32), C.byref(kw.get("P", P)), C.byref(W),
        0x20000, 0x30000, kw.get("ldmv", 512), C.byref(kw.get("h", h)), kw.get("ws", 0x40000), kw.get("wsb", ws),
        None, None, None)
    assert call(G=None) == B.QG_INVALID_ARGUMENT
    assert call(G=0x10002) == B.QG_MISALIGNED
    assert call(ldg=516) == B.QG_MISALIGNED
    assert call(ldmv=514) == B.QG_MISALIGNED
    assert call(wsb=ws - 1) == B.QG_WORKSPACE_TOO_SMALL
    assert call(ws=0x40010) == B.QG_MISALIGNED
    assert call(h=B._CHyper(0.004, 0.25, 0.9, 0.999, 1e-8, 0.0, 0, 0)) == B.QG_INVALID_ARGUMENT      # step 0
    P48 = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 48, 64, 4, 256)
    assert call(P=P48, r=48) == B.QG_UNSUPPORTED_SHAPE                                               # r % 32
    P96 = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 96, 128, 4, 256)
    assert call(P=P96, r=96) == B.QG_UNSUPPORTED_SHAPE                                               # r > m
    assert call(r=64) == B.QG_INVALID_ARGUMENT                                                       # P.cols != r
    # similarity
    A = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 32, 64, 4, 256)
    Bq = B._CQTensor(0x1000, 0x2000, 0x3000, 64, 64, 64, 4, 256)
    assert L.qgalore_subspace_similarity(C.byref(A), C.byref(Bq), 0, 0x5000, 0x6000, 1 << 20, None) == B.QG_INVALID_ARGUMENT
    assert L.qgalore_subspace_similarity(C.byref(A), C.byref(A), 0, 0x5000, 0x6000, 8, None) == B.QG_WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("k", [1, 2, 3])
def test_gate_matches_oracle_on_random_sequences(k):
    rng = np.random.default_rng(k)
    sims = rng.uniform(0.2, 0.7, size=200).astype(np.float32)
    sims[::17] = np.float32(0.4)                       # equality with the threshold counts as reached
    gate = B.Gate(interval=200, threshold=0.4, k=k)
    st = O.GateState(interval=200)
    for s in sims:
        if st.interval > (1 << 20):
            st, gate = O.GateState(interval=200), B.Gate(interval=200, threshold=0.4, k=k)
        want = O.gate_update(st, float(s), float(np.float32(0.4)), k)
        got = gate.update(float(s))
        assert got == want and gate.interval == st.interval


def test_gate_rejects_bad_arguments():
    L = B.lib()
    iv, cnt = C.c_int32(200), C.c_int32(0)
    hist = (C.c_float * 2)()
    assert L.qgalore_gate_update(0.5, 0.4, 0, C.byref(iv), hist, C.byref(cnt)) == B.QG_INVALID_ARGUMENT
    assert L.qgalore_gate_update(0.5, 0.4, 2, None, hist, C.byref(cnt)) == B.QG_INVALID_ARGUMENT
    cnt = C.c_int32(5)
    assert L.qgalore_gate_update(0.5, 0.4, 2, C.byref(iv), hist, C.byref(cnt)) == B.QG_INVALID_ARGUMENT


def test_both_similarity_entry_points_apply_the_same_pointer_rules():
    # host-only: nothing is dereferenced, every call is refused before a launch
    L = B.lib()
    small = lambda scales=0x2000, zeros=0x3000: B._CQTensor(0x1000, scales, zeros, 64, 256, 256, 4, 256)
    ok, bad_s, bad_z = small(), small(scales=0x2002), small(zeros=0x3001)
    for fn, extra in ((L.qgalore_subspace_similarity_static, ()), (L.qgalore_subspace_similarity, (0x8000, 1 << 20))):
        assert fn(C.byref(bad_s), C.byref(ok), 0, 0x4000, *extra, None) == B.QG_MISALIGNED
        assert fn(C.byref(ok), C.byref(bad_z), 0, 0x4000, *extra, None) == B.QG_MISALIGNED
        assert fn(C.byref(ok), C.byref(ok), 0, 0x4002, *extra, None) == B.QG_MISALIGNED
        assert fn(C.byref(ok), C.byref(small()), 0, None, *extra, None) == B.QG_INVALID_ARGUMENT


def test_wait_expiry_aid_validates_on_the_host():
    L = B.lib()
    assert L.qgalore_debug_expire_wait(0, 0x1000, None, None) == B.QG_INVALID_ARGUMENT
    assert L.qgalore_debug_expire_wait(8, None, None, None) == B.QG_INVALID_ARGUMENT
    assert L.qgalore_debug_expire_wait(8, 0x1002, None, None) == B.QG_MISALIGNED
