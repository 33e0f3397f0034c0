"""The similarity entry point for callers that cannot allocate device memory.

An optimizer hook inside a training framework, or a process whose device memory was parcelled out at
start-up, cannot hand the library a freshly allocated workspace.  qgalore_subspace_similarity_static keeps
its scratch in a fixed array inside the library; this file checks, through the C ABI, that it returns what
the workspace-taking entry point returns, twice in a row (the array keeps the previous call's contents),
and that it refuses shapes that do not fit the array.  Collected last on purpose."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle as O
from paper_2407_08296_b200 import binding as B
from paper_2407_08296_b200 import synth

from parity_utils import to_device_q

pytestmark = pytest.mark.gpu


def _pair(m, r, seed):
    base = synth.random_orthonormal(m, r, seed=seed, stream=1)
    rng = np.random.default_rng(seed)
    other = base + 0.5 * rng.standard_normal((m, r)).astype(np.float32) / np.sqrt(m)
    return O.quantize_rtn(base, 4), O.quantize_rtn(other.astype(np.float32), 4)


def test_static_similarity_matches_workspace_entry_point_twice_in_a_row():
    out_static = torch.full((1,), -7.0, dtype=torch.float32, device="cuda")   # allocated before the calls under test
    # a large case first, then a small one with fewer columns: the second call finds the first one's leftovers
    for (m, r, c, seed) in [(4096, 1024, 0, 1), (768, 256, 8, 2)]:
        A, Bq = _pair(m, r, seed)
        dA, dB = to_device_q(A), to_device_q(Bq)
        want = float(B.subspace_similarity(dA, dB, c).item())
        got = float(B.subspace_similarity_static(dA, dB, c, out=out_static).item())
        assert abs(got - want) <= 1e-6
        assert abs(got - O.subspace_similarity(A, Bq, c if c > 0 else None)) <= 1e-5   # the tolerance of the other tests
        again = float(B.subspace_similarity_static(dA, dB, c, out=out_static).item())
        assert again == got


def test_static_similarity_refuses_what_does_not_fit():
    L = B.lib()
    limit = int(L.qgalore_subspace_similarity_static_max_bytes())
    assert limit == 2 << 20
    rows, cols = 16384, 2048
    assert B.workspace_bytes(B.QG_OP_SIMILARITY, rows, 0, cols) > limit
    q = B._CQTensor(0x1000, 0x2000, 0x3000, rows, cols, cols, 4, 256)       # never dereferenced: rejected on the host
    assert L.qgalore_subspace_similarity_static(C.byref(q), C.byref(q), 0, 0x4000, None) == B.QG_WORKSPACE_TOO_SMALL
    assert L.qgalore_subspace_similarity_static(None, C.byref(q), 0, 0x4000, None) == B.QG_INVALID_ARGUMENT
    # the same pointer rules as the workspace-taking entry point, checked on the host: scales, zero points and the
    # result word are read and written as 4-byte words
    small = lambda scales=0x2000, zeros=0x3000: B._CQTensor(0x1000, scales, zeros, 64, 256, 256, 4, 256)
    ok, bad_s, bad_z = small(), small(scales=0x2002), small(zeros=0x3001)
    for fn, extra in ((L.qgalore_subspace_similarity_static, ()), (L.qgalore_subspace_similarity, (0x8000, 1 << 20))):
        assert fn(C.byref(bad_s), C.byref(ok), 0, 0x4000, *extra, None) == B.QG_MISALIGNED
        assert fn(C.byref(ok), C.byref(bad_z), 0, 0x4000, *extra, None) == B.QG_MISALIGNED
        assert fn(C.byref(ok), C.byref(ok), 0, 0x4002, *extra, None) == B.QG_MISALIGNED
