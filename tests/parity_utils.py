"""Helpers shared by the GPU parity tests: moving quantized tensors between the oracle's numpy
form and the library's device form, and the comparison rules for one step."""
import numpy as np
import torch

import oracle as O
from paper_2407_08296_b200 import binding as B


def to_device_q(q: O.QTensor, device="cuda") -> B.QTensor:
    rows, cols = q.codes.shape
    out = B.QTensor.empty(rows, cols, q.bits, device)
    if q.bits == 8:
        out.codes[:, :cols] = torch.from_numpy(q.codes).to(device)
    else:
        packed = O.pack_int4(q.codes)
        out.codes[:, :packed.shape[1]] = torch.from_numpy(packed).to(device)
    out.scales.copy_(torch.from_numpy(q.scales))
    out.zeros.copy_(torch.from_numpy(q.zeros))
    return out


def from_device_q(q: B.QTensor) -> O.QTensor:
    if q.bits == 8:
        codes = q.codes[:, :q.cols].cpu().numpy().astype(np.int8)
    else:
        codes = O.unpack_int4(q.codes.cpu().numpy(), q.cols)
    return O.QTensor(codes, q.scales.cpu().numpy(), q.zeros.cpu().numpy(), q.bits)


def g_to_device(g_bits: np.ndarray, device="cuda") -> torch.Tensor:
    m, n = g_bits.shape
    buf = B.zeros_matrix(m, n, torch.int16, device)
    buf.copy_(torch.from_numpy(g_bits.view(np.int16)).to(device))
    return buf


def f32_to_device(x: np.ndarray, device="cuda") -> torch.Tensor:
    buf = B.zeros_matrix(x.shape[0], x.shape[1], torch.float32, device)
    buf.copy_(torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device))
    return buf


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def check_moments(gpu, ref, name, tol=2e-3):
    """||gpu - oracle||_F <= tol ||oracle||_F and max|gpu - oracle| <= tol max|oracle|."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert np.all(np.isfinite(gpu)), f"{name}: non-finite values"
    assert rel_fro(gpu, ref) <= tol, f"{name}: relative Frobenius error {rel_fro(gpu, ref):.3e}"
    assert np.abs(gpu - ref).max() <= tol * max(np.abs(ref).max(), 1e-300), f"{name}: max error"


def check_direction(gpu, ref, name="N", tol=2e-3):
    """The Adam direction N = M^ / (sqrt(V^) + eps) is ill-conditioned where the projected gradient
    is within a few eps of zero (at t = 1 it is R / (|R| + eps)), so it is held to the Frobenius bound
    and to an element-wise bound on all but a vanishing fraction of the elements."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert np.all(np.isfinite(gpu)), f"{name}: non-finite values"
    assert rel_fro(gpu, ref) <= tol, f"{name}: relative Frobenius error {rel_fro(gpu, ref):.3e}"
    off = np.abs(gpu - ref) > tol * np.abs(ref).max()
    assert off.mean() <= 1e-4, f"{name}: {off.mean():.2e} of the elements off by more than {tol}"


def check_weight_codes(gpu_w: O.QTensor, out: dict, seed: int, step: int, max_frac=1e-3):
    """INT8 weights after one step against the oracle's.

    Scales agree to 1e-5 relative and zero points exactly wherever the group's scaled minimum is
    not at a rounding tie; codes agree except by exactly one level, in at most ``max_frac`` of the
    elements, and only where the oracle's scaled value T lies within 1e-3 of the element's
    rounding boundary (frac * 65536 within 65.536 of its Philox lane) or of the clamp edge.
    Returns the mismatch fraction.
    """
    ref_w = out["W"]
    m, n = ref_w.codes.shape
    assert np.allclose(gpu_w.scales, ref_w.scales, rtol=1e-5, atol=0), "W scales"
    zdiff = gpu_w.zeros != ref_w.zeros
    gcols = np.repeat(np.arange(ref_w.scales.shape[1]), 256)[:n]
    zd_el = zdiff[:, gcols]
    if zdiff.any():
        # a zero point may differ by one only when min * inv sits on a tie of rint
        assert np.all(np.abs(gpu_w.zeros - ref_w.zeros)[zdiff] == 1), "zero points differ by more than one"
        assert zdiff.mean() < 1e-3, "too many zero-point differences"
    diff = gpu_w.codes.astype(np.int32) - ref_w.codes.astype(np.int32)
    bad = (diff != 0) & ~zd_el
    frac_bad = bad.mean()
    assert np.all(np.abs(diff[bad]) == 1), "a weight code differs by more than one level"
    assert frac_bad <= max_frac, f"{frac_bad:.2e} of the weight codes differ"
    if bad.any():
        T = out["T"].astype(np.float64)
        h = O.sr_uniform16(seed, step, m, n).astype(np.float64)
        fr = (T - np.floor(T)) * 65536.0
        near_draw = np.abs(fr - h) <= 1e-3 * 65536 + 1
        near_int = (fr <= 1e-3 * 65536) | (fr >= (1 - 1e-3) * 65536)
        zeros_el = ref_w.zeros[:, gcols]
        lvl = np.floor(T) + zeros_el
        near_clamp = (lvl <= -128) | (lvl >= 126)
        ok = near_draw | near_int | near_clamp
        assert np.all(ok[bad]), f"{(bad & ~ok).sum()} code mismatches away from any rounding boundary"
    return float(frac_bad)
