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
        packed = O.pack_int4(q.codes) if q.bits == 4 else O.pack_int2(q.codes)
        out.codes[:, :packed.shape[1]] = torch.from_numpy(packed).to(device)
    out.scales.copy_(torch.from_numpy(q.scales))
    out.zeros.copy_(torch.from_numpy(q.zeros))
    return out


def from_device_q(q: B.QTensor) -> O.QTensor:
    if q.bits == 8:
        codes = q.codes[:, :q.cols].cpu().numpy().astype(np.int8)
    elif q.bits == 4:
        codes = O.unpack_int4(q.codes.cpu().numpy(), q.cols)
    else:
        codes = O.unpack_int2(q.codes.cpu().numpy(), q.cols)
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


def ill_conditioned(ref: dict, hyp) -> np.ndarray:
    """Elements of the low-rank state where the Adam direction N = M^ / (sqrt(V^) + eps) is
    ill-conditioned: sqrt(V^) within a factor 1000 of eps.  There a rounding difference dR of the
    projected gradient moves N by up to eps * dR / (sqrt(V^) + eps)^2, i.e. by O(1) when |R| ~ eps
    (at t = 1, N = R / (|R| + eps)).  Elsewhere dN <= 1e-6 * dR / eps is far below the tolerance."""
    _, _, _, b2, eps, _ = hyp.as_f32()
    v_hat = ref["V"].astype(np.float64) / (1.0 - b2 ** int(hyp.step))
    return np.sqrt(v_hat) < 1e3 * eps


def check_direction(gpu, ref, hyp, name="N", tol=2e-3):
    """N against the oracle: Frobenius bound on the whole matrix, element-wise bound wherever the
    direction is well conditioned; the ill-conditioned elements must be rare and of ordinary size."""
    gpu = np.asarray(gpu, dtype=np.float64)
    want = np.asarray(ref["N"], dtype=np.float64)
    assert np.all(np.isfinite(gpu)), f"{name}: non-finite values"
    ill = ill_conditioned(ref, hyp)
    assert ill.mean() <= 2e-2, f"{name}: {ill.mean():.2e} of the elements are ill-conditioned"
    good = ~ill
    err = np.abs(gpu - want)
    assert np.linalg.norm(err[good]) <= tol * np.linalg.norm(want[good]), f"{name}: relative Frobenius error"
    assert err[good].max() <= tol * np.abs(want).max(), f"{name}: max error {err[good].max():.3e}"
    assert np.abs(gpu).max() <= 10.0 * max(np.abs(want).max(), 1.0), f"{name}: out of range"
    return float(ill.mean())


def check_weight_codes(gpu_w: O.QTensor, out: dict, seed: int, step: int, max_frac=1e-3, col0=0, rounding="sr"):
    """INT8 weights after one step against the oracle's (same direction N_b on both sides).

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
        fr = (T - np.floor(T)) * 65536.0
        if rounding == "rtn":                                  # the boundary of round-to-nearest is the half
            near_draw = np.abs(fr - 32768.0) <= 1e-3 * 65536
        else:
            h = O.sr_uniform16(seed, step, m, n, col0=col0).astype(np.float64)
            near_draw = np.abs(fr - h) <= 1e-3 * 65536 + 1
        near_int = (fr <= 1e-3 * 65536) | (fr >= (1 - 1e-3) * 65536)
        zeros_el = ref_w.zeros[:, gcols]
        lvl = np.floor(T) + zeros_el
        near_clamp = (lvl <= -128) | (lvl >= 126)
        ok = near_draw | near_int | near_clamp
        assert np.all(ok[bad]), f"{(bad & ~ok).sum()} code mismatches away from any rounding boundary"
    return float(frac_bad)


def check_weight_codes_unforced(gpu_w: O.QTensor, ref: dict, max_frac=5e-3):
    """End-to-end sanity bound with the oracle's own direction: a handful of ill-conditioned N
    elements shift whole columns of W' by a few 1e-3 LSB, so codes may differ by one level in
    slightly more places than with the direction forced; never by more than one level."""
    ref_w = ref["W"]
    assert np.allclose(gpu_w.scales, ref_w.scales, rtol=1e-3, atol=0), "W scales (unforced)"
    diff = np.abs(gpu_w.codes.astype(np.int32) - ref_w.codes.astype(np.int32))
    n = ref_w.codes.shape[1]
    gcols = np.repeat(np.arange(ref_w.scales.shape[1]), 256)[:n]
    same_zero = (gpu_w.zeros == ref_w.zeros)[:, gcols]
    assert diff[same_zero].max(initial=0) <= 1, "a weight code differs by more than one level (unforced)"
    frac = float((diff[same_zero] != 0).mean()) if same_zero.any() else 0.0
    assert frac <= max_frac, f"{frac:.2e} of the weight codes differ (unforced)"
    return frac


class StepTaps:
    """Device buffers for the optional intermediates of qgalore_project_step."""

    def __init__(self, m, n, r, w_ld, side="left"):
        sc = m if side == "right" else n                # columns of the low-rank state
        self.R = B.zeros_matrix(r, sc, torch.float32)
        self.N = B.zeros_matrix(r, sc, torch.float32)
        self.W_pre = torch.zeros((m, w_ld), dtype=torch.float32, device="cuda")[:, :n]

    def as_dict(self):
        return {"R": self.R, "N": self.N, "W_pre": self.W_pre}


def run_and_check_step(gb, P: O.QTensor, W: O.QTensor, M, V, hyp: O.Hyper, tol=2e-3, impl=None, side="left"):
    """Teacher-forced single-step parity of qgalore_project_step against the oracle.

    Stage 1 (steps 1-4): M', V', R and the direction N against the oracle's own.
    Stage 2 (steps 5-6): the oracle recomputes the weight update from the GPU's bf16 direction, and
    W', scales, zero points and codes are held to the strict rule of check_weight_codes.
    Plus the looser end-to-end bound against the oracle's unforced result.  Returns a dict of statistics.
    """
    m, n = gb.shape
    r = P.codes.shape[1]
    ref = O.project_step(gb, P, W, M, V, hyp, side=side)
    dG, dP, dW = g_to_device(gb), to_device_q(P), to_device_q(W)
    dM, dV = f32_to_device(M), f32_to_device(V)
    taps = StepTaps(m, n, r, dW.ld, side)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if impl is not None:
        B.debug_set_step_impl(impl)
    try:
        B.project_step(dG, dP, dW, dM, dV,
                       B.Hyper(lr=hyp.lr, alpha=hyp.alpha, beta1=hyp.beta1, beta2=hyp.beta2, eps=hyp.eps,
                               weight_decay=hyp.weight_decay, step=hyp.step, seed=hyp.seed,
                               rounding=B.QG_ROUND_NEAREST if hyp.rounding == "rtn" else B.QG_ROUND_STOCHASTIC),
                       status=status, debug=taps.as_dict(), side=side)
        torch.cuda.synchronize()
    finally:
        if impl is not None:
            B.debug_set_step_impl(0)
    assert int(status.item()) == 0, "device status word"
    # stage 1
    check_moments(dM.cpu().numpy(), ref["M"], "M", tol)
    check_moments(dV.cpu().numpy(), ref["V"], "V", tol)
    check_moments(taps.R.cpu().numpy(), ref["R32"], "R", tol)
    n_gpu = taps.N.cpu().numpy()
    ill = check_direction(n_gpu, ref, hyp, "N", tol)
    # stage 2: same direction on both sides
    forced = O.project_step(gb, P, W, M, V, hyp, N_b_override=O.bf16_round(n_gpu), side=side)
    lsb = np.repeat(forced["W"].scales, 256, axis=1)[:, :n]
    wpre_err = float((np.abs(taps.W_pre.cpu().numpy() - forced["W_pre"]) / lsb).max())
    assert wpre_err <= 1e-3, f"pre-rounding weight off by {wpre_err:.2e} LSB"
    gw = from_device_q(dW)
    frac = check_weight_codes(gw, forced, hyp.seed, hyp.step, rounding=hyp.rounding)
    frac_unforced = check_weight_codes_unforced(gw, ref)
    # padding of the rows is never written
    if dW.ld > n:
        assert int(dW.codes[:, n:].abs().max().item()) == 0, "padding of the code rows was written"
    for t in (dM, dV):
        base = t._base
        sc = m if side == "right" else n
        if base is not None and base.shape[1] > sc:
            assert float(base[:, sc:].abs().max().item()) == 0.0, "padding of the moment rows was written"
    return {"mismatch": frac, "mismatch_unforced": frac_unforced, "ill": ill, "wpre_err_lsb": wpre_err,
            "W": gw, "M": dM.cpu().numpy(), "V": dV.cpu().numpy(), "ref": ref}


def column_block(q: O.QTensor, a: int, b: int) -> O.QTensor:
    """Columns [a, b) of a quantized matrix, a on a group boundary, b on one or at the end."""
    g = q.group
    assert a % g == 0 and (b % g == 0 or b == q.codes.shape[1])
    return O.QTensor(q.codes[:, a:b].copy(), q.scales[:, a // g:(b + g - 1) // g].copy(),
                     q.zeros[:, a // g:(b + g - 1) // g].copy(), q.bits, g)


def check_step_on_column_blocks(blocks, gb, P, W, M, V, hyp, gpu, tol=2e-3):
    """Parity of one step of a large matrix on a few column blocks the oracle can afford.

    Column j of every result of the step depends on column j of G, M, V, W only (and on P), so the
    oracle runs on the blocks alone.  ``gpu`` holds the library's results for the whole matrix:
    M, V, R, N, W_pre (numpy) and W (oracle QTensor).  Same two stages and rules as run_and_check_step.
    """
    stats = []
    for (a, b) in blocks:
        Wb = column_block(W, a, b)
        ref = O.project_step(gb[:, a:b], P, Wb, M[:, a:b], V[:, a:b], hyp, col0=a)
        check_moments(gpu["M"][:, a:b], ref["M"], f"M[:, {a}:{b}]", tol)
        check_moments(gpu["V"][:, a:b], ref["V"], f"V[:, {a}:{b}]", tol)
        check_moments(gpu["R"][:, a:b], ref["R32"], f"R[:, {a}:{b}]", tol)
        n_gpu = gpu["N"][:, a:b]
        check_direction(n_gpu, ref, hyp, f"N[:, {a}:{b}]", tol)
        forced = O.project_step(gb[:, a:b], P, Wb, M[:, a:b], V[:, a:b], hyp, N_b_override=O.bf16_round(n_gpu), col0=a)
        lsb = np.repeat(forced["W"].scales, 256, axis=1)[:, :b - a]
        wpre_err = float((np.abs(gpu["W_pre"][:, a:b] - forced["W_pre"]) / lsb).max())
        assert wpre_err <= 1e-3, f"pre-rounding weight off by {wpre_err:.2e} LSB in columns {a}:{b}"
        gw = column_block(gpu["W"], a, b)
        frac = check_weight_codes(gw, forced, hyp.seed, hyp.step, col0=a)
        check_weight_codes_unforced(gw, ref)
        stats.append((a, b, frac, wpre_err))
    return stats
