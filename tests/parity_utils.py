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


def _group_of_column(n, ngroups):
    return np.repeat(np.arange(ngroups), 256)[:n]


def _near_boundary(out: dict, ref_w: O.QTensor, seed: int, step: int, col0: int, rounding: str) -> np.ndarray:
    """Elements whose rounding decision sits within 1e-3 of a level of a boundary: the oracle's scaled value T
    within 1e-3 of the element's draw (frac * 65536 within 65.536 of its Philox lane; of one half for round to
    nearest), of an integer, or at a clamp edge."""
    m, n = ref_w.codes.shape
    gcols = _group_of_column(n, ref_w.scales.shape[1])
    T = out["T"].astype(np.float64)
    fr = (T - np.floor(T)) * 65536.0
    if rounding == "rtn":
        near_draw = np.abs(fr - 32768.0) <= 1e-3 * 65536
    else:
        h = O.sr_uniform16(seed, step, m, n, col0=col0).astype(np.float64)
        near_draw = np.abs(fr - h) <= 1e-3 * 65536 + 1
    near_int = (fr <= 1e-3 * 65536) | (fr >= (1 - 1e-3) * 65536)
    lvl = np.floor(T) + ref_w.zeros[:, gcols]
    near_clamp = (lvl <= -128) | (lvl >= 126)
    return near_draw | near_int | near_clamp


def _code_and_level_diff(gpu_w: O.QTensor, ref_w: O.QTensor):
    """Difference of the stored codes and, in groups whose zero points differ, of the represented levels
    q - z instead (a zero point one apart shifts every code of the group by one without changing what the
    codes stand for).  Returns (difference, mask of the elements of such groups)."""
    n = ref_w.codes.shape[1]
    gcols = _group_of_column(n, ref_w.scales.shape[1])
    zd_el = (gpu_w.zeros != ref_w.zeros)[:, gcols]
    diff = gpu_w.codes.astype(np.int64) - ref_w.codes.astype(np.int64)
    lvl = (gpu_w.codes.astype(np.int64) - gpu_w.zeros[:, gcols].astype(np.int64)) - \
          (ref_w.codes.astype(np.int64) - ref_w.zeros[:, gcols].astype(np.int64))
    return np.where(zd_el, lvl, diff), zd_el


def check_weight_codes(gpu_w: O.QTensor, out: dict, seed: int, step: int, max_frac=1e-3, col0=0, rounding="sr"):
    """INT8 weights after one step against the oracle's (same direction N_b on both sides).

    Scales agree to 1e-5 relative.  Zero points are equal except, rarely, one apart (the scaled group minimum
    at a tie of the rounding).  Codes agree except by exactly one level, in at most ``max_frac`` of the
    elements, and only where the oracle's scaled value T lies within 1e-3 of the element's rounding boundary
    or of the clamp edge; in a group whose zero points differ the represented levels q - z are held to the
    same rule, with one more excuse: an element at the clamp edge of either side's grid.
    Returns the mismatch fraction.
    """
    ref_w = out["W"]
    n = ref_w.codes.shape[1]
    assert np.allclose(gpu_w.scales, ref_w.scales, rtol=1e-5, atol=0), "W scales"
    zdiff = gpu_w.zeros != ref_w.zeros
    if zdiff.any():
        assert np.all(np.abs(gpu_w.zeros - ref_w.zeros)[zdiff] == 1), "zero points differ by more than one"
        assert zdiff.mean() < 1e-3, "too many zero-point differences"
    diff, zd_el = _code_and_level_diff(gpu_w, ref_w)
    bad = diff != 0
    frac_bad = bad.mean()
    assert np.all(np.abs(diff[bad]) == 1), "a weight code (or level) differs by more than one"
    assert frac_bad <= max_frac, f"{frac_bad:.2e} of the weight codes differ"
    if bad.any():
        ok = _near_boundary(out, ref_w, seed, step, col0, rounding)
        # where the grids are one apart, the end codes of either grid clamp differently
        edge = zd_el & ((gpu_w.codes <= -127) | (gpu_w.codes >= 126) | (ref_w.codes <= -127) | (ref_w.codes >= 126))
        assert np.all((ok | edge)[bad]), f"{(bad & ~(ok | edge)).sum()} code mismatches away from any rounding boundary"
    return float(frac_bad)


def check_weight_codes_unforced(gpu_w: O.QTensor, ref: dict, nb_gpu_bits, seed: int, step: int, side="left", col0=0,
                                rounding="sr", max_frac=1e-3):
    """The same weights against the oracle's own, unforced, result.

    The only licence beyond check_weight_codes is the direction: where the GPU's bfloat16 direction equals the
    oracle's N_b bit for bit in a whole column of the low-rank state, that column of the weight update (that
    row, for the right-hand projection) is the same product on both sides, and its codes obey the strict rule.
    Where a column's N_b differs (an ill-conditioned element, or one rounded the other way within the stated
    distance of a bfloat16 midpoint), its codes may differ by one level; and a group whose scale or zero point
    differs because its minimum or maximum moved (it holds such a column) is excused as a whole.  Nothing
    may differ by more than one level.  Returns (mismatch fraction in the strict part, share of columns whose
    direction is identical)."""
    ref_w = ref["W"]
    m, n = ref_w.codes.shape
    nb_ref_bits = O.f32_to_bf16_bits(ref["N_b"])
    same_vec = (np.asarray(nb_gpu_bits).view(np.uint16) == nb_ref_bits).all(axis=0)      # per column of the state
    gcols = _group_of_column(n, ref_w.scales.shape[1])
    if side == "right":
        el_same = np.repeat(same_vec[:, None], n, axis=1)                                # state column i = weight row i
        group_has_diff = np.repeat((~same_vec)[:, None], ref_w.scales.shape[1], axis=1)
    else:
        el_same = np.repeat(same_vec[None, :], m, axis=0)
        per_group = np.array([(~same_vec[gcols == g]).any() for g in range(ref_w.scales.shape[1])])
        group_has_diff = np.repeat(per_group[None, :], m, axis=0)
    grid_moved = ((gpu_w.scales != ref_w.scales) | (gpu_w.zeros != ref_w.zeros)) & group_has_diff
    assert np.allclose(gpu_w.scales, ref_w.scales, rtol=1e-3, atol=0), "W scales (unforced)"
    assert np.abs(gpu_w.zeros - ref_w.zeros).max(initial=0) <= 1, "zero points differ by more than one (unforced)"
    diff, _ = _code_and_level_diff(gpu_w, ref_w)
    assert np.abs(diff).max(initial=0) <= 1, "a weight code differs by more than one level (unforced)"
    strict = el_same & ~grid_moved[:, gcols]
    bad = (diff != 0) & strict
    frac = float(bad.sum() / max(strict.sum(), 1))
    assert frac <= max_frac, f"{frac:.2e} of the weight codes differ where the direction is identical"
    if bad.any():
        ok = _near_boundary(ref, ref_w, seed, step, col0, rounding)
        assert np.all(ok[bad]), f"{(bad & ~ok).sum()} code mismatches away from any rounding boundary in columns whose " \
                                "direction is identical"
    return frac, float(same_vec.mean())


# ----------------------------------------------------------------------------- the direction, bit for bit
def direction_error_bound(ref: dict, abs_sum: np.ndarray, K: int, hyp) -> np.ndarray:
    """Bound on |N_gpu - N_oracle| per element: the measured accumulation error of R, propagated through the
    arithmetic of the two sides to first order.

    R: the tensor core adds the 16 exact products of one instruction to the binary32 accumulator and truncates
    the aligned sum; against fp64 on the oracle's side the error is biased toward zero and grows like sqrt(K)
    relative to S = sum_k |P~_ki| |G_kj| (``abs_sum``): the partial sums it scales with are a random walk over the
    K / 16 instructions.  Measured on B200 for K = 512 ... 11008 over 1e6 elements each, with a random
    projection: at most 0.16 sqrt(K) 2^-24 S.  Allowed here: three times that, plus the coherent part: where the
    products of a row add up instead of cancelling (a projection column along a planted direction), the partial
    sums grow linearly to R and K / 16 truncations of up to 2^-23 |partial sum| add up to 2^-24 (K / 16) |R|.
    So |dR| <= 2^-24 (0.5 sqrt(K) S + (K / 16) |R|), plus the final rounding.  (The worst case of the same
    arithmetic, (K / 16 + 1) 2^-23 S everywhere, is 11 to 26 times wider at these K on the incoherent rows and
    would leave most elements of a 7B-sized matrix undecided.)
    M', V': both sides round to binary32; the GPU rounds (1 - b) R (and its square) before a fused multiply-add,
    the oracle rounds the exact expression once: two and three units in the last place apart at most, plus what
    dR carries in.  N = M^ / (sqrt(V^) + eps): propagated to first order, plus 2^-20 |N| for the
    approximate square root and division and the binary32 constants of the GPU's form of the expression.
    Where sqrt(V^) is of the order of eps the bound is large: such elements are simply not decidable."""
    _, _, b1, b2, eps, _ = hyp.as_f32()
    t = int(hyp.step)
    u = 2.0 ** -24
    R = np.abs(ref["R32"].astype(np.float64))
    Mn = np.abs(ref["M"].astype(np.float64))
    Vn = ref["V"].astype(np.float64)
    bias1, bias2 = 1.0 - b1 ** t, 1.0 - b2 ** t
    dR = u * (0.5 * np.sqrt(float(K)) * abs_sum + (K / 16.0) * R) + u * R
    dM = (1.0 - b1) * dR + 4.0 * u * Mn
    dV = (1.0 - b2) * (2.0 * R * dR + dR * dR) + 6.0 * u * Vn
    sv = np.sqrt(Vn / bias2)
    sv_lo = np.sqrt(np.maximum(Vn - dV, 0.0) / bias2)
    dsv = (dV / bias2) / np.maximum(sv + sv_lo, 1e-300)
    den_lo = sv_lo + eps
    Nabs = np.abs(ref["N"].astype(np.float64))
    return (dM / bias1) / den_lo + (Mn / bias1) * dsv / (den_lo * (sv + eps)) + 2.0 ** -20 * Nabs + 1e-38


def check_direction_bits(n_gpu: np.ndarray, nb_gpu_bits: np.ndarray, ref: dict, abs_sum: np.ndarray, K: int, hyp,
                         name="N_b", min_decidable=0.6):
    """The GPU's bfloat16 direction against the oracle's N_b, bit for bit.

    (1) The kernel's N_b is the round-to-nearest-even bfloat16 of its own binary32 N, everywhere.
    (2) |N_gpu - N_oracle| stays within direction_error_bound everywhere.
    (3) Wherever the oracle's N is further from the nearest bfloat16 rounding midpoint than that bound, the
        two N_b are the same 16 bits.  (Closer than that, either rounding is a correct result.)
    Returns (share of elements decided by (3), share of elements whose bits agree)."""
    nb_gpu_bits = np.asarray(nb_gpu_bits).view(np.uint16)
    assert np.array_equal(nb_gpu_bits, O.f32_to_bf16_bits(n_gpu)), f"{name}: not the bfloat16 rounding of the kernel's own N"
    want = ref["N"].astype(np.float32)
    bound = direction_error_bound(ref, abs_sum, K, hyp)
    err = np.abs(n_gpu.astype(np.float64) - want.astype(np.float64))
    worst = float((err / bound).max())
    assert worst <= 1.0, f"{name}: |N_gpu - N_oracle| exceeds the arithmetic's bound by a factor {worst:.2f}"
    bits = want.view(np.uint32)
    low = (bits & np.uint32(0xFFFF)).astype(np.float64)
    expo = ((bits >> np.uint32(23)) & np.uint32(0xFF)).astype(np.int64)
    ulp32 = np.ldexp(1.0, np.maximum(expo, 1) - 127 - 23)          # spacing of binary32 at the oracle's N
    dist_mid = np.abs(low - 32768.0) * ulp32                        # distance to the nearest bfloat16 midpoint
    decidable = dist_mid > bound
    share = float(decidable.mean())
    assert share >= min_decidable, f"{name}: only {share:.3f} of the elements are decidable"
    nb_ref_bits = O.f32_to_bf16_bits(want)
    wrong = decidable & (nb_gpu_bits != nb_ref_bits)
    assert not wrong.any(), f"{name}: {int(wrong.sum())} elements away from a bfloat16 midpoint differ from the oracle's bits"
    return share, float((nb_gpu_bits == nb_ref_bits).mean())


def projection_abs_sum(gb: np.ndarray, P: O.QTensor, side="left", cols=None) -> np.ndarray:
    """sum_k |P~_ki| |G_kj| in the layout of the low-rank state (r x n; r x m for the right-hand projection)."""
    G = np.abs(O.bf16_bits_to_f32(gb).astype(np.float64))
    Pt = np.abs(O.bf16_round(O.dequantize(P)).astype(np.float64))
    return (G @ Pt).T if side == "right" else Pt.T @ G


class StepTaps:
    """Device buffers for the optional intermediates of qgalore_project_step."""

    def __init__(self, m, n, r, w_ld, side="left"):
        sc = m if side == "right" else n                # columns of the low-rank state
        self.R = B.zeros_matrix(r, sc, torch.float32)
        self.N = B.zeros_matrix(r, sc, torch.float32)
        self.N_b = B.zeros_matrix(r, sc, torch.int16)     # bfloat16 bit patterns, the pitch of R and N
        self.W_pre = torch.zeros((m, w_ld), dtype=torch.float32, device="cuda")[:, :n]

    def as_dict(self):
        return {"R": self.R, "N": self.N, "W_pre": self.W_pre, "N_b": self.N_b}


def run_and_check_step(gb, P: O.QTensor, W: O.QTensor, M, V, hyp: O.Hyper, tol=2e-3, impl=None, side="left", ref=None):
    """Teacher-forced single-step parity of qgalore_project_step against the oracle.

    Stage 1 (steps 1-4): M', V', R and the direction N against the oracle's own.
    Stage 2 (steps 5-6): the oracle recomputes the weight update from the GPU's bf16 direction, and
    W', scales, zero points and codes are held to the strict rule of check_weight_codes.
    Plus the looser end-to-end bound against the oracle's unforced result.  Returns a dict of statistics.
    """
    m, n = gb.shape
    r = P.codes.shape[1]
    if ref is None:                                     # the caller may hand in the oracle's step if it has made it already
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
    nb_gpu = taps.N_b.cpu().numpy().view(np.uint16)
    ill = check_direction(n_gpu, ref, hyp, "N", tol)
    decided, nb_same = check_direction_bits(n_gpu, nb_gpu, ref, projection_abs_sum(gb, P, side), n if side == "right" else m, hyp)
    # stage 2: same direction on both sides (the bits the kernel's back-projection read)
    forced = O.project_step(gb, P, W, M, V, hyp, N_b_override=O.bf16_bits_to_f32(nb_gpu), side=side)
    lsb = np.repeat(forced["W"].scales, 256, axis=1)[:, :n]
    wpre_err = float((np.abs(taps.W_pre.cpu().numpy() - forced["W_pre"]) / lsb).max())
    assert wpre_err <= 1e-3, f"pre-rounding weight off by {wpre_err:.2e} LSB"
    gw = from_device_q(dW)
    frac = check_weight_codes(gw, forced, hyp.seed, hyp.step, rounding=hyp.rounding)
    frac_unforced, same_cols = check_weight_codes_unforced(gw, ref, nb_gpu, hyp.seed, hyp.step, side=side,
                                                            rounding=hyp.rounding)
    # padding of the rows is never written
    if dW.ld > n:
        assert int(dW.codes[:, n:].abs().max().item()) == 0, "padding of the code rows was written"
    for t in (dM, dV):
        base = t._base
        sc = m if side == "right" else n
        if base is not None and base.shape[1] > sc:
            assert float(base[:, sc:].abs().max().item()) == 0.0, "padding of the moment rows was written"
    return {"mismatch": frac, "mismatch_unforced": frac_unforced, "ill": ill, "wpre_err_lsb": wpre_err,
            "nb_decided": decided, "nb_same": nb_same, "columns_with_identical_direction": same_cols,
            "W": gw, "M": dM.cpu().numpy(), "V": dV.cpu().numpy(), "ref": ref}


def check_weights_loosely(gw: O.QTensor, ref_w: O.QTensor, max_frac=2e-2):
    """What holds for the weights without knowing the GPU's direction: scales to 1e-3, zero points and levels at
    most one apart, differences in at most ``max_frac`` of the elements."""
    assert np.allclose(gw.scales, ref_w.scales, rtol=1e-3, atol=0), "W scales"
    diff, _ = _code_and_level_diff(gw, ref_w)
    assert np.abs(diff).max(initial=0) <= 1 and np.abs(gw.zeros - ref_w.zeros).max(initial=0) <= 1
    frac = float((diff != 0).mean())
    assert frac <= max_frac, f"{frac:.2e} of the weight codes differ"
    return frac


def run_and_check_step_light(gb, P: O.QTensor, W: O.QTensor, M, V, hyp: O.Hyper, ref: dict, tol=2e-3):
    """The inexpensive form for the many steps of a long run: one GPU step from the oracle's pre-step state,
    the moments against the oracle's post-step moments by the usual rule; the weights only by what holds without
    knowing the GPU's direction: scales to 1e-3, zero points and levels at most one apart, mismatches in at most
    2 % of the elements.  (The strict weight rules run at the fully checked steps.)"""
    dG, dP, dW = g_to_device(gb), to_device_q(P), to_device_q(W)
    dM, dV = f32_to_device(M), f32_to_device(V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.project_step(dG, dP, dW, dM, dV,
                   B.Hyper(lr=hyp.lr, alpha=hyp.alpha, beta1=hyp.beta1, beta2=hyp.beta2, eps=hyp.eps,
                           weight_decay=hyp.weight_decay, step=hyp.step, seed=hyp.seed), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status word"
    check_moments(dM.cpu().numpy(), ref["M"], "M", tol)
    check_moments(dV.cpu().numpy(), ref["V"], "V", tol)
    return check_weights_loosely(from_device_q(dW), ref["W"])


def column_block(q: O.QTensor, a: int, b: int) -> O.QTensor:
    """Columns [a, b) of a quantized matrix, a on a group boundary, b on one or at the end."""
    g = q.group
    assert a % g == 0 and (b % g == 0 or b == q.codes.shape[1])
    return O.QTensor(q.codes[:, a:b].copy(), q.scales[:, a // g:(b + g - 1) // g].copy(),
                     q.zeros[:, a // g:(b + g - 1) // g].copy(), q.bits, g)


def check_step_on_column_blocks(blocks, gb, P, W, M, V, hyp, gpu, tol=2e-3, col0=0):
    """Parity of one step of a large matrix on a few column blocks the oracle can afford.

    Column j of every result of the step depends on column j of G, M, V, W only (and on P), so the
    oracle runs on the blocks alone.  ``gpu`` holds the library's results for the whole matrix:
    M, V, R, N, N_b, W_pre (numpy) and W (oracle QTensor).  Same two stages and rules as run_and_check_step.
    ``col0``: the arrays handed in are themselves the columns [col0, ...) of a wider matrix (col0 on a group
    boundary); it only enters the Philox lanes.
    """
    stats = []
    for (a, b) in blocks:
        Wb = column_block(W, a, b)
        ref = O.project_step(gb[:, a:b], P, Wb, M[:, a:b], V[:, a:b], hyp, col0=col0 + a)
        check_moments(gpu["M"][:, a:b], ref["M"], f"M[:, {a}:{b}]", tol)
        check_moments(gpu["V"][:, a:b], ref["V"], f"V[:, {a}:{b}]", tol)
        check_moments(gpu["R"][:, a:b], ref["R32"], f"R[:, {a}:{b}]", tol)
        n_gpu = gpu["N"][:, a:b]
        nb_gpu = np.ascontiguousarray(gpu["N_b"][:, a:b]).view(np.uint16)
        check_direction(n_gpu, ref, hyp, f"N[:, {a}:{b}]", tol)
        check_direction_bits(n_gpu, nb_gpu, ref, projection_abs_sum(gb[:, a:b], P), gb.shape[0], hyp, f"N_b[:, {a}:{b}]")
        forced = O.project_step(gb[:, a:b], P, Wb, M[:, a:b], V[:, a:b], hyp, N_b_override=O.bf16_bits_to_f32(nb_gpu), col0=col0 + a)
        lsb = np.repeat(forced["W"].scales, 256, axis=1)[:, :b - a]
        wpre_err = float((np.abs(gpu["W_pre"][:, a:b] - forced["W_pre"]) / lsb).max())
        assert wpre_err <= 1e-3, f"pre-rounding weight off by {wpre_err:.2e} LSB in columns {a}:{b}"
        gw = column_block(gpu["W"], a, b)
        frac = check_weight_codes(gw, forced, hyp.seed, hyp.step, col0=col0 + a)
        check_weight_codes_unforced(gw, ref, nb_gpu, hyp.seed, hyp.step, col0=col0 + a)
        stats.append((a, b, frac, wpre_err))
    return stats
