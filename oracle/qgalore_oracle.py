"""Plain CPU statement of the Q-GaLore per-matrix optimizer step.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
bench's CPU-baseline leg, never by the product path.  numpy/scipy only, fp64
arithmetic except at the rounding points written out below (``fl32`` = round to
IEEE binary32, ``bf16`` = round binary32 to bfloat16, both round-to-nearest-even).
No blocking, fusion or reordering: each function follows the paper's passage it
cites, one step after the other.

Pinned by tests/test_oracle_*.py against facts that do not come from this file:
published Philox known answers, the half-step error bound of the quantizer,
E[W_q] = W for stochastic rounding, reduction to dense Adam at full rank, a
hand-written Jacobi eigen-solver on 8x8 inputs, closed forms of the similarity
statistic and scripted gate sequences; the INT8 linear layer of App. A by index
loops on a tiny case, a permutation weight, the adjoint identity and autograd.

Parity unpinned: the 8-bit storage of the Adam moments (``Moments8``,
``quantize_m8``, ``quantize_v8`` and their inverses): the paper names 8-bit Adam
without a format, so the format is a choice and only its own promises are pinned.
The right-hand projection is pinned against the left-hand form on the
transposed gradient; the 2-bit quantizer and the round-to-nearest step by the
same bounds as the 4- and 8-bit quantizers.

Conventions
-----------
* Matrices are row-major numpy arrays.  W, G are m x n; P is m x r; M, V are r x n.
* Quantization groups are runs of ``group`` consecutive elements along a row and
  restart at every row; a row whose length is not a multiple of ``group`` ends in
  one shorter group (Sec. 3.1: "block-wise", block size 256).
* A quantized tensor is the triple (codes int8 [rows, cols], scales fp32
  [rows, ngroups], zeros fp32 [rows, ngroups]); INT4 codes are kept unpacked in
  int8 here, ``pack_int4`` gives the byte layout of the C boundary.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import scipy.linalg

__all__ = [
    "GROUP", "fl32", "bf16_round", "bf16_bits_to_f32", "f32_to_bf16_bits",
    "philox4x32_10", "sr_uniform16", "group_params", "quantize_rtn", "quantize_sr",
    "dequantize", "pack_int4", "unpack_int4", "pack_int2", "unpack_int2", "QTensor", "Hyper", "project_step",
    "refresh_subspace", "subspace_similarity", "GateState", "gate_update",
    "principal_angle", "int8_linear_forward", "int8_linear_backward", "STATE_BLOCK", "Moments8", "quantize_m8", "quantize_v8", "dequantize_m8", "dequantize_v8",
]

GROUP = 256  # Sec. 3.1: block size 256 in all implementations
_MIN_NORMAL = np.float32(2.0 ** -126)


# --------------------------------------------------------------------------- rounding helpers
def fl32(x):
    """Round to IEEE binary32 (numpy's float64 -> float32 cast is round-to-nearest-even)."""
    return np.asarray(x, dtype=np.float64).astype(np.float32)


def f32_to_bf16_bits(x32):
    """binary32 -> bfloat16 bit patterns (uint16), round-to-nearest-even on the dropped 16 bits."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = u + np.uint64(0x7FFF) + lsb
    return ((u >> np.uint64(16)) & np.uint64(0xFFFF)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    """bfloat16 bit patterns (uint16) -> the binary32 values they denote (exact)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def bf16_round(x32):
    """Round binary32 values to the nearest bfloat16, returned as binary32."""
    x32 = np.asarray(x32, dtype=np.float32)
    return bf16_bits_to_f32(f32_to_bf16_bits(x32)).reshape(x32.shape)


# --------------------------------------------------------------------------- Philox4x32-10
_PH_M0 = np.uint64(0xD2511F53)
_PH_M1 = np.uint64(0xCD9E8D57)
_PH_W0 = 0x9E3779B9
_PH_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11).

    ``counter``: four uint32 arrays (broadcastable), ``key``: two uint32 scalars.
    Returns four uint32 arrays.  The paper names no generator for Sec. 3.4's
    stochastic rounding; this counter-based one is the reading both sides use.
    """
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & _MASK32 for c in counter)
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(key[0]) & 0xFFFFFFFF
    k1 = int(key[1]) & 0xFFFFFFFF
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PH_W0) & 0xFFFFFFFF
            k1 = (k1 + _PH_W1) & 0xFFFFFFFF
        p0 = _PH_M0 * c0  # 32x32 -> 64 bit products, no overflow in uint64
        p1 = _PH_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0)
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def sr_uniform16(seed, step, rows, cols, row0=0, col0=0):
    """16-bit uniforms h[i, j] for the elements (row0+i, col0+j) of one matrix at one step.

    Element (i, j): counter = (j >> 3, i, lo32(step), hi32(step)), key = (lo32(seed),
    hi32(seed)); the four 32-bit outputs hold eight 16-bit lanes, lane l = j & 7 is
    bits [16*(l&1), 16*(l&1)+16) of output word l >> 1.
    """
    i = (np.arange(rows, dtype=np.uint64) + np.uint64(row0))[:, None]
    j = (np.arange(cols, dtype=np.uint64) + np.uint64(col0))[None, :]
    nblk = (int(col0) + cols + 7) // 8 - int(col0) // 8
    blk = np.arange(nblk, dtype=np.uint64)[None, :] + np.uint64(int(col0) // 8)
    step = int(step)
    seed = int(seed)
    x = philox4x32_10(
        (blk, i, np.uint64(step & 0xFFFFFFFF), np.uint64((step >> 32) & 0xFFFFFFFF)),
        (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF),
    )
    words = np.stack(x, axis=-1)  # [rows, nblk, 4]
    lanes = np.empty(words.shape[:2] + (8,), dtype=np.uint32)
    lanes[..., 0::2] = words & np.uint32(0xFFFF)
    lanes[..., 1::2] = words >> np.uint32(16)
    lanes = lanes.reshape(rows, nblk * 8)
    off = int(col0) % 8
    return lanes[:, off:off + cols]


# --------------------------------------------------------------------------- quantizer (Sec. 3.1)
@dataclass
class QTensor:
    codes: np.ndarray   # int8 [rows, cols], INT4 values lie in [-8, 7]
    scales: np.ndarray  # float32 [rows, ngroups]
    zeros: np.ndarray   # float32 [rows, ngroups], integer valued
    bits: int
    group: int = GROUP

    @property
    def shape(self):
        return self.codes.shape

    def copy(self):
        return QTensor(self.codes.copy(), self.scales.copy(), self.zeros.copy(), self.bits, self.group)


def group_params(seg, bits):
    """Scale s, its reciprocal and zero point z of each row of ``seg`` (one group per row).

    Sec. 3.1: W_q = clamp(round(W / s) + z, -2^(n-1), 2^(n-1) - 1) with s and z
    "calculated within each block".  Reading: affine min-max, s = (max - min) / (2^n - 1)
    in binary32, z the integer that sends the group minimum to the lowest code.
    A constant group, or one whose s is not a normal number, takes z = 0 and
    s = |max| (1 if that is not a normal number either).
    """
    seg = np.asarray(seg, dtype=np.float32)
    qlo = np.float32(-(1 << (bits - 1)))
    levels = np.float32((1 << bits) - 1)
    mn = seg.min(axis=1)
    mx = seg.max(axis=1)
    with np.errstate(over="ignore", invalid="ignore", divide="ignore"):
        s = (mx - mn) / levels                                   # binary32 subtract, binary32 divide
        degenerate = (mx == mn) | ~np.isfinite(s) | (s < _MIN_NORMAL)
        amx = np.abs(mx)
        s_deg = np.where(np.isfinite(amx) & (amx >= _MIN_NORMAL), amx, np.float32(1)).astype(np.float32)
        s = np.where(degenerate, s_deg, s).astype(np.float32)
        inv = (np.float32(1) / s).astype(np.float32)             # one IEEE divide per group
        z = (qlo - np.rint(mn * inv)).astype(np.float32)         # binary32 multiply, ties to even
        z = np.where(degenerate, np.float32(0), z).astype(np.float32)
    return s, inv, z


def _group_slices(cols, group):
    return [(c, min(c + group, cols)) for c in range(0, cols, group)]


def quantize_rtn(x, bits, group=GROUP, return_scaled=False):
    """Round-to-nearest block-wise uniform quantization Quant_n (Sec. 3.1)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, cols = x.shape
    sl = _group_slices(cols, group)
    codes = np.empty((rows, cols), dtype=np.int8)
    scales = np.empty((rows, len(sl)), dtype=np.float32)
    zeros = np.empty((rows, len(sl)), dtype=np.float32)
    scaled = np.empty((rows, cols), dtype=np.float32)
    qlo = np.float32(-(1 << (bits - 1)))
    qhi = np.float32((1 << (bits - 1)) - 1)
    for k, (a, b) in enumerate(sl):
        seg = x[:, a:b]
        s, inv, z = group_params(seg, bits)
        t = seg * inv[:, None]                                   # binary32 multiply
        q = np.clip(np.rint(t) + z[:, None], qlo, qhi)           # binary32 add of integers
        codes[:, a:b] = q.astype(np.int8)
        scales[:, k] = s
        zeros[:, k] = z
        scaled[:, a:b] = t
    qt = QTensor(codes, scales, zeros, bits, group)
    return (qt, scaled) if return_scaled else qt


def quantize_sr(x, seed, step, group=GROUP, return_scaled=False, col0=0):
    """INT8 block-wise quantization with stochastic rounding F_SR (Sec. 3.4).

    The scaled value t = x / s is rounded down with probability ceil(t) - t and up
    with probability t - floor(t); the draw is the element's 16-bit Philox lane h:
    round up iff frac(t) * 65536 > h.  Scale and zero point are recomputed from the
    updated group (Sec. 3.5: the weight update needs "an additional quantization step").
    ``col0``: x is the column block [col0, col0 + cols) of a wider matrix (col0 a multiple of the
    group size); it only shifts the column index that selects each element's Philox lane.
    """
    assert col0 % group == 0
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, cols = x.shape
    sl = _group_slices(cols, group)
    codes = np.empty((rows, cols), dtype=np.int8)
    scales = np.empty((rows, len(sl)), dtype=np.float32)
    zeros = np.empty((rows, len(sl)), dtype=np.float32)
    scaled = np.empty((rows, cols), dtype=np.float32)
    h = sr_uniform16(seed, step, rows, cols, col0=col0).astype(np.float32)
    for k, (a, b) in enumerate(sl):
        seg = x[:, a:b]
        s, inv, z = group_params(seg, 8)
        t = seg * inv[:, None]                                   # binary32 multiply
        f = np.floor(t)
        frac = t - f                                             # exact in binary32
        up = (frac * np.float32(65536.0) > h[:, a:b]).astype(np.float32)
        q = np.clip(f + up + z[:, None], np.float32(-128), np.float32(127))
        codes[:, a:b] = q.astype(np.int8)
        scales[:, k] = s
        zeros[:, k] = z
        scaled[:, a:b] = t
    qt = QTensor(codes, scales, zeros, 8, group)
    return (qt, scaled) if return_scaled else qt


def dequantize(qt: QTensor):
    """W = (q - zeros) * scales in binary32 (App. A listing, the dequantization line)."""
    rows, cols = qt.codes.shape
    out = np.empty((rows, cols), dtype=np.float32)
    for k, (a, b) in enumerate(_group_slices(cols, qt.group)):
        q = qt.codes[:, a:b].astype(np.float32)
        out[:, a:b] = (q - qt.zeros[:, k:k + 1]) * qt.scales[:, k:k + 1]
    return out


def pack_int4(codes):
    """Two INT4 codes per byte: byte k of a row = (q[2k] + 8) | (q[2k+1] + 8) << 4."""
    rows, cols = codes.shape
    u = (codes.astype(np.int16) + 8).astype(np.uint8)
    if cols % 2:
        u = np.concatenate([u, np.full((rows, 1), 8, dtype=np.uint8)], axis=1)
    return (u[:, 0::2] | (u[:, 1::2] << np.uint8(4))).astype(np.uint8)


def unpack_int4(packed, cols):
    packed = np.asarray(packed, dtype=np.uint8)
    rows = packed.shape[0]
    out = np.empty((rows, packed.shape[1] * 2), dtype=np.int16)
    out[:, 0::2] = packed & np.uint8(0xF)
    out[:, 1::2] = packed >> np.uint8(4)
    return (out[:, :cols] - 8).astype(np.int8)


def pack_int2(codes):
    """Four INT2 codes per byte: column 4k + i of a row in bits 2i, 2i + 1 of byte k, stored as q + 2."""
    rows, cols = codes.shape
    u = (codes.astype(np.int16) + 2).astype(np.uint8)
    pad = (-cols) % 4
    if pad:
        u = np.concatenate([u, np.full((rows, pad), 2, dtype=np.uint8)], axis=1)
    return (u[:, 0::4] | (u[:, 1::4] << np.uint8(2)) | (u[:, 2::4] << np.uint8(4)) | (u[:, 3::4] << np.uint8(6))).astype(np.uint8)


def unpack_int2(packed, cols):
    packed = np.asarray(packed, dtype=np.uint8)
    out = np.empty((packed.shape[0], packed.shape[1] * 4), dtype=np.int16)
    for i in range(4):
        out[:, i::4] = (packed >> np.uint8(2 * i)) & np.uint8(3)
    return (out[:, :cols] - 2).astype(np.int8)


# --------------------------------------------------------------------------- 8-bit moments (Sec. 3.5 "8-bit Adam")
# The paper keeps the Adam states of the low-rank subspace in 8 bits and cites block-wise 8-bit optimizers
# for it without giving a format.  PARITY UNPINNED: there is no definition in the paper to check this against;
# the format below is a choice (pinned only by what it promises: error bounds, exact block maximum, idempotence).
# Blocks of STATE_BLOCK consecutive elements along a row (restarting at every row, a shorter block at a ragged
# end), one binary32 scale per block.
#   first moment  (signed):   s = max |x|;  code = rint(x * (1 / (s / 127))) in [-127, 127];  x^ = code * (s / 127)
#   second moment (>= 0):     s = max x;    code = rint(255 * sqrt(x * (1 / s))) in [0, 255];  x^ = (code / 255)^2 * s
# (the square-root law gives small second moments the relative precision a linear code would not).  Every
# operation is a single binary32 operation in the order written; an all-zero block has scale 0 and codes 0.
STATE_BLOCK = 32


@dataclass
class Moments8:
    codes: np.ndarray    # int8 (first moment) or uint8 (second moment) [rows, cols]
    scales: np.ndarray   # float32 [rows, ceil(cols / STATE_BLOCK)]


def _state_blocks(cols):
    return [(a, min(a + STATE_BLOCK, cols)) for a in range(0, cols, STATE_BLOCK)]


def quantize_m8(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, cols = x.shape
    bl = _state_blocks(cols)
    codes = np.zeros((rows, cols), np.int8)
    scales = np.zeros((rows, len(bl)), np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        for k, (a, b) in enumerate(bl):
            seg = x[:, a:b]
            s = np.abs(seg).max(axis=1).astype(np.float32)
            step = (s / np.float32(127.0)).astype(np.float32)
            inv = np.where(step > 0, np.float32(1.0) / step, np.float32(0.0)).astype(np.float32)
            q = np.rint((seg * inv[:, None]).astype(np.float32))
            codes[:, a:b] = np.clip(q, -127, 127).astype(np.int8)
            scales[:, k] = s
    return Moments8(codes, scales)


def dequantize_m8(q: Moments8):
    rows, cols = q.codes.shape
    out = np.empty((rows, cols), np.float32)
    for k, (a, b) in enumerate(_state_blocks(cols)):
        step = (q.scales[:, k] / np.float32(127.0)).astype(np.float32)
        out[:, a:b] = (q.codes[:, a:b].astype(np.float32) * step[:, None]).astype(np.float32)
    return out


def quantize_v8(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, cols = x.shape
    bl = _state_blocks(cols)
    codes = np.zeros((rows, cols), np.uint8)
    scales = np.zeros((rows, len(bl)), np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        for k, (a, b) in enumerate(bl):
            seg = x[:, a:b]
            s = seg.max(axis=1).astype(np.float32)
            inv = np.where(s > 0, np.float32(1.0) / s, np.float32(0.0)).astype(np.float32)
            t = (seg * inv[:, None]).astype(np.float32)
            u = np.sqrt(np.maximum(t, np.float32(0.0))).astype(np.float32)
            q = np.rint((u * np.float32(255.0)).astype(np.float32))
            codes[:, a:b] = np.clip(q, 0, 255).astype(np.uint8)
            scales[:, k] = s
    return Moments8(codes, scales)


def dequantize_v8(q: Moments8):
    rows, cols = q.codes.shape
    out = np.empty((rows, cols), np.float32)
    c = np.float32(1.0) / np.float32(255.0)
    for k, (a, b) in enumerate(_state_blocks(cols)):
        w = (q.codes[:, a:b].astype(np.float32) * c).astype(np.float32)
        out[:, a:b] = ((w * w).astype(np.float32) * q.scales[:, k:k + 1]).astype(np.float32)
    return out


# --------------------------------------------------------------------------- the step (Sec. 3.5)
@dataclass
class Hyper:
    lr: float = 0.004        # the one learning rate the paper prints (7B run)
    alpha: float = 0.25      # GaLore scale factor, Sec. 4.1 baselines (vi)
    beta1: float = 0.9       # Adam constants: Kingma & Ba defaults (the paper says "Adam")
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    step: int = 1            # t >= 1
    seed: int = 0
    rounding: str = "sr"     # "sr": stochastic rounding F_SR (Sec. 3.4); "rtn": round to nearest (the Fig. 6 ablation)

    def as_f32(self):
        """The values as the C boundary carries them (binary32), widened back to Python floats."""
        g = lambda v: float(np.float32(v))
        return g(self.lr), g(self.alpha), g(self.beta1), g(self.beta2), g(self.eps), g(self.weight_decay)


def project_step(G_bits, P_q: QTensor, W_q: QTensor, M, V, h: Hyper, P_override=None, N_b_override=None, col0=0,
                 side="left"):
    """One Q-GaLore update of one weight matrix (Sec. 3.5, Fig. 4; GaLore projection as cited there).

    G_bits : uint16 [m, n] bfloat16 gradient.         P_q : INT4 m x r projection.
    W_q    : INT8 m x n weight.                       M, V: float32 r x n Adam moments.
    Returns a dict with the new W (QTensor), M, V and the intermediates R32, N, N_b,
    W_pre (pre-rounding weight) and T (= W_pre scaled by the new group reciprocal).
    ``P_override`` (float64 m x r) bypasses the INT4 dequantization and the bfloat16
    rounding of P and N; it exists only for the full-rank pin.
    ``N_b_override`` (float32 r x n, bfloat16-representable) replaces the direction that enters
    steps 5-6; steps 1-4 are still carried out and returned.  A staged comparison uses it: the
    direction N = M^ / (sqrt(V^) + eps) amplifies rounding differences of R without bound where
    sqrt(V^) is of the order of eps, so the weight update of another implementation is checked
    against steps 5-6 applied to that implementation's own direction.
    ``col0``: G, W, M, V are the column block starting at column col0 (a multiple of the group
    size) of a wider matrix; every column of the step depends on its own column of G, M, V, W only
    (and on P), so the block's results are those of the full matrix.  col0 enters the Philox lanes.
    ``side``: "left" is R = P^T G with P m x r and the moments r x n (what the rest of this docstring
    describes).  "right" is GaLore's other form, R = G Q with Q = P_q of shape n x r: the low-rank state is
    m x r, and M, V, R32, N, N_b are kept and returned TRANSPOSED (r x m, row-major) so that both forms
    hand the same kind of array around; the update is D = N Q^T.  (col0 is for the left form only.)
    M and V may also be Moments8 (the 8-bit block-wise storage defined above): they are dequantized on the
    way in, the step runs on binary32 moments as written, the direction N is taken from the binary32 M', V',
    and the result also carries their 8-bit form as "M8", "V8" ("M", "V" stay the binary32 values before storage).
    """
    state8 = isinstance(M, Moments8)
    if state8:
        M, V = dequantize_m8(M), dequantize_v8(V)
    if side == "right":
        assert col0 == 0
        out = _project_step_right(G_bits, P_q, W_q, M, V, h, N_b_override)
    else:
        out = _project_step_left(G_bits, P_q, W_q, M, V, h, P_override, N_b_override, col0)
    if state8:
        out["M8"], out["V8"] = quantize_m8(out["M"]), quantize_v8(out["V"])
    return out


def _project_step_left(G_bits, P_q, W_q, M, V, h, P_override, N_b_override, col0):
    lr, alpha, b1, b2, eps, wd = h.as_f32()
    t = int(h.step)
    G = bf16_bits_to_f32(G_bits).astype(np.float64)
    # 1. dequantize the projection matrix; it enters the contraction as bfloat16
    if P_override is None:
        Pt = bf16_round(dequantize(P_q)).astype(np.float64)
    else:
        Pt = np.asarray(P_override, dtype=np.float64)
    # 2. project the gradient into the subspace: R = P^T G
    R32 = fl32(Pt.T @ G)
    R = R32.astype(np.float64)
    # 3. Adam moments on the low-rank state
    M_new = fl32(b1 * M.astype(np.float64) + (1.0 - b1) * R)
    V_new = fl32(b2 * V.astype(np.float64) + (1.0 - b2) * R * R)
    # 4. bias-corrected direction, epsilon outside the square root
    m_hat = M_new.astype(np.float64) / (1.0 - b1 ** t)
    v_hat = V_new.astype(np.float64) / (1.0 - b2 ** t)
    N = m_hat / (np.sqrt(v_hat) + eps)
    N32 = fl32(N)
    N_b = bf16_round(N32) if P_override is None else N32
    if N_b_override is not None:
        N_b = np.asarray(N_b_override, dtype=np.float32)
    # 5. project back, scale, add to the dequantized weight (no high-precision master copy)
    D = Pt @ N_b.astype(np.float64)
    W_hat = dequantize(W_q).astype(np.float64)
    W_pre = fl32(W_hat - (lr * alpha) * D - (lr * wd) * W_hat)
    # 6. requantize every group: stochastic rounding (Sec. 3.4), or round to nearest for the ablation of Fig. 6
    if h.rounding == "rtn":
        W_new, T = quantize_rtn(W_pre, 8, W_q.group, return_scaled=True)
    else:
        W_new, T = quantize_sr(W_pre, h.seed, t, W_q.group, return_scaled=True, col0=col0)
    return dict(W=W_new, M=M_new, V=V_new, R32=R32, N=N32, N_b=N_b, W_pre=W_pre, T=T, P_tilde=Pt)


def _project_step_right(G_bits, Q_q: QTensor, W_q: QTensor, Mt, Vt, h: Hyper, N_b_override=None):
    """The step with the projection on the right (Sec. 3.5 defers the choice of side to GaLore):
    R = G Q~ (m x r), Adam on the m x r state, D = N_b Q~^T.  Mt, Vt and every returned low-rank array are
    the transposes (r x m)."""
    lr, alpha, b1, b2, eps, wd = h.as_f32()
    t = int(h.step)
    G = bf16_bits_to_f32(G_bits).astype(np.float64)
    Qt = bf16_round(dequantize(Q_q)).astype(np.float64)              # n x r, enters the contraction as bfloat16
    R32 = fl32((G @ Qt).T)                                            # r x m
    R = R32.astype(np.float64)
    M_new = fl32(b1 * Mt.astype(np.float64) + (1.0 - b1) * R)
    V_new = fl32(b2 * Vt.astype(np.float64) + (1.0 - b2) * R * R)
    m_hat = M_new.astype(np.float64) / (1.0 - b1 ** t)
    v_hat = V_new.astype(np.float64) / (1.0 - b2 ** t)
    N32 = fl32(m_hat / (np.sqrt(v_hat) + eps))
    N_b = bf16_round(N32)
    if N_b_override is not None:
        N_b = np.asarray(N_b_override, dtype=np.float32)
    D = N_b.astype(np.float64).T @ Qt.T                               # m x n
    W_hat = dequantize(W_q).astype(np.float64)
    W_pre = fl32(W_hat - (lr * alpha) * D - (lr * wd) * W_hat)
    if h.rounding == "rtn":
        W_new, T = quantize_rtn(W_pre, 8, W_q.group, return_scaled=True)
    else:
        W_new, T = quantize_sr(W_pre, h.seed, t, W_q.group, return_scaled=True)
    return dict(W=W_new, M=M_new, V=V_new, R32=R32, N=N32, N_b=N_b, W_pre=W_pre, T=T, P_tilde=Qt)


# --------------------------------------------------------------------------- refresh (Sec. 3.5, Sec. 1)
def refresh_subspace(G_bits, r, group=GROUP, bits=4, side="left"):
    """Projection matrix from the SVD of the gradient: the top-r left singular vectors.

    Exact LAPACK SVD (gesdd) of the gradient widened to fp64.  Each column's sign is
    fixed so that its largest-magnitude entry is positive.  Returns (P float32 m x r,
    its quantization (INT4 is the method, Sec. 3.3; 2 and 8 bits are the ablation of Sec. 4.4), singular values).
    """
    G = bf16_bits_to_f32(G_bits).astype(np.float64)
    if side == "right":          # the right singular vectors of G are the left ones of its transpose
        G = np.ascontiguousarray(G.T)
    U, S, _ = scipy.linalg.svd(G, full_matrices=False, lapack_driver="gesdd")
    P = U[:, :r].copy()
    piv = np.argmax(np.abs(P), axis=0)
    sgn = np.sign(P[piv, np.arange(P.shape[1])])
    sgn[sgn == 0] = 1.0
    P = fl32(P * sgn[None, :])
    return P, quantize_rtn(P, bits, group), S


def principal_angle(P_ref, P_test):
    """Largest principal angle between span(P_ref) and span(P_test), via asin of the residual norm.

    Both bases are orthonormalised in fp64 first; asin ||(I - Q_ref Q_ref^T) Q_test||_2 is
    accurate for small angles where acos of the smallest cosine is not.
    """
    Qr, _ = np.linalg.qr(np.asarray(P_ref, dtype=np.float64))
    Qt, _ = np.linalg.qr(np.asarray(P_test, dtype=np.float64))
    resid = Qt - Qr @ (Qr.T @ Qt)
    s = np.linalg.norm(resid, 2)
    return float(np.arcsin(min(1.0, s)))


# --------------------------------------------------------------------------- similarity and gate (Sec. 3.2)
def subspace_similarity(A_q: QTensor, B_q: QTensor, sim_cols=None):
    """Cosine similarity between two adjacent (INT4) projection matrices.

    sim = sum_{j<c} |<a_j, b_j>| / (||A[:, :c]||_F * ||B[:, :c]||_F) over the leading
    c columns of the dequantized matrices; the absolute value removes the sign freedom
    of singular vectors.  Returns a Python float (fp64 arithmetic).
    """
    A = dequantize(A_q).astype(np.float64)
    B = dequantize(B_q).astype(np.float64)
    c = A.shape[1] if sim_cols is None else int(sim_cols)
    A, B = A[:, :c], B[:, :c]
    num = np.abs((A * B).sum(axis=0)).sum()
    den = np.sqrt((A * A).sum()) * np.sqrt((B * B).sum())
    return float(num / den) if den > 0 else 0.0


@dataclass
class GateState:
    interval: int = 200
    history: list = field(default_factory=list)


def gate_update(state: GateState, sim, threshold=0.4, k=1):
    """Adaptive lazy update (Sec. 3.2): keep the last k similarities of this layer; once
    k are held and all are >= threshold, double the refresh interval and clear the history.
    Returns True when the interval was doubled.
    """
    state.history.append(float(sim))
    if len(state.history) > k:
        state.history = state.history[-k:]
    if len(state.history) == k and all(s >= threshold for s in state.history):
        state.interval *= 2
        state.history = []
        return True
    return False


# --------------------------------------------------------------------------- App. A: the INT8 linear layer
def _weight_operand(W_q: QTensor):
    """The weight as the products see it: dequantized in binary32 (App. A, the dequantization line), then
    rounded once to the activations' type, bfloat16.  Returned in float64."""
    return bf16_bits_to_f32(f32_to_bf16_bits(dequantize(W_q))).astype(np.float64)


def int8_linear_forward(X_bits, W_q: QTensor):
    """App. A, forward: Y = X W^T with W dequantized on the fly.  X is T x n (bfloat16 bit patterns), W is
    m x n, Y is T x m.  No bias (the listing names one without defining it; the LLaMA layers have none).
    Returns (Y exact in float64, Y rounded to bfloat16 bit patterns)."""
    X = bf16_bits_to_f32(X_bits).astype(np.float64)
    Y = X @ _weight_operand(W_q).T
    return Y, f32_to_bf16_bits(fl32(Y))


def int8_linear_backward(dY_bits, X_bits, W_q: QTensor):
    """App. A, backward: grad_input = dY W (T x n) and grad_W = dY^T X (m x n), the latter being the gradient
    G the optimizer step consumes.  Returns (dX exact, dX bf16 bits, G exact, G bf16 bits)."""
    dY = bf16_bits_to_f32(dY_bits).astype(np.float64)
    X = bf16_bits_to_f32(X_bits).astype(np.float64)
    dX = dY @ _weight_operand(W_q)
    G = dY.T @ X
    return dX, f32_to_bf16_bits(fl32(dX)), G, f32_to_bf16_bits(fl32(G))
