"""Pins of the CPU oracle against facts that do not come from the oracle itself.

Each test fixes a part of oracle/qgalore_oracle.py to something the paper or the
mathematics determines: published known answers, error bounds, expectations,
reductions to textbook routines written out here independently, brute force on
tiny inputs.  CPU only.
"""
import math
import os

import numpy as np
import pytest

import oracle as O
from paper_2407_08296_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- bfloat16 rounding
def test_bf16_rounding_is_nearest_with_ties_to_even():
    """The rounding point the step crosses twice (P~ and N_b).  bfloat16 keeps the top 16 bits of a binary32;
    hand-made cases: exact values stay; 1 + 2^-8 lies midway between 0x3F80 and 0x3F81 and goes to the even
    one, 0x3F80; 1 + 3 * 2^-8 lies midway between 0x3F81 and 0x3F82 and goes to 0x3F82 (truncation would give
    0x3F81, round-half-up would give 0x3F81 for the first); just above and below a midpoint; negative values
    mirror; the largest binary32 below 2 rounds up into the next binade.  Then torch's own conversion on
    random values and on every midpoint of one binade."""
    import torch
    cases = [
        (1.0, 0x3F80), (1.0 + 2.0 ** -7, 0x3F81), (-2.5, 0xC020), (0.0, 0x0000),
        (1.0 + 2.0 ** -8, 0x3F80), (1.0 + 3 * 2.0 ** -8, 0x3F82),
        (1.0 + 2.0 ** -8 + 2.0 ** -23, 0x3F81), (1.0 + 2.0 ** -8 - 2.0 ** -23, 0x3F80),
        (-(1.0 + 2.0 ** -8), 0xBF80), (-(1.0 + 3 * 2.0 ** -8), 0xBF82),
        (2.0 - 2.0 ** -23, 0x4000), (3.0e-3, 0x3B45),     # 3.0e-3 = 0x3B449BA6 in binary32: low half above 0x8000, up
    ]
    for value, bits in cases:
        x = np.array([value], np.float32)
        assert int(O.f32_to_bf16_bits(x)[0]) == bits, (value, hex(int(O.f32_to_bf16_bits(x)[0])))
        assert int(synth.to_bf16_bits(x)[0]) == bits
        back = O.bf16_round(x)
        assert back.dtype == np.float32 and back.view(np.uint32)[0] == bits << 16
        assert O.bf16_bits_to_f32(np.array([bits], np.uint16)).view(np.uint32)[0] == bits << 16
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(200000).astype(np.float32) * np.float32(s) for s in (1.0, 1e-3, 1e-20, 1e20)])
    mids = ((np.arange(0x3F80, 0x4000, dtype=np.uint32) << np.uint32(16)) | np.uint32(0x8000)).view(np.float32)
    x = np.concatenate([x, mids, -mids])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f32_to_bf16_bits(x), want)
    assert np.array_equal(synth.to_bf16_bits(x), want)


# ----------------------------------------------------------------------------- Philox
def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([int(w, 16) for w in line.split()])
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for w in rows:
        out = O.philox4x32_10([np.array([c], dtype=np.uint32) for c in w[:4]], w[4:6])
        assert [int(o[0]) for o in out] == w[6:10]


def test_sr_uniform16_lane_mapping():
    seed, step = (0x1234 << 32) | 0xABCDEF01, (7 << 32) | 99
    h = O.sr_uniform16(seed, step, 5, 37)
    for i, j in [(0, 0), (0, 1), (3, 7), (4, 8), (2, 36), (1, 22)]:
        x = O.philox4x32_10(
            [np.array([v], dtype=np.uint32) for v in (j >> 3, i, step & 0xFFFFFFFF, step >> 32)],
            (seed & 0xFFFFFFFF, seed >> 32))
        lane = j & 7
        want = (int(x[lane >> 1][0]) >> (16 * (lane & 1))) & 0xFFFF
        assert int(h[i, j]) == want
    # a window taken with (row0, col0) is the same as slicing the whole field
    win = O.sr_uniform16(seed, step, 2, 11, row0=2, col0=13)
    assert np.array_equal(win, h[2:4, 13:24])
    assert h.max() <= 0xFFFF


def test_sr_uniform16_is_uniform():
    h = O.sr_uniform16(5, 3, 2000, 512).astype(np.float64)
    assert abs(h.mean() - 32767.5) < 4 * 65536 / math.sqrt(12 * h.size)
    hist = np.bincount((h // 4096).astype(np.int64).ravel(), minlength=16)
    expect = h.size / 16
    assert np.all(np.abs(hist - expect) < 5 * math.sqrt(expect))


# ----------------------------------------------------------------------------- quantizer (Sec. 3.1)
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("cols", [256, 1376, 85, 600])
def test_quantizer_half_step_bound_and_range(bits, cols):
    rng = np.random.default_rng(bits * 1000 + cols)
    x = (rng.standard_normal((64, cols)) * 0.02).astype(np.float32)
    q = O.quantize_rtn(x, bits)
    qlo, qhi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1          # clamp range of the Quant_n equation
    assert q.codes.min() >= qlo and q.codes.max() <= qhi
    ngroups = (cols + 255) // 256
    assert q.scales.shape == (64, ngroups) and q.zeros.shape == (64, ngroups)
    xh = O.dequantize(q)
    for k in range(ngroups):
        a, b = k * 256, min(cols, k * 256 + 256)
        s = q.scales[:, k:k + 1].astype(np.float64)
        err = np.abs(xh[:, a:b].astype(np.float64) - x[:, a:b])
        assert np.all(err <= 0.5 * s * (1 + 1e-3))                  # half a group step
        seg, cod = x[:, a:b], q.codes[:, a:b]
        rows = np.arange(64)
        assert np.all(cod[rows, seg.argmin(axis=1)] == qlo)         # group minimum -> lowest code
        assert np.all(cod[rows, seg.argmax(axis=1)] == qhi)         # group maximum -> highest code
        # the scale is (max - min) / (2^n - 1)
        want = (seg.max(axis=1).astype(np.float64) - seg.min(axis=1)) / ((1 << bits) - 1)
        assert np.allclose(q.scales[:, k], want, rtol=3e-7)
    assert np.all(q.zeros == np.rint(q.zeros))


@pytest.mark.parametrize("bits", [4, 8])
def test_requantizing_a_dequantized_tensor_reproduces_codes(bits):
    rng = np.random.default_rng(11 + bits)
    x = rng.standard_normal((32, 700)).astype(np.float32)
    q1 = O.quantize_rtn(x, bits)
    q2 = O.quantize_rtn(O.dequantize(q1), bits)
    assert np.array_equal(q1.codes, q2.codes)
    assert np.allclose(q1.scales, q2.scales, rtol=2.5e-7)
    assert np.array_equal(q1.zeros, q2.zeros)


def test_quantizer_hand_example():
    # group {0, 1, ..., 255} / 4: min 0, max 63.75, s = 0.25 exactly, z = -128, code = k - 128
    x = (np.arange(256, dtype=np.float32) / 4)[None, :]
    q = O.quantize_rtn(x, 8)
    assert q.scales[0, 0] == np.float32(0.25) and q.zeros[0, 0] == -128
    assert np.array_equal(q.codes[0], np.arange(256) - 128)
    assert np.array_equal(O.dequantize(q), x)
    # INT4: {-7.5, -6.5, ..., 7.5}: s = 1, min * inv = -7.5 -> rint -8 (ties to even), z = 0
    x4 = (np.arange(16, dtype=np.float32) - 7.5)[None, :]
    q4 = O.quantize_rtn(x4, 4)
    assert q4.scales[0, 0] == 1 and q4.zeros[0, 0] == 0
    # rint(-7.5) = -8, rint(-6.5) = -6, rint(-5.5) = -6 ... ties to even
    assert np.array_equal(q4.codes[0], np.clip(np.rint(x4[0]), -8, 7).astype(np.int8))


def test_quantizer_degenerate_groups():
    x = np.zeros((3, 300), dtype=np.float32)
    x[1, :] = 0.5
    x[2, :256] = -3.0
    x[2, 256:] = np.linspace(-1, 1, 44, dtype=np.float32)
    q = O.quantize_rtn(x, 8)
    assert q.scales[0, 0] == 1 and q.zeros[0, 0] == 0 and np.all(q.codes[0] == 0)
    assert q.scales[1, 0] == np.float32(0.5) and np.all(q.codes[1] == 1)
    assert q.scales[2, 0] == 3 and np.all(q.codes[2, :256] == -1)
    assert np.array_equal(O.dequantize(q)[:, :256], x[:, :256])
    # a group symmetric about 0 puts min/s and max/s on rounding ties (-127.5, 127.5); with the
    # reciprocal rounded to binary32 the top code may come out one below the clamp edge
    assert q.codes[2, 256] == -128 and q.codes[2, 299] in (126, 127)
    assert np.all(np.abs(O.dequantize(q)[2, 256:] - x[2, 256:]) <= 0.5 * q.scales[2, 1] * (1 + 1e-3))


def test_int4_packing_layout():
    codes = np.array([[-8, 7, 0, -1, 3]], dtype=np.int8)
    p = O.pack_int4(codes)
    # byte k = (q[2k] + 8) | (q[2k+1] + 8) << 4 ; odd tail padded with code 0
    assert p.tolist() == [[0 | (15 << 4), 8 | (7 << 4), 11 | (8 << 4)]]
    assert np.array_equal(O.unpack_int4(p, 5), codes)
    rng = np.random.default_rng(0)
    c = rng.integers(-8, 8, size=(7, 130)).astype(np.int8)
    assert np.array_equal(O.unpack_int4(O.pack_int4(c), 130), c)


# ----------------------------------------------------------------------------- stochastic rounding (Sec. 3.4)
FRACS = [0.0, 2.0 ** -16, 0.01, 0.25, 0.5, 0.75, 0.99]


def _sr_field(rows):
    """Groups whose scale is exactly 1: element 0 = -100 (min), element 1 = 155 (max), the rest
    k + frac with 36 columns per fraction.  Two groups per row."""
    g = np.zeros(256, dtype=np.float32)
    g[0], g[1] = -100.0, 155.0
    fr = np.zeros(256, dtype=np.float32)
    for f_i, f in enumerate(FRACS):
        cols = 2 + f_i * 36 + np.arange(36)
        ints = (np.arange(36) * 5 - 90).astype(np.float32)
        g[cols] = ints + np.float32(f)
        fr[cols] = f
    g[2 + 7 * 36:] = 3.0
    x = np.tile(np.concatenate([g, g])[None, :], (rows, 1))
    return x, np.concatenate([fr, fr])


def test_sr_expectation_equals_input():
    rows = 100_000                                    # 10^5 draws per element
    x, _ = _sr_field(rows)
    q = O.quantize_sr(x, seed=42, step=3)
    assert np.all(q.scales == 1) and np.all(q.zeros == -28)
    val = O.dequantize(q).astype(np.float64)          # = floor(x) + up
    lo = np.floor(x[0].astype(np.float64))
    assert np.all((val == lo) | (val == lo + 1))      # only floor or ceil ever appear
    mean = val.mean(axis=0)
    xt = x[0].astype(np.float64)
    frac = xt - lo
    # per element: 4 sigma of a binomial mean; 16-bit draws add a bias below 2^-16
    sigma = np.sqrt(np.maximum(frac * (1 - frac), 1e-12) / rows)
    assert np.all(np.abs(mean - xt) <= 4 * sigma + 2.0 ** -16 + 1e-9)
    # pooled over the 72 columns that share a fraction: E[W_q] = W to 1e-3 LSB
    for f_i in range(len(FRACS)):
        cols = np.concatenate([2 + f_i * 36 + np.arange(36), 256 + 2 + f_i * 36 + np.arange(36)])
        assert abs((mean[cols] - xt[cols]).mean()) < 1e-3
    # exact integers never move
    zc = np.concatenate([2 + np.arange(36), 256 + 2 + np.arange(36)])
    assert np.all(val[:, zc] == xt[zc])


def test_sr_accumulates_sub_lsb_updates_where_rtn_loses_them():
    # Sec. 3.4: a small update vanishes under round-to-nearest and survives, in expectation, under SR.
    rows = 4
    base = np.zeros((rows, 256), dtype=np.float32)
    base[:, 0], base[:, 1] = -100.0, 155.0            # pins the scale at 1
    base[:, 2:] = 10.0
    w_rtn, w_sr = base.copy(), base.copy()
    for step in range(1, 201):
        for w, fn in ((w_rtn, lambda v: O.quantize_rtn(v, 8)), (w_sr, lambda v: O.quantize_sr(v, 9, step))):
            upd = w.copy()
            upd[:, 2:] += np.float32(0.1)             # a tenth of one LSB
            w[:] = O.dequantize(fn(upd))
    assert np.all(w_rtn[:, 2:] == 10.0)
    drift = w_sr[:, 2:].astype(np.float64).mean() - 10.0
    assert abs(drift - 20.0) < 1.0                    # 200 * 0.1 LSB, std error about 0.13


# ----------------------------------------------------------------------------- the step (Sec. 3.5)
def _dense_adam(grads, lr, b1=0.9, b2=0.999, eps=1e-8):
    """Textbook Adam (Kingma & Ba, Algorithm 1) on a dense parameter; returns the summed update."""
    b1, b2, eps, lr = (float(np.float32(v)) for v in (b1, b2, eps, lr))
    m = np.zeros_like(grads[0], dtype=np.float64)
    v = np.zeros_like(m)
    total = np.zeros_like(m)
    for t, g in enumerate(grads, start=1):
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g * g
        total += lr * (m / (1 - b1 ** t)) / (np.sqrt(v / (1 - b2 ** t)) + eps)
    return total, m, v


def _w_q(m, n, seed=0):
    return O.quantize_rtn(synth.initial_weight(m, n, seed), 8)


def _dummy_p(m, r):
    return O.quantize_rtn(np.zeros((m, r), dtype=np.float32), 4)


def test_full_rank_signed_permutation_reduces_to_dense_adam():
    m, n = 24, 300
    rng = np.random.default_rng(3)
    perm = rng.permutation(m)
    P = np.zeros((m, m))
    P[perm, np.arange(m)] = rng.choice([-1.0, 1.0], size=m)       # orthonormal, r = m
    gm = synth.GradientModel(m, n, seed=1)
    W = _w_q(m, n)
    M = np.zeros((m, n), dtype=np.float32)
    V = np.zeros((m, n), dtype=np.float32)
    grads, w_hat0 = [], O.dequantize(W).astype(np.float64)
    h = O.Hyper(lr=0.004, alpha=0.25)
    acc = np.zeros((m, n))
    for t in (1, 2, 3):
        gb = gm.sample(t)
        grads.append(synth.bf16_bits_to_float(gb).astype(np.float64))
        h.step = t
        w_before = O.dequantize(W).astype(np.float64)
        out = O.project_step(gb, _dummy_p(m, m), W, M, V, h, P_override=P)
        acc += out["W_pre"].astype(np.float64) - w_before              # the applied (pre-rounding) update
        W, M, V = out["W"], out["M"], out["V"]
    total, m_d, v_d = _dense_adam(grads, lr=float(np.float32(0.004)) * 0.25)
    assert np.allclose(-acc, total, rtol=2e-5, atol=3e-8)      # W_pre is binary32: ulp(0.06) = 4e-9 per step
    # moments live in the rotated basis: P M = dense first moment, |P| V = dense second moment
    assert np.allclose(P @ M.astype(np.float64), m_d, rtol=1e-5, atol=1e-12)
    assert np.allclose(np.abs(P) @ V.astype(np.float64), v_d, rtol=1e-5, atol=1e-15)
    assert w_hat0.shape == (m, n)


def test_full_rank_rotation_is_adam_in_rotated_coordinates():
    m, n = 16, 260
    Q, _ = np.linalg.qr(np.random.default_rng(5).standard_normal((m, m)))
    gb = synth.GradientModel(m, n, seed=2).sample(1)
    G = synth.bf16_bits_to_float(gb).astype(np.float64)
    W = _w_q(m, n)
    out = O.project_step(gb, _dummy_p(m, m), W, np.zeros((m, n), np.float32), np.zeros((m, n), np.float32),
                         O.Hyper(step=1), P_override=Q)
    total, _, _ = _dense_adam([Q.T @ G], lr=float(np.float32(0.004)) * 0.25)
    lhs = Q.T @ (out["W_pre"].astype(np.float64) - O.dequantize(W))
    assert np.allclose(-lhs, total, rtol=1e-4, atol=1e-8)


def test_step_tiny_orientation_example():
    # m = 2, n = 3, r = 1, P = e_1: R is G's first row, the update touches row 0 only.
    P = O.quantize_rtn(np.array([[1.0], [0.0]], dtype=np.float32), 4)
    assert np.array_equal(O.dequantize(P), [[1.0], [0.0]])
    G = np.array([[0.5, -0.25, 2.0], [4.0, 8.0, -16.0]], dtype=np.float32)
    W = O.quantize_rtn(np.array([[0.0, 0.5, 1.0], [-1.0, 0.0, 1.0]], dtype=np.float32), 8, group=256)
    out = O.project_step(synth.to_bf16_bits(G), P, W, np.zeros((1, 3), np.float32), np.zeros((1, 3), np.float32),
                         O.Hyper(lr=0.5, alpha=0.25, step=1))
    assert np.array_equal(out["R32"], G[:1])
    assert np.allclose(out["M"], (1 - float(np.float32(0.9))) * G[:1], rtol=1e-6)
    assert np.allclose(out["V"], (1 - float(np.float32(0.999))) * G[:1] ** 2, rtol=1e-6)  # beta2 travels as binary32
    assert np.allclose(out["N"], np.sign(G[:1]), atol=1e-6)            # t = 1: N = R / (|R| + eps)
    w_hat = O.dequantize(W)
    assert np.allclose(out["W_pre"][0], w_hat[0] - 0.125 * np.sign(G[0]), atol=1e-6)
    assert np.array_equal(out["W_pre"][1], w_hat[1])


def test_step_closed_form_at_t1_and_linearity():
    m, n, r = 64, 512, 16
    gb = synth.GradientModel(m, n, seed=4).sample(1)
    Pq = O.quantize_rtn(synth.random_orthonormal(m, r, seed=4), 4)
    W = _w_q(m, n, 4)
    z = np.zeros((r, n), np.float32)
    out = O.project_step(gb, Pq, W, z, z, O.Hyper(step=1))
    Pt = O.bf16_round(O.dequantize(Pq)).astype(np.float64)
    G = synth.bf16_bits_to_float(gb).astype(np.float64)
    R = Pt.T @ G
    assert np.allclose(out["R32"], R, rtol=1e-6, atol=1e-12)
    eps = float(np.float32(1e-8))
    assert np.allclose(out["N"], R / (np.abs(R) + eps), rtol=1e-5, atol=1e-7)
    Nb = O.bf16_round(out["N"]).astype(np.float64)
    want = O.dequantize(W).astype(np.float64) - float(np.float32(0.004)) * 0.25 * (Pt @ Nb)
    assert np.allclose(out["W_pre"], want, rtol=1e-6, atol=1e-9)
    # linearity of the projection in G: doubling G (exact in bfloat16) doubles R exactly
    G2 = synth.to_bf16_bits(2 * synth.bf16_bits_to_float(gb))
    out2 = O.project_step(G2, Pq, W, z, z, O.Hyper(step=1))
    assert np.array_equal(out2["R32"], 2 * out["R32"])
    # and the sum of two integer-valued gradients projects to the sum of the projections
    rng = np.random.default_rng(8)
    Ga = rng.integers(-8, 9, size=(m, n)).astype(np.float32)
    Gb = rng.integers(-8, 9, size=(m, n)).astype(np.float32)
    Ra, Rb, Rab = (O.project_step(synth.to_bf16_bits(g), Pq, W, z, z, O.Hyper(step=1))["R32"].astype(np.float64)
                   for g in (Ga, Gb, Ga + Gb))
    assert np.allclose(Rab, Ra + Rb, rtol=0, atol=2e-5)


def test_step_zero_gradient_decays_moments_and_keeps_weights():
    m, n, r = 32, 600, 8
    rng = np.random.default_rng(6)
    Pq = O.quantize_rtn(synth.random_orthonormal(m, r, seed=6), 4)
    W = _w_q(m, n, 6)
    M = rng.standard_normal((r, n)).astype(np.float32)
    V = (rng.standard_normal((r, n)) ** 2).astype(np.float32)
    # moments that make N = 0 as well: M = 0
    out = O.project_step(np.zeros((m, n), np.uint16), Pq, W, np.zeros_like(M), V, O.Hyper(step=5, seed=1))
    assert np.all(out["R32"] == 0) and np.all(out["M"] == 0) and np.all(out["N"] == 0)
    assert np.array_equal(out["V"], O.fl32(float(np.float32(0.999)) * V.astype(np.float64)))
    assert np.array_equal(out["W_pre"], O.dequantize(W))
    mism = out["W"].codes != W.codes
    assert mism.mean() < 1e-3
    assert np.all(np.abs(out["W"].codes.astype(int) - W.codes.astype(int)) <= 1)
    out_m = O.project_step(np.zeros((m, n), np.uint16), Pq, W, M, V, O.Hyper(step=5, seed=1))
    assert np.array_equal(out_m["M"], O.fl32(float(np.float32(0.9)) * M.astype(np.float64)))


def test_step_sr_codes_follow_the_philox_lanes():
    # the weight codes are floor(T) + [frac(T) * 65536 > h] + z, with h the element's Philox lane
    m, n, r = 16, 700, 8
    gb = synth.GradientModel(m, n, seed=7).sample(1)
    Pq = O.quantize_rtn(synth.random_orthonormal(m, r, seed=7), 4)
    W = _w_q(m, n, 7)
    z = np.zeros((r, n), np.float32)
    seed, t = synth.matrix_seed(3, 5), 17
    out = O.project_step(gb, Pq, W, z, z, O.Hyper(step=t, seed=seed))
    T = out["T"].astype(np.float64)
    h = O.sr_uniform16(seed, t, m, n).astype(np.float64)
    up = ((T - np.floor(T)) * 65536 > h)
    zeros = np.repeat(out["W"].zeros, 256, axis=1)[:, :n]
    want = np.clip(np.floor(T) + up + zeros, -128, 127)
    assert np.array_equal(out["W"].codes, want.astype(np.int8))
    assert 0.3 < up.mean() < 0.7


# ----------------------------------------------------------------------------- refresh (Sec. 3.5)
def _jacobi_eigh(A, sweeps=30):
    """Cyclic Jacobi eigenvalue iteration for a small symmetric matrix (textbook, written out)."""
    A = A.copy()
    n = A.shape[0]
    Vv = np.eye(n)
    for _ in range(sweeps):
        off = 0.0
        for p in range(n - 1):
            for q in range(p + 1, n):
                off += A[p, q] ** 2
                if abs(A[p, q]) < 1e-300:
                    continue
                theta = (A[q, q] - A[p, p]) / (2 * A[p, q])
                tt = math.copysign(1.0, theta) / (abs(theta) + math.sqrt(theta * theta + 1))
                c = 1 / math.sqrt(tt * tt + 1)
                s = tt * c
                J = np.eye(n)
                J[p, p] = J[q, q] = c
                J[p, q], J[q, p] = s, -s
                A = J.T @ A @ J
                Vv = Vv @ J
        if off < 1e-30:
            break
    w = np.diag(A)
    order = np.argsort(-w)
    return w[order], Vv[:, order]


def test_refresh_matches_brute_force_jacobi_on_8x8():
    rng = np.random.default_rng(12)
    G = synth.bf16_bits_to_float(synth.to_bf16_bits(rng.standard_normal((8, 8)))).astype(np.float64)
    w, Vv = _jacobi_eigh(G @ G.T)
    for r in (1, 3, 8):
        P, Pq, S = O.refresh_subspace(synth.to_bf16_bits(G), r)
        assert np.allclose(S[:8] ** 2, w, rtol=1e-10)
        for j in range(r):                                         # distinct singular values: columns match up to sign
            assert abs(abs(P[:, j].astype(np.float64) @ Vv[:, j]) - 1) < 1e-5
        piv = np.argmax(np.abs(P), axis=0)
        assert np.all(P[piv, np.arange(r)] > 0)                    # canonical sign
        assert Pq.bits == 4 and Pq.codes.shape == (8, r)


def test_refresh_orthonormal_energy_and_rank_one():
    m, n, r = 96, 200, 24
    gb = synth.GradientModel(m, n, seed=13).sample(1)
    G = synth.bf16_bits_to_float(gb).astype(np.float64)
    P, Pq, S = O.refresh_subspace(gb, r)
    assert np.abs(P.astype(np.float64).T @ P - np.eye(r)).max() <= 1e-5
    ev = np.sort(np.linalg.eigvalsh(G.T @ G))[::-1]                # singular values by another route
    captured = np.linalg.norm(P.astype(np.float64).T @ G, "fro") ** 2
    assert abs(captured - ev[:r].sum()) <= 1e-5 * ev[:r].sum()
    # INT4 copy stays within half a step of P
    assert np.all(np.abs(O.dequantize(Pq) - P) <= 0.5 * Pq.scales.max() * (1 + 1e-3))
    # rank one: G = sigma u v^T gives +-u as the first column
    rng = np.random.default_rng(14)
    u = rng.standard_normal(m); u /= np.linalg.norm(u)
    v = rng.standard_normal(n); v /= np.linalg.norm(v)
    gb1 = synth.to_bf16_bits(3.0 * np.outer(u, v))
    P1, _, S1 = O.refresh_subspace(gb1, 2)
    assert abs(abs(P1[:, 0].astype(np.float64) @ u) - 1) < 1e-4     # bfloat16 rounding of G perturbs u slightly
    assert abs(S1[0] - 3.0) < 2e-2
    assert O.principal_angle(P, P) < 1e-7
    assert abs(O.principal_angle(np.eye(4)[:, :2], np.eye(4)[:, [0, 2]]) - math.pi / 2) < 1e-7
    c, s = math.cos(0.01), math.sin(0.01)
    assert abs(O.principal_angle(np.eye(3)[:, :1], np.array([[c], [s], [0.0]])) - 0.01) < 1e-9


# ----------------------------------------------------------------------------- similarity and gate (Sec. 3.2)
def _negated(q):
    # -(q - z) s = (q' - z') s with q' = -q - 1, z' = -z - 1: stays inside [-8, 7]
    return O.QTensor((-q.codes.astype(np.int16) - 1).astype(np.int8), q.scales.copy(), -q.zeros - 1, q.bits, q.group)


def test_similarity_closed_forms():
    m, r = 512, 64
    A = O.quantize_rtn(synth.random_orthonormal(m, r, seed=1, stream=1), 4)
    B = O.quantize_rtn(synth.random_orthonormal(m, r, seed=1, stream=2), 4)
    assert abs(O.subspace_similarity(A, A) - 1) < 1e-12
    nA = _negated(A)
    assert np.array_equal(O.dequantize(nA), -O.dequantize(A))
    assert abs(O.subspace_similarity(A, nA) - 1) < 1e-12
    indep = O.subspace_similarity(A, B)
    assert abs(indep - math.sqrt(2 / (math.pi * m))) < 0.01         # E|cos| of independent unit vectors
    perm = O.QTensor(np.roll(A.codes, 1, axis=1), np.roll(A.scales, 0), A.zeros.copy(), 4)
    assert O.subspace_similarity(A, perm) < 0.1
    # the leading-columns variant ignores the tail
    mix = O.QTensor(np.concatenate([A.codes[:, :8], B.codes[:, 8:]], axis=1), A.scales, A.zeros, 4)
    assert abs(O.subspace_similarity(A, mix, sim_cols=8) - 1) < 1e-12
    # hand example: a = (1, 0), b = (1, 1)/.. through exact codes
    a = O.QTensor(np.array([[1], [0]], np.int8), np.ones((2, 1), np.float32), np.zeros((2, 1), np.float32), 4)
    b = O.QTensor(np.array([[1], [1]], np.int8), np.ones((2, 1), np.float32), np.zeros((2, 1), np.float32), 4)
    assert abs(O.subspace_similarity(a, b) - 1 / math.sqrt(2)) < 1e-12


def test_gate_scripted_sequences():
    # k = 1: every similarity >= threshold doubles the interval (Sec. 3.2: t -> 2t)
    st = O.GateState(interval=200)
    assert O.gate_update(st, 0.39999, 0.4, 1) is False and st.interval == 200
    assert O.gate_update(st, 0.4, 0.4, 1) is True and st.interval == 400      # ">= 40%": equality counts
    assert O.gate_update(st, 0.9, 0.4, 1) is True and st.interval == 800
    # k = 2: needs two in a row, history cleared after a doubling
    st = O.GateState(interval=200)
    seq = [0.5, 0.3, 0.5, 0.6, 0.7, 0.8]
    got = [O.gate_update(st, s, 0.4, 2) for s in seq]
    assert got == [False, False, False, True, False, True] and st.interval == 800
    # k = 3 with a dip resets nothing but delays the doubling
    st = O.GateState(interval=100)
    got = [O.gate_update(st, s, 0.4, 3) for s in [0.9, 0.9, 0.1, 0.9, 0.9, 0.9]]
    assert got == [False, False, False, False, False, True] and st.interval == 200


# ----------------------------------------------------------------------------- inputs
def test_synthetic_gradient_recipe():
    gm = synth.GradientModel(256, 384, seed=0)
    g = synth.bf16_bits_to_float(gm.sample(1)).astype(np.float64)
    s = np.linalg.svd(g, compute_uv=False)
    assert abs(s[0] - 1.0) < 0.02 and abs(s[1] - 0.5) < 0.02       # planted 1/k spectrum on top
    assert 0.8e-3 < np.std(g - gm.signal()) < 1.2e-3                # noise level 1e-3
    assert np.array_equal(gm.sample(3), synth.GradientModel(256, 384, seed=0).sample(3))
    assert not np.array_equal(gm.sample(3), gm.sample(4))
    assert len(synth.stack_matrices("llama130m")) == 84 and len(synth.stack_matrices("llama7b")) == 224
    assert sum(s.m * s.n for s in synth.stack_matrices("llama1b")) == 24 * (4 * 2048 * 2048 + 3 * 2048 * 5461)
    shapes = {(m, n, r): c for m, n, r, c in synth.distinct_shapes("llama1b")}
    assert shapes == {(2048, 2048, 512): 96, (2048, 5461, 512): 48, (5461, 2048, 512): 24}


def test_step_of_a_column_block_equals_the_block_of_the_full_step():
    # Sec. 3.5: R = P^T G, Adam, P N and the row-wise groups act on each column block on its own, so the
    # oracle may be run on a few blocks of a matrix too large to run whole; col0 only moves the Philox lanes.
    from paper_2407_08296_b200 import synth
    m, n, r = 96, 256 * 2 + 85, 32
    gb = synth.GradientModel(m, n, seed=3, matrix_index=0).sample(2)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=3), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 3), 8)
    rng = np.random.default_rng(7)
    M = rng.normal(0, 1e-3, (r, n)).astype(np.float32)
    V = (rng.normal(0, 1e-3, (r, n)) ** 2).astype(np.float32)
    hyp = O.Hyper(step=2, seed=11)
    full = O.project_step(gb, P, W, M, V, hyp)
    for (a, b) in [(0, 256), (256, 512), (512, n)]:
        Wb = O.QTensor(W.codes[:, a:b], W.scales[:, a // 256:(b + 255) // 256], W.zeros[:, a // 256:(b + 255) // 256], 8)
        blk = O.project_step(gb[:, a:b], P, Wb, M[:, a:b], V[:, a:b], hyp, col0=a)
        assert np.array_equal(blk["W"].codes, full["W"].codes[:, a:b])
        assert np.array_equal(blk["W"].scales, full["W"].scales[:, a // 256:(b + 255) // 256])
        assert np.array_equal(blk["M"], full["M"][:, a:b]) and np.array_equal(blk["V"], full["V"][:, a:b])
        assert np.array_equal(blk["W_pre"], full["W_pre"][:, a:b])
    # without the offset the second block draws other uniforms
    Wb = O.QTensor(W.codes[:, 256:512], W.scales[:, 1:2], W.zeros[:, 1:2], 8)
    assert not np.array_equal(O.project_step(gb[:, 256:512], P, Wb, M[:, 256:512], V[:, 256:512], hyp)["W"].codes,
                              full["W"].codes[:, 256:512])


def test_round_to_nearest_step_is_the_same_step_with_quant8_at_the_end():
    # Sec. 4.4 (Fig. 6) ablates stochastic rounding against round to nearest: everything before the last
    # quantization is untouched by the choice, the nearest codes are Quant_8 of the pre-rounding weight, no
    # code is further than one level from the stochastic one, and the seed no longer matters.
    from paper_2407_08296_b200 import synth
    m, n, r = 64, 256 + 85, 32
    gb = synth.GradientModel(m, n, seed=5, matrix_index=0).sample(1)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=5), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 5), 8)
    z = np.zeros((r, n), np.float32)
    sr = O.project_step(gb, P, W, z, z, O.Hyper(step=1, seed=3))
    rtn = O.project_step(gb, P, W, z, z, O.Hyper(step=1, seed=3, rounding="rtn"))
    rtn2 = O.project_step(gb, P, W, z, z, O.Hyper(step=1, seed=4, rounding="rtn"))
    sr2 = O.project_step(gb, P, W, z, z, O.Hyper(step=1, seed=4))
    assert np.array_equal(sr["W_pre"], rtn["W_pre"]) and np.array_equal(sr["M"], rtn["M"]) and np.array_equal(sr["V"], rtn["V"])
    assert np.array_equal(sr["W"].scales, rtn["W"].scales) and np.array_equal(sr["W"].zeros, rtn["W"].zeros)
    q8 = O.quantize_rtn(rtn["W_pre"], 8)
    assert np.array_equal(rtn["W"].codes, q8.codes)
    d = np.abs(rtn["W"].codes.astype(np.int32) - sr["W"].codes.astype(np.int32))
    assert d.max() == 1 and 0.2 < (d != 0).mean() < 0.8          # a coin per element, never two levels
    assert np.array_equal(rtn["W"].codes, rtn2["W"].codes) and not np.array_equal(sr["W"].codes, sr2["W"].codes)
    # nearest: the dequantized result is within half a level of the pre-rounding weight inside the clamp range
    lsb = np.repeat(rtn["W"].scales, 256, axis=1)[:, :n]
    assert np.all(np.abs(O.dequantize(rtn["W"]) - rtn["W_pre"]) <= 0.5 * lsb * (1 + 1e-5) + 1e-12)


def test_int2_quantizer_levels_bound_and_packing():
    # Quant_n of Sec. 3.1 with n = 2 (the 2-bit projection of Sec. 4.4): four levels per group, the group's
    # minimum and maximum take the end codes, every value lands within half a step, packing round-trips.
    rng = np.random.default_rng(3)
    x = rng.normal(0, 0.03, (16, 256 * 2 + 40)).astype(np.float32)
    q = O.quantize_rtn(x, 2)
    assert q.codes.min() == -2 and q.codes.max() == 1
    xh = O.dequantize(q)
    step = np.repeat(q.scales, 256, axis=1)[:, :x.shape[1]]
    assert np.all(np.abs(xh - x) <= 0.5 * step * (1 + 1e-5) + 1e-12)
    for g, (a, b) in enumerate([(0, 256), (256, 512), (512, 552)]):
        seg, codes = x[:, a:b], q.codes[:, a:b]
        rows = np.arange(16)
        assert np.all(codes[rows, seg.argmin(axis=1)] == -2) and np.all(codes[rows, seg.argmax(axis=1)] == 1)
        assert np.allclose(q.scales[:, g], (seg.max(axis=1) - seg.min(axis=1)) / 3.0, rtol=1e-6)
    packed = O.pack_int2(q.codes)
    assert packed.shape == (16, (552 + 3) // 4)
    assert np.array_equal(O.unpack_int2(packed, 552), q.codes)
    # byte layout: column 4k + i in bits 2i, 2i + 1, stored as code + 2
    c = np.array([[-2, -1, 0, 1, 1, 0, -1, -2]], dtype=np.int8)
    assert O.pack_int2(c).tolist() == [[0b11100100, 0b00011011]]


def test_coarser_projection_loses_more_of_the_subspace():
    # Sec. 3.3 / Fig. 3: the projection tolerates 4 bits; fewer bits reproduce the orthonormal basis worse.
    from paper_2407_08296_b200 import synth
    P = synth.random_orthonormal(512, 128, seed=1)
    err = {}
    for bits in (2, 4, 8):
        Ph = O.dequantize(O.quantize_rtn(P, bits)).astype(np.float64)
        err[bits] = np.linalg.norm(Ph.T @ Ph - np.eye(128)) / np.sqrt(128)
    assert err[8] < err[4] < err[2] and err[8] < 1e-2 and err[2] > 0.1


def test_right_projection_is_the_left_projection_of_the_transposed_gradient():
    # GaLore projects on the side of the shorter dimension; R = G Q is (Q^T G^T)^T, so the low-rank state of the
    # right form on G is that of the left form on G^T, and the two updates are transposes of each other.  The
    # weights differ (quantization groups run along the rows of W either way), so they are compared through D.
    from paper_2407_08296_b200 import synth
    m, n, r = 300, 128, 32
    gb = synth.GradientModel(m, n, seed=8, matrix_index=0).sample(1)
    Q = O.quantize_rtn(synth.random_orthonormal(n, r, seed=8), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 8), 8)
    Wt = O.quantize_rtn(synth.initial_weight(n, m, 8), 8)
    rng = np.random.default_rng(8)
    Mt = rng.normal(0, 1e-3, (r, m)).astype(np.float32)
    Vt = (rng.normal(0, 1e-3, (r, m)) ** 2).astype(np.float32)
    hyp = O.Hyper(step=3, seed=1)
    right = O.project_step(gb, Q, W, Mt, Vt, hyp, side="right")
    left = O.project_step(np.ascontiguousarray(gb.T), Q, Wt, Mt, Vt, hyp)
    assert right["M"].shape == (r, m)
    for k in ("R32", "M", "V"):
        assert np.allclose(right[k], left[k], rtol=1e-6, atol=1e-12), k
    good = np.sqrt(left["V"].astype(np.float64) / (1 - 0.999 ** 3)) > 1e-5
    assert np.allclose(right["N"][good], left["N"][good], rtol=1e-4)
    # with the same direction on both sides the two updates are transposes
    right_f = O.project_step(gb, Q, W, Mt, Vt, hyp, side="right", N_b_override=left["N_b"])
    d_right = (O.dequantize(W).astype(np.float64) - right_f["W_pre"]) / (0.004 * 0.25)
    d_left = (O.dequantize(Wt).astype(np.float64) - left["W_pre"]) / (0.004 * 0.25)
    scale = np.abs(d_left).max()
    assert np.abs(d_right - d_left.T).max() <= 1e-3 * scale       # fp32 rounding of W' on either side
    # and the definition itself on a tiny case: R = G Q~
    Qt = O.bf16_round(O.dequantize(Q)).astype(np.float64)
    G = O.bf16_bits_to_f32(gb).astype(np.float64)
    assert np.allclose(right["R32"], (G @ Qt).T.astype(np.float32), rtol=1e-6, atol=1e-12)


# ----------------------------------------------------------------------------- 8-bit moments (a format of the library)
def test_8bit_moment_formats_bounds_idempotence_and_zero_blocks():
    # Sec. 3.5 keeps the Adam states in 8 bits without giving a format; the one built here is pinned by what it
    # promises: the first moment is off by at most half a step s/127, the square root of the second by at most
    # half of sqrt(s)/255 (the square-root law), the largest element of a block is exact, storing a stored
    # value again changes nothing, codes are monotone, zero blocks stay zero, ragged rows end in a short block.
    rng = np.random.default_rng(11)
    rows, cols = 9, 3 * 32 + 7
    x = (rng.normal(0, 1e-3, (rows, cols)) * rng.lognormal(0, 2, (rows, 1))).astype(np.float32)
    x[2, 32:64] = 0.0
    q = O.quantize_m8(x)
    assert q.scales.shape == (rows, 4) and q.codes.dtype == np.int8 and np.abs(q.codes.astype(int)).max() == 127
    xh = O.dequantize_m8(q)
    step = np.repeat(q.scales / 127.0, 32, axis=1)[:, :cols]
    assert np.all(np.abs(xh - x) <= 0.5 * step * (1 + 1e-5))
    assert np.all(q.codes[2, 32:64] == 0) and q.scales[2, 1] == 0.0 and np.all(xh[2, 32:64] == 0.0)
    for k, (a, b) in enumerate([(0, 32), (32, 64), (64, 96), (96, cols)]):
        top = np.abs(x[:, a:b]).argmax(axis=1)
        assert np.array_equal(np.abs(xh[np.arange(rows), a + top]), q.scales[:, k])       # the block maximum is exact
    again = O.quantize_m8(xh)
    assert np.array_equal(again.codes, q.codes) and np.allclose(again.scales, q.scales, rtol=2e-7)
    order = np.argsort(x[0, :32])
    assert np.all(np.diff(q.codes[0, :32][order].astype(int)) >= 0)                        # monotone

    v = (x.astype(np.float64) ** 2).astype(np.float32)
    qv = O.quantize_v8(v)
    assert qv.codes.dtype == np.uint8 and qv.codes.max() == 255
    vh = O.dequantize_v8(qv)
    root = np.repeat(np.sqrt(qv.scales.astype(np.float64)) / 255.0, 32, axis=1)[:, :cols]
    assert np.all(np.abs(np.sqrt(vh.astype(np.float64)) - np.sqrt(v.astype(np.float64))) <= 0.5 * root * (1 + 1e-4))
    assert np.all(qv.codes[2, 32:64] == 0) and np.all(vh[2, 32:64] == 0.0)
    assert np.array_equal(O.quantize_v8(vh).codes, qv.codes)
    # the square-root law: an element 10^4 times smaller than the block maximum still has a code
    t = np.full((1, 32), 1e-12, np.float32)
    t[0, 0] = 1e-8
    assert O.quantize_v8(t).codes[0, 1] >= 2 and O.dequantize_v8(O.quantize_v8(t))[0, 1] > 0


def test_step_on_8bit_moments_is_the_step_on_their_values_and_tracks_the_fp32_run():
    from paper_2407_08296_b200 import synth
    m, n, r = 96, 2 * 32 + 20, 32
    gm = synth.GradientModel(m, n, seed=6, matrix_index=0)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=6), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 6), 8)
    z = np.zeros((r, n), np.float32)
    M8, V8 = O.quantize_m8(z), O.quantize_v8(z)
    Mf, Vf, Wf, W8 = z, z, W, W
    for t in range(1, 6):
        hyp = O.Hyper(step=t, seed=2)
        a = O.project_step(gm.sample(t), P, W8, M8, V8, hyp)
        b = O.project_step(gm.sample(t), P, W8, O.dequantize_m8(M8), O.dequantize_v8(V8), hyp)
        assert np.array_equal(a["M"], b["M"]) and np.array_equal(a["W"].codes, b["W"].codes)      # same step
        assert np.array_equal(a["M8"].codes, O.quantize_m8(a["M"]).codes)
        f = O.project_step(gm.sample(t), P, Wf, Mf, Vf, hyp)
        M8, V8, W8 = a["M8"], a["V8"], a["W"]
        Mf, Vf, Wf = f["M"], f["V"], f["W"]
    # five steps on: the stored moments stay close to the binary32 ones (no drift from the rounding of the state)
    assert np.linalg.norm(O.dequantize_m8(M8) - Mf) <= 0.02 * np.linalg.norm(Mf)
    assert np.linalg.norm(np.sqrt(O.dequantize_v8(V8)) - np.sqrt(Vf)) <= 0.02 * np.linalg.norm(np.sqrt(Vf))


# ----------------------------------------------------------------------------- App. A: the INT8 linear layer
def _small_linear_case(T=5, m=3, n=260, seed=3):
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((m, n)).astype(np.float32) * 0.05
    W_q = O.quantize_rtn(W, 8)
    X_bits = O.f32_to_bf16_bits(rng.standard_normal((T, n)).astype(np.float32))
    dY_bits = O.f32_to_bf16_bits(rng.standard_normal((T, m)).astype(np.float32))
    return W_q, X_bits, dY_bits


def test_int8_linear_matches_index_loops_on_a_tiny_case():
    """App. A written out index by index in Python floats: y[t][i] = sum_j x[t][j] w[i][j],
    dx[t][j] = sum_i dy[t][i] w[i][j], g[i][j] = sum_t dy[t][i] x[t][j], with w the INT8 weight
    dequantized per group of 256 and rounded to bfloat16."""
    T, m, n = 5, 3, 260                     # two groups per row, the second one 4 wide
    W_q, X_bits, dY_bits = _small_linear_case(T, m, n)
    x = O.bf16_bits_to_f32(X_bits).tolist()
    dy = O.bf16_bits_to_f32(dY_bits).tolist()
    w = [[0.0] * n for _ in range(m)]
    for i in range(m):
        for j in range(n):
            g = j // 256
            v = np.float32(np.float32(float(W_q.codes[i, j]) - float(W_q.zeros[i, g])) * W_q.scales[i, g])
            w[i][j] = float(O.bf16_bits_to_f32(O.f32_to_bf16_bits(np.array([v], np.float32)))[0])
    Y, Yb = O.int8_linear_forward(X_bits, W_q)
    dX, dXb, G, Gb = O.int8_linear_backward(dY_bits, X_bits, W_q)
    assert Y.shape == (T, m) and dX.shape == (T, n) and G.shape == (m, n)
    for t in range(T):
        for i in range(m):
            assert Y[t, i] == pytest.approx(math.fsum(x[t][j] * w[i][j] for j in range(n)), rel=1e-12, abs=1e-14)
        for j in range(0, n, 37):
            assert dX[t, j] == pytest.approx(math.fsum(dy[t][i] * w[i][j] for i in range(m)), rel=1e-12, abs=1e-14)
    for i in range(m):
        for j in range(0, n, 37):
            assert G[i, j] == pytest.approx(math.fsum(dy[t][i] * x[t][j] for t in range(T)), rel=1e-12, abs=1e-14)
    # the bfloat16 outputs are the exact ones rounded once
    np.testing.assert_array_equal(Yb, O.f32_to_bf16_bits(Y.astype(np.float32)))
    np.testing.assert_array_equal(Gb, O.f32_to_bf16_bits(G.astype(np.float32)))


def test_int8_linear_with_a_permutation_weight_moves_columns():
    """A weight whose dequantized value is exactly a permutation matrix (Quant_8 of a 0/1 row represents 0
    and 1 exactly): the forward pass permutes the columns of X one way, the input gradient permutes dY the
    other way.  A transposed operand in either product fails this."""
    n = 256
    perm = np.roll(np.arange(n), 5)                  # not an involution
    Wm = np.zeros((n, n), np.float32)
    Wm[np.arange(n), perm] = 1.0                     # row i has its one in column perm[i]
    W_q = O.quantize_rtn(Wm, 8)
    np.testing.assert_array_equal(O.dequantize(W_q), Wm)
    rng = np.random.default_rng(0)
    X_bits = O.f32_to_bf16_bits(rng.standard_normal((4, n)).astype(np.float32))
    dY_bits = O.f32_to_bf16_bits(rng.standard_normal((4, n)).astype(np.float32))
    Y, Yb = O.int8_linear_forward(X_bits, W_q)
    dX, dXb, G, _ = O.int8_linear_backward(dY_bits, X_bits, W_q)
    np.testing.assert_array_equal(Yb, X_bits[:, perm])               # y[:, i] = x[:, perm[i]]
    inv = np.argsort(perm)
    np.testing.assert_array_equal(dXb, dY_bits[:, inv])              # dx[:, perm[i]] = dy[:, i]
    assert not np.array_equal(Yb, X_bits[:, inv])


def test_int8_linear_adjoint_identity_and_autograd():
    """<dY, X W^T> = <dY W, X> = <dY^T X, W> (the three products are one trilinear form), and torch's
    autograd on y = x @ w.t() returns the same two gradients."""
    torch = pytest.importorskip("torch")
    W_q, X_bits, dY_bits = _small_linear_case(T=7, m=6, n=300, seed=11)
    Y, _ = O.int8_linear_forward(X_bits, W_q)
    dX, _, G, _ = O.int8_linear_backward(dY_bits, X_bits, W_q)
    X = O.bf16_bits_to_f32(X_bits).astype(np.float64)
    dY = O.bf16_bits_to_f32(dY_bits).astype(np.float64)
    Wt = O.bf16_bits_to_f32(O.f32_to_bf16_bits(O.dequantize(W_q))).astype(np.float64)
    a, b, c = np.sum(dY * Y), np.sum(dX * X), np.sum(G * Wt)
    assert a == pytest.approx(b, rel=1e-12) and a == pytest.approx(c, rel=1e-12)
    xt = torch.tensor(X, requires_grad=True)
    wt = torch.tensor(Wt, requires_grad=True)
    y = xt @ wt.t()
    y.backward(torch.tensor(dY))
    np.testing.assert_allclose(y.detach().numpy(), Y, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(xt.grad.numpy(), dX, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(wt.grad.numpy(), G, rtol=1e-12, atol=1e-14)
