"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Quantizer output is compared bit for bit; the step within the tolerances below."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2407_08296_b200 import binding as B
from paper_2407_08296_b200 import synth

from parity_utils import (StepTaps, check_step_on_column_blocks, f32_to_device, from_device_q, g_to_device,
                          run_and_check_step, to_device_q)

pytestmark = pytest.mark.gpu

MOMENT_TOL = 2e-3        # relative, for M, V, N and R (bf16 operands, fp32 accumulation)


# ----------------------------------------------------------------------------- quantizer: bit-exact
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("shape", [(1, 1), (3, 7), (5, 256), (64, 1376), (33, 5461), (128, 128), (17, 600)])
def test_quantize_bit_exact(bits, shape):
    rows, cols = shape
    rng = np.random.default_rng(rows * 7919 + cols + bits)
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    if rows > 4:
        x[1, :] = 0.0                 # constant-zero groups
        x[2, :] = -1.25               # constant groups
        x[3, : min(cols, 256)] = np.linspace(-1, 1, min(cols, 256), dtype=np.float32)   # symmetric: ties
        x[4, :] = 1e-41               # subnormal values: scale not a normal number
    ref = O.quantize_rtn(x, bits)
    fn = B.quantize_int4 if bits == 4 else B.quantize_int8
    got = from_device_q(fn(f32_to_device(x)))
    assert np.array_equal(got.scales.view(np.uint32), ref.scales.view(np.uint32))
    assert np.array_equal(got.zeros.view(np.uint32), ref.zeros.view(np.uint32))
    assert np.array_equal(got.codes, ref.codes)


@pytest.mark.parametrize("bits", [4, 8])
def test_int4_padding_nibble_and_dequantize(bits):
    rows, cols = 9, 301
    x = (np.random.default_rng(5).standard_normal((rows, cols))).astype(np.float32)
    ref = O.quantize_rtn(x, bits)
    dq = B.quantize_int4(f32_to_device(x)) if bits == 4 else B.quantize_int8(f32_to_device(x))
    if bits == 4:
        packed = dq.codes.cpu().numpy()[:, : (cols + 1) // 2]
        assert np.array_equal(packed, O.pack_int4(ref.codes))        # odd tail: high nibble holds code 0
    y = B.dequantize(dq).cpu().numpy()
    assert np.array_equal(y.view(np.uint32), O.dequantize(ref).view(np.uint32))
    # dequantize of codes uploaded from the oracle
    y2 = B.dequantize(to_device_q(ref)).cpu().numpy()
    assert np.array_equal(y2, O.dequantize(ref))


def test_quantize_large_matrix_bit_exact():
    x = synth.initial_weight(2048, 5461, seed=3)
    ref = O.quantize_rtn(x, 8)
    got = from_device_q(B.quantize_int8(f32_to_device(x)))
    assert np.array_equal(got.codes, ref.codes)
    assert np.array_equal(got.scales, ref.scales) and np.array_equal(got.zeros, ref.zeros)


# ----------------------------------------------------------------------------- similarity
@pytest.mark.parametrize("m,r,c", [(512, 128, 0), (768, 256, 8), (100, 32, 5), (2048, 512, 0), (4096, 1024, 100)])
def test_similarity_matches_oracle(m, r, c):
    A = O.quantize_rtn(synth.random_orthonormal(m, r, seed=m, stream=1), 4)
    rng = np.random.default_rng(m + r)
    mix = synth.random_orthonormal(m, r, seed=m, stream=1) + 0.5 * rng.standard_normal((m, r)).astype(np.float32) / np.sqrt(m)
    Bq = O.quantize_rtn(mix.astype(np.float32), 4)
    want = O.subspace_similarity(A, Bq, c if c > 0 else None)
    got = float(B.subspace_similarity(to_device_q(A), to_device_q(Bq), c).item())
    assert abs(got - want) <= 1e-5
    same = float(B.subspace_similarity(to_device_q(A), to_device_q(A), c).item())
    assert abs(same - 1.0) <= 1e-6


# ----------------------------------------------------------------------------- refresh
def run_refresh_case(m, n, r, seed=0, iters=12):
    gb = synth.GradientModel(m, n, seed=seed, matrix_index=0).sample(1)
    P_ref, _, sv = O.refresh_subspace(gb, r)
    dG = g_to_device(gb)
    P32 = torch.zeros((m, r), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    P_new = B.refresh_subspace(dG, r, iters=iters, seed=seed + 1, P_fp32=P32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status word"
    Pg = P32.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(Pg))
    # orthonormal columns, each with its largest entry positive
    assert np.abs(Pg.T @ Pg - np.eye(r)).max() <= 1e-4
    piv = np.argmax(np.abs(Pg), axis=0)
    assert np.all(Pg[piv, np.arange(r)] > 0)
    # the subspace is the oracle's (exact SVD) to a largest principal angle below 1e-2 rad
    angle = O.principal_angle(P_ref, Pg)
    assert angle < 1e-2, f"largest principal angle {angle:.3e} rad"
    # it captures the energy of the top-r singular values
    G = O.bf16_bits_to_f32(gb).astype(np.float64)
    energy = np.linalg.norm(Pg.T @ G) ** 2
    assert abs(energy - np.sum(sv[:r] ** 2)) <= 1e-5 * np.sum(sv[:r] ** 2)
    # the leading, well separated singular vectors agree one by one (up to the sign convention both sides share)
    lead = np.abs(np.sum(P_ref[:, :8].astype(np.float64) * Pg[:, :8], axis=0))
    assert lead.min() > 0.999, f"leading vectors: {lead}"
    # and what was stored is Quant_4 of exactly those vectors
    want = O.quantize_rtn(P32.cpu().numpy(), 4)
    got = from_device_q(P_new)
    assert np.array_equal(got.codes, want.codes) and np.array_equal(got.scales, want.scales)
    assert np.array_equal(got.zeros, want.zeros)
    return angle, P_new


@pytest.mark.parametrize("m,n,r", [(256, 320, 64), (320, 256, 64), (512, 1376, 128), (768, 768, 256), (2048, 2048, 512)])
def test_refresh_subspace_matches_exact_svd(m, n, r):
    # (the three LLaMA-7B shapes at r = 1024 run in test_gpu_configs.py, two gradients each)
    run_refresh_case(m, n, r, seed=m + r)


def test_refresh_with_the_row_by_row_eigen_iteration():
    # blocks wider than 2048 columns do not fit the block form of the Jacobi iteration and take the row-by-row form;
    # here the same form is selected on a small shape
    B.debug_set_jacobi_blocks(False)
    try:
        run_refresh_case(768, 768, 256, seed=1024)
        run_refresh_case(512, 1376, 128, seed=640)
    finally:
        B.debug_set_jacobi_blocks(True)


def test_refresh_reports_similarity_with_previous_projection():
    m, n, r = 256, 512, 64
    gm = synth.GradientModel(m, n, seed=9, matrix_index=0)
    dG = g_to_device(gm.sample(1))
    P1 = B.refresh_subspace(dG, r, seed=1)
    sim = torch.zeros(1, dtype=torch.float32, device="cuda")
    dG2 = g_to_device(gm.sample(2))                       # same planted subspace, fresh noise
    P2 = B.refresh_subspace(dG2, r, seed=2, P_prev=P1, sim_cols=8, sim=sim)
    torch.cuda.synchronize()
    want = O.subspace_similarity(from_device_q(P1), from_device_q(P2), 8)
    assert abs(float(sim.item()) - want) <= 1e-5
    assert float(sim.item()) > 0.9                         # the leading planted directions persist


def test_refresh_replayed_from_a_cuda_graph_gives_the_same_codes():
    """Nothing in the refresh decides on the host: a captured refresh (a few thousand launches, one of them
    cooperative) replays to the codes of the direct call, also on another gradient placed in the same buffer."""
    m, n, r = 512, 768, 128
    gm = synth.GradientModel(m, n, seed=4, matrix_index=0)
    dG = g_to_device(gm.sample(1))
    block = 2 * r
    ws = torch.empty(B.workspace_bytes(B.QG_OP_REFRESH, m, n, block), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    direct = B.refresh_subspace(dG, r, seed=3, workspace=ws, status=status)
    torch.cuda.synchronize()
    P_new = B.QTensor.empty(m, r, 4, "cuda")
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        B.refresh_subspace(dG, r, seed=3, P_new=P_new, workspace=ws, status=status, stream=torch.cuda.current_stream())
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(P_new.codes, direct.codes) and torch.equal(P_new.scales, direct.scales)
    g2 = g_to_device(gm.sample(2))
    want = B.refresh_subspace(g2, r, seed=3, workspace=ws, status=status)
    torch.cuda.synchronize()
    dG.copy_(g2)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(P_new.codes, want.codes) and torch.equal(P_new.zeros, want.zeros)


@pytest.mark.parametrize("side,m,n,r,max_batch", [("left", 512, 768, 128, 8), ("left", 320, 256, 64, 2), ("right", 768, 320, 64, 3)])
def test_batched_refresh_equals_single_calls(side, m, n, r, max_batch):
    """Five matrices of one shape refreshed in one call (in batches of max_batch: 5, 2 + 2 + 1, 3 + 2) give, matrix by
    matrix, the codes, the vectors and the similarity of five single calls."""
    right = side == "right"
    pm = n if right else m
    gms = [synth.GradientModel(m, n, seed=40, matrix_index=i) for i in range(5)]
    Gs = [g_to_device(gm.sample(1)) for gm in gms]
    prev = [B.refresh_subspace(g_to_device(gm.sample(2)), r, seed=9, side=side) for gm in gms]
    single, items = [], []
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for i, G in enumerate(Gs):
        P32 = torch.zeros((pm, r), dtype=torch.float32, device="cuda")
        sim = torch.zeros(1, dtype=torch.float32, device="cuda")
        Pn = B.refresh_subspace(G, r, seed=100 + i, P_fp32=P32, P_prev=prev[i], sim_cols=8, sim=sim, status=status, side=side)
        single.append((Pn, P32, sim))
        items.append({"G": G, "seed": 100 + i, "P_fp32": torch.zeros((pm, r), dtype=torch.float32, device="cuda"), "P_prev": prev[i],
                      "sim": torch.zeros(1, dtype=torch.float32, device="cuda")})
    got = B.refresh_subspace_batched(items, r, sim_cols=8, max_batch=max_batch, status=status, side=side)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for (Pn, P32, sim), it, Pb in zip(single, items, got):
        assert torch.equal(Pn.codes, Pb.codes) and torch.equal(Pn.scales, Pb.scales) and torch.equal(Pn.zeros, Pb.zeros)
        assert torch.equal(P32, it["P_fp32"]) and torch.equal(sim, it["sim"])
    with pytest.raises((B.QgError, ValueError)):      # one shape per call
        B.refresh_subspace_batched([items[0], {"G": g_to_device(synth.GradientModel(m, n + 64, seed=1).sample(1)), "seed": 1}], r)


def test_refresh_rejects_bad_block_widths():
    dG = torch.zeros((128, 256), dtype=torch.int16, device="cuda")
    with pytest.raises(B.QgError) as e:
        B.refresh_subspace(dG, 64, oversample_cols=32)     # block of 96 columns: not a multiple of 64
    assert e.value.status == B.QG_UNSUPPORTED_SHAPE
    with pytest.raises(B.QgError) as e:
        B.refresh_subspace(dG, 64, oversample_cols=128)    # block wider than the matrix is tall
    assert e.value.status == B.QG_UNSUPPORTED_SHAPE


# ----------------------------------------------------------------------------- the step
def run_step_case(m, n, r, seed=0, step=1, steps_before=0, wd=0.0, impl=None, P=None, matrix_index=1):
    """Teacher-forced single-step parity: upload the oracle's pre-step state, run one GPU step, compare."""
    gm = synth.GradientModel(m, n, seed=seed, matrix_index=matrix_index)
    if P is None:
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=seed, stream=9), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, seed=seed, matrix_index=matrix_index), 8)
    M = np.zeros((r, n), np.float32)
    V = np.zeros((r, n), np.float32)
    sr_seed = synth.matrix_seed(seed, matrix_index)
    for t in range(step - steps_before, step):          # advance the oracle so that M, V are not trivial
        out = O.project_step(gm.sample(t), P, W, M, V, O.Hyper(step=t, seed=sr_seed, weight_decay=wd))
        W, M, V = out["W"], out["M"], out["V"]
    return run_and_check_step(gm.sample(step), P, W, M, V, O.Hyper(step=step, seed=sr_seed, weight_decay=wd),
                              tol=MOMENT_TOL, impl=impl)


SMALL_CASES = [
    (64, 256, 32), (128, 512, 64), (96, 300, 32), (160, 1376, 64), (512, 1376, 128),
    (300, 777, 96), (768, 768, 256), (1000, 85, 128), (130, 2736, 128), (64, 3, 32), (200, 17, 64),
    (257, 1025, 160),
]


@pytest.mark.parametrize("m,n,r", SMALL_CASES)
def test_step_parity_small_and_ragged(m, n, r):
    run_step_case(m, n, r, seed=m + n + r, step=1)


@pytest.mark.parametrize("m,n,r", [(128, 512, 64), (512, 1376, 128)])
def test_step_parity_cuda_core_kernels(m, n, r):
    run_step_case(m, n, r, seed=3, step=2, steps_before=1, impl=1)


def test_step_parity_after_several_steps_with_weight_decay():
    run_step_case(256, 1376, 64, seed=11, step=4, steps_before=3, wd=0.1)


def test_step_config1_llama60m_mlp():
    # configs[0]: 512 x 1376, r = 128, one step, seed 0, P from the oracle's refresh of that gradient
    spec = synth.stack_matrices("llama60m_mlp")[0]
    gb = synth.GradientModel(spec.m, spec.n, seed=0, matrix_index=0).sample(1)
    _, P, _ = O.refresh_subspace(gb, spec.r)
    run_step_case(spec.m, spec.n, spec.r, seed=0, step=1, P=P, matrix_index=0)


@pytest.mark.parametrize("m,n,r", [(2048, 2048, 512), (2048, 5461, 512), (5461, 2048, 512)])
def test_step_parity_llama1b_shapes(m, n, r):
    # the three distinct shapes of the LLaMA-1B stack at full size, second step (non-trivial moments)
    run_step_case(m, n, r, seed=4, step=2, steps_before=1)


def test_step_is_deterministic_and_seeded():
    m, n, r = 128, 512, 64
    gb = synth.GradientModel(m, n, seed=1).sample(1)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=1), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 1), 8)
    z = np.zeros((r, n), np.float32)
    outs = []
    for seed in (5, 5, 6):
        dW, dM, dV = to_device_q(W), f32_to_device(z), f32_to_device(z)
        B.project_step(g_to_device(gb), to_device_q(P), dW, dM, dV, B.Hyper(step=3, seed=seed))
        outs.append(dW.codes.cpu().numpy().copy())
    assert np.array_equal(outs[0], outs[1])           # counter-based randomness: same (seed, step) -> same codes
    assert not np.array_equal(outs[0], outs[2])


# ----------------------------------------------------------------------------- plans (grouped launches)
def _plan_items(shapes, seed=0, steps_before=1):
    """Host-side state of a few matrices after ``steps_before`` oracle steps, as (gm, P, W, M, V, sr_seed)."""
    out = []
    for idx, (m, n, r) in enumerate(shapes):
        gm = synth.GradientModel(m, n, seed=seed, matrix_index=idx)
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=seed, stream=idx), 4)
        W = O.quantize_rtn(synth.initial_weight(m, n, seed, idx), 8)
        M = np.zeros((r, n), np.float32)
        V = np.zeros((r, n), np.float32)
        sr = synth.matrix_seed(seed, idx)
        for t in range(1, steps_before + 1):
            o = O.project_step(gm.sample(t), P, W, M, V, O.Hyper(step=t, seed=sr))
            W, M, V = o["W"], o["M"], o["V"]
        out.append((gm, P, W, M, V, sr))
    return out


@pytest.mark.parametrize("workspace_bytes", [None, 0])
def test_plan_step_equals_single_matrix_calls(workspace_bytes):
    # a plan over ragged and regular shapes gives bit for bit what qgalore_project_step gives per matrix
    shapes = [(256, 512, 64), (300, 777, 96), (512, 1376, 128), (128, 85, 32), (768, 768, 256), (1024, 2736, 256)]
    state = _plan_items(shapes, seed=2, steps_before=1)
    step = 2
    single, items = [], []
    for (gm, P, W, M, V, sr) in state:
        gb = gm.sample(step)
        dG, dP = g_to_device(gb), to_device_q(P)
        dW1, dM1, dV1 = to_device_q(W), f32_to_device(M), f32_to_device(V)
        B.project_step(dG, dP, dW1, dM1, dV1, B.Hyper(step=step, seed=sr))
        single.append((dW1, dM1, dV1))
        items.append({"G": dG, "P": dP, "W": to_device_q(W), "M": f32_to_device(M), "V": f32_to_device(V), "seed": sr})
    if workspace_bytes == 0:     # the minimum: one matrix per chunk
        workspace_bytes = max(B.workspace_bytes(B.QG_OP_PROJECT_STEP, m, n, r) for (m, n, r) in shapes)
    plan = B.StepPlan(items, workspace_bytes=workspace_bytes)
    plan.step(B.Hyper(step=step))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    for (dW1, dM1, dV1), it in zip(single, items):
        assert torch.equal(dW1.codes, it["W"].codes)
        assert torch.equal(dW1.scales, it["W"].scales) and torch.equal(dW1.zeros, it["W"].zeros)
        assert torch.equal(dM1._base, it["M"]._base) and torch.equal(dV1._base, it["V"]._base)
    plan.close()


def test_plan_free_run_tracks_oracle_moments():
    # three free-running steps of a small stack: M and V do not depend on W, so they stay on the oracle's trajectory
    shapes = [(256, 512, 64), (512, 1376, 128)]
    state = _plan_items(shapes, seed=5, steps_before=0)
    items = [{"G": g_to_device(gm.sample(1)), "P": to_device_q(P), "W": to_device_q(W), "M": f32_to_device(M),
              "V": f32_to_device(V), "seed": sr} for (gm, P, W, M, V, sr) in state]
    plan = B.StepPlan(items)
    ref = [(W, M, V) for (_, _, W, M, V, _) in state]
    for t in (1, 2, 3):
        for k, (gm, P, _, _, _, sr) in enumerate(state):
            gb = gm.sample(t)
            items[k]["G"].copy_(torch.from_numpy(gb.view(np.int16)).cuda())
            o = O.project_step(gb, P, ref[k][0], ref[k][1], ref[k][2], O.Hyper(step=t, seed=sr))
            ref[k] = (o["W"], o["M"], o["V"])
        plan.step(B.Hyper(step=t))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    for k in range(len(state)):
        m_gpu, v_gpu = items[k]["M"].cpu().numpy(), items[k]["V"].cpu().numpy()
        assert np.linalg.norm(m_gpu - ref[k][1]) <= MOMENT_TOL * np.linalg.norm(ref[k][1])
        assert np.linalg.norm(v_gpu - ref[k][2]) <= MOMENT_TOL * np.linalg.norm(ref[k][2])
        # weights: free-running trajectories differ by re-rolled roundings, but stay within a few levels
        w_gpu, w_ref = O.dequantize(from_device_q(items[k]["W"])), O.dequantize(ref[k][0])
        lsb = float(ref[k][0].scales.max())
        assert np.abs(w_gpu - w_ref).max() <= 4 * lsb


def _clone_items(items):
    return [{"G": it["G"], "P": it["P"], "W": it["W"].clone(), "M": it["M"]._base.clone()[:, :it["M"].shape[1]],
             "V": it["V"]._base.clone()[:, :it["V"].shape[1]], "seed": it["seed"]} for it in items]


@pytest.mark.parametrize("mask", [1, 2, 3])   # compared with mask 0
def test_cta_pair_kernels_equal_single_cta_kernels(mask):
    # two layers of the LLaMA-1B stack (14 matrices, r = 512): the cta_group::2 variants of the two GEMM kernels
    # must reproduce the one-CTA kernels bit for bit (same products, same accumulation order, same epilogues)
    from paper_2407_08296_b200.synth_device import build_stack
    _, base = build_stack("llama1b", torch.device("cuda", 0), seed=3, layers=2)
    set_mode = B.debug_set_pair_mode
    results = []
    try:
        for m in (0, mask):
            set_mode(m)
            items = _clone_items(base)
            plan = B.StepPlan(items)
            for t in (1, 2):
                plan.step(B.Hyper(step=t))
            torch.cuda.synchronize()
            assert int(plan.status.item()) == 0
            plan.close()
            results.append(items)
    finally:
        set_mode(B.DEFAULT_PAIR_MODE)
    for a, b in zip(*results):
        assert torch.equal(a["W"].codes, b["W"].codes)
        assert torch.equal(a["W"].scales, b["W"].scales) and torch.equal(a["W"].zeros, b["W"].zeros)
        assert torch.equal(a["M"], b["M"]) and torch.equal(a["V"], b["V"])


def test_projection_dequantized_inside_the_kernel_equals_the_separate_launch():
    """The converter warps of the projection kernel form the same bf16 operand as the dequantize-P launch: two
    steps of a stack that mixes 1B shapes (ragged K: 5461 rows), small ranks, a right-hand item and a rank that is
    not a multiple of 128 (which keeps the separate launch either way) give the same bits in both modes, as single
    calls and as a plan."""
    from paper_2407_08296_b200.synth_device import build_stack
    _, base = build_stack("llama1b", torch.device("cuda", 0), seed=5, layers=1)
    base = [{k: v for k, v in it.items() if k != "spec"} for it in base]
    for idx, ((m, n, r), side) in enumerate([((512, 1376, 128), "left"), ((1376, 512, 256), "right"), ((300, 777, 96), "left"),
                                              ((257, 1025, 128), "left")]):
        right = side == "right"
        gb = synth.GradientModel(m, n, seed=23, matrix_index=idx).sample(1)
        P = O.quantize_rtn(synth.random_orthonormal(n if right else m, r, seed=23, stream=idx), 4)
        sc = m if right else n
        base.append({"G": g_to_device(gb), "P": to_device_q(P), "W": to_device_q(O.quantize_rtn(synth.initial_weight(m, n, 23, idx), 8)),
                     "M": f32_to_device(np.zeros((r, sc), np.float32)), "V": f32_to_device(np.zeros((r, sc), np.float32)),
                     "seed": 100 + idx, "side": side})
    results = {}
    try:
        for fused in (True, False):
            B.debug_set_fused_dequant(fused)
            items = [{**it, "W": it["W"].clone(), "M": it["M"]._base.clone()[:, :it["M"].shape[1]],
                      "V": it["V"]._base.clone()[:, :it["V"].shape[1]]} for it in base]
            plan = B.StepPlan(items)
            for t in (1, 2):
                plan.step(B.Hyper(step=t))
            torch.cuda.synchronize()
            assert int(plan.status.item()) == 0
            plan.close()
            singles = [{**it, "W": it["W"].clone(), "M": it["M"]._base.clone()[:, :it["M"].shape[1]],
                        "V": it["V"]._base.clone()[:, :it["V"].shape[1]]} for it in base[-4:]]
            for it in singles:
                for t in (1, 2):
                    B.project_step_item(it, B.Hyper(step=t))
            torch.cuda.synchronize()
            results[fused] = items + singles
    finally:
        B.debug_set_fused_dequant(True)
    for a, b in zip(results[True], results[False]):
        assert torch.equal(a["W"].codes, b["W"].codes) and torch.equal(a["W"].scales, b["W"].scales)
        assert torch.equal(a["W"].zeros, b["W"].zeros) and torch.equal(a["M"], b["M"]) and torch.equal(a["V"], b["V"])
    for a, b in zip(results[True][-8:-4], results[True][-4:]):       # plan == single calls, in the fused mode too
        assert torch.equal(a["W"].codes, b["W"].codes) and torch.equal(a["M"], b["M"])


# ----------------------------------------------------------------------------- full sizes, as the bench runs them
def _full_size_case(shapes, blocks_of, seed):
    """A plan over full-size matrices (the launch configuration bench.py times: grouped launches, CTA pairs,
    host-made tile lists) against (a) per-matrix calls, bit for bit, and (b) the oracle on a few column blocks."""
    step = 3
    host, items, singles = [], [], []
    rng = np.random.default_rng(seed)
    for idx, (m, n, r) in enumerate(shapes):
        gb = synth.GradientModel(m, n, seed=seed, matrix_index=idx).sample(step)
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=seed, stream=idx), 4)
        W = O.quantize_rtn(synth.initial_weight(m, n, seed, idx), 8)
        M = rng.normal(0, 1e-3, (r, n)).astype(np.float32)
        V = (rng.normal(0, 1e-3, (r, n)) ** 2).astype(np.float32)
        sr = synth.matrix_seed(seed, idx)
        host.append((gb, P, W, M, V, sr))
        dG, dP = g_to_device(gb), to_device_q(P)
        items.append({"G": dG, "P": dP, "W": to_device_q(W), "M": f32_to_device(M), "V": f32_to_device(V), "seed": sr})
        dW1, dM1, dV1 = to_device_q(W), f32_to_device(M), f32_to_device(V)
        taps = StepTaps(m, n, r, dW1.ld)
        B.project_step(dG, dP, dW1, dM1, dV1, B.Hyper(step=step, seed=sr), debug=taps.as_dict())
        singles.append((dW1, dM1, dV1, taps))
    plan = B.StepPlan(items)
    plan.step(B.Hyper(step=step))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    for (dW1, dM1, dV1, taps), it, (gb, P, W, M, V, sr), (m, n, r) in zip(singles, items, host, shapes):
        assert torch.equal(dW1.codes, it["W"].codes)
        assert torch.equal(dW1.scales, it["W"].scales) and torch.equal(dW1.zeros, it["W"].zeros)
        assert torch.equal(dM1._base, it["M"]._base) and torch.equal(dV1._base, it["V"]._base)
        gpu = {"M": it["M"].cpu().numpy(), "V": it["V"].cpu().numpy(), "R": taps.R.cpu().numpy(),
               "N": taps.N.cpu().numpy(), "N_b": taps.N_b.cpu().numpy(), "W_pre": taps.W_pre.cpu().numpy(),
               "W": from_device_q(it["W"])}
        check_step_on_column_blocks(blocks_of(n), gb, P, W, M, V, O.Hyper(step=step, seed=sr), gpu)
    plan.close()


def test_plan_at_llama1b_sizes_on_sampled_column_blocks():
    # the three LLaMA-1B shapes (r = 512) in one plan; first, a middle and the ragged last group of columns
    def blocks(n):
        last = (n - 1) // 256 * 256
        return [(0, 256), (last // 2 // 256 * 256, last // 2 // 256 * 256 + 256), (last, n)]
    _full_size_case([(2048, 2048, 512), (2048, 5461, 512), (5461, 2048, 512)], blocks, seed=21)


def test_plan_at_llama7b_sizes_on_sampled_column_blocks():
    # the three LLaMA-7B shapes (r = 1024) in one plan, two column groups each
    def blocks(n):
        return [(0, 256), (n - 256, n)]
    _full_size_case([(4096, 4096, 1024), (4096, 11008, 1024), (11008, 4096, 1024)], blocks, seed=22)


# ----------------------------------------------------------------------------- round to nearest (Sec. 4.4 ablation)
@pytest.mark.parametrize("shape", [(512, 1376, 128), (300, 777, 96), (2048, 2048, 512)])
@pytest.mark.parametrize("impl", [None, 1])
def test_step_with_round_to_nearest(shape, impl):
    m, n, r = shape
    if impl == 1 and m > 1024:
        pytest.skip("the CUDA-core cross-check is run on the small shapes")
    gm = synth.GradientModel(m, n, seed=9, matrix_index=0)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=9), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 9), 8)
    M = np.zeros((r, n), np.float32)
    V = np.zeros((r, n), np.float32)
    o = O.project_step(gm.sample(1), P, W, M, V, O.Hyper(step=1, seed=2, rounding="rtn"))
    stats = run_and_check_step(gm.sample(2), P, o["W"], o["M"], o["V"], O.Hyper(step=2, seed=2, rounding="rtn"), impl=impl)
    assert stats["mismatch"] <= 1e-3


def test_round_to_nearest_ignores_the_seed_and_a_bad_mode_is_refused():
    m, n, r = 256, 512, 64
    gb = synth.GradientModel(m, n, seed=4, matrix_index=0).sample(1)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=4), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 4), 8)
    z = np.zeros((r, n), np.float32)
    outs = []
    for seed in (5, 6):
        dW, dM, dV = to_device_q(W), f32_to_device(z), f32_to_device(z)
        B.project_step(g_to_device(gb), to_device_q(P), dW, dM, dV, B.Hyper(step=3, seed=seed, rounding=B.QG_ROUND_NEAREST))
        outs.append(dW.codes.cpu().numpy().copy())
    assert np.array_equal(outs[0], outs[1])
    with pytest.raises(B.QgError):
        B.project_step(g_to_device(gb), to_device_q(P), to_device_q(W), f32_to_device(z), f32_to_device(z),
                       B.Hyper(step=1, rounding=7))


# ----------------------------------------------------------------------------- projection bit width (Sec. 4.4, Fig. 3)
@pytest.mark.parametrize("shape", [(64, 256), (33, 777), (512, 128)])
def test_int2_quantizer_is_bit_exact(shape):
    rows, cols = shape
    x = np.random.default_rng(rows + cols).normal(0, 0.05, (rows, cols)).astype(np.float32)
    x[0, :] = 0.25                                    # a constant group
    ref = O.quantize_rtn(x, 2)
    q = B.quantize_int2(f32_to_device(x))
    got = from_device_q(q)
    assert np.array_equal(got.codes, ref.codes) and np.array_equal(got.scales, ref.scales) and np.array_equal(got.zeros, ref.zeros)
    assert np.array_equal(B.dequantize(q).cpu().numpy(), O.dequantize(ref))
    assert np.array_equal(B.dequantize(to_device_q(ref)).cpu().numpy(), O.dequantize(ref))


@pytest.mark.parametrize("bits", [2, 8])
@pytest.mark.parametrize("impl", [None, 1])
def test_step_with_a_2_or_8_bit_projection(bits, impl):
    m, n, r = 512, 1376, 128
    gm = synth.GradientModel(m, n, seed=12, matrix_index=0)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=12), bits)
    W = O.quantize_rtn(synth.initial_weight(m, n, 12), 8)
    z = np.zeros((r, n), np.float32)
    o = O.project_step(gm.sample(1), P, W, z, z, O.Hyper(step=1, seed=8))
    stats = run_and_check_step(gm.sample(2), P, o["W"], o["M"], o["V"], O.Hyper(step=2, seed=8), impl=impl)
    assert stats["mismatch"] <= 1e-3


def test_plan_mixes_projection_bit_widths_and_similarity_takes_them():
    shapes = [(256, 512, 64), (512, 1376, 128), (768, 768, 256)]
    step = 2
    single, items = [], []
    for idx, ((m, n, r), bits) in enumerate(zip(shapes, (2, 8, 4))):
        gm = synth.GradientModel(m, n, seed=13, matrix_index=idx)
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=13, stream=idx), bits)
        W = O.quantize_rtn(synth.initial_weight(m, n, 13, idx), 8)
        M = np.zeros((r, n), np.float32)
        V = np.zeros((r, n), np.float32)
        gb = gm.sample(step)
        dG, dP = g_to_device(gb), to_device_q(P)
        dW1, dM1, dV1 = to_device_q(W), f32_to_device(M), f32_to_device(V)
        B.project_step(dG, dP, dW1, dM1, dV1, B.Hyper(step=step, seed=idx))
        single.append((dW1, dM1, dV1))
        items.append({"G": dG, "P": dP, "W": to_device_q(W), "M": f32_to_device(M), "V": f32_to_device(V), "seed": idx})
        # similarity of the projection with a perturbed copy of itself, both at this bit width
        P2 = O.quantize_rtn(O.dequantize(P) + np.random.default_rng(idx).normal(0, 0.01, (m, r)).astype(np.float32), bits)
        sim = B.subspace_similarity(dP, to_device_q(P2))
        assert abs(float(sim.item()) - O.subspace_similarity(P, P2)) <= 1e-5
    plan = B.StepPlan(items)
    plan.step(B.Hyper(step=step))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    for (dW1, dM1, dV1), it in zip(single, items):
        assert torch.equal(dW1.codes, it["W"].codes) and torch.equal(dM1._base, it["M"]._base) and torch.equal(dV1._base, it["V"]._base)
    plan.close()


def test_refresh_writes_an_8_bit_projection_when_asked():
    m, n, r = 512, 1376, 128
    gb = synth.GradientModel(m, n, seed=14, matrix_index=0).sample(1)
    P32 = torch.zeros((m, r), dtype=torch.float32, device="cuda")
    P8 = B.QTensor(torch.zeros((m, r), dtype=torch.int8, device="cuda"), torch.zeros((m, 1), dtype=torch.float32, device="cuda"),
                   torch.zeros((m, 1), dtype=torch.float32, device="cuda"), m, r, r, 8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.refresh_subspace(g_to_device(gb), r, P_new=P8, P_fp32=P32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = O.quantize_rtn(P32.cpu().numpy(), 8)
    got = from_device_q(P8)
    assert np.array_equal(got.codes, ref.codes) and np.array_equal(got.scales, ref.scales)


# ----------------------------------------------------------------------------- degenerate and limiting cases
def test_zero_gradient_and_constant_groups_are_bit_exact():
    # G = 0 at t = 1: R = M' = V' = 0 and N = 0 / (0 + eps) = 0 exactly, so W' is the dequantized weight and every
    # bit of the requantization is decided by identical inputs; one row of W is constant (a degenerate group:
    # z = 0, s = |max|), one is all zero.
    m, n, r = 128, 256 + 85, 32
    gb = np.zeros((m, n), np.uint16)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=2), 4)
    w = synth.initial_weight(m, n, 2).copy()
    w[3, :] = 0.0125
    w[5, :] = 0.0
    W = O.quantize_rtn(w, 8)
    z = np.zeros((r, n), np.float32)
    hyp = O.Hyper(step=1, seed=77)
    ref = O.project_step(gb, P, W, z, z, hyp)
    dW, dM, dV = to_device_q(W), f32_to_device(z), f32_to_device(z)
    taps = StepTaps(m, n, r, dW.ld)
    B.project_step(g_to_device(gb), to_device_q(P), dW, dM, dV, B.Hyper(step=1, seed=77), debug=taps.as_dict())
    torch.cuda.synchronize()
    assert float(dM.abs().max().item()) == 0.0 and float(dV.abs().max().item()) == 0.0
    assert float(taps.N.abs().max().item()) == 0.0 and float(taps.R.abs().max().item()) == 0.0
    got = from_device_q(dW)
    assert np.array_equal(taps.W_pre.cpu().numpy(), ref["W_pre"])
    assert np.array_equal(got.codes, ref["W"].codes)
    assert np.array_equal(got.scales, ref["W"].scales) and np.array_equal(got.zeros, ref["W"].zeros)


def test_step_at_the_largest_rank():
    # r = 2048 is the limit of the step (r <= m, r % 32 == 0)
    run_step_case(2048, 600, 2048, seed=6, step=1)


def test_step_refuses_empty_oversized_and_misshapen_problems():
    m, n, r = 128, 256, 32
    gb = synth.GradientModel(m, n, seed=1, matrix_index=0).sample(1)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=1), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 1), 8)
    z = np.zeros((r, n), np.float32)
    dG, dP, dW, dM, dV = g_to_device(gb), to_device_q(P), to_device_q(W), f32_to_device(z), f32_to_device(z)
    L, C = B.lib(), B.C
    ws = torch.empty(B.workspace_bytes(B.QG_OP_PROJECT_STEP, m, n, r), dtype=torch.uint8, device="cuda")
    h = B.Hyper().c_struct()
    pc, wc = dP.c_struct(), dW.c_struct()

    def call(mm, nn, rr, hyper=h, ws_bytes=ws.numel()):
        return L.qgalore_project_step(dG.data_ptr(), dG.stride(0), mm, nn, rr, C.byref(pc), C.byref(wc), dM.data_ptr(),
                                      dV.data_ptr(), dM.stride(0), C.byref(hyper), ws.data_ptr(), ws_bytes, None, None, None)

    before = dW.codes.clone()
    assert call(0, n, r) == B.QG_INVALID_ARGUMENT           # empty
    assert call(m, 0, r) == B.QG_INVALID_ARGUMENT
    assert call(m, n, 0) == B.QG_INVALID_ARGUMENT
    assert call(m, n, 64) == B.QG_INVALID_ARGUMENT          # P is m x 32
    assert call(m, n, r, ws_bytes=16) == B.QG_WORKSPACE_TOO_SMALL
    bad = B.Hyper(step=0).c_struct()
    assert call(m, n, r, hyper=bad) == B.QG_INVALID_ARGUMENT
    torch.cuda.synchronize()
    assert torch.equal(before, dW.codes)                    # nothing was enqueued
    # rank limits are shape errors
    big = B.QTensor.empty(4096, 4096, 4)
    bc = big.c_struct()
    assert L.qgalore_project_step(dG.data_ptr(), 4096, 4096, 256, 4096, C.byref(bc), C.byref(wc), dM.data_ptr(), dV.data_ptr(),
                                  256, C.byref(h), ws.data_ptr(), ws.numel(), None, None, None) in (B.QG_UNSUPPORTED_SHAPE,
                                                                                                    B.QG_INVALID_ARGUMENT)


# ----------------------------------------------------------------------------- projection on the right (GaLore's other side)
def _right_case(m, n, r, seed, step=2):
    gm = synth.GradientModel(m, n, seed=seed, matrix_index=0)
    Q = O.quantize_rtn(synth.random_orthonormal(n, r, seed=seed), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, seed), 8)
    Mt = np.zeros((r, m), np.float32)
    Vt = np.zeros((r, m), np.float32)
    for t in range(1, step):
        o = O.project_step(gm.sample(t), Q, W, Mt, Vt, O.Hyper(step=t, seed=seed), side="right")
        W, Mt, Vt = o["W"], o["M"], o["V"]
    return gm.sample(step), Q, W, Mt, Vt


@pytest.mark.parametrize("m,n,r", [(512, 256, 64), (777, 300, 96), (1376, 512, 128), (85, 1000, 32), (2736, 1024, 256)])
def test_step_with_the_projection_on_the_right(m, n, r):
    gb, Q, W, Mt, Vt = _right_case(m, n, r, seed=m + n)
    stats = run_and_check_step(gb, Q, W, Mt, Vt, O.Hyper(step=2, seed=m + n), side="right")
    assert stats["mismatch"] <= 1e-3


def test_right_projection_at_a_llama1b_size():
    m, n, r = 5461, 2048, 512                            # the down projection: m > n
    gb, Q, W, Mt, Vt = _right_case(m, n, r, seed=31)
    run_and_check_step(gb, Q, W, Mt, Vt, O.Hyper(step=2, seed=31), side="right")


def test_plan_mixes_projection_sides():
    cases = [((512, 256, 64), "right"), ((256, 512, 64), "left"), ((1376, 512, 256), "right"), ((768, 768, 256), "left"),
             ((2048, 1024, 512), "right")]
    step = 2
    single, items = [], []
    for idx, ((m, n, r), side) in enumerate(cases):
        right = side == "right"
        gb = synth.GradientModel(m, n, seed=17, matrix_index=idx).sample(step)
        P = O.quantize_rtn(synth.random_orthonormal(n if right else m, r, seed=17, stream=idx), 4)
        W = O.quantize_rtn(synth.initial_weight(m, n, 17, idx), 8)
        rng = np.random.default_rng(idx)
        sc = m if right else n
        M = rng.normal(0, 1e-3, (r, sc)).astype(np.float32)
        V = (rng.normal(0, 1e-3, (r, sc)) ** 2).astype(np.float32)
        dG, dP = g_to_device(gb), to_device_q(P)
        dW1, dM1, dV1 = to_device_q(W), f32_to_device(M), f32_to_device(V)
        B.project_step(dG, dP, dW1, dM1, dV1, B.Hyper(step=step, seed=idx), side=side)
        single.append((dW1, dM1, dV1))
        items.append({"G": dG, "P": dP, "W": to_device_q(W), "M": f32_to_device(M), "V": f32_to_device(V), "seed": idx,
                      "side": side})
    for pair_mode in (2, 0, 1, 3, 6):   # 1 and 3 ask for the paired back-projection, which a chunk with a right-hand item declines
        B.debug_set_pair_mode(pair_mode)
        try:
            fresh = [{**it, "W": it["W"].clone(), "M": it["M"]._base.clone()[:, :it["M"].shape[1]],
                      "V": it["V"]._base.clone()[:, :it["V"].shape[1]]} for it in items]
            plan = B.StepPlan(fresh)
            plan.step(B.Hyper(step=step))
            torch.cuda.synchronize()
            assert int(plan.status.item()) == 0
            for (dW1, dM1, dV1), it in zip(single, fresh):
                assert torch.equal(dW1.codes, it["W"].codes)
                assert torch.equal(dM1._base, it["M"]._base) and torch.equal(dV1._base, it["V"]._base)
            plan.close()
        finally:
            B.debug_set_pair_mode(B.DEFAULT_PAIR_MODE)


@pytest.mark.parametrize("m,n,r", [(320, 256, 64), (1376, 512, 128), (5461, 2048, 512)])
def test_refresh_of_the_right_singular_subspace(m, n, r):
    gb = synth.GradientModel(m, n, seed=5, matrix_index=2).sample(1)
    Q_ref, _, _ = O.refresh_subspace(gb, r, side="right")
    Q32 = torch.zeros((n, r), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Qq = B.refresh_subspace(g_to_device(gb), r, P_fp32=Q32, status=status, side="right")
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and (Qq.rows, Qq.cols) == (n, r)
    q = Q32.cpu().numpy()
    assert O.principal_angle(Q_ref, q) < 1e-2
    assert np.abs(q.T.astype(np.float64) @ q - np.eye(r)).max() < 1e-4
    ref_q = O.quantize_rtn(q, 4)
    got = from_device_q(Qq)
    assert np.array_equal(got.codes, ref_q.codes) and np.array_equal(got.scales, ref_q.scales)


# ----------------------------------------------------------------------------- checkpoint: save, load, continue
def test_saved_and_reloaded_state_continues_bit_for_bit():
    """The whole state of a run is plain buffers plus (seed, step index): k steps, every buffer copied to the host
    and back into fresh allocations (a new plan over them), k more steps, against 2k uninterrupted steps."""
    shapes = [(256, 512, 64), (300, 777, 96), (768, 768, 256)]
    k = 3
    grads = [[synth.GradientModel(m, n, seed=8, matrix_index=i).sample(t) for t in range(1, 2 * k + 1)]
             for i, (m, n, r) in enumerate(shapes)]

    def fresh_items():
        out = []
        for i, (m, n, r) in enumerate(shapes):
            out.append({"G": g_to_device(grads[i][0]), "P": to_device_q(O.quantize_rtn(synth.random_orthonormal(m, r, seed=8, stream=i), 4)),
                        "W": to_device_q(O.quantize_rtn(synth.initial_weight(m, n, 8, i), 8)),
                        "M": f32_to_device(np.zeros((r, n), np.float32)), "V": f32_to_device(np.zeros((r, n), np.float32)),
                        "seed": synth.matrix_seed(8, i)})
        return out

    def run(items, first, last):
        plan = B.StepPlan(items)
        for t in range(first, last + 1):
            for i, it in enumerate(items):
                it["G"].copy_(torch.from_numpy(grads[i][t - 1].view(np.int16)).cuda())
            plan.step(B.Hyper(step=t))
        torch.cuda.synchronize()
        assert int(plan.status.item()) == 0
        plan.close()

    straight = fresh_items()
    run(straight, 1, 2 * k)
    first_half = fresh_items()
    run(first_half, 1, k)
    saved = [{"P": from_device_q(it["P"]), "W": from_device_q(it["W"]), "M": it["M"].cpu().numpy(), "V": it["V"].cpu().numpy(),
              "seed": it["seed"]} for it in first_half]
    del first_half
    torch.cuda.empty_cache()
    resumed = [{"G": g_to_device(grads[i][k]), "P": to_device_q(s["P"]), "W": to_device_q(s["W"]), "M": f32_to_device(s["M"]),
                "V": f32_to_device(s["V"]), "seed": s["seed"]} for i, s in enumerate(saved)]
    run(resumed, k + 1, 2 * k)
    for a, b in zip(straight, resumed):
        assert torch.equal(a["W"].codes, b["W"].codes) and torch.equal(a["W"].scales, b["W"].scales)
        assert torch.equal(a["W"].zeros, b["W"].zeros) and torch.equal(a["M"], b["M"]) and torch.equal(a["V"], b["V"])


# ----------------------------------------------------------------------------- bounded waits
def test_a_bounded_barrier_wait_runs_out_and_reports_it():
    """Every barrier wait of the tensor-core kernels has a poll limit; a wait that runs out raises
    QG_DEV_WAIT_EXPIRED in the status word and the kernel returns.  The harmless form of that event: a one-warp
    kernel waits on a barrier nothing signals (no copy in flight, no tensor memory held); the context stays usable."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    used = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.debug_expire_wait(64, status, used)
    torch.cuda.synchronize()
    assert int(status.item()) == B.QG_DEV_WAIT_EXPIRED and int(used.item()) == 64
    status.fill_(2)                                    # flags are OR-ed in, never cleared
    B.debug_expire_wait(1, status, used)
    torch.cuda.synchronize()
    assert int(status.item()) == (2 | B.QG_DEV_WAIT_EXPIRED) and int(used.item()) == 1
    with pytest.raises(B.QgError):
        B.debug_expire_wait(0, status)
    # the device still works: a step right after it is clean
    run_step_case(128, 512, 64, seed=1, step=1)


# ----------------------------------------------------------------------------- 8-bit moments
def _codes_to_device(codes: np.ndarray) -> torch.Tensor:
    rows, cols = codes.shape
    ld = (cols + 63) // 64 * 64                      # the pitch the fp32 test taps get, which the taps share
    buf = torch.zeros((rows, ld), dtype=torch.int8 if codes.dtype == np.int8 else torch.uint8, device="cuda")
    buf[:, :cols] = torch.from_numpy(codes).to("cuda")
    return buf[:, :cols]


def _check_state8(gpu_codes, gpu_scales, ref8, deq, name, max_frac=2e-3):
    """Stored moments against the oracle's: scales to 1e-5, codes equal except by one level in a small fraction
    (the binary32 moments entering the storage differ in their last bits between fp32 and fp64 accumulation)."""
    assert np.allclose(gpu_scales, ref8.scales, rtol=1e-5, atol=0), f"{name} scales"
    d = np.abs(gpu_codes.astype(np.int32) - ref8.codes.astype(np.int32))
    assert d.max() <= 1, f"{name}: a code differs by more than one level"
    assert (d != 0).mean() <= max_frac, f"{name}: {(d != 0).mean():.2e} of the codes differ"


@pytest.mark.parametrize("m,n,r,side", [(256, 512, 64, "left"), (300, 777, 96, "left"), (512, 1376, 128, "left"),
                                        (777, 300, 96, "right"), (2048, 2048, 512, "left")])
def test_step_with_8bit_moments(m, n, r, side):
    right = side == "right"
    sc = m if right else n
    gm = synth.GradientModel(m, n, seed=m + r, matrix_index=0)
    P = O.quantize_rtn(synth.random_orthonormal(n if right else m, r, seed=m + r), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, m + r), 8)
    z = np.zeros((r, sc), np.float32)
    M8, V8 = O.quantize_m8(z), O.quantize_v8(z)
    for t in (1, 2):                                   # two oracle steps so that the stored moments are not trivial
        o = O.project_step(gm.sample(t), P, W, M8, V8, O.Hyper(step=t, seed=5), side=side)
        W, M8, V8 = o["W"], o["M8"], o["V8"]
    hyp = O.Hyper(step=3, seed=5)
    gb = gm.sample(3)
    ref = O.project_step(gb, P, W, M8, V8, hyp, side=side)
    dM, dV = _codes_to_device(M8.codes), _codes_to_device(V8.codes)
    dMs, dVs = torch.from_numpy(M8.scales).cuda().contiguous(), torch.from_numpy(V8.scales).cuda().contiguous()
    dW = to_device_q(W)
    taps = StepTaps(m, n, r, dW.ld, side)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    item = {"G": g_to_device(gb), "P": to_device_q(P), "W": dW, "M": dM, "V": dV, "M_scale": dMs, "V_scale": dVs,
            "seed": 5, "side": side}
    B.project_step_item(item, B.Hyper(step=3), status=status, debug=taps.as_dict())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the direction comes from the binary32 moments: same rules as for fp32 storage
    from parity_utils import check_direction, check_moments, check_weight_codes
    check_moments(taps.R.cpu().numpy(), ref["R32"], "R")
    n_gpu = taps.N.cpu().numpy()
    check_direction(n_gpu, ref, hyp, "N")
    forced = O.project_step(gb, P, W, M8, V8, hyp, side=side, N_b_override=O.bf16_bits_to_f32(taps.N_b.cpu().numpy().view(np.uint16)))
    check_weight_codes(from_device_q(dW), forced, 5, 3)
    # the stored moments
    _check_state8(dM.cpu().numpy(), dMs.cpu().numpy(), ref["M8"], O.dequantize_m8, "M")
    _check_state8(dV.cpu().numpy(), dVs.cpu().numpy(), ref["V8"], O.dequantize_v8, "V")
    assert int(dM._base[:, sc:].abs().max().item()) == 0 if dM._base.shape[1] > sc else True


def test_plan_mixes_fp32_and_8bit_moments():
    shapes = [(256, 512, 64), (512, 1376, 128), (768, 768, 256)]
    step = 2
    single, items = [], []
    for idx, (m, n, r) in enumerate(shapes):
        gb = synth.GradientModel(m, n, seed=19, matrix_index=idx).sample(step)
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=19, stream=idx), 4)
        W = O.quantize_rtn(synth.initial_weight(m, n, 19, idx), 8)
        rng = np.random.default_rng(idx)
        M = rng.normal(0, 1e-3, (r, n)).astype(np.float32)
        V = (rng.normal(0, 1e-3, (r, n)) ** 2).astype(np.float32)
        dG, dP = g_to_device(gb), to_device_q(P)
        pair = []
        for _ in range(2):                              # one copy for the single call, one for the plan
            if idx == 1:
                it = {"G": dG, "P": dP, "W": to_device_q(W), "M": f32_to_device(M), "V": f32_to_device(V), "seed": idx}
            else:
                M8, V8 = O.quantize_m8(M), O.quantize_v8(V)
                it = {"G": dG, "P": dP, "W": to_device_q(W), "M": _codes_to_device(M8.codes), "V": _codes_to_device(V8.codes),
                      "M_scale": torch.from_numpy(M8.scales).cuda().contiguous(),
                      "V_scale": torch.from_numpy(V8.scales).cuda().contiguous(), "seed": idx}
            pair.append(it)
        B.project_step_item(pair[0], B.Hyper(step=step))
        single.append(pair[0])
        items.append(pair[1])
    plan = B.StepPlan(items)
    plan.step(B.Hyper(step=step))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    for a, b in zip(single, items):
        assert torch.equal(a["W"].codes, b["W"].codes) and torch.equal(a["M"]._base, b["M"]._base)
        assert torch.equal(a["V"]._base, b["V"]._base)
        if "M_scale" in a:
            assert torch.equal(a["M_scale"], b["M_scale"]) and torch.equal(a["V_scale"], b["V_scale"])
    plan.close()


def test_8bit_moments_through_a_plan_at_a_7b_shape():
    """The 8-bit moment storage in the launch configuration the throughput run uses at 7B size (a plan, CTA pairs,
    r = 1024): one 4096 x 4096 matrix stepped twice as a plan and twice by single calls, bit for bit."""
    m, n, r = 4096, 4096, 1024
    gb = synth.GradientModel(m, n, seed=33, matrix_index=0).sample(1)
    P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=33), 4)
    W = O.quantize_rtn(synth.initial_weight(m, n, 33), 8)
    rng = np.random.default_rng(33)
    M8 = O.quantize_m8(rng.normal(0, 1e-3, (r, n)).astype(np.float32))
    V8 = O.quantize_v8((rng.normal(0, 1e-3, (r, n)) ** 2).astype(np.float32))
    dG, dP = g_to_device(gb), to_device_q(P)
    pair = []
    for _ in range(2):
        pair.append({"G": dG, "P": dP, "W": to_device_q(W), "M": _codes_to_device(M8.codes), "V": _codes_to_device(V8.codes),
                     "M_scale": torch.from_numpy(M8.scales).cuda().contiguous(),
                     "V_scale": torch.from_numpy(V8.scales).cuda().contiguous(), "seed": 3})
    plan = B.StepPlan([pair[1]])
    for t in (1, 2):
        B.project_step_item(pair[0], B.Hyper(step=t))
        plan.step(B.Hyper(step=t))
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0
    a, b = pair
    assert torch.equal(a["W"].codes, b["W"].codes) and torch.equal(a["W"].scales, b["W"].scales)
    assert torch.equal(a["M"]._base, b["M"]._base) and torch.equal(a["V"]._base, b["V"]._base)
    assert torch.equal(a["M_scale"], b["M_scale"]) and torch.equal(a["V_scale"], b["V_scale"])
    assert int(a["M"].abs().max().item()) > 0
    plan.close()


# ----------------------------------------------------------------------------- App. A: the INT8 linear layer
def _linear_case(T, m, n, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((m, n)) * 0.02).astype(np.float32)
    W[:, : min(n, 256)] += 0.5                    # a group far from zero: large zero points
    W_q = O.quantize_rtn(W, 8)
    X_bits = O.f32_to_bf16_bits(rng.standard_normal((T, n)).astype(np.float32))
    dY_bits = O.f32_to_bf16_bits((rng.standard_normal((T, m)) * 0.1).astype(np.float32))
    return W_q, X_bits, dY_bits


def _check_product(got: torch.Tensor, exact: np.ndarray, ref_bits: np.ndarray, abs_sum: np.ndarray, K: int, name: str):
    """bf16 operands are exact on both sides, so the only differences are the binary32 accumulation of the
    tensor core (each of the K / 16 instructions adds its products to the accumulator with an error of at most
    one unit in the last place of the running sum: (K / 16 + 1) * 2^-22 of the sum of magnitudes bounds it with a
    factor two to spare) and the final rounding to bfloat16 (half a unit in the last place, 2^-9 relative; 2^-8
    allows the rounding to fall the other way)."""
    got_bits = got.view(torch.int16).cpu().numpy().view(np.uint16)
    assert got_bits.shape == ref_bits.shape, name
    val = O.bf16_bits_to_f32(got_bits).astype(np.float64)
    tol = 2.0 ** -8 * np.abs(exact) + (K / 16 + 1) * 2.0 ** -22 * abs_sum + 1e-30
    bad = np.abs(val - exact) > tol
    assert not bad.any(), f"{name}: {int(bad.sum())} of {bad.size} outside the tolerance"
    same = np.mean(got_bits == ref_bits)
    assert same >= 0.98, f"{name}: only {same:.4f} of the outputs round to the same bfloat16"


@pytest.mark.parametrize("shape", [(300, 520, 1376), (1, 256, 256), (130, 300, 5461), (1000, 2048, 2048), (257, 64, 200),
                                   (1, 1, 1), (7, 9, 17), (129, 127, 63)])
def test_int8_linear_forward_and_backward(shape):
    T, m, n = shape
    W_q, X_bits, dY_bits = _linear_case(T, m, n, seed=T + 3 * m + 7 * n)
    Wd, Xd, dYd = to_device_q(W_q), g_to_device(X_bits), g_to_device(dY_bits)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    w_before = Wd.codes.clone()
    Y = B.int8_linear_forward(Xd, Wd, status=status)
    dX = B.int8_linear_backward_input(dYd, Wd, status=status)
    G = B.int8_linear_backward_weight(dYd, Xd, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(w_before, Wd.codes)          # the weight is only read

    Y_ref, Y_bits = O.int8_linear_forward(X_bits, W_q)
    dX_ref, dX_bits, G_ref, G_bits = O.int8_linear_backward(dY_bits, X_bits, W_q)
    X = np.abs(O.bf16_bits_to_f32(X_bits).astype(np.float64))
    dY = np.abs(O.bf16_bits_to_f32(dY_bits).astype(np.float64))
    Wt = np.abs(O.bf16_bits_to_f32(O.f32_to_bf16_bits(O.dequantize(W_q))).astype(np.float64))
    _check_product(Y, Y_ref, Y_bits, X @ Wt.T, n, "Y")
    _check_product(dX, dX_ref, dX_bits, dY @ Wt, m, "dX")
    _check_product(G, G_ref, G_bits, dY.T @ X, T, "G")


def test_int8_linear_backward_feeds_the_optimizer_step():
    """One training step of one layer on the device, no host copy in between: the weight gradient the layer's
    backward pass writes is the G the optimizer step reads (same buffer, same pitch).  The oracle runs the same
    chain on its own: its G differs from the device's in the last bfloat16 bit of a few entries, which the
    moments see as noise far below their tolerance; the stochastic rounding of the weights is compared in
    bulk only (a changed G moves some elements across a rounding boundary)."""
    from parity_utils import check_moments
    T, m, n, r = 640, 256, 768, 64
    W_q, X_bits, dY_bits = _linear_case(T, m, n, seed=21)
    rng = np.random.default_rng(2)
    P = O.quantize_rtn(np.linalg.qr(rng.standard_normal((m, r)))[0].astype(np.float32), 4)
    M0 = (rng.standard_normal((r, n)) * 1e-3).astype(np.float32)
    V0 = (rng.random((r, n)) * 1e-6).astype(np.float32)
    hyp = O.Hyper(lr=1e-3, step=3, seed=77)
    _, _, _, G_bits = O.int8_linear_backward(dY_bits, X_bits, W_q)
    ref = O.project_step(G_bits, P, W_q, M0, V0, hyp)

    Wd, Xd, dYd, Pd = to_device_q(W_q), g_to_device(X_bits), g_to_device(dY_bits), to_device_q(P)
    Md, Vd = f32_to_device(M0), f32_to_device(V0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    G = B.int8_linear_backward_weight(dYd, Xd, status=status)
    B.project_step(G, Pd, Wd, Md, Vd, B.Hyper(lr=hyp.lr, step=hyp.step, seed=hyp.seed), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_moments(Md.cpu().numpy(), ref["M"], "M", MOMENT_TOL)
    check_moments(Vd.cpu().numpy(), ref["V"], "V", MOMENT_TOL)
    got = from_device_q(Wd)
    diff = np.abs(got.codes.astype(np.int32) - ref["W"].codes.astype(np.int32))
    assert diff.max() <= 1 and np.mean(diff != 0) <= 0.02
    np.testing.assert_allclose(got.scales, ref["W"].scales, rtol=1e-4)


def test_int8_linear_refusals():
    W_q, X_bits, dY_bits = _linear_case(8, 64, 256, seed=0)
    Wd, Xd, dYd = to_device_q(W_q), g_to_device(X_bits), g_to_device(dY_bits)
    with pytest.raises(B.QgError):                   # X with the wrong inner extent for W: pitch shorter than n
        B.int8_linear_forward(Xd[:, :64].contiguous(), Wd)
    narrow = torch.zeros((8, 72), dtype=torch.int16, device="cuda")[:, :70]
    with pytest.raises(B.QgError):                   # the pitch (72) does not cover the last 64-column slab of 70 columns
        B.int8_linear_backward_weight(narrow, Xd)
