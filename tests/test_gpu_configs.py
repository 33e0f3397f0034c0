"""The layer-stack configurations as RUNS: step -> refresh -> INT4 -> similarity -> gate -> step on the new
projection, chained by a small host loop that is the consumer of the C ABI (Sec. 3.2 adaptive lazy update,
Sec. 3.5 / Fig. 4 the per-layer pipeline, Sec. 4.1 the 130M / 350M / 7B setups).

Protocol (teacher-forced).  The oracle advances its own trajectory.  At a checked step the oracle's pre-step
state (W codes / scales / zero points, M, V, P) is uploaded, one GPU step runs, and the result is compared
with the oracle's post-step state.  At a refresh both sides compute a new projection from the same gradient;
the subspaces are compared by their largest principal angle, the similarity statistic and the gate are
compared on the ORACLE's projection pair (identical inputs on both sides), and the run continues on the
oracle's INT4 codes.  A matrix is refreshed at step t when t - t_last >= interval, and always at its first
step; the gate (threshold 0.4) doubles the interval when the last k similarities are all above the threshold.

What is scaled down, so that the CPU oracle finishes in minutes: which matrices run how many steps (stated at
each test).  Shapes, ranks, group sizes, hyper-parameters and the gradient model are the configurations' own.
"""
import math

import numpy as np
import pytest
import torch

import oracle as O
from paper_2407_08296_b200 import binding as B
from paper_2407_08296_b200 import synth

from parity_utils import (StepTaps, check_moments, check_step_on_column_blocks, check_weights_loosely, column_block, f32_to_device, from_device_q,
                          g_to_device, run_and_check_step, run_and_check_step_light, to_device_q)

pytestmark = pytest.mark.gpu

THRESHOLD = 0.4          # Sec. 3.2: similarity above which a layer's subspace counts as stable
ANGLE_BAR = 1e-2         # largest principal angle between the refreshed subspaces, rad
SIM_TOL = 1e-5


def refresh_is_due(t, t_last, interval):
    return t_last is None or t - t_last >= interval


class MatrixRun:
    """One matrix of a stack on both sides: the oracle's state, and the host state (gate, last refresh) of the
    loop that drives the library."""

    def __init__(self, spec, seed=0, base_interval=200, k=1, sim_cols=0, forced_refresh=()):
        self.spec, self.k, self.sim_cols = spec, k, sim_cols
        self.gm = synth.GradientModel(spec.m, spec.n, seed=seed, matrix_index=spec.index)
        self.sr_seed = synth.matrix_seed(seed, spec.index)
        self.W = O.quantize_rtn(synth.initial_weight(spec.m, spec.n, seed, spec.index), 8)
        self.M = np.zeros((spec.r, spec.n), np.float32)
        self.V = np.zeros((spec.r, spec.n), np.float32)
        self.P = None
        self.forced = set(forced_refresh)
        # oracle side of the lazy update
        self.gate_ref, self.t_last_ref = O.GateState(interval=base_interval), None
        # library side: the C gate and the loop's own bookkeeping
        self.gate_lib, self.t_last_lib = B.Gate(interval=base_interval, threshold=THRESHOLD, k=k), None
        self.log = []                                   # (step, similarity, doubled, interval after)

    def due(self, t):
        ref = refresh_is_due(t, self.t_last_ref, self.gate_ref.interval) or t in self.forced
        lib = refresh_is_due(t, self.t_last_lib, self.gate_lib.interval) or t in self.forced
        assert ref == lib, f"{self.spec.name}@{self.spec.layer} step {t}: refresh decisions differ"
        return ref

    def refresh(self, t, gb, check_gpu=True):
        """Both sides refresh from the gradient of step t; returns the largest principal angle (or None)."""
        r = self.spec.r
        P32_ref, P_new, _ = O.refresh_subspace(gb, r)
        angle = None
        dP_prev = to_device_q(self.P) if self.P is not None else None
        if check_gpu:
            P32 = torch.zeros((self.spec.m, r), dtype=torch.float32, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            sim_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
            got = B.refresh_subspace(g_to_device(gb), r, iters=12, seed=t, P_fp32=P32, P_prev=dP_prev,
                                     sim_cols=self.sim_cols, sim=sim_dev if dP_prev is not None else None, status=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, "refresh: device status word"
            Pg = P32.cpu().numpy()
            angle = O.principal_angle(P32_ref, Pg)
            assert angle < ANGLE_BAR, f"{self.spec.name}@{self.spec.layer} step {t}: largest principal angle {angle:.3e} rad"
            want = O.quantize_rtn(Pg, 4)                 # what the library stored is Quant_4 of its own vectors
            stored = from_device_q(got)
            assert np.array_equal(stored.codes, want.codes) and np.array_equal(stored.scales, want.scales)
            assert np.array_equal(stored.zeros, want.zeros)
        if self.P is not None:
            c = self.sim_cols if self.sim_cols > 0 else None
            sim_ref = O.subspace_similarity(self.P, P_new, c)
            # identical inputs on both sides: the oracle's previous and new codes
            sim_lib = float(B.subspace_similarity(dP_prev, to_device_q(P_new), self.sim_cols).item())
            assert abs(sim_lib - sim_ref) <= SIM_TOL, f"similarity {sim_lib} vs {sim_ref}"
            if check_gpu:                                # the refresh's own output: its projection, not the oracle's
                assert abs(float(sim_dev.item()) - sim_ref) <= 2e-2
            doubled_ref = O.gate_update(self.gate_ref, sim_ref, THRESHOLD, self.k)
            doubled_lib = self.gate_lib.update(sim_lib)
            assert doubled_ref == doubled_lib and self.gate_ref.interval == self.gate_lib.interval
            self.log.append((t, sim_ref, doubled_ref, self.gate_ref.interval))
        self.P = P_new                                   # teacher forcing: the run continues on the oracle's codes
        self.t_last_ref = self.t_last_lib = t
        return angle

    def step(self, t, gb, check="full"):
        hyp = O.Hyper(step=t, seed=self.sr_seed)
        ref = O.project_step(gb, self.P, self.W, self.M, self.V, hyp)
        stats = None
        if check == "full":
            stats = run_and_check_step(gb, self.P, self.W, self.M, self.V, hyp, ref=ref)
        elif check == "light":
            run_and_check_step_light(gb, self.P, self.W, self.M, self.V, hyp, ref)
        self.W, self.M, self.V = ref["W"], ref["M"], ref["V"]
        return stats


def _specs(workload, layers=None, names=None):
    out = synth.stack_matrices(workload)
    if layers is not None:
        out = [s for s in out if s.layer in layers]
    if names is not None:
        out = [s for s in out if s.name in names]
    return out


# ----------------------------------------------------------------------------- LLaMA-130M stack, r = 256, refresh every 200
def test_config2_every_matrix_through_its_first_steps():
    """All 84 matrices (12 layers x 7) at steps 1-3: the refresh at step 1 on both sides (GPU refresh compared
    for layers 0 and 11, two of each shape and more; every matrix continues on the oracle's codes), then step 1
    with every check, steps 2 and 3 for every matrix in ONE grouped launch sequence (a plan, teacher-forced,
    the configuration the throughput run uses) with the moments and weights compared, and layer 0 with every
    check as well."""
    runs = [MatrixRun(s, seed=0, base_interval=200) for s in _specs("llama130m")]
    assert len(runs) == 84
    worst_angle = 0.0
    for mr in runs:
        gb = mr.gm.sample(1)
        assert mr.due(1)
        a = mr.refresh(1, gb, check_gpu=mr.spec.layer in (0, 11))
        worst_angle = max(worst_angle, a or 0.0)
        st = mr.step(1, gb, "full")
        assert st["mismatch"] <= 1e-3
    for t in (2, 3):
        items, refs = [], []
        for mr in runs:
            assert not mr.due(t)
            gb = mr.gm.sample(t)
            hyp = O.Hyper(step=t, seed=mr.sr_seed)
            ref = O.project_step(gb, mr.P, mr.W, mr.M, mr.V, hyp)
            if mr.spec.layer == 0:
                run_and_check_step(gb, mr.P, mr.W, mr.M, mr.V, hyp, ref=ref)
            items.append({"G": g_to_device(gb), "P": to_device_q(mr.P), "W": to_device_q(mr.W), "M": f32_to_device(mr.M),
                          "V": f32_to_device(mr.V), "seed": mr.sr_seed})
            refs.append(ref)
        plan = B.StepPlan(items)
        plan.step(B.Hyper(step=t))
        torch.cuda.synchronize()
        assert int(plan.status.item()) == 0
        for mr, it, ref in zip(runs, items, refs):
            check_moments(it["M"].cpu().numpy(), ref["M"], "M")
            check_moments(it["V"].cpu().numpy(), ref["V"], "V")
            check_weights_loosely(from_device_q(it["W"]), ref["W"])
            mr.W, mr.M, mr.V = ref["W"], ref["M"], ref["V"]
        plan.close()
    assert worst_angle < ANGLE_BAR


def test_config2_one_matrix_of_each_shape_through_200_steps():
    """q, gate and down of layer 5 through all 200 steps of the configuration: the refresh at step 1, none
    after it (interval 200: the next one would fall on step 201), a GPU step from the oracle's state at EVERY
    step (moments by the 2e-3 rule, weights within one level), every check at steps 1-3, every 25th and the
    last two."""
    runs = [MatrixRun(s, seed=0, base_interval=200) for s in _specs("llama130m", layers=(5,), names=("q", "gate", "down"))]
    full_at = {1, 2, 3, 199, 200} | set(range(25, 200, 25))
    for t in range(1, 201):
        for mr in runs:
            gb = mr.gm.sample(t)
            if mr.due(t):
                assert t == 1
                mr.refresh(t, gb)
            mr.step(t, gb, "full" if t in full_at else "light")
    for mr in runs:
        assert mr.t_last_ref == 1 and mr.gate_ref.interval == 200 and not mr.log
        assert refresh_is_due(201, mr.t_last_lib, mr.gate_lib.interval)


# ----------------------------------------------------------------------------- LLaMA-350M stack, adaptive refresh, drifting subspaces
def _theta(layer):
    return (layer / 23.0) * math.pi / 2.0       # layer 0 never drifts ("early bird"), the last layer turns a quarter circle each time


def test_config3_gate_in_the_loop_with_drifting_subspaces():
    """Layers 0, 11 and 23, all seven matrices of each, over the 500 steps of the configuration: every 100 steps the
    planted left subspace of layer l turns by theta_l = (l / 23) pi / 2; base interval 200, k = 1, similarity over the 8
    leading columns.  The loop acts at the refresh steps (a refresh needs only that step's gradient): both
    sides refresh, the similarity and the gate are compared, and the step that follows runs on the new projection
    with every check (moments carried over from the matrix's previous checked step).  Both gate outcomes occur:
    layer 0 doubles its interval at step 201 and is not refreshed again, layer 23 keeps 200 and is refreshed at
    401 as well."""
    runs = [MatrixRun(s, seed=0, base_interval=200, k=1, sim_cols=8) for s in _specs("llama350m", layers=(0, 11, 23))]
    assert len(runs) == 21
    for t in range(1, 501):
        for mr in runs:
            if t > 1 and (t - 1) % 100 == 0:
                mr.gm.rotate(_theta(mr.spec.layer), (t - 1) // 100)
            if mr.due(t):
                gb = mr.gm.sample(t)
                mr.refresh(t, gb, check_gpu=mr.spec.name in ("q", "up", "down") or t == 1)
                st = mr.step(t, gb, "full")                # a step on the refreshed (teacher-forced) projection
                assert st["mismatch"] <= 1e-3
    doubled, kept = 0, 0
    for mr in runs:
        assert mr.gate_ref.interval == mr.gate_lib.interval
        steps = [e[0] for e in mr.log]
        if mr.spec.layer == 0:
            assert steps == [201] and mr.log[0][2] and mr.gate_ref.interval == 400, (mr.spec, mr.log)
            assert mr.log[0][1] > 0.9                      # no drift: the leading directions persist
            doubled += 1
        if mr.spec.layer == 23:
            assert steps == [201, 401] and not any(e[2] for e in mr.log) and mr.gate_ref.interval == 200, (mr.spec, mr.log)
            assert max(e[1] for e in mr.log) < THRESHOLD   # a quarter turn twice: nothing of the old subspace is left
            kept += 1
    assert doubled == 7 and kept == 7


def test_config3_a_drifting_matrix_through_500_steps():
    """q of layer 23 (1024 x 1024, r = 256) through all 500 steps with the loop of the test above and a GPU step
    from the oracle's state at every step: every check at steps 1-3, at each refresh step and the step after it
    and at every 50th step, the moment and one-level rules in between; q of layer 0 the same way through step 202
    (its refresh at 201 doubles the interval)."""
    long_run = MatrixRun(_specs("llama350m", layers=(23,), names=("q",))[0], seed=0, base_interval=200, k=1, sim_cols=8)
    short_run = MatrixRun(_specs("llama350m", layers=(0,), names=("q",))[0], seed=0, base_interval=200, k=1, sim_cols=8)
    for mr, last in ((long_run, 500), (short_run, 202)):
        after_refresh = set()
        for t in range(1, last + 1):
            if t > 1 and (t - 1) % 100 == 0:
                mr.gm.rotate(_theta(mr.spec.layer), (t - 1) // 100)
            gb = mr.gm.sample(t)
            full = t <= 3 or t % 50 == 0 or t in after_refresh
            if mr.due(t):
                mr.refresh(t, gb)
                after_refresh.add(t + 1)
                full = True
            mr.step(t, gb, "full" if full else "light")
    assert [e[0] for e in long_run.log] == [201, 401] and long_run.gate_lib.interval == 200
    assert [e[0] for e in short_run.log] == [201] and short_run.gate_lib.interval == 400


# ----------------------------------------------------------------------------- LLaMA-7B stack, r = 1024, forced refresh mid-run
def test_config5_forced_refresh_mid_run_at_full_size():
    """One matrix of each 7B shape (q of layer 0, gate of layer 15, down of layer 31; r = 1024) through the 50
    steps of the configuration with the forced refresh at step 26.  The oracle advances the first and the last
    column group (every column of a step depends on its own column of G, M, V, W only) through all 50 steps;
    the library runs the whole matrix at the checked steps 1, 2, 25, 26 (refresh, then the step on the refreshed
    and teacher-forced projection), 27 and 50, with the oracle's block state written into its buffers first.
    Both refreshes (steps 1 and 26: different noise, so a different bulk subspace) are compared with the exact
    SVD at full size.  The gradient's noise is drawn per 256-column block here, so that the 44 steps in
    between cost only the blocks."""
    picks = [(0, "q"), (15, "gate"), (31, "down")]
    checked = {1, 2, 25, 26, 27, 50}
    for layer, name in picks:
        spec = _specs("llama7b", layers=(layer,), names=(name,))[0]
        m, n, r = spec.m, spec.n, spec.r
        mr = MatrixRun(spec, seed=0, base_interval=200, k=1, sim_cols=8, forced_refresh=(26,))
        blocks = [(0, 256), (n - 256, n)]
        W0 = mr.W
        state = {blk: [column_block(W0, *blk), np.zeros((r, 256), np.float32), np.zeros((r, 256), np.float32)] for blk in blocks}
        mr.W = mr.M = mr.V = None                       # the full-size state lives on the device only
        dW, dM, dV = to_device_q(W0), f32_to_device(np.zeros((r, n), np.float32)), f32_to_device(np.zeros((r, n), np.float32))
        angles = []
        for t in range(1, 51):
            full_g = None
            if mr.due(t):
                assert t in (1, 26)
                full_g = mr.gm.sample_columns(t, 0, n)
                angles.append(mr.refresh(t, full_g))
                if t == 26:
                    assert len(mr.log) == 1 and mr.log[0][0] == 26
            hyp = O.Hyper(step=t, seed=mr.sr_seed)
            if t in checked:
                if full_g is None:
                    full_g = mr.gm.sample_columns(t, 0, n)
                # the oracle's pre-step block state into the device buffers
                Mh, Vh = dM.cpu().numpy(), dV.cpu().numpy()
                Wh = from_device_q(dW)
                for (a, b), (Wb, Mb, Vb) in state.items():
                    Mh[:, a:b], Vh[:, a:b] = Mb, Vb
                    Wh.codes[:, a:b] = Wb.codes
                    Wh.scales[:, a // 256:b // 256], Wh.zeros[:, a // 256:b // 256] = Wb.scales, Wb.zeros
                dW, dM, dV = to_device_q(Wh), f32_to_device(Mh), f32_to_device(Vh)
                taps = StepTaps(m, n, r, dW.ld)
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                B.project_step(g_to_device(full_g), to_device_q(mr.P), dW, dM, dV, B.Hyper(step=t, seed=mr.sr_seed),
                               status=status, debug=taps.as_dict())
                torch.cuda.synchronize()
                assert int(status.item()) == 0
                gpu = {"M": dM.cpu().numpy(), "V": dV.cpu().numpy(), "R": taps.R.cpu().numpy(), "N": taps.N.cpu().numpy(),
                       "N_b": taps.N_b.cpu().numpy(), "W_pre": taps.W_pre.cpu().numpy(), "W": from_device_q(dW)}
                del taps
                for (a, b), (Wb, Mb, Vb) in state.items():
                    check_step_on_column_blocks([(0, b - a)], full_g[:, a:b], mr.P, Wb, Mb, Vb, hyp,
                                                {k: (column_block(v, a, b) if k == "W" else v[:, a:b]) for k, v in gpu.items()},
                                                col0=a)
            for (a, b), st in state.items():
                gblk = full_g[:, a:b] if full_g is not None else mr.gm.sample_columns(t, a, b)
                out = O.project_step(gblk, mr.P, st[0], st[1], st[2], hyp, col0=a)
                state[(a, b)] = [out["W"], out["M"], out["V"]]
        assert len(angles) == 2 and max(angles) < ANGLE_BAR
        del dW, dM, dV
        torch.cuda.empty_cache()
