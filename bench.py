#!/usr/bin/env python
"""Throughput of the Q-GaLore optimizer step on a LLaMA-shaped layer stack (one B200 per rank).

A "step" is one pass of the whole hot path (dequantize P, project, Adam, project back, dequantize-
add, stochastic-rounding requantization) over every 2-D attention/MLP matrix of the stack.
Prints ONE JSON line: weight elements updated per second, with the per-step roofline, the end-to-end
figure (gradients copied from pinned host memory every step) and the CPU oracle timed beside it.

With no --workload the run times BOTH stacks the target is set on: LLaMA-7B (the largest single-GPU
configuration; the top-level keys of the line) and then LLaMA-1B (the same block under "also": {"llama1b": ...}).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama1b|llama7b|...] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "Q-GaLore optimizer step: weight elements updated/s"
UNIT = "elements/s"
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained")}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def matrix_flops(m, n, r):
    return 4.0 * m * n * r                      # two dense contractions of 2 m n r each


MOMENT_BYTES = 16.0      # M, V read + written per element of the low-rank state: 4 x 4 bytes in fp32,
                         # 4 x 1 byte + 4 scale words per 32 elements = 4.5 with --moments 8


def matrix_bytes(m, n, r):
    """Algorithmic HBM bytes of one step of one matrix: G (bf16), W codes read+write, W scale/zero
    read+write, P codes + scale/zero, M and V fp32 read+write."""
    ng_n = (n + 255) // 256
    ng_r = (r + 255) // 256
    return 2 * m * n + 2 * m * n + 16 * m * ng_n + m * r // 2 + 8 * m * ng_r + MOMENT_BYTES * r * n


# Algorithmic units of each kernel of the step, per matrix (what the method has to move or compute, not what
# the implementation happens to move): the projection reads G and reads+writes M, V and does half the flops;
# the back-projection reads+writes the INT8 codes and their scale/zero and does the other half; the bf16
# direction N_b between them and the bf16 copy of P are implementation traffic and are not counted.
def k1_units(m, n, r):
    return 2.0 * m * n * r, 2 * m * n + MOMENT_BYTES * r * n + m * r // 2 + 8 * m * ((r + 255) // 256)


def k2_units(m, n, r):
    return 2.0 * m * n * r, 2 * m * n + 16 * m * ((n + 255) // 256) + m * r // 2 + 8 * m * ((r + 255) // 256)


def dq_units(m, n, r):
    return 0.0, m * r // 2 + 8 * m * ((r + 255) // 256)


# Lane-operations per weight element that the requantizing epilogue of the back-projection cannot avoid,
# counted from the definitions (scalar 32-bit operations, no credit for packed pairs): Philox4x32-10 for
# eight 16-bit uniforms = 10 rounds x (2 wide multiplies + 2 three-input XORs) = 5 per element; byte -> float,
# minus zero point, times scale, minus lr*alpha*D = 4; minimum and maximum = 2; times 1/s', uniform -> float,
# subtract, round up, clamp, pack = 6.
K2_ALU_OPS_PER_ELEMENT = 17
ALU_LANES_PER_SM_CLOCK = 128            # 4 schedulers x 32 lanes issue one instruction per clock


def k2_alu_ops(m, n, r):
    return float(K2_ALU_OPS_PER_ELEMENT) * m * n


def load_ncu_traffic(kernel_revision):
    """Measured DRAM bytes over algorithmic bytes of each kernel, per workload, from the ncu captures summarised
    under profiles/ (read from the small table beside them).  A row counts only if it was taken on the kernels as
    they stand: its revision tag must equal the one the library reports.  The captures are of small cases (a few
    layers); every kernel streams each byte once, so its traffic grows in proportion to its algorithmic bytes and
    the ratio carries over to a full launch.  Returns {workload: {kernel: ratio}}."""
    table = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic_ratio.txt")
    if not os.path.exists(path):
        return table
    with open(path) as f:
        for line in f:
            f4 = line.split()
            if len(f4) < 4 or line.startswith("#"):
                continue
            workload, kernel, ratio, revision = f4[0], f4[1], float(f4[2]), f4[3]
            if revision == kernel_revision:
                table.setdefault(workload, {})[kernel] = ratio
    return table


def stack_roofline(specs, peaks):
    t = 0.0
    fl = by = 0.0
    for s in specs:
        f, b = matrix_flops(s.m, s.n, s.r), matrix_bytes(s.m, s.n, s.r)
        t += max(f / (peaks["bf16_tflops"] * 1e12), b / (peaks["hbm_gbs"] * 1e9))
        fl += f
        by += b
    return t, fl, by


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for (_, l) in self.lines]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------- reference arm
def oracle_sample(workload, steps, warmup):
    """Times the CPU oracle, as it stands, on one matrix of each distinct shape of the workload and
    extrapolates by the shape counts.  Returns (elements/s, seconds per stack step, description)."""
    import oracle as O
    from paper_2407_08296_b200 import synth
    shapes = synth.distinct_shapes(workload)
    per_step = 0.0
    elements = 0
    detail = []
    for (m, n, r, count) in shapes:
        gm = synth.GradientModel(m, n, seed=0, matrix_index=0)
        P = O.quantize_rtn(synth.random_orthonormal(m, r, seed=0), 4)
        W = O.quantize_rtn(synth.initial_weight(m, n, 0), 8)
        M = np.zeros((r, n), np.float32)
        V = np.zeros((r, n), np.float32)
        g = gm.sample(1)
        best = None
        for it in range(warmup + steps):
            t0 = time.perf_counter()
            out = O.project_step(g, P, W, M, V, O.Hyper(step=it + 1, seed=1))
            dt = time.perf_counter() - t0
            W, M, V = out["W"], out["M"], out["V"]
            if it >= warmup or dt > 2.0:
                best = dt if best is None else min(best, dt)
            if dt > 2.0:                                  # a 7B-sized matrix: one step is the bounded sample
                break
        per_step += best * count
        elements += m * n * count
        detail.append(f"{m}x{n} r{r}: {best:.3f}s x{count}")
    return (elements / per_step, per_step,
            f"best of up to {steps} oracle steps (after {warmup} warm-up; a single step where one takes over 2 s) on one matrix "
            "of each distinct shape, extrapolated by shape counts (" + "; ".join(detail) + ")")


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 2))
    args.workload = args.workload or "llama7b"
    value, per_step, sample = oracle_sample(args.workload, steps, 0 if args.warmup == 0 else 1)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "note": "CPU oracle (numpy/scipy fp64), not a GPU program"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------- our arm
def whole_job_throughput(ms_total, elements_per_rank, steps, world, device):
    """Every rank steps its own replica of the stack (matrices are independent units: no collective on the
    data path).  The job's time is the slowest rank's (MAX over ranks of the device-timed milliseconds), its
    throughput the elements all ranks updated in that time.  Returns (ms_total of the job, elements/s)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_total], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    return ms, elements_per_rank * world * steps / (ms * 1e-3)


def time_linear(items, device, tokens, peak_tflops):
    """The INT8 linear layer either side of the step (App. A), timed apart from it: forward, input gradient and
    weight gradient of one matrix of each distinct shape on `tokens` rows of synthetic activations, CUDA events
    around 10 calls after 3 warm-up calls.  TFLOP/s against the burst bf16 peak (each product is timed alone)."""
    import torch
    from paper_2407_08296_b200 import binding as B
    seen, out = set(), []
    status = torch.zeros(1, dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream()
    for it in items:
        sp = it["spec"]
        if (sp.m, sp.n) in seen:
            continue
        seen.add((sp.m, sp.n))
        gen = torch.Generator(device=device).manual_seed(sp.m * 31 + sp.n)
        X = B.zeros_matrix(tokens, sp.n, torch.bfloat16, device)
        X.copy_(torch.randn((tokens, sp.n), device=device, generator=gen))
        dY = B.zeros_matrix(tokens, sp.m, torch.bfloat16, device)
        dY.copy_(torch.randn((tokens, sp.m), device=device, generator=gen) * 0.1)
        Y = B.empty_matrix(tokens, sp.m, torch.bfloat16, device)
        dX = B.empty_matrix(tokens, sp.n, torch.bfloat16, device)
        G = B.empty_matrix(sp.m, sp.n, torch.bfloat16, device)
        calls = {"forward": lambda: B.int8_linear_forward(X, it["W"], out=Y, status=status),
                 "backward_input": lambda: B.int8_linear_backward_input(dY, it["W"], out=dX, status=status),
                 "backward_weight": lambda: B.int8_linear_backward_weight(dY, X, out=G, status=status)}
        row = {"shape": f"{sp.m}x{sp.n}"}
        flops = 2.0 * tokens * sp.m * sp.n
        for name, fn in calls.items():
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(10):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 10
            row[name] = {"ms": ms, "tflops": flops / ms / 1e9, "frac_of_peak": flops / ms / 1e9 / peak_tflops}
        out.append(row)
        del X, dY, Y, dX, G
    return {"tokens": tokens, "peak_tflops": peak_tflops, "per_shape": out, "device_status": int(status.item()),
            "note": "not part of the timed step; forward and backward_input dequantize the INT8 weight inside the GEMM"}


def time_refresh(items, device):
    """The occasional subspace refresh (Sec. 3.5), timed apart from the step (12 subspace iterations on a block of
    2r columns, Rayleigh-Ritz, INT4): per distinct shape, one matrix alone (the latency of a refresh) and a batch of
    up to eight matrices of that shape in one qgalore_refresh_subspace_batched call (how a stack is refreshed),
    CUDA events around the second of two calls each; extrapolated to the stack by the shape counts.  Also the
    similarity to the random projection the stack was built with, as the gate would see it."""
    import torch
    from paper_2407_08296_b200 import binding as B
    groups = {}
    for it in items:
        sp = it["spec"]
        groups.setdefault((sp.m, sp.n, sp.r), []).append(it)
    per_shape, total_single, total_batched = [], 0.0, 0.0
    stream = torch.cuda.current_stream()
    for (m, n, r), group in groups.items():
        block = min((2 * r + 63) // 64 * 64, min(m, n) // 64 * 64)
        nb = min(8, len(group))
        per = B.workspace_bytes(B.QG_OP_REFRESH, m, n, block)
        ws = torch.empty(per * nb, dtype=torch.uint8, device=device)
        sim = torch.zeros(1, dtype=torch.float32, device=device)
        status = torch.zeros(1, dtype=torch.int32, device=device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for rep in range(2):
            e0.record(stream)
            B.refresh_subspace(group[0]["G"], r, iters=12, seed=1, P_prev=group[0]["P"], sim=sim, workspace=ws, status=status)
            e1.record(stream)
            torch.cuda.synchronize()
        ms_single = e0.elapsed_time(e1)
        batch = [{"G": it["G"], "seed": 1 + k, "P_new": B.dense_projection(m, r, 4, device)} for k, it in enumerate(group[:nb])]
        for rep in range(2):
            e0.record(stream)
            B.refresh_subspace_batched(batch, r, iters=12, workspace=ws, status=status)
            e1.record(stream)
            torch.cuda.synchronize()
        ms_batch = e0.elapsed_time(e1)
        count = len(group)
        per_shape.append({"shape": f"{m}x{n} r{r}", "count": count, "ms": ms_single, "block": block, "batch": nb,
                          "batch_ms": ms_batch, "ms_per_matrix_batched": ms_batch / nb,
                          "similarity_to_previous": float(sim.item()), "device_status": int(status.item())})
        total_single += ms_single * count * 1e-3
        total_batched += ms_batch / nb * count * 1e-3
        del ws, batch
        torch.cuda.empty_cache()
    return {"iters": 12, "per_shape": per_shape, "stack_seconds": total_single, "stack_seconds_batched": total_batched,
            "stack_seconds_best": min(total_single, total_batched),
            "note": "not part of the timed step; per distinct shape one matrix alone and a batch of up to 8, extrapolated by shape counts"}


def bench_workload(workload, args, B, torch, dist, device, world, rank, local_rank, peaks, peak_kind, extras):
    """Times one stack and returns the keys of its result block (rank 0; None elsewhere)."""
    from paper_2407_08296_b200.synth_device import build_stack
    global MOMENT_BYTES
    MOMENT_BYTES = 4.5 if args.moments == 8 else 16.0
    # every rank holds and steps its own replica of the stack: matrices are independent units, no collective
    specs, items = build_stack(workload, device, seed=rank, layers=args.layers, moments=args.moments)
    batch = B.StepPlan(items)
    elements = batch.elements
    hyper = B.Hyper(rounding=B.QG_ROUND_NEAREST if args.rounding == "nearest" else B.QG_ROUND_STOCHASTIC)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_no = 0
    for _ in range(args.warmup):
        step_no += 1
        hyper.step = step_no
        batch.step(hyper)
    barrier()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.launch_count()
    barrier()
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step_no += 1
        hyper.step = step_no
        batch.step(hyper)
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    launches = B.launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    status = int(batch.status.item())

    ms_total, value = whole_job_throughput(ms_total, elements, args.steps, world, device)
    ms_per_step = ms_total / args.steps

    # ---- end to end: gradients arrive from pinned host memory every step, the status word is read back
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    h2d = sum(it["G"].shape[0] * it["G"].shape[1] * 2 for it in items)
    host_g = [torch.empty((it["G"].shape[0], it["G"].shape[1]), dtype=torch.bfloat16).pin_memory() for it in items]
    for hg, it in zip(host_g, items):
        hg.copy_(it["G"])
    host_status = torch.zeros(1, dtype=torch.int32).pin_memory()
    # two sets of device gradient buffers and a plan over each (same weights, moments, projections): the copy of
    # the next step's gradients runs on a second stream while this step computes, as a training loop whose
    # gradients arrive from the host would arrange it.  Every step still pays its whole copy and its read-back.
    alt_g = [B.empty_matrix(it["G"].shape[0], it["G"].shape[1], torch.bfloat16, device) for it in items]
    plan_alt = B.StepPlan([{**it, "G": g} for it, g in zip(items, alt_g)])
    plans, gsets = [batch, plan_alt], [[it["G"] for it in items], alt_g]
    copy_stream = torch.cuda.Stream(device=device)
    copied = [torch.cuda.Event(), torch.cuda.Event()]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    copy_stream.wait_event(e0)
    for k in range(e2e_steps):
        step_no += 1
        hyper.step = step_no
        b = k & 1
        with torch.cuda.stream(copy_stream):
            if k >= 2:
                copy_stream.wait_event(done[b])            # the step that read this set has finished
            for hg, g in zip(host_g, gsets[b]):
                g.copy_(hg, non_blocking=True)
            copied[b].record(copy_stream)
        stream.wait_event(copied[b])
        plans[b].step(hyper)
        host_status.copy_(plans[b].status, non_blocking=True)
        done[b].record(stream)
    e1.record(stream)
    stream.synchronize()
    barrier()
    _, e2e_value = whole_job_throughput(e0.elapsed_time(e1), elements, e2e_steps, world, device)
    status |= int(plan_alt.status.item())
    plan_alt.close()
    del host_g, alt_g, plan_alt, plans, gsets

    # ---- per-kernel device time: a second pass of the same steps with an event pair around every launch
    names = list(B.STEP_KERNEL_NAMES)
    kms = [0.0] * len(names)
    kcount = [0] * len(names)
    for _ in range(args.steps):
        step_no += 1
        hyper.step = step_no
        ms3, c3 = batch.step_timed(hyper)
        kms = [a + b for a, b in zip(kms, ms3)]
        kcount = [a + b for a, b in zip(kcount, c3)]
    barrier()

    block = None
    if rank == 0:
        t_roof, flops, nbytes = stack_roofline(specs, peaks)
        t_roof_nom, _, _ = stack_roofline(specs, NOMINAL)
        t_c = flops / (peaks["bf16_tflops"] * 1e12)
        t_m = nbytes / (peaks["hbm_gbs"] * 1e9)
        sec = ms_per_step * 1e-3
        # roofline of every kernel from its live-measured duration: the bound is the slowest of the tensor pipe
        # (burst bf16 peak: the primary denominator; the sustained figure is reported beside it), HBM (copy
        # peak) and, for the requantizing epilogue, the plain ALUs (lanes x SMs x the maximum SM clock)
        units = {"dequant_p_grouped": dq_units, "project_adam": k1_units, "backproject_sr": k2_units}
        peak_tf, peak_tf_sus = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
        sm_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        alu_peak = torch.cuda.get_device_properties(device).multi_processor_count * ALU_LANES_PER_SM_CLOCK * sm_mhz * 1e6
        per_kernel = {}
        for k, nm in enumerate(names):
            if kcount[k] == 0:
                continue
            kf = sum(units[nm](sp.m, sp.n, sp.r)[0] for sp in specs) * args.steps
            kb = sum(units[nm](sp.m, sp.n, sp.r)[1] for sp in specs) * args.steps
            ko = sum(k2_alu_ops(sp.m, sp.n, sp.r) for sp in specs) * args.steps if nm == "backproject_sr" else 0.0
            ksec = max(kms[k] * 1e-3, 1e-12)
            cand = {"tensor": (kf / (peak_tf * 1e12), kf / ksec / 1e12, peak_tf, "TFLOP/s"),
                    "hbm": (kb / (peaks["hbm_gbs"] * 1e9), kb / ksec / 1e9, peaks["hbm_gbs"], "GB/s"),
                    "alu": (ko / alu_peak, ko / ksec / 1e12, alu_peak / 1e12, "Tlane-op/s")}
            bound = max(cand, key=lambda c: cand[c][0])
            per_kernel[nm] = {"bound": bound, "achieved": cand[bound][1], "peak": cand[bound][2], "unit": cand[bound][3],
                              "frac": cand[bound][1] / cand[bound][2], "ms_per_step": kms[k] / args.steps,
                              "launches_per_step": kcount[k] / args.steps,
                              "bound_ms_per_step": {c: cand[c][0] * 1e3 / args.steps for c in cand},
                              "flops": kf / args.steps, "bytes": kb / args.steps, "alu_ops": ko / args.steps}
            if bound == "tensor":
                per_kernel[nm]["frac_of_sustained_peak"] = cand[bound][1] / peak_tf_sus
        # the dominant kernel is named by what the shapes demand, not by a timing: the one whose own bound is largest
        dom_name = max(per_kernel, key=lambda nm: max(per_kernel[nm]["bound_ms_per_step"].values()))
        dom = names.index(dom_name)
        k_flops = per_kernel[dom_name]["flops"] * args.steps
        k_bytes = per_kernel[dom_name]["bytes"] * args.steps
        roof = {key: per_kernel[dom_name][key] for key in ("bound", "achieved", "peak", "unit")}
        roof["frac"] = roof["achieved"] / roof["peak"]
        if roof["bound"] == "tensor":
            roof["frac_of_sustained_peak"] = roof["achieved"] / peak_tf_sus
            roof["sustained_peak"] = peak_tf_sus
        # measured DRAM traffic per launch = (ratio from the committed ncu capture) x (algorithmic bytes per launch)
        traffic = extras["traffic"].get(workload, {}) if args.moments == 32 else {}
        tpe = traffic.get(dom_name)
        roof["traffic"] = None if tpe is None else tpe * k_bytes / max(kcount[dom], 1)
        roof["traffic_over_algorithmic"] = tpe
        roof["traffic_per_kernel_per_launch"] = {nm: traffic[nm] * per_kernel[nm]["bytes"] * args.steps / max(kcount[names.index(nm)], 1)
                                                 for nm in per_kernel if nm in traffic} or None
        roof["kernel"] = dom_name
        roof["kernel_revision"] = extras["revision"]
        roof["launches"] = kcount[dom]
        roof["avg_launch_ms"] = kms[dom] / max(kcount[dom], 1)
        roof["algorithmic_bytes_per_launch"] = k_bytes / max(kcount[dom], 1)
        roof["algorithmic_flops_per_launch"] = k_flops / max(kcount[dom], 1)
        roof["peak_source"] = {"tensor": peak_kind + " (burst bf16; sustained beside it)", "hbm": peak_kind + " (copy)",
                               "alu": "derived: SMs x 128 lanes x maximum SM clock"}[roof["bound"]]
        roof["per_kernel"] = per_kernel
        roof["timing"] = "separate pass of the same steps with a CUDA event pair around every launch"
        roof["kernel_ms_per_step"] = {nm: kms[k] / args.steps for k, nm in enumerate(names) if kcount[k]}
        roof["kernel_share"] = {nm: kms[k] / max(sum(kms), 1e-12) for k, nm in enumerate(names) if kcount[k]}
        kernel_bound_ms = sum(max(per_kernel[nm]["bound_ms_per_step"].values()) for nm in per_kernel)
        roof["whole_step"] = {"per_matrix_roofline_ms": t_roof * 1e3, "frac_of_per_matrix_roofline": t_roof / sec,
                              "frac_of_nominal_roofline": t_roof_nom / sec,
                              "bound": "tensor" if t_c >= t_m else "hbm",
                              "achieved_tflops": flops / sec / 1e12, "achieved_gbs": nbytes / sec / 1e9,
                              # the kernels run one after the other: the sum of their own bounds (each the slowest
                              # of its tensor, HBM and ALU time) is what such a design can reach at best
                              "sum_of_kernel_rooflines_ms": kernel_bound_ms,
                              "frac_of_sum_of_kernel_rooflines": kernel_bound_ms / ms_per_step}
        refresh = None if args.no_refresh else time_refresh(items, device)
        if refresh is not None:
            # the step and the refresh blended at the base interval of Sec. 4.1 (a refresh every 200 steps)
            refresh["blended_ms_per_step_at_interval_200"] = ms_per_step + refresh["stack_seconds_best"] * 1e3 / 200.0
        linear = time_linear(items, device, args.linear_tokens, peaks["bf16_tflops"]) if args.linear_tokens > 0 else None
        cpu = None
        if not args.no_cpu_baseline:
            v, per_step, sample = oracle_sample(workload, 3, 1)
            cpu = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample,
                   "host_cpus": os.cpu_count()}
        block = {
            "value": value, "unit": UNIT, "ms_per_step": ms_per_step,
            "config": {"workload": workload + (f"[first {args.layers} layers]" if args.layers else ""), "matrices": len(specs),
                       "elements_per_step": elements, "rank": specs[0].r, "group": 256, "rounding": args.rounding,
                       "moments_bits": args.moments, "l2": "inputs larger than L2 (whole stack streams each step)",
                       "parallelism": f"replica per GPU x{world}, no collective"},
            "roofline": roof, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4,
                    "steps": e2e_steps},
            "gpu_launches": launches, "clocks": clocks, "device_status": status, "refresh": refresh,
            "int8_linear": linear,
        }
    batch.close()
    del batch, items
    torch.cuda.empty_cache()
    return block


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2407_08296_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Q-GaLore step has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    B.lib()                                                    # fail loudly if the library is missing
    peaks, peak_kind = load_peaks()
    revision = B.kernel_revision()
    extras = {"traffic": load_ncu_traffic(revision), "revision": revision}

    # both target stacks unless one is asked for: the largest single-GPU configuration first (top level of the
    # line), the other under "also"
    workloads = [args.workload] if args.workload else ["llama7b", "llama1b"]
    blocks = [bench_workload(w, args, B, torch, dist, device, world, rank, local_rank, peaks, peak_kind, extras)
              for w in workloads]
    if rank == 0:
        top = blocks[0]
        line = {"metric": METRIC, "value": top["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": top["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
        line.update({k: v for k, v in top.items() if k not in ("value", "unit", "ms_per_step")})
        if len(blocks) > 1:
            line["also"] = {w: b for w, b in zip(workloads[1:], blocks[1:])}
            line["gpu_launches"] = sum(b["gpu_launches"] for b in blocks)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None,
                    help="llama7b | llama1b | llama350m | llama130m | llama60m_mlp; default: llama7b, then llama1b under 'also'")
    ap.add_argument("--no-refresh", action="store_true", help="skip the separate timing of the subspace refresh")
    ap.add_argument("--linear-tokens", type=int, default=8192,
                    help="rows of activations for the separate timing of the INT8 linear layer's GEMMs (0: skip)")
    ap.add_argument("--moments", type=int, choices=[32, 8], default=32,
                    help="storage of the Adam moments: fp32 (the measured configuration) or the 8-bit block-wise form")
    ap.add_argument("--rounding", choices=["stochastic", "nearest"], default="stochastic",
                    help="requantization of the updated weight: the method's stochastic rounding, or the round-to-nearest ablation")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0,
                    help="keep only the first L layers of the stack (small cases for profiler captures); 0 = all")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
