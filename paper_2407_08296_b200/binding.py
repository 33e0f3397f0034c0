"""ctypes binding of libqgalore.so: one Python function per exported entry point.

Argument marshalling only.  torch is used for device memory and streams; every step of the
path runs in the library's CUDA kernels.  Matrices are 2-D torch tensors whose last stride is
1; the row pitch ("ld") handed to the library is ``tensor.stride(0)``, so a padded buffer is
passed as the view ``buf[:, :cols]``.  Loading fails loudly if the library is missing: there
is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqgalore.so")

QG_OK = 0
QG_INVALID_ARGUMENT, QG_UNSUPPORTED_SHAPE, QG_MISALIGNED = -1, -2, -3
QG_WORKSPACE_TOO_SMALL, QG_CUDA_ERROR, QG_NOT_CONVERGED = -4, -5, -6
QG_OP_PROJECT_STEP, QG_OP_REFRESH, QG_OP_SIMILARITY = 1, 2, 3
QG_DEV_WAIT_EXPIRED, QG_DEV_NOT_CONVERGED, QG_DEV_BAD_FACTOR = 1, 2, 4
GROUP = 256


class QgError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


class _CQTensor(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("zeros", C.c_void_p),
                ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("bits", C.c_int32), ("group", C.c_int32)]


QG_ROUND_STOCHASTIC, QG_ROUND_NEAREST = 0, 1
QG_SIDE_LEFT, QG_SIDE_RIGHT = 0, 1


class _CHyper(C.Structure):
    _fields_ = [("lr", C.c_float), ("alpha", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("weight_decay", C.c_float), ("step", C.c_int64), ("seed", C.c_uint64),
                ("rounding", C.c_int32), ("reserved", C.c_int32)]


class _CStepItem(C.Structure):
    _fields_ = [("G", C.c_void_p), ("ldg", C.c_int64), ("m", C.c_int64), ("n", C.c_int64), ("r", C.c_int64),
                ("P", _CQTensor), ("W", _CQTensor), ("M", C.c_void_p), ("V", C.c_void_p), ("ldmv", C.c_int64),
                ("seed", C.c_uint64), ("side", C.c_int32), ("state_bits", C.c_int32),
                ("M_scale", C.c_void_p), ("V_scale", C.c_void_p)]


class _CRefreshItem(C.Structure):
    _fields_ = [("G", C.c_void_p), ("ldg", C.c_int64), ("seed", C.c_uint64), ("P_new", _CQTensor), ("P_fp32", C.c_void_p),
                ("P_prev", C.POINTER(_CQTensor)), ("sim_dev", C.c_void_p)]


class _CDebug(C.Structure):
    _fields_ = [("R", C.c_void_p), ("N", C.c_void_p), ("W_pre", C.c_void_p), ("N_b", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2407_08296_b200.build` "
                "(there is no fallback implementation)")
        L = C.CDLL(LIB_PATH)
        i64, i32, vp, sz = C.c_int64, C.c_int32, C.c_void_p, C.c_size_t
        qp = C.POINTER(_CQTensor)
        L.qgalore_quantize_int4.argtypes = [vp, i64, i64, i64, qp, vp]
        L.qgalore_quantize_int8.argtypes = [vp, i64, i64, i64, qp, vp]
        L.qgalore_quantize_int2.argtypes = [vp, i64, i64, i64, qp, vp]
        L.qgalore_dequantize.argtypes = [qp, vp, i64, vp]
        L.qgalore_int8_linear_forward.argtypes = [vp, i64, i64, qp, vp, i64, vp, vp]
        L.qgalore_int8_linear_backward_input.argtypes = [vp, i64, i64, qp, vp, i64, vp, vp]
        L.qgalore_int8_linear_backward_weight.argtypes = [vp, i64, i64, vp, i64, i64, i64, vp, i64, vp, vp]
        L.qgalore_project_step.argtypes = [vp, i64, i64, i64, i64, qp, qp, vp, vp, i64, C.POINTER(_CHyper),
                                           vp, sz, vp, C.POINTER(_CDebug), vp]
        L.qgalore_project_step_right.argtypes = L.qgalore_project_step.argtypes
        L.qgalore_project_step_item.argtypes = [C.POINTER(_CStepItem), C.POINTER(_CHyper), vp, sz, vp, C.POINTER(_CDebug), vp]
        L.qgalore_project_step_batched.argtypes = [C.POINTER(_CStepItem), i32, C.POINTER(_CHyper), vp, sz, vp, vp]
        L.qgalore_workspace_bytes_batched.argtypes = [C.POINTER(_CStepItem), i32]
        L.qgalore_workspace_bytes_batched.restype = sz
        L.qgalore_plan_table_bytes.argtypes = [C.POINTER(_CStepItem), i32]
        L.qgalore_plan_table_bytes.restype = sz
        L.qgalore_plan_create.argtypes = [C.POINTER(_CStepItem), i32, vp, sz, vp, sz, C.POINTER(vp)]
        L.qgalore_plan_step.argtypes = [vp, C.POINTER(_CHyper), vp, vp]
        L.qgalore_plan_step_timed.argtypes = [vp, C.POINTER(_CHyper), vp, vp, C.POINTER(C.c_float), C.POINTER(i32)]
        L.qgalore_plan_destroy.argtypes = [vp]
        L.qgalore_plan_destroy.restype = None
        L.qgalore_refresh_subspace.argtypes = [vp, i64, i64, i64, i64, i32, i32, C.c_uint64, qp, vp, qp, i32, vp,
                                               vp, sz, vp, vp]
        L.qgalore_refresh_subspace_right.argtypes = L.qgalore_refresh_subspace.argtypes
        L.qgalore_refresh_subspace_batched.argtypes = [C.POINTER(_CRefreshItem), i32, i64, i64, i64, i32, i32, i32, i32, vp, sz,
                                                       vp, vp]
        L.qgalore_subspace_similarity.argtypes = [qp, qp, i32, vp, vp, sz, vp]
        L.qgalore_subspace_similarity_static.argtypes = [qp, qp, i32, vp, vp]
        L.qgalore_subspace_similarity_static_max_bytes.restype = sz
        L.qgalore_gate_update.argtypes = [C.c_float, C.c_float, i32, C.POINTER(i32), C.POINTER(C.c_float),
                                          C.POINTER(i32)]
        L.qgalore_workspace_bytes.argtypes = [C.c_int, i64, i64, i64]
        L.qgalore_workspace_bytes.restype = sz
        L.qgalore_status_string.argtypes = [C.c_int]
        L.qgalore_status_string.restype = C.c_char_p
        L.qgalore_last_cuda_error.restype = C.c_char_p
        L.qgalore_launch_count.restype = C.c_uint64
        L.qgalore_kernel_revision.restype = C.c_char_p
        L.qgalore_debug_set_step_impl.argtypes = [C.c_int]
        L.qgalore_debug_set_pair_mode.argtypes = [C.c_int]
        L.qgalore_debug_set_jacobi_blocks.argtypes = [C.c_int]
        L.qgalore_debug_set_fused_dequant.argtypes = [C.c_int]
        L.qgalore_debug_set_refresh_tensor_cores.argtypes = [C.c_int]
        L.qgalore_debug_set_chunk_budget.argtypes = [sz]
        L.qgalore_debug_expire_wait.argtypes = [i32, vp, vp, vp]
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status < 0:
        L = lib()
        msg = L.qgalore_status_string(status).decode()
        if status == QG_CUDA_ERROR:
            msg += ": " + L.qgalore_last_cuda_error().decode()
        raise QgError(status, f"{what}: {msg}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def round_up(x: int, mult: int) -> int:
    return (x + mult - 1) // mult * mult


def empty_matrix(rows: int, cols: int, dtype, device="cuda", pitch_multiple: int = 64) -> torch.Tensor:
    """A rows x cols view of a buffer whose row pitch is cols rounded up to ``pitch_multiple`` elements."""
    ld = round_up(cols, pitch_multiple)
    return torch.empty((rows, ld), dtype=dtype, device=device)[:, :cols]


def zeros_matrix(rows: int, cols: int, dtype, device="cuda", pitch_multiple: int = 64) -> torch.Tensor:
    ld = round_up(cols, pitch_multiple)
    return torch.zeros((rows, ld), dtype=dtype, device=device)[:, :cols]


def _matrix_ld(t: torch.Tensor, what: str) -> int:
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{what}: expected a 2-D tensor with unit column stride")
    return int(t.stride(0)) if t.shape[0] > 1 else max(int(t.stride(0)), int(t.shape[1]))


@dataclass
class QTensor:
    """A block-wise quantized matrix on the device (Sec. 3.1): codes, per-group scales and zeros.

    ``codes`` is int8 [rows, cols] (a view with pitch ld) for bits == 8, uint8 [rows, ld // 2]
    holding two codes per byte for bits == 4, uint8 [rows, ld // 4] holding four per byte for bits == 2.
    """
    codes: torch.Tensor
    scales: torch.Tensor
    zeros: torch.Tensor
    rows: int
    cols: int
    ld: int
    bits: int

    @staticmethod
    def empty(rows: int, cols: int, bits: int, device="cuda") -> "QTensor":
        ld = round_up(cols, 64)
        ng = (cols + GROUP - 1) // GROUP
        if bits == 8:
            codes = torch.zeros((rows, ld), dtype=torch.int8, device=device)
        elif bits == 4:
            codes = torch.full((rows, ld // 2), 0x88, dtype=torch.uint8, device=device)
        elif bits == 2:
            codes = torch.full((rows, ld // 4), 0xAA, dtype=torch.uint8, device=device)
        else:
            raise ValueError("bits must be 2, 4 or 8")
        return QTensor(codes, torch.zeros((rows, ng), dtype=torch.float32, device=device),
                       torch.zeros((rows, ng), dtype=torch.float32, device=device), rows, cols, ld, bits)

    def c_struct(self) -> _CQTensor:
        return _CQTensor(_ptr(self.codes), _ptr(self.scales), _ptr(self.zeros), self.rows, self.cols, self.ld,
                         self.bits, GROUP)

    def clone(self) -> "QTensor":
        return QTensor(self.codes.clone(), self.scales.clone(), self.zeros.clone(), self.rows, self.cols, self.ld,
                       self.bits)


@dataclass
class Hyper:
    lr: float = 0.004
    alpha: float = 0.25
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    step: int = 1
    seed: int = 0
    rounding: int = 0        # QG_ROUND_STOCHASTIC (Sec. 3.4) or QG_ROUND_NEAREST (the ablation of Fig. 6)

    def c_struct(self) -> _CHyper:
        return _CHyper(self.lr, self.alpha, self.beta1, self.beta2, self.eps, self.weight_decay, self.step, self.seed,
                       self.rounding, 0)


def workspace_bytes(op: int, m: int, n: int, r: int) -> int:
    return int(lib().qgalore_workspace_bytes(op, m, n, r))


# kernels of one plan step, in the order qgalore_plan_step_timed reports them
STEP_KERNEL_NAMES = ("dequant_p_grouped", "project_adam", "backproject_sr")


def kernel_revision() -> str:
    return lib().qgalore_kernel_revision().decode()


def launch_count() -> int:
    return int(lib().qgalore_launch_count())


def _quantize(fn_name: str, bits: int, src: torch.Tensor, out: QTensor | None, stream) -> QTensor:
    rows, cols = src.shape
    if src.dtype != torch.float32:
        raise ValueError("quantize: src must be float32")
    if out is None:
        out = QTensor.empty(rows, cols, bits, src.device)
    cs = out.c_struct()
    fn = getattr(lib(), fn_name)
    _check(fn(_ptr(src), rows, cols, _matrix_ld(src, "src"), C.byref(cs), _stream_ptr(stream)), fn_name)
    return out


def quantize_int4(src: torch.Tensor, out: QTensor | None = None, stream=None) -> QTensor:
    return _quantize("qgalore_quantize_int4", 4, src, out, stream)


def quantize_int8(src: torch.Tensor, out: QTensor | None = None, stream=None) -> QTensor:
    return _quantize("qgalore_quantize_int8", 8, src, out, stream)


def quantize_int2(src: torch.Tensor, out: QTensor | None = None, stream=None) -> QTensor:
    return _quantize("qgalore_quantize_int2", 2, src, out, stream)


def dequantize(q: QTensor, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if out is None:
        out = empty_matrix(q.rows, q.cols, torch.float32, q.codes.device, 4)
    cs = q.c_struct()
    _check(lib().qgalore_dequantize(C.byref(cs), _ptr(out), _matrix_ld(out, "out"), _stream_ptr(stream)),
           "qgalore_dequantize")
    return out


def _bf16_arg(t: torch.Tensor, what: str) -> torch.Tensor:
    if t.dtype not in (torch.bfloat16, torch.int16, torch.uint16):
        raise ValueError(f"{what} must hold bfloat16 values (bfloat16 / int16 / uint16 storage)")
    return t


def int8_linear_forward(X: torch.Tensor, W: QTensor, out: torch.Tensor | None = None,
                        status: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """App. A, forward: Y (T x m) = X (T x n) W~^T with the INT8 weight dequantized inside the GEMM."""
    T = X.shape[0]
    if out is None:
        out = empty_matrix(T, W.rows, torch.bfloat16, X.device, 64)
    cs = W.c_struct()
    _check(lib().qgalore_int8_linear_forward(_ptr(_bf16_arg(X, "X")), T, _matrix_ld(X, "X"), C.byref(cs),
                                             _ptr(_bf16_arg(out, "out")), _matrix_ld(out, "out"),
                                             _ptr(status), _stream_ptr(stream)),
           "qgalore_int8_linear_forward")
    return out


def int8_linear_backward_input(dY: torch.Tensor, W: QTensor, out: torch.Tensor | None = None,
                               status: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """App. A, backward: grad_input (T x n) = dY (T x m) W~."""
    T = dY.shape[0]
    if out is None:
        out = empty_matrix(T, W.cols, torch.bfloat16, dY.device, 64)
    cs = W.c_struct()
    _check(lib().qgalore_int8_linear_backward_input(_ptr(_bf16_arg(dY, "dY")), T, _matrix_ld(dY, "dY"), C.byref(cs),
                                                    _ptr(_bf16_arg(out, "out")), _matrix_ld(out, "out"),
                                                    _ptr(status),
                                                    _stream_ptr(stream)),
           "qgalore_int8_linear_backward_input")
    return out


def int8_linear_backward_weight(dY: torch.Tensor, X: torch.Tensor, out: torch.Tensor | None = None,
                                status: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """App. A, backward: grad_W (m x n) = dY^T (T x m) X (T x n): the gradient G of the optimizer step."""
    T, m = dY.shape
    n = X.shape[1]
    if X.shape[0] != T:
        raise ValueError("dY and X must have the same number of rows")
    if out is None:
        out = empty_matrix(m, n, torch.bfloat16, dY.device, 64)
    _check(lib().qgalore_int8_linear_backward_weight(_ptr(_bf16_arg(dY, "dY")), T, _matrix_ld(dY, "dY"),
                                                     _ptr(_bf16_arg(X, "X")), _matrix_ld(X, "X"), m, n,
                                                     _ptr(_bf16_arg(out, "out")), _matrix_ld(out, "out"),
                                                     _ptr(status),
                                                     _stream_ptr(stream)),
           "qgalore_int8_linear_backward_weight")
    return out


def _debug_struct(debug: dict) -> _CDebug:
    """Optional taps of one step: R, N (fp32), N_b (bf16 bit patterns, same pitch as R and N), W_pre (fp32)."""
    nb = debug.get("N_b")
    for key in ("R", "N"):
        if nb is not None and debug.get(key) is not None and debug[key].stride(0) != nb.stride(0):
            raise ValueError("the N_b tap must share the row pitch of the R and N taps")
    return _CDebug(_ptr(debug.get("R")), _ptr(debug.get("N")), _ptr(debug.get("W_pre")), _ptr(nb))


def project_step(G: torch.Tensor, P: QTensor, W: QTensor, M: torch.Tensor, V: torch.Tensor, hyper: Hyper,
                 workspace: torch.Tensor | None = None, status: torch.Tensor | None = None,
                 debug: dict | None = None, stream=None, side: str = "left") -> None:
    """One Q-GaLore step of one matrix (Sec. 3.5): W, M and V are updated in place.  ``side`` = "right" takes
    P as the n x r right-hand projection and M, V as the transposed (r x m) moments."""
    m, n = G.shape
    r = P.cols
    right = side == "right"
    if G.dtype not in (torch.bfloat16, torch.int16, torch.uint16):
        raise ValueError("G must hold bfloat16 values (bfloat16 / int16 / uint16 storage)")
    if M.dtype != torch.float32 or V.dtype != torch.float32:
        raise ValueError("M and V must be float32")
    if tuple(M.shape) != (r, m if right else n) or tuple(V.shape) != (r, m if right else n):
        raise ValueError("M and V must be r x n (r x m for the right-hand projection)")
    ldmv = _matrix_ld(M, "M")
    if _matrix_ld(V, "V") != ldmv:
        raise ValueError("M and V must share their row pitch")
    if workspace is None:
        workspace = torch.empty(workspace_bytes(QG_OP_PROJECT_STEP, m, n, r), dtype=torch.uint8, device=G.device)
    dbg = None
    if debug:
        dbg = _debug_struct(debug)
    pc, wc, hc = P.c_struct(), W.c_struct(), hyper.c_struct()
    fn = lib().qgalore_project_step_right if right else lib().qgalore_project_step
    _check(fn(_ptr(G), _matrix_ld(G, "G"), m, n, r, C.byref(pc), C.byref(wc), _ptr(M), _ptr(V),
              ldmv, C.byref(hc), _ptr(workspace), workspace.numel() * workspace.element_size(),
              _ptr(status), C.byref(dbg) if dbg is not None else None, _stream_ptr(stream)),
           "qgalore_project_step_right" if right else "qgalore_project_step")


def _c_step_item(it: dict) -> _CStepItem:
    """One matrix of a step as the C table holds it.  Keys: G, P, W, M, V, seed; optional side ("left" / "right")
    and, for 8-bit moments, M_scale and V_scale (then M is an int8 and V a uint8 tensor)."""
    G, P, W, M, V = it["G"], it["P"], it["W"], it["M"], it["V"]
    m, ncol = G.shape
    state8 = it.get("M_scale") is not None
    if state8 and (M.dtype != torch.int8 or V.dtype != torch.uint8):
        raise ValueError("8-bit moments: M must be int8 and V uint8")
    return _CStepItem(_ptr(G), _matrix_ld(G, "G"), m, ncol, P.cols, P.c_struct(), W.c_struct(),
                      _ptr(M), _ptr(V), _matrix_ld(M, "M"), int(it.get("seed", 0)),
                      QG_SIDE_RIGHT if it.get("side", "left") == "right" else QG_SIDE_LEFT, 8 if state8 else 0,
                      _ptr(it.get("M_scale")), _ptr(it.get("V_scale")))


def project_step_item(item: dict, hyper: "Hyper", workspace: torch.Tensor | None = None, status: torch.Tensor | None = None,
                      debug: dict | None = None, stream=None) -> None:
    """One step of one matrix described like an item of a plan (any side, fp32 or 8-bit moments)."""
    ci = _c_step_item(item)
    m, n = item["G"].shape
    if workspace is None:
        workspace = torch.empty(workspace_bytes(QG_OP_PROJECT_STEP, m, n, item["P"].cols), dtype=torch.uint8,
                                device=item["G"].device)
    dbg = None
    if debug:
        dbg = _debug_struct(debug)
    hc = hyper.c_struct()
    _check(lib().qgalore_project_step_item(C.byref(ci), C.byref(hc), _ptr(workspace), workspace.numel(), _ptr(status),
                                           C.byref(dbg) if dbg is not None else None, _stream_ptr(stream)),
           "qgalore_project_step_item")


class StepBatch:
    """A list of matrices stepped together by one call (a layer or a whole stack, Sec. 3.5).

    Holds references to the tensors and the marshalled item table; ``step`` enqueues one optimizer
    step of every matrix.
    """

    def __init__(self, items: list[dict], device=None):
        """items: dicts with G, P, W, M, V and seed."""
        self.items = items
        n = len(items)
        self._table = (_CStepItem * n)()
        for k, it in enumerate(items):
            G, P, W, M, V = it["G"], it["P"], it["W"], it["M"], it["V"]
            m, ncol = G.shape
            self._table[k] = _c_step_item(it)
        dev = device if device is not None else items[0]["G"].device
        nbytes = int(lib().qgalore_workspace_bytes_batched(self._table, n))
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.elements = sum(int(it["G"].shape[0]) * int(it["G"].shape[1]) for it in items)

    def step(self, hyper: Hyper, stream=None) -> None:
        hc = hyper.c_struct()
        _check(lib().qgalore_project_step_batched(self._table, len(self.items), C.byref(hc), _ptr(self.workspace),
                                                  self.workspace.numel(), _ptr(self.status), _stream_ptr(stream)),
               "qgalore_project_step_batched")


class StepPlan:
    """A fixed list of matrices prepared once and stepped many times with grouped launches (Sec. 3.5).

    ``items`` are dicts with G, P, W, M, V and seed.  The plan owns its device table and workspace (torch
    tensors) and keeps references to the items' tensors, which must not be reallocated while it lives.
    """

    PREFERRED_WORKSPACE = 264 << 20

    def __init__(self, items: list[dict], workspace_bytes: int | None = None, device=None):
        self.items = items
        n = len(items)
        self._table = (_CStepItem * n)()
        for k, it in enumerate(items):
            G, P, W, M, V = it["G"], it["P"], it["W"], it["M"], it["V"]
            m, ncol = G.shape
            self._table[k] = _c_step_item(it)
        dev = device if device is not None else items[0]["G"].device
        L = lib()
        need = int(L.qgalore_workspace_bytes_batched(self._table, n))
        if workspace_bytes is None:
            workspace_bytes = max(need, self.PREFERRED_WORKSPACE)
        self.workspace = torch.empty(max(int(workspace_bytes), 1024), dtype=torch.uint8, device=dev)
        self.table_dev = torch.empty(max(int(L.qgalore_plan_table_bytes(self._table, n)), 256), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.elements = sum(int(it["G"].shape[0]) * int(it["G"].shape[1]) for it in items)
        handle = C.c_void_p()
        _check(L.qgalore_plan_create(self._table, n, _ptr(self.table_dev), self.table_dev.numel(), _ptr(self.workspace),
                                     self.workspace.numel(), C.byref(handle)), "qgalore_plan_create")
        self._handle = handle

    def step(self, hyper: Hyper, stream=None) -> None:
        hc = hyper.c_struct()
        _check(lib().qgalore_plan_step(self._handle, C.byref(hc), _ptr(self.status), _stream_ptr(stream)),
               "qgalore_plan_step")

    def step_timed(self, hyper: Hyper, stream=None) -> tuple[list[float], list[int]]:
        """One step with events around every launch; returns (ms per kernel kind, launches per kernel kind)
        for [dequantize-P, projection+Adam, back-projection+requantize].  Blocks until the step is done."""
        hc = hyper.c_struct()
        ms = (C.c_float * 3)()
        cnt = (C.c_int32 * 3)()
        _check(lib().qgalore_plan_step_timed(self._handle, C.byref(hc), _ptr(self.status), _stream_ptr(stream), ms, cnt),
               "qgalore_plan_step_timed")
        return [float(x) for x in ms], [int(x) for x in cnt]

    def close(self) -> None:
        if self._handle is not None and self._handle.value:
            lib().qgalore_plan_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def refresh_subspace(G: torch.Tensor, r: int, iters: int = 12, oversample_cols: int | None = None, seed: int = 0,
                     P_new: QTensor | None = None, P_fp32: torch.Tensor | None = None, P_prev: QTensor | None = None,
                     sim_cols: int = 0, sim: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                     status: torch.Tensor | None = None, stream=None, side: str = "left") -> QTensor:
    """New INT4 projection matrix from the top-r left singular subspace of G (Sec. 3.5, Sec. 3.3); with
    ``side`` = "right" from its right singular subspace (an n x r matrix, for the right-hand projection)."""
    m, n = G.shape
    right = side == "right"
    pm, pn_ = (n, m) if right else (m, n)
    if oversample_cols is None:     # block of 2 r columns, in whole panels of 64, never wider than the matrix
        block = min((2 * r + 63) // 64 * 64, min(m, n) // 64 * 64)
        oversample_cols = max(block - r, 0)
    if P_new is None:
        P_new = QTensor.empty(pm, r, 4, G.device)
        if P_new.ld != r:               # the refresh writes a densely packed P (ld == r)
            ng = (r + GROUP - 1) // GROUP
            P_new = QTensor(torch.full((pm, r // 2), 0x88, dtype=torch.uint8, device=G.device),
                            torch.zeros((pm, ng), dtype=torch.float32, device=G.device),
                            torch.zeros((pm, ng), dtype=torch.float32, device=G.device), pm, r, r, 4)
    if workspace is None:
        workspace = torch.empty(workspace_bytes(QG_OP_REFRESH, pm, pn_, r + oversample_cols), dtype=torch.uint8,
                                device=G.device)
    pn = P_new.c_struct()
    pp = P_prev.c_struct() if P_prev is not None else None
    fn = lib().qgalore_refresh_subspace_right if right else lib().qgalore_refresh_subspace
    _check(fn(_ptr(G), _matrix_ld(G, "G"), m, n, r, iters, oversample_cols, seed,
              C.byref(pn), _ptr(P_fp32), C.byref(pp) if pp is not None else None,
              sim_cols, _ptr(sim), _ptr(workspace),
              workspace.numel() * workspace.element_size(), _ptr(status),
              _stream_ptr(stream)), "qgalore_refresh_subspace_right" if right else "qgalore_refresh_subspace")
    return P_new


def dense_projection(rows: int, r: int, bits: int = 4, device="cuda") -> QTensor:
    """An empty quantized rows x r projection with ld == r, the layout the refresh writes."""
    ng = (r + GROUP - 1) // GROUP
    per_byte = {8: 1, 4: 2, 2: 4}[bits]
    fill = {8: 0, 4: 0x88, 2: 0xAA}[bits]
    codes = torch.full((rows, r // per_byte), fill, dtype=torch.int8 if bits == 8 else torch.uint8, device=device)
    return QTensor(codes, torch.zeros((rows, ng), dtype=torch.float32, device=device),
                   torch.zeros((rows, ng), dtype=torch.float32, device=device), rows, r, r, bits)


def refresh_subspace_batched(items: list[dict], r: int, iters: int = 12, oversample_cols: int | None = None, sim_cols: int = 0,
                             workspace: torch.Tensor | None = None, max_batch: int = 8, status: torch.Tensor | None = None,
                             stream=None, side: str = "left") -> list[QTensor]:
    """The refresh of several matrices of one shape in one call (Sec. 3.5).  items: dicts with G and seed, and
    optionally P_new, P_fp32, P_prev and sim (a 1-element device tensor).  Returns the new projections."""
    m, n = items[0]["G"].shape
    right = side == "right"
    pm, pn_ = (n, m) if right else (m, n)
    if oversample_cols is None:
        block = min((2 * r + 63) // 64 * 64, min(m, n) // 64 * 64)
        oversample_cols = max(block - r, 0)
    dev = items[0]["G"].device
    table = (_CRefreshItem * len(items))()
    keep, out = [], []
    for k, it in enumerate(items):
        G = it["G"]
        if tuple(G.shape) != (m, n):
            raise ValueError("a batch holds matrices of one shape")
        P_new = it.get("P_new") or dense_projection(pm, r, 4, dev)
        out.append(P_new)
        prev = it.get("P_prev")
        prev_c = prev.c_struct() if prev is not None else None
        keep.append(prev_c)
        table[k] = _CRefreshItem(_ptr(G), _matrix_ld(G, "G"), int(it.get("seed", 0)), P_new.c_struct(), _ptr(it.get("P_fp32")),
                                 C.pointer(prev_c) if prev_c is not None else None, _ptr(it.get("sim")))
    if workspace is None:
        per = workspace_bytes(QG_OP_REFRESH, pm, pn_, r + oversample_cols)
        workspace = torch.empty(per * max(1, min(max_batch, len(items))), dtype=torch.uint8, device=dev)
    _check(lib().qgalore_refresh_subspace_batched(table, len(items), m, n, r, iters, oversample_cols,
                                                  QG_SIDE_RIGHT if right else QG_SIDE_LEFT, sim_cols, _ptr(workspace),
                                                  workspace.numel(), _ptr(status), _stream_ptr(stream)),
           "qgalore_refresh_subspace_batched")
    return out


def subspace_similarity(A: QTensor, B: QTensor, sim_cols: int = 0, out: torch.Tensor | None = None,
                        workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Cosine similarity between two adjacent INT4 projection matrices (Sec. 3.2); a 1-element device tensor."""
    if out is None:
        out = torch.zeros(1, dtype=torch.float32, device=A.codes.device)
    if workspace is None:
        workspace = torch.empty(workspace_bytes(QG_OP_SIMILARITY, A.rows, 0, A.cols), dtype=torch.uint8,
                                device=A.codes.device)
    ac, bc = A.c_struct(), B.c_struct()
    _check(lib().qgalore_subspace_similarity(C.byref(ac), C.byref(bc), sim_cols, _ptr(out), _ptr(workspace),
                                             workspace.numel(), _stream_ptr(stream)), "qgalore_subspace_similarity")
    return out


def subspace_similarity_static(A: QTensor, B: QTensor, sim_cols: int = 0, out: torch.Tensor | None = None,
                               stream=None) -> torch.Tensor:
    """Same result as subspace_similarity, for callers that may not allocate: the scratch is a fixed array
    inside the library (shapes needing more than 2 MiB are refused), so pass ``out`` and nothing is allocated.
    Calls on one device share that array and must not overlap."""
    if out is None:
        out = torch.zeros(1, dtype=torch.float32, device=A.codes.device)
    ac, bc = A.c_struct(), B.c_struct()
    _check(lib().qgalore_subspace_similarity_static(C.byref(ac), C.byref(bc), sim_cols, _ptr(out), _stream_ptr(stream)),
           "qgalore_subspace_similarity_static")
    return out


class Gate:
    """Host state of the adaptive lazy update (Sec. 3.2) for one matrix."""

    def __init__(self, interval: int = 200, threshold: float = 0.4, k: int = 1):
        self.threshold, self.k = float(threshold), int(k)
        self._interval = C.c_int32(interval)
        self._history = (C.c_float * max(1, k))()
        self._count = C.c_int32(0)

    @property
    def interval(self) -> int:
        return int(self._interval.value)

    def update(self, sim: float) -> bool:
        rc = lib().qgalore_gate_update(float(sim), self.threshold, self.k, C.byref(self._interval), self._history,
                                       C.byref(self._count))
        _check(rc, "qgalore_gate_update")
        return rc == 1


def debug_set_step_impl(impl: int) -> None:
    _check(lib().qgalore_debug_set_step_impl(impl), "qgalore_debug_set_step_impl")


DEFAULT_PAIR_MODE = 6


def debug_set_jacobi_blocks(on: bool) -> None:
    _check(lib().qgalore_debug_set_jacobi_blocks(1 if on else 0), "qgalore_debug_set_jacobi_blocks")


def debug_set_pair_mode(mask: int) -> None:
    _check(lib().qgalore_debug_set_pair_mode(mask), "qgalore_debug_set_pair_mode")


def debug_set_fused_dequant(on: bool) -> None:
    _check(lib().qgalore_debug_set_fused_dequant(1 if on else 0), "qgalore_debug_set_fused_dequant")


def debug_set_refresh_tensor_cores(on: bool) -> None:
    _check(lib().qgalore_debug_set_refresh_tensor_cores(1 if on else 0), "qgalore_debug_set_refresh_tensor_cores")


def debug_expire_wait(polls: int, status: torch.Tensor, polls_used: torch.Tensor | None = None, stream=None) -> None:
    """Test aid: one bounded barrier wait that nothing ever satisfies; ORs QG_DEV_WAIT_EXPIRED into ``status``."""
    _check(lib().qgalore_debug_expire_wait(polls, _ptr(status), _ptr(polls_used), _stream_ptr(stream)),
           "qgalore_debug_expire_wait")
