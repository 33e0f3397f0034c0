"""Seeded synthetic inputs for the Q-GaLore step: layer-stack shapes and gradient/weight generators.

This module holds none of the method's arithmetic (no quantizer, no projection, no
Adam, no rounding rule of the method).  It only produces inputs: LLaMA layer shapes
(Sec. 4.1 "Network Architecture", Table 1 ranks), a low-rank-plus-noise gradient in
bfloat16 and Gaussian initial weights.  Both the CUDA path's tests and the CPU oracle's
tests draw their inputs from here, so that they see identical bits.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

SIGNAL_RANK = 32        # planted singular values 1/k, k = 1..32
NOISE_STD = 1e-3        # i.i.d. Gaussian noise added to every gradient entry
WEIGHT_STD = 0.02       # initial weights ~ N(0, 0.02^2)


@dataclass(frozen=True)
class MatrixSpec:
    layer: int
    name: str
    index: int          # position in the stack; also selects the matrix's random streams
    m: int
    n: int
    r: int


@dataclass(frozen=True)
class StackSpec:
    name: str
    layers: int
    hidden: int
    mlp: int
    r: int


STACKS = {
    "llama60m_mlp": StackSpec("llama60m_mlp", 1, 512, 1376, 128),   # one 512 x 1376 matrix
    "llama130m": StackSpec("llama130m", 12, 768, 2048, 256),
    "llama350m": StackSpec("llama350m", 24, 1024, 2736, 256),
    "llama1b": StackSpec("llama1b", 24, 2048, 5461, 512),
    "llama7b": StackSpec("llama7b", 32, 4096, 11008, 1024),
}


def stack_matrices(name: str) -> list[MatrixSpec]:
    """Every 2-D attention/MLP weight of the named stack: per layer q,k,v,o (hidden x hidden),
    gate and up (hidden x mlp), down (mlp x hidden)."""
    s = STACKS[name]
    if name == "llama60m_mlp":
        return [MatrixSpec(0, "gate", 0, s.hidden, s.mlp, s.r)]
    out = []
    for layer in range(s.layers):
        for nm, m, n in (("q", s.hidden, s.hidden), ("k", s.hidden, s.hidden), ("v", s.hidden, s.hidden),
                         ("o", s.hidden, s.hidden), ("gate", s.hidden, s.mlp), ("up", s.hidden, s.mlp),
                         ("down", s.mlp, s.hidden)):
            out.append(MatrixSpec(layer, nm, len(out), m, n, s.r))
    return out


def distinct_shapes(name: str) -> list[tuple[int, int, int, int]]:
    """(m, n, r, count) of each distinct matrix shape of the stack."""
    counts: dict[tuple[int, int, int], int] = {}
    for s in stack_matrices(name):
        counts[(s.m, s.n, s.r)] = counts.get((s.m, s.n, s.r), 0) + 1
    return [(m, n, r, c) for (m, n, r), c in counts.items()]


def round_up(x: int, mult: int) -> int:
    return (x + mult - 1) // mult * mult


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float -> bfloat16 bit patterns (uint16), nearest-even.  Input formatting only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return ((u >> np.uint64(16)) & np.uint64(0xFFFF)).astype(np.uint16)


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(s) for s in stream]])


def _orthonormal(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    q, _ = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q


class GradientModel:
    """G_t = bf16( U diag(1/k) V^T + 1e-3 Z_t ): a rank-32 signal with fixed (or drifting)
    singular subspaces plus fresh Gaussian noise each step."""

    def __init__(self, m: int, n: int, seed: int = 0, matrix_index: int = 0):
        self.m, self.n, self.seed, self.index = m, n, seed, matrix_index
        k = min(SIGNAL_RANK, m, n)
        rng = _rng(seed, matrix_index, 0)
        self.U = _orthonormal(rng, m, k)
        self.V = _orthonormal(rng, n, k)
        self.sigma = 1.0 / np.arange(1, k + 1)

    def rotate(self, theta: float, epoch: int) -> None:
        """Drift of the left singular subspace: U <- orth(cos(theta) U + sin(theta) U_perp)."""
        rng = _rng(self.seed, self.index, 1, epoch)
        k = self.U.shape[1]
        X = rng.standard_normal((self.m, k))
        X -= self.U @ (self.U.T @ X)
        Uperp, _ = np.linalg.qr(X)
        self.U, _ = np.linalg.qr(np.cos(theta) * self.U + np.sin(theta) * Uperp)

    def signal(self) -> np.ndarray:
        return (self.U * self.sigma[None, :]) @ self.V.T

    def sample(self, step: int) -> np.ndarray:
        """bfloat16 bit patterns (uint16, m x n) of the gradient at ``step``."""
        z = _rng(self.seed, self.index, 2, step).standard_normal((self.m, self.n), dtype=np.float32)
        g = self.signal().astype(np.float32) + np.float32(NOISE_STD) * z
        return to_bf16_bits(g)


    def sample_columns(self, step: int, a: int, b: int, width: int = 256) -> np.ndarray:
        """Columns [a, b) of a gradient whose noise is drawn per block of ``width`` columns, each block from its
        own stream (seed, matrix, step, block): any column range costs only its own blocks, and the full matrix
        ``sample_columns(step, 0, n)`` is the concatenation of the ranges.  (A different gradient than
        ``sample(step)``, with the same model; used where only a few column blocks of a large matrix are needed
        at most steps.)  ``a`` must be a multiple of ``width``."""
        assert a % width == 0 and 0 <= a < b <= self.n
        sig_u = (self.U * self.sigma[None, :]).astype(np.float32)
        out = np.empty((self.m, b - a), np.uint16)
        for c0 in range(a, b, width):
            cw = min(width, self.n - c0)                # the whole block is formed, then cut: the same arithmetic
            z = _rng(self.seed, self.index, 5, step, c0 // width).standard_normal((self.m, cw), dtype=np.float32)
            g = to_bf16_bits(sig_u @ self.V[c0:c0 + cw].T.astype(np.float32) + np.float32(NOISE_STD) * z)
            c1 = min(c0 + cw, b)
            out[:, c0 - a:c1 - a] = g[:, :c1 - c0]
        return out


def initial_weight(m: int, n: int, seed: int = 0, matrix_index: int = 0) -> np.ndarray:
    """fp32 W0 ~ N(0, 0.02^2); the caller quantizes it."""
    return (_rng(seed, matrix_index, 3).standard_normal((m, n), dtype=np.float32) * np.float32(WEIGHT_STD))


def matrix_seed(base_seed: int, matrix_index: int) -> int:
    """Stochastic-rounding seed of one matrix of a stack."""
    return (int(base_seed) << 20) + int(matrix_index)


def random_orthonormal(m: int, r: int, seed: int = 0, stream: int = 0) -> np.ndarray:
    """An m x r matrix with orthonormal columns (fp32), e.g. a stand-in projection matrix."""
    return _orthonormal(_rng(seed, stream, 4), m, r).astype(np.float32)
