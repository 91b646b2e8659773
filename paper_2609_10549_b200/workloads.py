"""Seeded synthetic workloads: tensor shapes and BF16 input generation.

This module serves both the CUDA path and the CPU oracle used by the tests.
It contains no arithmetic of the method itself (no schedule, no GEMM, no
model): only shapes, random draws and the float32 -> BF16 bit conversion of
the drawn inputs.

Shapes stand in for tensor-parallel transformer layers (the paper's own grid,
Table IV, is a list of shapes and names no dataset):

* ``AG`` = AllGather+GEMM (Section II-A): rank r holds an activation shard
  A_r [M/P x K] and a weight shard B_r stored K-major as [N x K]
  (N = output columns *per rank*); result C_r [M x N].
* ``RS`` = GEMM+ReduceScatter: rank r holds A_r [M x K] (K = *per-rank*
  K-slice) and B_r [N x K]; result Out_r [M/P x N].

All tensors are carried as ``uint16`` arrays holding BF16 bit patterns so that
the very same host arrays feed both sides.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Tuple

import numpy as np

OP_AG_GEMM = 0
OP_GEMM_RS = 1


@dataclass(frozen=True)
class Workload:
    name: str
    op: int            # OP_AG_GEMM | OP_GEMM_RS
    P: int             # tensor-parallel size (logical ranks)
    M: int             # AG: gathered rows; RS: rows of every partial product
    N: int             # AG: columns per rank; RS: full output width
    K: int             # AG: full hidden size; RS: per-rank K slice
    a_dist: Tuple[str, float] = ("normal", 1.0)    # ("normal", std) | ("uniform", halfwidth)
    b_dist: Tuple[str, float] = ("normal", 0.02)
    seed: int = 0

    @property
    def m(self) -> int:
        """Rows per rank (chunk height)."""
        return self.M // self.P

    @property
    def a_shape(self) -> Tuple[int, int]:
        return (self.m, self.K) if self.op == OP_AG_GEMM else (self.M, self.K)

    @property
    def b_shape(self) -> Tuple[int, int]:
        return (self.N, self.K)

    @property
    def out_shape(self) -> Tuple[int, int]:
        return (self.M, self.N) if self.op == OP_AG_GEMM else (self.m, self.N)

    @property
    def flops(self) -> float:
        """FLOPs executed by all P logical ranks together."""
        return 2.0 * self.P * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> float:
        """Bytes the operator must move: every rank reads the whole gathered A
        (AG) or its own A (RS), its own B, and writes its own output."""
        if self.op == OP_AG_GEMM:
            a = self.P * self.M * self.K
        else:
            a = self.P * self.M * self.K
        b = self.P * self.N * self.K
        o = self.P * self.out_shape[0] * self.out_shape[1]
        return 2.0 * (a + b + o)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (1-based in the text, C1..C5 here).
C1_AG = Workload("C1-AG", OP_AG_GEMM, P=2, M=512, N=1024, K=1024,
                 a_dist=("uniform", 1.0), b_dist=("uniform", 1.0), seed=0)
C2_AG = Workload("C2-AG-QKV-7B", OP_AG_GEMM, P=4, M=4096, N=3072, K=4096)
C3_RS = Workload("C3-RS-MLPdown-7B", OP_GEMM_RS, P=8, M=8192, N=4096, K=1376)
C4_AG = replace(C2_AG, name="C4-AG")
C4_RS = Workload("C4-RS", OP_GEMM_RS, P=4, M=4096, N=4096, K=1024)
C5_AG = Workload("C5-AG-gateup-70B", OP_AG_GEMM, P=8, M=16384, N=7168, K=8192,
                 b_dist=("normal", 0.01))
C5_RS = Workload("C5-RS-down-70B", OP_GEMM_RS, P=8, M=16384, N=8192, K=3584,
                 b_dist=("normal", 0.01))

ALL = {w.name: w for w in (C1_AG, C2_AG, C3_RS, C4_AG, C4_RS, C5_AG, C5_RS)}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to BF16 (round-to-nearest-even) and return the
    16-bit patterns as uint16.  Inputs are finite by construction."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def _draw(shape, dist, seed) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    kind, scale = dist
    if kind == "normal":
        x = rng.standard_normal(shape, dtype=np.float32) * np.float32(scale)
    elif kind == "uniform":
        x = (rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)) * np.float32(scale)
    else:
        raise ValueError(f"unknown distribution {kind!r}")
    return f32_to_bf16_bits(x)


def tensor_seed(base_seed: int, rank: int, which: int) -> int:
    """Seed of one tensor: base*1000 + 10*rank + (0 for A, 1 for B)."""
    return base_seed * 1000 + 10 * rank + which


def make_inputs(w: Workload) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Return (A, B): per-rank lists of uint16 arrays holding BF16 bits."""
    A = [_draw(w.a_shape, w.a_dist, tensor_seed(w.seed, r, 0)) for r in range(w.P)]
    B = [_draw(w.b_shape, w.b_dist, tensor_seed(w.seed, r, 1)) for r in range(w.P)]
    return A, B


def make_structured_inputs(w: Workload, kind: str) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Inputs that expose layout mistakes: small exactly-representable integers.

    ``kind == "index"``: A[i, k] depends on (rank, i, k), B[n, k] on (rank, n, k),
    all values are small integers so every product and partial sum is exact.
    """
    if kind != "index":
        raise ValueError(kind)
    A, B = [], []
    for r in range(w.P):
        ra, ka = w.a_shape
        i = np.arange(ra, dtype=np.int64)[:, None]
        k = np.arange(ka, dtype=np.int64)[None, :]
        a = ((3 * i + 5 * k + 7 * r) % 5 - 2).astype(np.float32)
        rb, kb = w.b_shape
        n = np.arange(rb, dtype=np.int64)[:, None]
        k = np.arange(kb, dtype=np.int64)[None, :]
        b = ((2 * n + 3 * k + r) % 3 - 1).astype(np.float32)
        A.append(f32_to_bf16_bits(a))
        B.append(f32_to_bf16_bits(b))
    return A, B


# ---- the tensor-parallel MLP block (Section II-A) ---------------------------------

ACT_NONE, ACT_GELU_TANH, ACT_SWIGLU = 0, 1, 2


@dataclass(frozen=True)
class MlpWorkload:
    """X_r [M/P x hidden], W0_r [ffn x hidden] (column-parallel slice, K-major), W1_r [hidden x hc]
    (row-parallel slice, K-major); hc = ffn, or ffn / 2 when the activation pairs (gate, up) columns."""
    name: str
    P: int
    M: int
    hidden: int
    ffn: int                 # GEMM0 output columns per rank
    activation: int = ACT_NONE
    seed: int = 0

    @property
    def m(self) -> int:
        return self.M // self.P

    @property
    def hc(self) -> int:
        return self.ffn // 2 if self.activation == ACT_SWIGLU else self.ffn

    @property
    def flops(self) -> float:
        """FLOPs of both GEMMs over all P logical ranks."""
        return 2.0 * self.P * self.M * self.hidden * (self.ffn + self.hc)


def make_mlp_inputs(w: MlpWorkload) -> Tuple[List[np.ndarray], List[np.ndarray], List[np.ndarray]]:
    """(X, W0, W1) as BF16 bit patterns.  X ~ N(0, 1); the weights' standard deviations keep both GEMMs'
    outputs of order one: 1/sqrt(hidden) for W0, 1/sqrt(P * hc) for W1."""
    s0 = 1.0 / float(np.sqrt(w.hidden))
    s1 = 1.0 / float(np.sqrt(w.P * w.hc))
    X = [_draw((w.m, w.hidden), ("normal", 1.0), tensor_seed(w.seed, r, 0)) for r in range(w.P)]
    W0 = [_draw((w.ffn, w.hidden), ("normal", s0), tensor_seed(w.seed, r, 1)) for r in range(w.P)]
    W1 = [_draw((w.hidden, w.hc), ("normal", s1), tensor_seed(w.seed, r, 2)) for r in range(w.P)]
    return X, W0, W1


# LLaMA-7B MLP over 8 ranks: hidden 4096, 11008 / 8 = 1376 gate and up columns per rank (interleaved rows of
# W0_r), 8192 tokens.  Its second GEMM is the GEMM+ReduceScatter of configuration 3.
MLP_7B = MlpWorkload("MLP-7B-SwiGLU", P=8, M=8192, hidden=4096, ffn=2752, activation=ACT_SWIGLU)
