"""The tensor-parallel MLP block in FP64 (oracle; tests only).

Section II-A (the two-layer MLP figure): an AllGather brings the full input to
every rank, GEMM0 multiplies it by the rank's column-parallel slice of W0,
GEMM1 multiplies the result by the rank's row-parallel slice of W1, and a
ReduceScatter sums the ranks' partial products and leaves every rank its rows:

    H_r   = act( gather(X) * W0_r )          AllGather+GEMM, then an element-wise function
    Out_c = rows of chunk c of  sum_q H_q * W1_q      GEMM+ReduceScatter

The paper's text names no activation between the two GEMMs; ``ACT_NONE`` is
that literal chain.  An MLP has one, so two more are defined here:

* ``ACT_GELU_TANH``: 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) )).
* ``ACT_SWIGLU``: GEMM0's output columns hold (gate_j, up_j) pairs side by side
  (columns 2j and 2j+1); H[:, j] = gate_j / (1 + exp(-gate_j)) * up_j, so H has
  half as many columns as GEMM0's output.

H is a BF16 tensor (GEMM0's output type, GEMM1's input type): the function is
applied to the exact FP64 sum and the result rounded once to BF16, ties to
even.  Both collectives run in schedule order through ``operators``.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import operators as ops

ACT_NONE, ACT_GELU_TANH, ACT_SWIGLU = 0, 1, 2


def activation(c: np.ndarray, act: int) -> np.ndarray:
    """The element-wise function between GEMM0 and GEMM1, in FP64."""
    if act == ACT_NONE:
        return c
    if act == ACT_GELU_TANH:
        return 0.5 * c * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (c + 0.044715 * c ** 3)))
    if act == ACT_SWIGLU:
        assert c.shape[-1] % 2 == 0
        gate, up = c[..., 0::2], c[..., 1::2]
        with np.errstate(over="ignore"):
            return gate / (1.0 + np.exp(-gate)) * up
    raise ValueError(f"unknown activation {act}")


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round FP64 to the nearest BF16 (8 significant bits, ties to even) in one
    step and return the bit patterns.  Scaling by a power of two is exact, so
    ``rint`` of the scaled value is the correctly rounded significand."""
    x = np.asarray(x, dtype=np.float64)
    mant, exp = np.frexp(x)                       # x = mant * 2^exp, 0.5 <= |mant| < 1
    exp = np.maximum(exp, -125)                   # below 2^-126 the BF16 grid stops refining (subnormals)
    q = np.ldexp(1.0, exp - 8)                    # spacing of BF16 values in x's binade
    r = np.rint(x / q) * q                        # exact operations except the rint
    f = r.astype(np.float32)                      # exactly representable: no second rounding
    assert (f.astype(np.float64) == r)[np.isfinite(r)].all()
    bits = (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    assert ((f.view(np.uint32) & np.uint32(0xFFFF)) == 0).all()
    return bits


def hidden_columns(ffn: int, act: int) -> int:
    return ffn // 2 if act == ACT_SWIGLU else ffn


def mlp_block(X: Sequence[np.ndarray], W0: Sequence[np.ndarray], W1: Sequence[np.ndarray], act: int,
              rings: int = 2) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Returns (Out as FP64 per rank, H as BF16 bit patterns per rank).

    X[r]: [m x hidden], W0[r]: [ffn x hidden], W1[r]: [hidden x H columns], all
    BF16 bit patterns, weights K-major as everywhere in ``operators``."""
    C = ops.ag_gemm(X, W0, rings=rings)                                   # AllGather + GEMM0
    H = [f64_to_bf16_bits(activation(c, act)) for c in C]                 # what GEMM1 reads
    Out = ops.gemm_rs(H, W1, rings=rings)                                 # GEMM1 + ReduceScatter
    return Out, H


def mlp_block_rows(X: Sequence[np.ndarray], W0: Sequence[np.ndarray], W1: Sequence[np.ndarray], act: int,
                   rows: np.ndarray, rings: int = 2):
    """The block restricted to some rows of the gathered input (sorted global
    row indices), for sampling large cases: the rows of H and of the reduced
    output depend on the same rows of the gathered input only.  Returns
    (H rows as BF16 bits per rank, {owner chunk: (rows inside its block, FP64 values)})."""
    rows = np.asarray(rows, dtype=np.int64)
    P = len(X)
    C = ops.ag_gemm(X, W0, rings=rings, rows=rows)
    H_rows = [f64_to_bf16_bits(activation(c, act)) for c in C]
    M = P * X[0].shape[0]
    # GEMM1 + ReduceScatter on full-height tensors that hold only the sampled rows
    H_full = []
    for r in range(P):
        h = np.zeros((M, H_rows[r].shape[1]), dtype=np.uint16)
        h[rows] = H_rows[r]
        H_full.append(h)
    return H_rows, ops.gemm_rs_rows(H_full, W1, rows, rings=rings)
