"""AllGather+GEMM, GEMM+ReduceScatter and InterDecom in FP64 (oracle; tests only).

Inputs are BF16 bit patterns (uint16).  A product of two BF16 values has at
most 16 significant bits, so every product is exact in FP64 and a K-term sum
carries a relative error of about K * 2^-53: the FP64 result is "the exact
result" at the scale of a BF16 output.

Definitions followed (Section II-A):

* AllGather+GEMM: the column-parallel GEMM needs the full input, so rank r
  first gathers G = [A_0; A_1; ...; A_{P-1}] and then computes C_r = G * B_r.
* GEMM+ReduceScatter: rank q computes the partial Z_q = A_q * B_q of the
  row-parallel GEMM; the partials are summed and rank c keeps rows
  [c*m, (c+1)*m) of the sum.

The gather and the reduce-scatter are carried out explicitly, partition by
partition, in the order of a schedule table (Section III-B), so that a wrong
table breaks these functions' own invariants.

B_r is stored K-major, i.e. as an [N x K] array (the layout of a linear
layer's weight), so "A * B" below is ``A @ B.T``.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from . import OP_AG_GEMM, OP_GEMM_RS
from .schedule import RANK, STEP, RING, PART, CHUNK, ROW_BEGIN, ROW_COUNT, schedule


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen BF16 bit patterns to FP64 exactly."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_f64(x: np.ndarray) -> np.ndarray:
    """Round FP64 values to the nearest BF16 (ties to even); result as FP64.
    Used only for statistics, never for the acceptance rule."""
    f = x.astype(np.float32)                      # double rounding is harmless for statistics
    u = f.view(np.uint32)
    u = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def fp32_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round FP32 values to the nearest BF16, ties to even (exact: one rounding
    of a binary32 value); result as FP64."""
    assert x.dtype == np.float32
    u = x.view(np.uint32)
    u = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def hop_in_bf16(running: np.ndarray, partial: np.ndarray) -> np.ndarray:
    """One hop of a reduce-scatter ring whose messages have the output's type,
    BF16 (Section III-B: a rank adds its partial to the sum it received and
    sends the result on; the paper does not state the type of the message, this
    is the reading in which the ring moves tensors of the operator's own type).
    The arriving sum is a BF16 value, the rank's own partial an FP32
    accumulator; they are added in FP32 and the sum is rounded to BF16 for the
    next message.  This decides a rounding, so it is taken in that precision
    and not in FP64."""
    s = running.astype(np.float32) + partial.astype(np.float32)
    return fp32_to_bf16_rne(s)


def gather_in_schedule_order(A: Sequence[np.ndarray], table: np.ndarray, rank: int) -> np.ndarray:
    """Rank `rank`'s private gather buffer, filled partition by partition in
    the order of its schedule entries.  Every row must be written exactly once."""
    P = len(A)
    m, K = A[0].shape
    G = np.full((P * m, K), np.nan)
    written = np.zeros(P * m, dtype=np.int64)
    mine = table[table[:, RANK] == rank]
    assert (np.diff(mine[:, STEP]) >= 0).all(), "entries of a rank must be in step order"
    for e in mine:
        c, rb, rc = int(e[CHUNK]), int(e[ROW_BEGIN]), int(e[ROW_COUNT])
        lo = rb - c * m                      # first row inside shard c
        assert 0 <= lo and lo + rc <= m
        G[rb:rb + rc] = bf16_bits_to_f64(A[c][lo:lo + rc])
        written[rb:rb + rc] += 1
    assert (written == 1).all(), "a rank must consume every partition exactly once"
    return G


def ag_gemm(A: Sequence[np.ndarray], B: Sequence[np.ndarray], table: Optional[np.ndarray] = None,
            rings: int = 2, ranks: Optional[Sequence[int]] = None,
            rows: Optional[np.ndarray] = None) -> List[np.ndarray]:
    """C_r = gather(A) * B_r for every rank r (FP64).

    ``ranks`` restricts the computation to some ranks; ``rows`` to some rows of
    the gathered tensor (used to sample large cases: the gather still runs in
    full, only the GEMM is restricted)."""
    P = len(A)
    m, K = A[0].shape
    if table is None:
        table = schedule(OP_AG_GEMM, P, rings, P * m)
    out = []
    for r in (range(P) if ranks is None else ranks):
        G = gather_in_schedule_order(A, table, r)
        if rows is not None:
            G = G[rows]
        out.append(G @ bf16_bits_to_f64(B[r]).T)
    return out


def gemm_rs(A: Sequence[np.ndarray], B: Sequence[np.ndarray], table: Optional[np.ndarray] = None,
            rings: int = 2, chunks: Optional[Sequence[int]] = None, bf16_hops: bool = False,
            hop_group: int = 1) -> List[np.ndarray]:
    """Out_c = rows [c*m,(c+1)*m) of sum_q A_q * B_q, reduced along the ring.

    For every partition the running sum starts at the rank whose table lists
    that partition at step 0 and visits the ranks in step order; the last
    contributor must be the owner (Section III-B: local partition last).

    ``bf16_hops=False``: the sum itself (FP64), whatever the ring carries.
    ``bf16_hops=True``: the result of a ring whose messages are BF16 -- the sum
    is rounded once per contributor (``hop_in_bf16``), so the result depends on
    the ORDER of the contributors; the values returned are BF16 values.
    ``hop_group=G`` (a divisor of P): a ring between P/G nodes of G ranks each --
    G consecutive contributors add up their partials exactly before the node's
    one hop, so the sum is rounded P/G times."""
    P = len(A)
    M, K = A[0].shape
    N = B[0].shape[0]
    m = M // P
    if table is None:
        table = schedule(OP_GEMM_RS, P, rings, M)
    Bf = [bf16_bits_to_f64(b) for b in B]
    out = {}
    parts = {}
    for e in table:
        parts.setdefault(int(e[PART]), []).append(e)
    for part, entries in sorted(parts.items()):
        entries = sorted(entries, key=lambda e: int(e[STEP]))
        assert [int(e[STEP]) for e in entries] == list(range(P)), "one contributor per step"
        assert sorted(int(e[RANK]) for e in entries) == list(range(P)), "every rank contributes once"
        c = int(entries[0][CHUNK])
        if chunks is not None and c not in chunks:
            continue
        rb, rc = int(entries[0][ROW_BEGIN]), int(entries[0][ROW_COUNT])
        running = np.zeros((rc, N))
        for e in entries:
            assert int(e[ROW_BEGIN]) == rb and int(e[ROW_COUNT]) == rc and int(e[CHUNK]) == c
            q = int(e[RANK])
            partial = bf16_bits_to_f64(A[q][rb:rb + rc]) @ Bf[q].T
            node = partial if int(e[STEP]) % hop_group == 0 else node + partial
            if not bf16_hops:
                running = running + partial
            elif int(e[STEP]) % hop_group == hop_group - 1:
                running = hop_in_bf16(running, node)
        assert P % hop_group == 0
        assert int(entries[-1][RANK]) == c, "the running sum must end at the owner"
        if c not in out:
            out[c] = np.full((m, N), np.nan)
        lo = rb - c * m
        assert np.isnan(out[c][lo:lo + rc]).all(), "output rows written twice"
        out[c][lo:lo + rc] = running
    result = [out[c] for c in sorted(out)]
    for o in result:
        assert not np.isnan(o).any(), "output rows never written"
    return result


def gemm_rs_rows(A: Sequence[np.ndarray], B: Sequence[np.ndarray], rows: np.ndarray,
                 table: Optional[np.ndarray] = None, rings: int = 2, bf16_hops: bool = False, hop_group: int = 1):
    """GEMM+ReduceScatter restricted to some rows of the reduced [M x N] tensor
    (sorted global row indices), for sampling large cases.  Same ring order as
    ``gemm_rs``.  Returns {owner chunk: (rows inside the owner's block, values)}."""
    P = len(A)
    M, K = A[0].shape
    m = M // P
    if table is None:
        table = schedule(OP_GEMM_RS, P, rings, M)
    rows = np.asarray(rows, dtype=np.int64)
    Bf = [bf16_bits_to_f64(b) for b in B]
    parts = {}
    for e in table:
        parts.setdefault(int(e[PART]), []).append(e)
    found = {}
    for part, entries in sorted(parts.items()):
        entries = sorted(entries, key=lambda e: int(e[STEP]))
        c, rb, rc = int(entries[0][CHUNK]), int(entries[0][ROW_BEGIN]), int(entries[0][ROW_COUNT])
        sel = rows[(rows >= rb) & (rows < rb + rc)]
        if sel.size == 0:
            continue
        running = np.zeros((sel.size, Bf[0].shape[0]))
        for e in entries:
            q = int(e[RANK])
            partial = bf16_bits_to_f64(A[q][sel]) @ Bf[q].T
            node = partial if int(e[STEP]) % hop_group == 0 else node + partial
            if not bf16_hops:
                running = running + partial
            elif int(e[STEP]) % hop_group == hop_group - 1:
                running = hop_in_bf16(running, node)
        assert int(entries[-1][RANK]) == c
        found.setdefault(c, []).append((sel - c * m, running))
    return {c: (np.concatenate([x[0] for x in v]), np.concatenate([x[1] for x in v])) for c, v in found.items()}


def decomp_ag_gemm(A: Sequence[np.ndarray], B: Sequence[np.ndarray], d: int) -> List[np.ndarray]:
    """InterDecom of AllGather+GEMM into d sub-operators (Section II-B).

    Reading: the operator is split along rows; sub-operator j gathers row
    slice j of every rank's shard (a sub-AllGather) and multiplies those rows
    (a sub-GEMM).  d = 1 is sequential execution."""
    P = len(A)
    m, K = A[0].shape
    assert m % d == 0
    sl = m // d
    C = [np.full((P * m, B[r].shape[0]), np.nan) for r in range(P)]
    for j in range(d):
        for r in range(P):
            Gj = np.concatenate([bf16_bits_to_f64(A[q][j * sl:(j + 1) * sl]) for q in range(P)])   # sub-AllGather
            Cj = Gj @ bf16_bits_to_f64(B[r]).T                                                        # sub-GEMM
            for q in range(P):
                C[r][q * m + j * sl:q * m + (j + 1) * sl] = Cj[q * sl:(q + 1) * sl]
    return C


def decomp_gemm_rs(A: Sequence[np.ndarray], B: Sequence[np.ndarray], d: int) -> List[np.ndarray]:
    """InterDecom of GEMM+ReduceScatter: sub-operator j computes, on every
    rank, the partial rows of slice j of every owner's block (a sub-GEMM) and
    a sub-ReduceScatter sums them into the owners' rows."""
    P = len(A)
    M, K = A[0].shape
    N = B[0].shape[0]
    m = M // P
    assert m % d == 0
    sl = m // d
    Out = [np.full((m, N), np.nan) for _ in range(P)]
    Bf = [bf16_bits_to_f64(b) for b in B]
    for j in range(d):
        rows = np.concatenate([np.arange(c * m + j * sl, c * m + (j + 1) * sl) for c in range(P)])
        partial = [bf16_bits_to_f64(A[q][rows]) @ Bf[q].T for q in range(P)]      # sub-GEMMs
        total = np.zeros_like(partial[0])
        for q in range(P):                                                         # sub-ReduceScatter
            total += partial[q]
        for c in range(P):
            Out[c][j * sl:(j + 1) * sl] = total[c * sl:(c + 1) * sl]
    return Out


def unsharded_gemm(A_full_bits: np.ndarray, B_bits: np.ndarray) -> np.ndarray:
    """Plain C = A * B^T in FP64 on BF16 bit inputs, no sharding, no schedule."""
    return bf16_bits_to_f64(A_full_bits) @ bf16_bits_to_f64(B_bits).T
