"""Ring chunk schedule, closed form (oracle; test infrastructure only).

What the paper fixes (Section III-A, III-B):

* the gathered / reduced tensor is cut into P chunks, one per GPU, and with
  the double ring every chunk is cut again into a backward-ring and a
  forward-ring component: 2P logical partitions (8 at 4 GPUs);
* the backward ring circulates the even-indexed partitions, the forward ring
  the odd-indexed ones, in opposite directions;
* AllGather+GEMM starts with the local data (step 1 of the paper = step 0
  here) and a partition is processed on arrival;
* GEMM+ReduceScatter reverses the dependency and schedules the partition that
  stays on the local device last;
* a ring over P GPUs takes P-1 transfer steps.

Readings where the text is silent (the worked 4-GPU figure is not available):

* forward ring sends r -> r+1, backward ring r -> r-1 (mod P);
* a chunk is split along rows; the even (backward-ring) partition is the
  first half of the chunk's rows, the odd (forward-ring) one the second half;
* inside one step the ring-0 entry precedes the ring-1 entry;
* the ReduceScatter order is the ring reduce-scatter in which every partition
  finishes at its owner at the last step: at step s rank r works on the
  partition whose owner is P-1-s hops downstream of r on that ring;
* with a single ring the only ring is the forward one.

Table layout: int32 array [count, 8], columns
``rank, step, ring, part, chunk, peer, row_begin, row_count``; order is
rank-major, then step, then ring.  ``part = rings*chunk + ring``.  ``peer`` is
the neighbour the partition arrives from (AG) or is sent to (RS), and equals
``rank`` for the local entry.  ``row_begin/row_count`` address rows of the
gathered (AG) or of the full reduced (RS) tensor.
"""
from __future__ import annotations

import numpy as np

from . import OP_AG_GEMM, OP_GEMM_RS

COLS = ("rank", "step", "ring", "part", "chunk", "peer", "row_begin", "row_count")
RANK, STEP, RING, PART, CHUNK, PEER, ROW_BEGIN, ROW_COUNT = range(8)


def ring_direction(rings: int, ring: int) -> int:
    """+1 for the forward ring (r -> r+1), -1 for the backward ring."""
    if rings == 1:
        return +1
    return -1 if ring == 0 else +1


def schedule(op: int, P: int, rings: int, M: int) -> np.ndarray:
    if op not in (OP_AG_GEMM, OP_GEMM_RS):
        raise ValueError("op")
    if P < 1 or rings not in (1, 2):
        raise ValueError("P / rings")
    if M <= 0 or M % P != 0 or (M // P) % rings != 0:
        raise ValueError("M must split into P chunks of `rings` equal parts")
    m = M // P          # rows per chunk
    h = m // rings      # rows per partition
    rows = []
    for r in range(P):
        for s in range(P):
            for g in range(rings):
                direction = ring_direction(rings, g)
                if op == OP_AG_GEMM:
                    # After s hops along the ring, rank r holds what started
                    # s positions upstream of it.
                    chunk = (r - direction * s) % P
                    local = (s == 0)
                    peer = r if local else (r - direction) % P      # arrives from upstream
                else:
                    # The partition worked on at step s still has P-1-s hops
                    # to go downstream before it reaches its owner.
                    chunk = (r + direction * (P - 1 - s)) % P
                    local = (s == P - 1)
                    peer = r if local else (r + direction) % P      # sent downstream
                part = rings * chunk + g
                rows.append((r, s, g, part, chunk, peer, chunk * m + g * h, h))
    return np.asarray(rows, dtype=np.int32).reshape(-1, 8)


def entries_of_rank(table: np.ndarray, rank: int) -> np.ndarray:
    return table[table[:, RANK] == rank]
