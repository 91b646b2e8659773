"""Second, independent enumeration of the ring schedule (oracle; tests only).

Instead of a closed form this module *plays the rings*: every rank starts
with a token for each of its own partitions and at every step hands the token
it obtained last to its downstream neighbour (Section III-B, "rolling wave").

* AllGather+GEMM: what a rank holds after step s is what it processes at s.
* GEMM+ReduceScatter: run the reduce-scatter backwards in time.  At the last
  step every rank holds the running sum of its own partitions; one step
  earlier that running sum sat at the upstream neighbour, and so on.

It also counts, per step, the rows crossing every directed link, from which
the effective-bandwidth factors printed in Section III-A follow.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

from . import OP_AG_GEMM, OP_GEMM_RS


def simulate(op: int, P: int, rings: int, M: int) -> np.ndarray:
    m = M // P
    h = m // rings
    # downstream neighbour of rank r on ring g
    if rings == 2:
        downstream = [lambda r: (r - 1) % P, lambda r: (r + 1) % P]
    else:
        downstream = [lambda r: (r + 1) % P]
    # holder[g][r] = chunk id of the token that rank r holds on ring g
    per_rank = {r: [] for r in range(P)}
    for g in range(rings):
        holder = list(range(P))             # everybody holds its own chunk
        came_from = list(range(P))          # local
        history = []
        for s in range(P):
            history.append((list(holder), list(came_from)))
            nxt = [None] * P
            src = [None] * P
            for r in range(P):
                d = downstream[g](r)
                nxt[d] = holder[r]
                src[d] = r
            holder, came_from = nxt, src
        if op == OP_AG_GEMM:
            for s, (hold, frm) in enumerate(history):
                for r in range(P):
                    per_rank[r].append((s, g, hold[r], frm[r]))
        else:
            # Time reversal.  At the last step every rank holds the running
            # sum of its own partition.  The running sum that rank r holds at
            # step s was, at step s-1, at the rank u whose downstream
            # neighbour is r; so holder_{s-1}[u] = holder_s[downstream(u)].
            hold = list(range(P))
            for s in range(P - 1, -1, -1):
                for r in range(P):
                    to = r if s == P - 1 else downstream[g](r)
                    per_rank[r].append((s, g, hold[r], to))
                hold = [hold[downstream[g](u)] for u in range(P)]
    rows = []
    for r in range(P):
        for (s, g, chunk, peer) in sorted(per_rank[r], key=lambda t: (t[0], t[1])):
            rows.append((r, s, g, rings * chunk + g, chunk, peer, chunk * m + g * h, h))
    return np.asarray(rows, dtype=np.int32).reshape(-1, 8)


def link_rows_per_step(table: np.ndarray, op: int, P: int):
    """For every step, a dict {(src, dst): rows carried} derived from a table.

    AG: an entry with peer != rank at step s was carried peer -> rank to be
    ready at step s.  RS: an entry with peer != rank at step s is sent
    rank -> peer after step s.
    """
    steps = [dict() for _ in range(P)]
    for rank, step, ring, part, chunk, peer, row_begin, row_count in table.tolist():
        if peer == rank:
            continue
        link = (peer, rank) if op == OP_AG_GEMM else (rank, peer)
        steps[step][link] = steps[step].get(link, 0) + row_count
    return steps


def effective_bandwidth_factor(table: np.ndarray, op: int, P: int, M: int) -> Fraction:
    """Collective size / (sum over steps of the busiest link's load), in units
    of one link's bandwidth: the quantity Section III-A quotes as (8/7)B,
    (4/3)B and (8/3)B."""
    busiest = 0
    for links in link_rows_per_step(table, op, P):
        if links:
            busiest += max(links.values())
    return Fraction(M, busiest)
