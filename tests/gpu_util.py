"""Helpers of the GPU parity tests: move seeded inputs to the device, run the
library through its C ABI, bring the BF16 outputs back as bit patterns.

Outputs are pre-filled with a NaN pattern and allocated with guard rows in
front and behind, so that a tile that is never written or a store outside the
tensor is caught without a memory checker."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_10549_b200 import api
from paper_2609_10549_b200 import workloads as wl

NAN_BITS = 0x7FC0
GUARD_BITS = 0x4B4B
GUARD_ROWS = 8


class Guarded:
    """A [rows x cols] BF16 device tensor with guard rows around it."""

    def __init__(self, rows: int, cols: int):
        self.rows, self.cols = rows, cols
        self.full = torch.full((rows + 2 * GUARD_ROWS, cols), GUARD_BITS, dtype=torch.int16, device="cuda")
        self.full[GUARD_ROWS:GUARD_ROWS + rows] = NAN_BITS
        self.view = self.full[GUARD_ROWS:GUARD_ROWS + rows].view(torch.bfloat16)

    def bits(self) -> np.ndarray:
        return self.full[GUARD_ROWS:GUARD_ROWS + self.rows].cpu().numpy().view(np.uint16)

    def guards_intact(self) -> bool:
        g = torch.cat([self.full[:GUARD_ROWS], self.full[GUARD_ROWS + self.rows:]])
        return bool((g == GUARD_BITS).all().item())


def device_inputs(A_bits, B_bits):
    return [api.to_device(a) for a in A_bits], [api.to_device(b) for b in B_bits]


def problem_of(w: wl.Workload, rings=2, d=1, rs_variant=api.RS_SEGMENTED_K, copy_mode=api.COPY_KERNEL) -> api.Problem:
    return api.make_problem(w.op, w.P, w.M, w.N, w.K, rings=rings, d=d, rs_variant=rs_variant, copy_mode=copy_mode)


def run_fused(w: wl.Workload, A_bits, B_bits, rings=2, rs_variant=api.RS_SEGMENTED_K):
    """Returns (list of uint16 outputs, status, guards ok)."""
    pr = problem_of(w, rings=rings, rs_variant=rs_variant)
    A, B = device_inputs(A_bits, B_bits)
    outs = [Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr, api.WS_FUSED)
    if w.op == wl.OP_AG_GEMM:
        api.compass_ag_gemm(pr, A, B, [o.view for o in outs], ws)
    else:
        api.compass_gemm_rs(pr, A, B, [o.view for o in outs], ws)
    status, detail = api.compass_read_status(ws)
    torch.cuda.synchronize()
    return [o.bits() for o in outs], (status, detail), all(o.guards_intact() for o in outs)


def run_decomp(w: wl.Workload, A_bits, B_bits, d: int, two_streams=True, copy_mode=api.COPY_KERNEL):
    pr = problem_of(w, d=d, copy_mode=copy_mode)
    A, B = device_inputs(A_bits, B_bits)
    outs = [Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr, api.WS_DECOMP)
    torch.cuda.synchronize()
    side = torch.cuda.Stream() if two_streams else None
    api.compass_decomp(pr, A, B, [o.view for o in outs], ws, torch.cuda.current_stream(), side)
    status, detail = api.compass_read_status(ws)
    torch.cuda.synchronize()
    return [o.bits() for o in outs], (status, detail), all(o.guards_intact() for o in outs)


def sample_rows(M: int, P: int, rings: int, tile: int = 128, frac: float = 0.01, seed: int = 0) -> np.ndarray:
    """Rows next to every partition and tile boundary plus a random sample."""
    h = M // P // rings
    rows = {0, M - 1}
    for b in range(0, M, h):
        for t in range(b, b + h, tile):
            rows.update(r for r in (t - 1, t, t + 1) if 0 <= r < M)
        rows.update(r for r in (b + h - 1,) if 0 <= r < M)
    rng = np.random.default_rng(seed)
    rows.update(int(r) for r in rng.integers(0, M, size=max(1, int(M * frac))))
    return np.array(sorted(rows), dtype=np.int64)
