"""The schedule tables executed as a real ring exchange between processes (gloo on CPU).

On one GPU the P logical ranks share a device and the fused kernels gather by address.  What the tables mean for P
separate devices -- a rank forwards, at every step and on every ring, the partition it obtained one step earlier, and
receives the partition its own entry names from the neighbour the entry names -- is run here with one process per rank:
the tables come from the library (compass_schedule through the C ABI), the transport is torch.distributed
send/recv, the arithmetic is numpy FP64 on the BF16 inputs.  AllGather+GEMM must end with every rank holding the whole
gathered input (and C_r equal to the oracle's); GEMM+ReduceScatter must end with every owner holding its rows of the
sum, accumulated hop by hop in ring order (equal to the oracle's, which adds in the same order)."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import numpy as np
import torch
import torch.distributed as dist
from oracle import operators as ops
from paper_2609_10549_b200 import api, workloads as wl

op, P, rings, m, N, K = {op}, {P}, {rings}, {m}, {N}, {K}
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=P)
r = dist.get_rank()
M = P * m
h = m // rings
table = api.compass_schedule(op, P, rings, M)                       # columns: rank, step, ring, part, chunk, peer, row_begin, row_count
mine = table[table[:, 0] == r]
entry = lambda s, g: mine[(mine[:, 1] == s) & (mine[:, 2] == g)][0]
w = wl.Workload("ring", op, P=P, M=M, N=N, K=K, b_dist=("normal", 0.1), seed=5)
A_bits, B_bits = wl.make_inputs(w)                                  # every process draws the same seeded inputs; it USES only its own shard
f64 = ops.bf16_bits_to_f64
down = lambda g: (r - 1) % P if (rings == 2 and g == 0) else (r + 1) % P      # ring 0 runs backward, ring 1 (or the single ring) forward
up = lambda g: (r + 1) % P if (rings == 2 and g == 0) else (r - 1) % P

pending = []                                                        # sends in flight: (request, buffer kept alive)

def exchange(send_to, send_arr, recv_from, shape, tag):
    # a send completes once its receiver has posted the matching receive, which may be a step later:
    # sends are left in flight and collected at the end
    got = None
    if send_arr is not None:
        buf = torch.from_numpy(np.ascontiguousarray(send_arr))
        pending.append((dist.isend(buf, dst=send_to, tag=tag), buf))
    if recv_from is not None:
        got = torch.empty(shape, dtype=torch.float64)
        dist.irecv(got, src=recv_from, tag=tag).wait()
    return None if got is None else got.numpy()

ok = True
if op == wl.OP_AG_GEMM:
    G = np.full((M, K), np.nan)
    held = {{}}                                                      # ring -> rows obtained at the previous step
    for s in range(P):
        for g in range(rings):
            e = entry(s, g)
            rb, rc, peer = int(e[6]), int(e[7]), int(e[5])
            if s == 0:
                ok &= peer == r and int(e[4]) == r                  # the local chunk first
                rows = f64(A_bits[r][rb - r * m: rb - r * m + rc])
            else:
                ok &= peer == up(g)                                 # arrives from the upstream neighbour of that ring
                rows = exchange(down(g), held[g], peer, (rc, K), tag=s * 2 + g)
            ok &= bool(np.isnan(G[rb:rb + rc]).all())               # every partition exactly once
            G[rb:rb + rc] = rows
            held[g] = rows
    ok &= not np.isnan(G).any()
    ok &= bool(np.array_equal(G, np.concatenate([f64(a) for a in A_bits])))
    C = G @ f64(B_bits[r]).T
    ok &= bool(np.array_equal(C, ops.ag_gemm(A_bits, B_bits, rings=rings, ranks=[r])[0]))
else:
    Bf = f64(B_bits[r])
    Out = np.full((m, N), np.nan)
    for s in range(P):
        for g in range(rings):
            e = entry(s, g)
            rb, rc, peer, chunk = int(e[6]), int(e[7]), int(e[5]), int(e[4])
            partial = f64(A_bits[r][rb:rb + rc]) @ Bf.T             # this rank's contribution to the partition
            # the running sum of THIS partition arrives from upstream (which worked on it one step earlier) ...
            running = exchange(None, None, up(g) if s > 0 else None, (rc, N), tag=(s - 1) * 2 + g)
            running = partial if running is None else running + partial
            if s < P - 1:
                ok &= peer == down(g)                               # ... and travels on to the neighbour the entry names
                exchange(peer, running, None, None, tag=s * 2 + g)
            else:
                ok &= peer == r and chunk == r                      # the local partition last: the sum ends at its owner
                Out[rb - r * m: rb - r * m + rc] = running
    ok &= not np.isnan(Out).any()
    ok &= bool(np.array_equal(Out, ops.gemm_rs(A_bits, B_bits, rings=rings, chunks=[r])[0]))
for req, _buf in pending:
    req.wait()
dist.barrier()
print(json.dumps({{"rank": r, "ok": bool(ok)}}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("op,P,rings,m,N,K", [
    (0, 2, 2, 16, 24, 32), (0, 4, 2, 8, 16, 24), (0, 4, 1, 6, 16, 24), (0, 3, 2, 4, 8, 16),
    (1, 2, 2, 16, 24, 32), (1, 4, 2, 8, 16, 24), (1, 4, 1, 6, 16, 24), (1, 3, 2, 4, 8, 16),
])
def test_tables_run_as_a_ring_exchange_between_processes(op, P, rings, m, N, K):
    port = _free_port()
    procs = []
    for rank in range(P):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(P), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="1")
        code = WORKER.format(root=ROOT, op=op, P=P, rings=rings, m=m, N=N, K=K)
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for rank, p in enumerate(procs):
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-3000:]
        assert json.loads(out.strip().splitlines()[-1]) == {"rank": rank, "ok": True}
