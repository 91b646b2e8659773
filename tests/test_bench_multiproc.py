"""The multi-process side of bench.py on CPU (gloo, world size 2): device timings
are reduced with MAX over ranks, launch counts with SUM, the aggregate counts
every replica's FLOPs, and the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
timings, launches = bench.reduce_over_ranks(dist, [1.0 + rank, 5.0 - rank, 0.25 * (rank + 1)], 200 + rank, "cpu")
dist.barrier()
print(json.dumps({{"rank": rank, "timings": timings, "launches": launches,
                  "value": bench.aggregate_tflops(dist.get_world_size(), 2.0e12, timings[0])}}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_timings_max_and_launches_sum_over_two_ranks():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT)], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["timings"] == [2.0, 5.0, 0.5]          # max over ranks, element by element
        assert o["launches"] == 401                       # sum over ranks
        # two replicas of 2 TFLOP per step in 2 ms: 2 * 2e12 / 2e-3 = 2000 TFLOP/s
        assert abs(o["value"] - 2000.0) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
