"""Times one operator of the library on one shape (a small command-line tool).

    python -m paper_2609_10549_b200.run_case --op ag --P 8 --M 16384 --N 7168 --K 8192
    python -m paper_2609_10549_b200.run_case --op rs --variant ring --P 8 --M 8192 --N 4096 --K 1376
    python -m paper_2609_10549_b200.run_case --op ag --variant decomp --d 4 --P 4 --M 4096 --N 3072 --K 4096

--op ag|rs: AllGather+GEMM (N per rank, K full) or GEMM+ReduceScatter (K per rank, N full).
--variant fused|ring|ring32|push|decomp|comm: the fused kernel (gather by address / segmented K), the ring
read-modify-write GEMM+ReduceScatter (running sum in the BF16 output rows, or in FP32 scratch), the readiness-driven AllGather+GEMM, InterDecom with --d stages, or the --d
sub-collectives of InterDecom alone (gather / reduce kernels on one stream; reported in GB/s of their algorithmic bytes).
Inputs are drawn on the device (seeded); every launch is timed between its own pair of CUDA events on the
launching stream after --warmup untimed launches.  Prints one JSON line: median / best milliseconds,
TFLOP/s over the FLOPs of all P logical ranks, the host time of one call, and the SM clock the last kernel
recorded.  It is also the command the ncu summaries under profiles/ were captured with.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=["ag", "rs"], required=True)
    ap.add_argument("--variant", choices=["fused", "ring", "ring32", "push", "decomp", "comm"], default="fused")
    ap.add_argument("--P", type=int, required=True)
    ap.add_argument("--M", type=int, required=True)
    ap.add_argument("--N", type=int, required=True)
    ap.add_argument("--K", type=int, required=True)
    ap.add_argument("--d", type=int, default=1)
    ap.add_argument("--rings", type=int, default=2)
    ap.add_argument("--ring-group", type=int, default=0, help="ring / ring32: contributors fused per read-modify-write pass")
    ap.add_argument("--order", choices=["rank", "step"], default="rank")
    ap.add_argument("--layout", choices=["nk", "kn"], default="nk")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--b-std", type=float, default=0.02)
    args = ap.parse_args()

    import torch

    from . import api
    from . import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("run_case needs a CUDA device: the library has no CPU fallback")
    op = wl.OP_AG_GEMM if args.op == "ag" else wl.OP_GEMM_RS
    if args.variant in ("ring", "ring32") and op != wl.OP_GEMM_RS:
        raise SystemExit("--variant ring / ring32 is a GEMM+ReduceScatter variant")
    if args.variant == "push" and op != wl.OP_AG_GEMM:
        raise SystemExit("--variant push is an AllGather+GEMM variant")
    w = wl.Workload("case", op, P=args.P, M=args.M, N=args.N, K=args.K)
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    mk = lambda shape, std: (torch.randn(shape, device="cuda", dtype=torch.float32, generator=g) * std).to(torch.bfloat16)
    A = [mk(w.a_shape, 1.0) for _ in range(w.P)]
    b_shape = w.b_shape if args.layout == "nk" else (w.b_shape[1], w.b_shape[0])
    B = [mk(b_shape, args.b_std) for _ in range(w.P)]
    out = [torch.empty(w.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(w.P)]
    pr = api.make_problem(op, w.P, w.M, w.N, w.K, rings=args.rings, d=args.d,
                          rs_variant={"ring": api.RS_RING_RMW, "ring32": api.RS_RING_RMW_F32}.get(args.variant, api.RS_SEGMENTED_K),
                          order=api.ORDER_RANK_MAJOR if args.order == "rank" else api.ORDER_STEP_MAJOR,
                          b_layout=api.B_NK if args.layout == "nk" else api.B_KN, ring_group=args.ring_group)
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    if args.variant in ("fused", "ring", "ring32"):
        ws = api.alloc_workspace(pr)
        call = api.compass_ag_gemm if op == wl.OP_AG_GEMM else api.compass_gemm_rs
        run = lambda: call(pr, A, B, out, ws, stream)
    elif args.variant == "push":
        ws = api.alloc_workspace(pr, api.WS_PUSH)
        run = lambda: api.compass_ag_gemm_push(pr, A, B, out, ws, stream, side)
    elif args.variant == "comm":
        ws = api.alloc_workspace(pr, api.WS_DECOMP)
        run = lambda: api.compass_decomp_comm(pr, A, B, out, ws, stream, None)
    else:
        ws = api.alloc_workspace(pr, api.WS_DECOMP)
        run = lambda: api.compass_decomp(pr, A, B, out, ws, stream, side)
    for _ in range(args.warmup):
        run()
    torch.cuda.synchronize()
    ts, host = [], []
    for _ in range(args.iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        h0 = time.perf_counter()
        run()
        host.append(time.perf_counter() - h0)
        e1.record(stream)
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    status = api.compass_read_status(ws)
    if status != (api.OK, 0):
        raise SystemExit(f"device-side status {status}")
    cycles, ns = api.compass_read_kernel_clock(ws)
    med = float(np.median(ts))
    if args.variant == "comm":
        # AllGather: every shard read once, written to the P gather buffers; ReduceScatter: P partials read, one result written
        nbytes = 2.0 * w.M * w.K * (1 + w.P) if op == wl.OP_AG_GEMM else 2.0 * w.M * w.N * (w.P + 1)
        print(json.dumps({"op": args.op, "variant": "comm", "P": w.P, "M": w.M, "N": w.N, "K": w.K, "d": args.d,
                          "ms_median": med, "ms_best": float(np.min(ts)), "algorithmic_bytes": nbytes,
                          "gbs_median": nbytes / (med * 1e-3) / 1e9}), flush=True)
        return
    print(json.dumps({
        "op": args.op, "variant": args.variant, "P": w.P, "M": w.M, "N": w.N, "K": w.K, "d": args.d, "rings": args.rings, "ring_group": args.ring_group,
        "order": args.order, "layout": args.layout, "iters": args.iters,
        "ms_median": med, "ms_best": float(np.min(ts)), "tflops_median": w.flops / (med * 1e-3) / 1e12,
        "tflops_best": w.flops / (float(np.min(ts)) * 1e-3) / 1e12,
        "host_us_per_call_median": float(np.median(host)) * 1e6,
        "kernel_sm_mhz": round(cycles / ns * 1e3, 1) if ns else None,
        "algorithmic_bytes": w.algorithmic_bytes}), flush=True)


if __name__ == "__main__":
    main()
