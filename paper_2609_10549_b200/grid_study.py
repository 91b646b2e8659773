"""Scores the performance models and the selector over the paper's parameter grid.

Table IV spans hidden size K x intermediate size N x world size x sequence
length M x pattern = 288 cases, with the decomposition degree swept inside
each case.  For every case this script times, through the C ABI,

  * the fused kernel (gather by address / segmented K),
  * for AllGather+GEMM the readiness-driven variant (pushed partitions + flags),
  * the decomposed pipeline for d in {1, 2, 4, 8, 16},

then fits the models' parameters on half of the cases (Section IV-C: one-time
offline regression) and scores them on the other half: mean absolute error of
the decomposition model with and without the overhead factor (the comparison
of Table II), of the fusion model with and without its overhead term, how often
Eq. 4-5 pick the measured-best degree, what a fixed d = 4 costs, and how often
Algorithm 1 picks the measured-faster strategy.

Mapping of Table IV onto the two operators of one MLP block (Section II-A):
AllGather+GEMM multiplies [M x K] by the column-parallel [K x N/P];
GEMM+ReduceScatter multiplies [M x N/P] by the row-parallel [N/P x K].

    python -m paper_2609_10549_b200.grid_study measure --out grid.jsonl [--shard i/n] [--max-m 32768] [--limit n]
    python -m paper_2609_10549_b200.grid_study analyze --inp grid.jsonl [--report report.json] [--summary summary.md]
                                                       [--calib-out calib.json]

`measure` appends one JSON line per case and skips cases already in the file.
`analyze` needs no GPU (host arithmetic through the C ABI); `--calib-out`
stores the fitted compass_calib of both patterns with its provenance, in the
form `load_calibration` reads back (bench.py uses it instead of refitting).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

from . import api
from . import workloads as wl

HIDDEN = (4096, 8192, 16384)
INTER = (2048, 4096, 8192, 16384)
WORLD = (4, 8)
SEQ = (2048, 4096, 8192, 12288, 16384, 32768)
DEGREES = (1, 2, 4, 8, 16)


def grid(max_m=32768):
    cases = []
    for op in (wl.OP_AG_GEMM, wl.OP_GEMM_RS):
        for P in WORLD:
            for K in HIDDEN:
                for N in INTER:
                    for M in SEQ:
                        if M > max_m:
                            continue
                        if op == wl.OP_AG_GEMM:
                            shape = dict(op=op, P=P, M=M, N=N // P, K=K)
                        else:
                            shape = dict(op=op, P=P, M=M, N=K, K=N // P)
                        cases.append(dict(shape, table_K=K, table_N=N))
    return cases


def case_key(c):
    return f"{c['op']}-{c['P']}-{c['M']}-{c['table_N']}-{c['table_K']}"


def measure_cases(cases, out_path, iters=5, log=print):
    """Times every case in `cases` (dicts as `grid` makes them) and appends one JSON line per case to `out_path`;
    cases already in the file are skipped.  Returns the number of cases measured."""
    import torch

    done = set()
    if os.path.exists(out_path):
        with open(out_path) as f:
            done = {case_key(json.loads(line)) for line in f if line.strip()}
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()

    def timed_in_turn(fns, iters, warm=1):
        """Median time of every variant, the variants timed in turn inside one loop: the board's power state drifts
        while a case runs, and variants timed one after the other would not be compared at the same clock."""
        for _ in range(warm):
            for fn in fns.values():
                fn()
        torch.cuda.synchronize()
        ts = {k: [] for k in fns}
        for _ in range(iters):
            for k, fn in fns.items():
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                torch.cuda.synchronize()
                ts[k].append(e0.elapsed_time(e1))
        return {k: float(np.median(v)) for k, v in ts.items()}

    measured = 0
    for c in cases:
        if case_key(c) in done:
            continue
        w = wl.Workload("grid", c["op"], P=c["P"], M=c["M"], N=c["N"], K=c["K"])
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        mk = lambda shape, std: (torch.randn(shape, device="cuda", dtype=torch.float32, generator=g) * std).to(torch.bfloat16)
        A = [mk(w.a_shape, 1.0) for _ in range(w.P)]
        B = [mk(w.b_shape, 0.02) for _ in range(w.P)]
        out = [torch.empty(w.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(w.P)]
        pr = api.make_problem(w.op, w.P, w.M, w.N, w.K)
        ws = api.alloc_workspace(pr)
        fused = api.compass_ag_gemm if w.op == wl.OP_AG_GEMM else api.compass_gemm_rs
        rec = dict(c, flops=w.flops, m_rows=w.m)
        fns = {"fused": lambda: fused(pr, A, B, out, ws, stream)}
        pws = None
        if w.op == wl.OP_AG_GEMM:
            pws = torch.empty(api.compass_workspace_bytes(pr, api.WS_PUSH), dtype=torch.uint8, device="cuda")
            api.compass_workspace_init(pws)
            fns["push"] = lambda: api.compass_ag_gemm_push(pr, A, B, out, pws, stream, side)
        dws = None
        for d in DEGREES:
            if w.m % d:
                continue
            prd = api.make_problem(w.op, w.P, w.M, w.N, w.K, d=d)
            if dws is None:
                dws = api.alloc_workspace(prd, api.WS_DECOMP)
            fns[str(d)] = (lambda prd: lambda: api.compass_decomp(prd, A, B, out, dws, stream, side))(prd)
        ms = timed_in_turn(fns, iters)
        rec["fused_ms"] = ms["fused"]
        if "push" in ms:
            rec["push_ms"] = ms["push"]
        rec["decomp_ms"] = {k: v for k, v in ms.items() if k not in ("fused", "push")}
        status = api.compass_read_status(ws)
        if status != (api.OK, 0):
            raise SystemExit(f"device status {status} on {c}")
        with open(out_path, "a") as f:
            f.write(json.dumps(rec) + "\n")
        log(case_key(c), round(rec["fused_ms"], 3), {k: round(v, 3) for k, v in rec["decomp_ms"].items()})
        measured += 1
        del A, B, out, ws, dws, pws, fns
        torch.cuda.empty_cache()
    return measured


def measure(args):
    cases = grid(args.max_m)
    i, n = (int(x) for x in args.shard.split("/"))
    cases = [c for k, c in enumerate(cases) if k % n == i]
    if args.limit:
        cases = cases[:args.limit]
    measure_cases(cases, args.out, log=lambda *a: print(*a, flush=True))


CALIB_FIELDS = ("comp_a", "comp_b", "comm_a", "comm_b", "alpha_decomp", "beta_decomp", "alpha_fusion", "beta_fusion")
PATTERNS = ((wl.OP_AG_GEMM, "AG+GEMM"), (wl.OP_GEMM_RS, "GEMM+RS"))


def analyze_records(recs):
    """Fit on every other case, score on the rest; host arithmetic only (the C ABI's model and regression calls).
    `recs`: the dicts `measure_cases` writes.  Returns the report dict."""
    recs = [dict(r) for r in recs]
    report = {"cases": len(recs)}
    for op, name in PATTERNS:
        rs = sorted((r for r in recs if r["op"] == op), key=case_key)
        if len(rs) < 4:
            continue
        for r in rs:
            r["t_comp"] = r["fused_ms"]                                      # same FLOPs, no sub-collective
            r["t_comm"] = max(r["decomp_ms"]["1"] - r["fused_ms"], 1e-4)     # T(1) = T_comp + T_comm
            r["t_intra"] = r.get("push_ms") or r["fused_ms"]
            r["volume"] = float(r["M"]) * (r["K"] if op == wl.OP_AG_GEMM else r["N"])
            r["bytes"] = 2.0 * r["P"] * r["volume"]
        cal, test = rs[0::2], rs[1::2]
        ca, cb = api.compass_calib_fit_line([r["flops"] for r in cal], [r["t_comp"] for r in cal])
        ma, mb = api.compass_calib_fit_line([r["bytes"] for r in cal], [r["t_comm"] for r in cal])
        tc, tm, dd, tt = [], [], [], []
        for r in cal:
            for d, t in r["decomp_ms"].items():
                if int(d) > 1:
                    tc.append(r["t_comp"]); tm.append(r["t_comm"]); dd.append(int(d)); tt.append(t)
        alpha, beta = api.compass_calib_fit_decomp(tc, tm, dd, tt)
        af, bf = api.compass_calib_fit_fusion([r["t_comp"] for r in cal], [r["t_comm"] for r in cal], [r["P"] for r in cal],
                                              [r["volume"] for r in cal], [r["t_intra"] for r in cal])
        calib = api.Calib(ca, cb, ma, mb, alpha, beta, af, bf)
        mae_aware = {d: [] for d in DEGREES[1:]}
        mae_agn = {d: [] for d in DEGREES[1:]}
        fus_aware, fus_agn, d_hits, strat_hits, fixed4_penalty, pred_penalty = [], [], [], [], [], []
        best_hist = {}
        for r in test:
            for d in DEGREES[1:]:
                if str(d) in r["decomp_ms"]:
                    meas = r["decomp_ms"][str(d)]
                    mae_aware[d].append(abs(api.compass_model_decomp_time(r["t_comp"], r["t_comm"], alpha, beta, d) - meas))
                    mae_agn[d].append(abs(api.compass_model_decomp_time(r["t_comp"], r["t_comm"], 1.0, 0.0, d) - meas))
            fus_aware.append(abs(api.compass_model_fusion_time(r["t_comp"], r["t_comm"], r["P"], af, bf, r["volume"]) - r["t_intra"]))
            fus_agn.append(abs(api.compass_model_fusion_time(r["t_comp"], r["t_comm"], r["P"], 0.0, 0.0, r["volume"]) - r["t_intra"]))
            best_d = min(r["decomp_ms"], key=lambda k: r["decomp_ms"][k])
            best_hist[best_d] = best_hist.get(best_d, 0) + 1
            choice = api.compass_select(api.make_problem(op, r["P"], r["M"], r["N"], r["K"]), calib)
            d_hits.append(int(str(choice.d_star) == best_d))
            t_best = r["decomp_ms"][best_d]
            pred_penalty.append(r["decomp_ms"].get(str(choice.d_star), t_best) / t_best - 1.0)
            if "4" in r["decomp_ms"]:
                fixed4_penalty.append(r["decomp_ms"]["4"] / t_best - 1.0)
            winner = api.STRATEGY_INTRAFUSION if r["t_intra"] < t_best else api.STRATEGY_INTERDECOM
            strat_hits.append(int(choice.strategy == winner))
        mean = lambda xs: float(np.mean(xs)) if xs else None
        report[name] = {
            "calibration_cases": len(cal), "test_cases": len(test),
            "calib": dict(zip(CALIB_FIELDS, (ca, cb, ma, mb, alpha, beta, af, bf))),
            "decomp_mae_ms_overhead_aware": {str(d): mean(v) for d, v in mae_aware.items()},
            "decomp_mae_ms_overhead_agnostic": {str(d): mean(v) for d, v in mae_agn.items()},
            "decomp_mae_ms_overall": {"aware": mean(sum(mae_aware.values(), [])), "agnostic": mean(sum(mae_agn.values(), []))},
            "mean_decomp_time_ms": mean([t for r in test for t in r["decomp_ms"].values()]),
            "fusion_mae_ms": {"aware": mean(fus_aware), "agnostic": mean(fus_agn)},
            "measured_best_d_histogram": best_hist,
            "predicted_d_is_best": mean(d_hits),
            "penalty_of_predicted_d": mean(pred_penalty), "penalty_of_fixed_d4": mean(fixed4_penalty),
            "selector_accuracy": mean(strat_hits),
            "intrafusion_wins": int(sum(1 for r in test if r["t_intra"] < min(r["decomp_ms"].values()))),
        }
    return report


def calibration_of(report, provenance):
    """The fitted parameters of both patterns in the form `load_calibration` reads (times in milliseconds)."""
    return {"unit": "ms", "provenance": provenance,
            "patterns": {name: report[name]["calib"] for _op, name in PATTERNS if name in report}}


def load_calibration(path):
    """{pattern name: api.Calib} from a file `analyze --calib-out` wrote, plus its provenance string."""
    with open(path) as f:
        doc = json.load(f)
    calibs = {name: api.Calib(*[float(c[k]) for k in CALIB_FIELDS]) for name, c in doc["patterns"].items()}
    return calibs, doc.get("provenance", "")


def summary_markdown(report, source):
    """The comparison of Table II / Section V-B / Section VI-C as a small table."""
    rows = [("cases scored (fit on every other case)", lambda r: f"{r['test_cases']} (fit on {r['calibration_cases']})"),
            ("decomposition model MAE, overhead-agnostic -> aware (ms; mean time)",
             lambda r: f"{r['decomp_mae_ms_overall']['agnostic']:.2f} -> {r['decomp_mae_ms_overall']['aware']:.2f} "
                       f"({r['mean_decomp_time_ms']:.2f})"),
            ("per d = 2 / 4 / 8 / 16, aware (ms)",
             lambda r: " / ".join(f"{r['decomp_mae_ms_overhead_aware'][d]:.2f}" for d in ("2", "4", "8", "16"))),
            ("per d = 2 / 4 / 8 / 16, agnostic (ms)",
             lambda r: " / ".join(f"{r['decomp_mae_ms_overhead_agnostic'][d]:.2f}" for d in ("2", "4", "8", "16"))),
            ("fusion model MAE, agnostic -> aware (ms)",
             lambda r: f"{r['fusion_mae_ms']['agnostic']:.2f} -> {r['fusion_mae_ms']['aware']:.2f}"),
            ("fitted (alpha, beta) of Eq. 3", lambda r: f"{r['calib']['alpha_decomp']:.3f}, {r['calib']['beta_decomp']:.3f}"),
            ("measured-best d: 1 / 2 / 4 / 8 / 16",
             lambda r: " / ".join(str(r['measured_best_d_histogram'].get(d, 0)) for d in ("1", "2", "4", "8", "16"))),
            ("Eq. 4-5 pick the measured best", lambda r: f"{100 * r['predicted_d_is_best']:.1f} %"),
            ("cost of the predicted d / of fixed d = 4 over the best",
             lambda r: f"{100 * r['penalty_of_predicted_d']:.1f} % / {100 * r['penalty_of_fixed_d4']:.1f} %"),
            ("Algorithm 1 picks the faster strategy", lambda r: f"{100 * r['selector_accuracy']:.1f} %"),
            ("IntraFusion faster in", lambda r: f"{r['intrafusion_wins']} of {r['test_cases']}")]
    names = [name for _op, name in PATTERNS if name in report]
    lines = [f"Grid study over {report['cases']} cases ({source}).", "",
             "| | " + " | ".join(names) + " |", "|---|" + "---|" * len(names)]
    for label, fn in rows:
        lines.append(f"| {label} | " + " | ".join(fn(report[n]) for n in names) + " |")
    return "\n".join(lines) + "\n"


def analyze(args):
    with open(args.inp) as f:
        recs = [json.loads(line) for line in f if line.strip()]
    report = analyze_records(recs)
    text = json.dumps(report, indent=1)
    print(text)
    if args.report:
        with open(args.report, "w") as f:
            f.write(text + "\n")
    if args.summary:
        with open(args.summary, "w") as f:
            f.write(summary_markdown(report, args.provenance or os.path.basename(args.inp)))
    if args.calib_out:
        with open(args.calib_out, "w") as f:
            json.dump(calibration_of(report, args.provenance or os.path.basename(args.inp)), f, indent=1)
            f.write("\n")


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    m = sub.add_parser("measure")
    m.add_argument("--out", required=True)
    m.add_argument("--shard", default="0/1")
    m.add_argument("--max-m", type=int, default=32768)
    m.add_argument("--limit", type=int, default=0, help="measure only the first n cases of the shard")
    a = sub.add_parser("analyze")
    a.add_argument("--inp", required=True)
    a.add_argument("--report", help="write the report (JSON) here")
    a.add_argument("--summary", help="write the comparison table (markdown) here")
    a.add_argument("--calib-out", help="write the fitted calibration of both patterns (JSON) here")
    a.add_argument("--provenance", default="", help="where and how the timings were taken (stored with the outputs)")
    args = ap.parse_args()
    (measure if args.cmd == "measure" else analyze)(args)


if __name__ == "__main__":
    sys.exit(main())
