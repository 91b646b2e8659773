"""The grid study (the models and the selector scored over Table IV's 288 cases).

`analyze_records` is host arithmetic over recorded timings, so it is tested
without a GPU: timings are synthesised from PLANTED parameters through the
oracle's own model functions (Eq. 2-3, Eq. 7-8), and the analysis -- which
runs the library's regressions, models and selector through the C ABI -- must
recover the parameters, predict every timing, and pick the best degree and
strategy in every case.  A GPU test measures a few small grid cases for real.
"""
import json
import math

import pytest

from oracle import models as omo
from paper_2609_10549_b200 import api
from paper_2609_10549_b200 import grid_study as gs
from paper_2609_10549_b200 import workloads as wl

PLANTED = {
    wl.OP_AG_GEMM: omo.Calib(0.011, 7.3e-13, 0.004, 2.9e-10, 0.62, 0.021, 0.0031, 1.7e-9),
    wl.OP_GEMM_RS: omo.Calib(0.013, 6.9e-13, 0.006, 4.1e-10, 0.48, 0.034, 0.0007, 0.6e-9),
}


def synthetic_records():
    recs = []
    for c in gs.grid():
        cal = PLANTED[c["op"]]
        P, M, N, K = c["P"], c["M"], c["N"], c["K"]
        t_comp = cal.comp_a + cal.comp_b * omo.workload_flops(P, M, N, K)
        t_comm = cal.comm_a + cal.comm_b * omo.workload_comm_bytes(c["op"], P, M, N, K)
        rec = dict(c, flops=omo.workload_flops(P, M, N, K), m_rows=M // P, fused_ms=t_comp)
        rec["decomp_ms"] = {str(d): omo.decomp_time(t_comp, t_comm, cal.alpha_decomp, cal.beta_decomp, d)
                            for d in gs.DEGREES if (M // P) % d == 0}
        t_fusion = omo.fusion_time(t_comp, t_comm, P, cal.alpha_fusion, cal.beta_fusion, omo.message_volume(c["op"], M, N, K))
        if c["op"] == wl.OP_AG_GEMM:
            rec["push_ms"] = t_fusion
        else:
            rec["fused_ms"] = t_comp      # GEMM+ReduceScatter has no push variant: its fused time stands for IntraFusion
        recs.append(rec)
    return recs


def test_the_grid_is_the_papers():
    cases = gs.grid()
    assert len(cases) == 288 and len({gs.case_key(c) for c in cases}) == 288          # Table IV: 3 x 4 x 2 x 6 x 2
    assert sum(1 for c in cases if c["op"] == wl.OP_AG_GEMM) == 144


def test_analysis_recovers_planted_parameters_and_scores_perfectly():
    recs = synthetic_records()
    assert recs[0]["decomp_ms"]["1"] == pytest.approx(recs[0]["fused_ms"] + 0.004 + 2.9e-10 * 2 * recs[0]["P"] * recs[0]["M"] * recs[0]["K"])
    report = gs.analyze_records(recs)
    assert report["cases"] == 288
    for op, name in gs.PATTERNS:
        r, planted = report[name], PLANTED[op]
        assert r["calibration_cases"] == 72 and r["test_cases"] == 72
        for field in ("comp_a", "comp_b", "comm_a", "comm_b", "alpha_decomp", "beta_decomp"):
            assert r["calib"][field] == pytest.approx(getattr(planted, field), rel=1e-6, abs=1e-12), field
        assert r["decomp_mae_ms_overall"]["aware"] < 1e-9
        assert r["decomp_mae_ms_overall"]["agnostic"] > 1e-3          # eta = 1 is not the planted overhead
        assert all(v < 1e-9 for v in r["decomp_mae_ms_overhead_aware"].values())
        assert r["predicted_d_is_best"] == 1.0 and r["penalty_of_predicted_d"] == pytest.approx(0.0, abs=1e-12)
        assert r["penalty_of_fixed_d4"] > 0.0
        assert sum(r["measured_best_d_histogram"].values()) == 72
    ag = report["AG+GEMM"]
    # the push timings carry the planted fusion overhead: the regression finds it and the aware model is exact
    assert ag["calib"]["alpha_fusion"] == pytest.approx(PLANTED[wl.OP_AG_GEMM].alpha_fusion, rel=1e-6)
    assert ag["calib"]["beta_fusion"] == pytest.approx(PLANTED[wl.OP_AG_GEMM].beta_fusion, rel=1e-6)
    assert ag["fusion_mae_ms"]["aware"] < 1e-9 < ag["fusion_mae_ms"]["agnostic"]
    # ... so Algorithm 1 compares two exact predictions and is right every time.  (GEMM+ReduceScatter has no
    # transfer-carrying variant: its IntraFusion time is the fused kernel's, which Eq. 7 does not describe.)
    assert ag["selector_accuracy"] == 1.0


def test_calibration_round_trip_and_summary(tmp_path):
    report = gs.analyze_records(synthetic_records())
    path = tmp_path / "calib.json"
    path.write_text(json.dumps(gs.calibration_of(report, "synthetic, planted parameters")))
    calibs, provenance = gs.load_calibration(str(path))
    assert provenance == "synthetic, planted parameters" and sorted(calibs) == ["AG+GEMM", "GEMM+RS"]
    for name, cal in calibs.items():
        for field in gs.CALIB_FIELDS:
            assert getattr(cal, field) == report[name]["calib"][field]
    # the stored calibration drives the selector exactly as the in-memory one
    pr = api.make_problem(wl.OP_AG_GEMM, 8, 16384, 2048, 8192)
    a = api.compass_select(pr, calibs["AG+GEMM"])
    b = api.compass_select(pr, api.Calib(*[report["AG+GEMM"]["calib"][f] for f in gs.CALIB_FIELDS]))
    assert (a.strategy, a.d_star, a.t_star) == (b.strategy, b.d_star, b.t_star) and math.isfinite(a.t_star)
    text = gs.summary_markdown(report, "synthetic")
    assert "| Algorithm 1 picks the faster strategy | 100.0 % |" in text
    assert text.count("\n|") >= 12


@pytest.mark.gpu
def test_measure_a_few_small_cases(tmp_path):
    """`measure_cases` on three small cases of the grid: every timing present and positive, resumable."""
    small = [c for c in gs.grid(max_m=2048) if c["table_K"] == 4096 and c["table_N"] == 2048]
    cases = [small[0], small[-1], small[len(small) // 2]]
    out = tmp_path / "grid.jsonl"
    assert gs.measure_cases(cases, str(out), iters=2, log=lambda *a: None) == 3
    recs = [json.loads(line) for line in out.read_text().splitlines()]
    assert [gs.case_key(r) for r in recs] == [gs.case_key(c) for c in cases]
    for r in recs:
        assert r["fused_ms"] > 0 and set(r["decomp_ms"]) == {"1", "2", "4", "8", "16"}
        assert all(t > 0 for t in r["decomp_ms"].values())
        assert ("push_ms" in r) == (r["op"] == wl.OP_AG_GEMM)
    assert gs.measure_cases(cases, str(out), iters=2, log=lambda *a: None) == 0         # already in the file
