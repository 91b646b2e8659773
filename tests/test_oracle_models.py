"""Pins for the oracle's performance models and selector (CPU only).

The paper prints no calibrated parameters, so these are the algebraic facts it
states (Section IV-B/IV-C/V-B, Algorithm 1) plus hand-evaluated examples.
"""
import math

import pytest
from hypothesis import given, settings, strategies as st

from oracle import OP_AG_GEMM, OP_GEMM_RS
from oracle import models as mo

pos = st.floats(min_value=1e-3, max_value=1e4, allow_nan=False, allow_infinity=False)


@given(pos, pos, st.floats(0.0, 3.0), st.floats(0.0, 1.0))
def test_sequential_case_is_sum(tc, tm, a, b):
    # Section IV-C: at d = 1 the overlapped term vanishes
    assert mo.decomp_time(tc, tm, a, b, 1) == pytest.approx(tc + tm, rel=1e-15)


@given(pos, pos, st.sampled_from([2, 4, 8, 16]))
def test_unit_overhead_is_the_overhead_agnostic_model(tc, tm, d):
    # Section IV-B: eta = 1 degenerates to (d-1) stages + first/last sub-operator
    want = (d - 1) * max(tc, tm) / d + (tc + tm) / d
    assert mo.decomp_time(tc, tm, 1.0, 0.0, d) == pytest.approx(want, rel=1e-14)


def test_hand_evaluated_decomposition_example():
    tc, tm, a, b = 250.0, 50.0, 1.0, 0.01
    # (d-1) * 250/d * (1 + 0.01 d) + 300/d, evaluated by hand
    assert mo.decomp_time(tc, tm, a, b, 1) == pytest.approx(300.0)
    assert mo.decomp_time(tc, tm, a, b, 2) == pytest.approx(277.5)
    assert mo.decomp_time(tc, tm, a, b, 4) == pytest.approx(270.0)
    assert mo.decomp_time(tc, tm, a, b, 8) == pytest.approx(273.75)
    assert mo.decomp_time(tc, tm, a, b, 16) == pytest.approx(290.625)
    # Eq. 5: sqrt((1 - 1 + 1/5)/0.01) = sqrt(20) = 4.47 -> 4
    assert mo.d_continuous(tc, tm, a, b) == pytest.approx(math.sqrt(20.0))
    assert mo.d_continuous(tc, tm, a, b, as_printed=True) == pytest.approx(math.sqrt(20.0))
    assert mo.d_candidate(tc, tm, a, b) == 4
    assert mo.optimal_degree(tc, tm, a, b) == 4
    assert mo.optimal_degree(tc, tm, a, b, d_max=2) == 2


def test_printed_formula_is_the_compute_bound_regime():
    # lambda < 1: the derivative condition uses lambda, the printed formula 1/lambda
    tc, tm, a, b = 50.0, 250.0, 1.0, 0.01
    assert mo.d_continuous(tc, tm, a, b) == pytest.approx(math.sqrt(0.2 / 0.01))
    assert mo.d_continuous(tc, tm, a, b, as_printed=True) == pytest.approx(math.sqrt(5.0 / 0.01))


@pytest.mark.parametrize("x,want", [(1.0, 1), (1.4, 1), (1.42, 2), (2.0, 2), (2.82, 2), (2.83, 4),
                                    (5.6, 4), (5.7, 8), (11.3, 8), (11.4, 16), (100.0, 128), (0.3, 1)])
def test_nearest_power_of_two_is_log_nearest(x, want):
    assert mo.nearest_power_of_two(x) == want


@settings(max_examples=300, deadline=None)
@given(pos, pos, st.floats(0.2, 1.8), st.floats(1e-4, 0.5))
def test_analytic_candidate_minimises_over_powers_of_two(tc, tm, a, b):
    """Section IV-C: the model is convex in d, so the (log-nearest) rounding of
    the stationary point is the best power of two in the candidate set."""
    cand = mo.d_candidate(tc, tm, a, b)
    times = {d: mo.decomp_time(tc, tm, a, b, d) for d in mo.CANDIDATE_DEGREES}
    best = min(times.values())
    assert times[cand] <= best * (1 + 1e-9) + 1e-12
    # Eq. 4: the final degree never loses to sequential execution
    d_final = mo.optimal_degree(tc, tm, a, b)
    assert d_final in (1,) + mo.CANDIDATE_DEGREES
    t_seq = tc + tm
    assert mo.decomp_time(tc, tm, a, b, d_final) <= t_seq * (1 + 1e-12)
    if d_final == 1:
        assert not (times[cand] < mo.decomp_time(tc, tm, a, b, 1))


def test_degenerate_inputs():
    assert mo.optimal_degree(10.0, 0.0, 1.0, 0.01) == 1          # nothing to hide
    assert mo.d_continuous(10.0, 5.0, 1.0, 0.0) is None
    assert mo.d_continuous(10.0, 5.0, 3.0, 0.1) is None           # radicand <= 0
    # no analytic candidate: enumerate.  eta = 1 exactly -> deeper is better up to 16
    assert mo.d_candidate(100.0, 100.0, 1.0, 0.0) == 16
    assert mo.optimal_degree(100.0, 100.0, 1.0, 0.0) == 16
    # overhead so large that decomposition never pays
    assert mo.optimal_degree(100.0, 1.0, 5.0, 1.0) == 1
    assert mo.d_candidate(1.0, 1.0, 1.0, 0.1, d_max=1) is None
    assert mo.optimal_degree(1.0, 1.0, 1.0, 0.1, d_max=1) == 1


def test_fusion_model_special_cases():
    # no communication: compute plus (n-1) synchronisation points
    assert mo.fusion_time(80.0, 0.0, 4, 2.0, 1e-3, 1000.0) == pytest.approx(80.0 + 3 * (2.0 + 1.0))
    # no overhead and communication hidden: exactly the compute time
    assert mo.fusion_time(80.0, 30.0, 4, 0.0, 0.0, 1.0) == pytest.approx(80.0)
    # communication-bound: (n-1) comm steps plus the exposed first chunk
    assert mo.fusion_time(40.0, 90.0, 4, 0.0, 0.0, 1.0) == pytest.approx(90.0 + 10.0)
    # one GPU: nothing to overlap, no synchronisation point
    assert mo.fusion_time(50.0, 0.0, 1, 3.0, 1.0, 10.0) == pytest.approx(50.0)
    # hand-evaluated: sum_{i=2..4} max(62.5, 16.67) + 62.5 + 3*2 = 256
    assert mo.fusion_time(250.0, 50.0, 4, 2.0, 0.0, 123.0) == pytest.approx(256.0)
    assert mo.fusion_overhead(8, 1.5, 2e-6, 1e6) == pytest.approx(7 * 3.5)


def test_message_volume_follows_eq8():
    assert mo.message_volume(OP_AG_GEMM, 4096, 3072, 4096) == 4096 * 4096
    assert mo.message_volume(OP_GEMM_RS, 8192, 4096, 1376) == 8192 * 4096


def _calib(alpha_f):
    # T_comp = 250, T_comm = 50 for the workload below
    P, M, N, K = 4, 4096, 1024, 1024
    return (P, M, N, K), mo.Calib(comp_a=0.0, comp_b=250.0 / mo.workload_flops(P, M, N, K),
                                  comm_a=0.0, comm_b=50.0 / mo.workload_comm_bytes(OP_AG_GEMM, P, M, N, K),
                                  alpha_decomp=1.0, beta_decomp=0.01, alpha_fusion=alpha_f, beta_fusion=0.0)


def test_selector_follows_algorithm_1():
    shape, calib = _calib(2.0)
    c = mo.select(OP_AG_GEMM, *shape, calib)
    assert c.t_comp == pytest.approx(250.0) and c.t_comm == pytest.approx(50.0) and c.lam == pytest.approx(5.0)
    assert c.d_star == 4 and c.t_decomp == pytest.approx(270.0) and c.t_fusion == pytest.approx(256.0)
    assert c.strategy == mo.STRATEGY_INTRAFUSION and c.t_star == pytest.approx(256.0)
    shape, calib = _calib(7.0)                 # 250 + 21 = 271 > 270
    c = mo.select(OP_AG_GEMM, *shape, calib)
    assert c.strategy == mo.STRATEGY_INTERDECOM and c.t_star == pytest.approx(270.0)


def test_selector_tie_goes_to_interdecom():
    # alpha_f chosen so that T_fusion == T_decomp exactly: 250 + 3*alpha_f = 270
    shape, calib = _calib(20.0 / 3.0)
    c = mo.select(OP_AG_GEMM, *shape, calib)
    if c.t_fusion == c.t_decomp:
        assert c.strategy == mo.STRATEGY_INTERDECOM
    # an exactly representable tie
    calib = mo.Calib(comp_a=8.0, comp_b=0.0, comm_a=0.0, comm_b=0.0, alpha_decomp=1.0, beta_decomp=0.1)
    c = mo.select(OP_GEMM_RS, 2, 64, 64, 64, calib)
    assert c.d_star == 1 and c.t_fusion == c.t_decomp == 8.0 and c.strategy == mo.STRATEGY_INTERDECOM


def test_max_degree():
    assert mo.max_degree(4096, 4) == 16
    assert mo.max_degree(4 * 24, 4) == 8
    assert mo.max_degree(4 * 7, 4) == 1
    assert mo.max_degree(4 * 64, 4) == 16


def test_calibration_recovers_planted_parameters():
    alpha, beta = 1.1, 0.03
    samples = []
    for (tc, tm) in [(100.0, 40.0), (30.0, 90.0), (55.0, 55.0)]:
        for d in (2, 4, 8, 16):
            samples.append((tc, tm, d, mo.decomp_time(tc, tm, alpha, beta, d)))
    a, b = mo.fit_decomp_overhead(samples)
    assert a == pytest.approx(alpha, rel=1e-10) and b == pytest.approx(beta, rel=1e-10)
    af, bf = 3.0, 2e-6
    fs = [(tc, tm, n, vol, mo.fusion_time(tc, tm, n, af, bf, vol))
          for (tc, tm, n, vol) in [(100.0, 40.0, 4, 1e6), (30.0, 90.0, 8, 4e6), (55.0, 55.0, 4, 2e6)]]
    a, b = mo.fit_fusion_overhead(fs)
    assert a == pytest.approx(af, rel=1e-9) and b == pytest.approx(bf, rel=1e-9)
    assert mo.ols([1.0, 2.0, 3.0], [3.0, 5.0, 7.0]) == (pytest.approx(1.0), pytest.approx(2.0))
    assert mo.ols([2.0, 2.0], [1.0, 3.0]) == (2.0, 0.0)


def test_table_iv_grid_counts():
    from tests.test_oracle_schedule import paper_pins
    pins = paper_pins()
    K = (4096, 8192, 16384); N = (2048, 4096, 8192, 16384); W = (4, 8)
    M = (2048, 4096, 8192, 12288, 16384, 32768); pat = (OP_AG_GEMM, OP_GEMM_RS)
    grid = [(k, n, w, m, p) for k in K for n in N for w in W for m in M for p in pat]
    assert len(grid) == pins["grid_cases"]
    assert sum(1 for g in grid if g[4] == OP_AG_GEMM) == pins["grid_cases_ag"]
    assert sum(1 for g in grid if g[4] == OP_AG_GEMM and g[2] == 8) == pins["grid_cases_ag_tp8"]
