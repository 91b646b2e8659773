"""Host-side tests of the C ABI (no GPU): the library loads and exports every
declared symbol; the schedule, the models and the selector of the library
agree with the oracle; bad arguments are refused with the documented codes;
the launch plan keeps every rank's schedule order."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import OP_AG_GEMM, OP_GEMM_RS
from oracle import models as omo
from oracle.schedule import schedule as oracle_schedule
from paper_2609_10549_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "compass.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(compass_[a-z_0-9]+)\s*\(", header))
    assert declared == set(api.EXPORTS)
    lib = api.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header():
    assert C.sizeof(api.Problem) == 4 * 4 + 3 * 8 + 6 * 4
    assert api.Problem.b_layout.offset == 56
    assert C.sizeof(api.SchedEntry) == 32
    assert C.sizeof(api.Calib) == 64
    assert C.sizeof(api.Choice) == 8 + 6 * 8
    assert C.sizeof(api.PlanBlock) == 44
    assert C.sizeof(api.Mlp) == 2 * 4 + 3 * 8 + 4 * 4
    assert api.Mlp.M.offset == 8 and api.Mlp.activation.offset == 32


@pytest.mark.parametrize("op", [OP_AG_GEMM, OP_GEMM_RS])
@pytest.mark.parametrize("rings", [1, 2])
def test_schedule_bit_exact_against_oracle(op, rings):
    for P in range(1, api.MAX_P + 1):
        for rows in (rings, 6 * rings, 1024):
            M = P * rows
            got = api.compass_schedule(op, P, rings, M)
            want = oracle_schedule(op, P, rings, M)
            assert got.dtype == want.dtype and got.shape == want.shape
            assert np.array_equal(got, want), (op, P, rings, M)


def test_schedule_argument_errors():
    lib = api.lib()
    n = C.c_size_t(0)
    buf = (api.SchedEntry * 8)()
    f = lib.compass_schedule
    assert f(0, 2, 2, 512, buf, 8, None) == api.ERR_INVALID_ARG
    assert f(5, 2, 2, 512, buf, 8, C.byref(n)) == api.ERR_INVALID_ARG
    assert f(0, 0, 2, 512, buf, 8, C.byref(n)) == api.ERR_INVALID_ARG
    assert f(0, 2, 3, 512, buf, 8, C.byref(n)) == api.ERR_INVALID_ARG
    assert f(0, 17, 2, 17 * 2, buf, 8, C.byref(n)) == api.ERR_UNSUPPORTED
    assert f(0, 3, 2, 512, buf, 8, C.byref(n)) == api.ERR_SHAPE           # M % P
    assert f(0, 2, 2, 6, buf, 8, C.byref(n)) == api.ERR_SHAPE             # (M/P) % rings
    assert f(0, 2, 2, 0, buf, 8, C.byref(n)) == api.ERR_SHAPE
    assert f(0, 2, 2, 512, buf, 7, C.byref(n)) == api.ERR_BUFFER_TOO_SMALL and n.value == 8
    assert f(0, 2, 2, 512, None, 0, C.byref(n)) == api.OK and n.value == 8
    assert f(0, 2, 2, 512, buf, 8, C.byref(n)) == api.OK


pos = st.floats(min_value=1e-3, max_value=1e4, allow_nan=False, allow_infinity=False)


@settings(max_examples=300, deadline=None)
@given(pos, pos, st.floats(0.0, 3.0), st.floats(-0.1, 0.6), st.sampled_from([1, 2, 4, 8, 16]), st.booleans())
def test_decomposition_model_matches_oracle(tc, tm, a, b, d_max, printed):
    for d in (1, 2, 4, 8, 16):
        assert api.compass_model_decomp_time(tc, tm, a, b, d) == pytest.approx(omo.decomp_time(tc, tm, a, b, d),
                                                                               rel=1e-12)
    d_lib, x_lib = api.compass_model_optimal_degree(tc, tm, a, b, d_max, printed)
    assert d_lib == omo.optimal_degree(tc, tm, a, b, d_max, printed)
    x_ref = omo.d_continuous(tc, tm, a, b, printed)
    if x_ref is None:
        assert x_lib is None
    else:
        assert x_lib == pytest.approx(x_ref, rel=1e-12)


@settings(max_examples=200, deadline=None)
@given(pos, st.floats(0.0, 1e4), st.integers(1, 16), st.floats(0.0, 10.0), st.floats(0.0, 1e-5), st.floats(1.0, 1e9))
def test_fusion_model_matches_oracle(tc, tm, n, af, bf, vol):
    assert api.compass_model_fusion_time(tc, tm, n, af, bf, vol) == pytest.approx(
        omo.fusion_time(tc, tm, n, af, bf, vol), rel=1e-12)


@settings(max_examples=200, deadline=None)
@given(st.sampled_from([OP_AG_GEMM, OP_GEMM_RS]), st.sampled_from([1, 2, 4, 8]), st.sampled_from([8, 24, 56, 128, 1024]),
       st.sampled_from([64, 4096]), st.sampled_from([64, 1376, 8192]),
       st.floats(0.0, 50.0), st.floats(1e-13, 1e-9), st.floats(0.0, 50.0), st.floats(1e-10, 1e-6),
       st.floats(0.5, 1.5), st.floats(0.0, 0.2), st.floats(0.0, 10.0), st.floats(0.0, 1e-6))
def test_selector_matches_oracle(op, P, rows, N, K, ca, cb, ma, mb, ad, bd, af, bf):
    M = P * rows
    calib_o = omo.Calib(ca, cb, ma, mb, ad, bd, af, bf)
    want = omo.select(op, P, M, N, K, calib_o)
    got = api.compass_select(api.make_problem(op, P, M, N, K), api.Calib(ca, cb, ma, mb, ad, bd, af, bf))
    assert got.strategy == want.strategy and got.d_star == want.d_star
    for name_l, name_o in (("t_fusion", "t_fusion"), ("t_decomp", "t_decomp"), ("t_comp", "t_comp"),
                           ("t_comm", "t_comm"), ("lam", "lam"), ("t_star", "t_star")):
        assert getattr(got, name_l) == pytest.approx(getattr(want, name_o), rel=1e-12)


def test_selector_on_eq5_as_printed():
    """In the communication-bound regime (lambda < 1) the printed Eq. 5 and the regime-aware form pick different
    degrees; compass_select_ex runs Algorithm 1 on either, and both agree with the oracle."""
    P, M, N, K = 4, 4096, 1024, 1024
    flops, nbytes = 2.0 * P * M * N * K, 2.0 * P * M * K
    args = (0.0, 10.0 / flops, 0.0, 100.0 / nbytes, 0.9, 0.004, 50.0, 0.0)      # T_comp 10, T_comm 100: lambda = 0.1
    pr = api.make_problem(OP_AG_GEMM, P, M, N, K)
    aware = api.compass_select(pr, api.Calib(*args))
    printed = api.compass_select(pr, api.Calib(*args), eq5_as_printed=True)
    want_aware = omo.select(OP_AG_GEMM, P, M, N, K, omo.Calib(*args))
    want_printed = omo.select(OP_AG_GEMM, P, M, N, K, omo.Calib(*args), as_printed=True)
    assert (aware.d_star, printed.d_star) == (want_aware.d_star, want_printed.d_star)
    assert aware.d_star != printed.d_star
    assert aware.t_decomp == pytest.approx(want_aware.t_decomp, rel=1e-12)
    assert printed.t_decomp == pytest.approx(want_printed.t_decomp, rel=1e-12)
    assert aware.t_decomp <= printed.t_decomp            # the regime-aware degree is never the worse of the two here


def test_selector_hand_example_and_errors():
    P, M, N, K = 4, 4096, 1024, 1024
    cal = api.Calib(0.0, 250.0 / (2.0 * P * M * N * K), 0.0, 50.0 / (2.0 * P * M * K), 1.0, 0.01, 2.0, 0.0)
    c = api.compass_select(api.make_problem(OP_AG_GEMM, P, M, N, K), cal)
    assert c.d_star == 4 and c.t_decomp == pytest.approx(270.0) and c.t_fusion == pytest.approx(256.0)
    assert c.strategy == api.STRATEGY_INTRAFUSION
    lib = api.lib()
    out = api.Choice()
    pr = api.make_problem(OP_AG_GEMM, P, M, N, K)
    assert lib.compass_select(None, C.byref(cal), C.byref(out)) == api.ERR_INVALID_ARG
    assert lib.compass_select(C.byref(pr), None, C.byref(out)) == api.ERR_INVALID_ARG
    bad = api.make_problem(OP_AG_GEMM, 3, 4096, N, K)
    assert lib.compass_select(C.byref(bad), C.byref(cal), C.byref(out)) == api.ERR_SHAPE


def test_mlp_block_argument_checks_run_on_the_host():
    lib = api.lib()
    n = C.c_size_t(0)

    def code(**kw):
        base = dict(P=4, M=4096, hidden=1024, ffn=2048, activation=api.ACT_SWIGLU)
        base.update(kw)
        return lib.compass_mlp_workspace_bytes(C.byref(api.make_mlp(**base)), C.byref(n))

    assert code() == api.OK and n.value >= api.STATUS_BYTES
    # the workspace serves both kernels: at least what each needs on its own
    ag = api.make_problem(OP_AG_GEMM, 4, 4096, 2048, 1024)
    rs = api.make_problem(OP_GEMM_RS, 4, 4096, 1024, 1024, rs_variant=api.RS_RING_RMW)
    assert code(rs_variant=api.RS_RING_RMW) == api.OK
    assert n.value == max(api.compass_workspace_bytes(ag, api.WS_FUSED), api.compass_workspace_bytes(rs, api.WS_FUSED))
    assert lib.compass_mlp_workspace_bytes(None, C.byref(n)) == api.ERR_INVALID_ARG
    assert lib.compass_mlp_workspace_bytes(C.byref(api.make_mlp(4, 4096, 1024, 2048)), None) == api.ERR_INVALID_ARG
    assert code(activation=3) == api.ERR_INVALID_ARG
    assert code(P=0) == api.ERR_INVALID_ARG
    assert code(rings=3) == api.ERR_INVALID_ARG
    assert code(rs_variant=5) == api.ERR_INVALID_ARG
    assert code(P=3) == api.ERR_SHAPE                       # 4096 rows do not split over 3 ranks
    assert code(hidden=0) == api.ERR_SHAPE
    assert code(ffn=2056) == api.ERR_ALIGNMENT              # SwiGLU needs (gate, up) pairs and 16-byte rows of H
    assert code(ffn=2056, activation=api.ACT_GELU_TANH) == api.OK
    assert code(hidden=1020) == api.ERR_ALIGNMENT
    assert code(P=32, M=8192) == api.ERR_UNSUPPORTED
    assert code(b_layout=api.B_KN) == api.OK
    assert code(b_layout=2) == api.ERR_INVALID_ARG
    # the block itself refuses NULL pointer arrays before any CUDA call
    mp = api.make_mlp(4, 4096, 1024, 2048)
    assert lib.compass_mlp_block(C.byref(mp), None, None, None, None, None, None, 0, None) == api.ERR_INVALID_ARG
    assert lib.compass_mlp_block(None, None, None, None, None, None, None, 0, None) == api.ERR_INVALID_ARG


def test_read_kernel_clock_rejects_null_arguments_before_touching_a_device():
    lib = api.lib()
    cycles, ns = C.c_uint64(7), C.c_uint64(7)
    assert lib.compass_read_kernel_clock(None, None, C.byref(cycles), C.byref(ns)) == api.ERR_INVALID_ARG
    fake_ws = C.c_void_p(4096)                       # never dereferenced: the NULL checks come first
    assert lib.compass_read_kernel_clock(fake_ws, None, None, C.byref(ns)) == api.ERR_INVALID_ARG
    assert lib.compass_read_kernel_clock(fake_ws, None, C.byref(cycles), None) == api.ERR_INVALID_ARG
    assert (cycles.value, ns.value) == (7, 7)


def test_calibration_matches_oracle():
    alpha, beta = 1.07, 0.025
    tc, tm, d, t = [], [], [], []
    rng = np.random.default_rng(0)
    for (c, m) in [(100.0, 40.0), (30.0, 90.0), (55.0, 55.0)]:
        for dd in (2, 4, 8, 16):
            tc.append(c); tm.append(m); d.append(dd)
            t.append(omo.decomp_time(c, m, alpha, beta, dd) * (1 + 0.01 * rng.standard_normal()))
    a_lib, b_lib = api.compass_calib_fit_decomp(tc, tm, d, t)
    a_ref, b_ref = omo.fit_decomp_overhead(list(zip(tc, tm, d, t)))
    assert a_lib == pytest.approx(a_ref, rel=1e-10) and b_lib == pytest.approx(b_ref, rel=1e-10)
    n = [4, 8, 4, 8]; vol = [1e6, 4e6, 2e6, 8e6]; c4 = [100.0, 30.0, 55.0, 70.0]; m4 = [40.0, 90.0, 55.0, 10.0]
    tf = [omo.fusion_time(c, m, nn, 3.0, 2e-6, v) * (1 + 0.01 * rng.standard_normal())
          for c, m, nn, v in zip(c4, m4, n, vol)]
    assert api.compass_calib_fit_line([1.0, 2.0, 4.0], [3.5, 5.0, 8.0]) == (pytest.approx(omo.ols([1.0, 2.0, 4.0], [3.5, 5.0, 8.0])[0]),
                                                                            pytest.approx(omo.ols([1.0, 2.0, 4.0], [3.5, 5.0, 8.0])[1]))
    assert api.compass_calib_fit_line([2.0, 2.0], [1.0, 3.0]) == (2.0, 0.0)
    a_lib, b_lib = api.compass_calib_fit_fusion(c4, m4, n, vol, tf)
    a_ref, b_ref = omo.fit_fusion_overhead(list(zip(c4, m4, n, vol, tf)))
    assert a_lib == pytest.approx(a_ref, rel=1e-9) and b_lib == pytest.approx(b_ref, rel=1e-9)


def _codes(pr, which=api.WS_FUSED):
    n = C.c_size_t(0)
    return api.lib().compass_workspace_bytes(C.byref(pr), which, C.byref(n)), n.value


def test_problem_validation_codes():
    ok = dict(op=OP_AG_GEMM, P=4, M=4096, N=3072, K=4096)
    assert _codes(api.make_problem(**ok))[0] == api.OK
    assert _codes(api.make_problem(**{**ok, "op": 9}))[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**{**ok, "b_layout": api.B_KN}))[0] == api.OK
    assert _codes(api.make_problem(**{**ok, "b_layout": 2}))[0] == api.ERR_INVALID_ARG
    # contributors fused per read-modify-write pass: ring variants of GEMM+ReduceScatter only, a divisor of P
    assert _codes(api.make_problem(**ok, ring_group=2))[0] == api.ERR_INVALID_ARG
    rs = dict(op=OP_GEMM_RS, P=8, M=8192, N=4096, K=1376)
    assert _codes(api.make_problem(**rs, ring_group=1))[0] == api.OK
    assert _codes(api.make_problem(**rs, ring_group=2))[0] == api.ERR_INVALID_ARG                   # segmented K
    for variant in (api.RS_RING_RMW, api.RS_RING_RMW_F32):
        assert [_codes(api.make_problem(**rs, rs_variant=variant, ring_group=g))[0] for g in (0, 1, 2, 4, 8)] == [api.OK] * 5
        assert [_codes(api.make_problem(**rs, rs_variant=variant, ring_group=g))[0] for g in (-1, 3, 16)] == [api.ERR_INVALID_ARG] * 3
    assert _codes(api.make_problem(**{**ok, "P": 0}))[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**ok, rings=3))[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**{**ok, "P": 32, "M": 4096}))[0] == api.ERR_UNSUPPORTED
    assert _codes(api.make_problem(**ok, dtype=1))[0] == api.ERR_UNSUPPORTED
    assert _codes(api.make_problem(**{**ok, "M": 4098}))[0] == api.ERR_SHAPE
    assert _codes(api.make_problem(**{**ok, "P": 4, "M": 4 * 7}))[0] == api.ERR_SHAPE      # odd rows, two rings
    assert _codes(api.make_problem(**{**ok, "K": 0}))[0] == api.ERR_SHAPE
    assert _codes(api.make_problem(**{**ok, "K": 4100}))[0] == api.ERR_ALIGNMENT           # row pitch % 16 bytes
    assert _codes(api.make_problem(**{**ok, "N": 3076}))[0] == api.ERR_ALIGNMENT
    assert _codes(api.make_problem(**ok, d=0), api.WS_DECOMP)[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**ok, d=3), api.WS_DECOMP)[0] == api.ERR_SHAPE
    assert _codes(api.make_problem(**ok), 7)[0] == api.ERR_INVALID_ARG
    rs = api.make_problem(OP_GEMM_RS, 8, 8192, 4096, 1376, rs_variant=5)
    assert _codes(rs)[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**ok, order=2))[0] == api.ERR_INVALID_ARG
    assert _codes(api.make_problem(**ok, copy_mode=2))[0] == api.ERR_INVALID_ARG


def test_workspace_sizes():
    ag = api.make_problem(OP_AG_GEMM, 4, 4096, 3072, 4096, d=4)
    assert _codes(ag) == (api.OK, api.STATUS_BYTES)
    assert _codes(ag, api.WS_DECOMP) == (api.OK, api.STATUS_BYTES + 4 * 4096 * 4096 * 2)
    rs = api.make_problem(OP_GEMM_RS, 4, 4096, 4096, 1024, d=2)
    assert _codes(rs, api.WS_DECOMP) == (api.OK, api.STATUS_BYTES + 4 * 4096 * 4096 * 2)
    assert _codes(ag, api.WS_PUSH) == (api.OK, api.STATUS_BYTES + 256 + 4 * 4096 * 4096 * 2)     # 32 flags + 4 gather buffers
    assert _codes(rs, api.WS_PUSH)[0] == api.ERR_INVALID_ARG
    ring = api.make_problem(OP_GEMM_RS, 8, 8192, 4096, 1376, rs_variant=api.RS_RING_RMW)
    # 16 partitions x 4 fragments of 128 rows x 16 column tiles: one counter and one BF16 fragment (128 x 256) of
    # running sum each
    counters = 16 * 4 * 16
    assert _codes(ring) == (api.OK, api.STATUS_BYTES + counters * 4 + counters * 128 * 256 * 2)
    # the same with the running sum in FP32
    ring32 = api.make_problem(OP_GEMM_RS, 8, 8192, 4096, 1376, rs_variant=api.RS_RING_RMW_F32)
    assert _codes(ring32) == (api.OK, api.STATUS_BYTES + counters * 4 + counters * 128 * 256 * 4)
    # ragged: 2 partitions x P = 3 of 136 rows (2 fragments) x 520 columns (3 tiles); counters padded to 256 bytes
    ragged = api.make_problem(OP_GEMM_RS, 3, 3 * 272, 520, 64, rs_variant=api.RS_RING_RMW)
    assert _codes(ragged) == (api.OK, api.STATUS_BYTES + 256 + 36 * 128 * 256 * 2)
    assert _codes(api.make_problem(OP_GEMM_RS, 8, 8192, 4096, 1376, rs_variant=3))[0] == api.ERR_INVALID_ARG
    plan32 = api.compass_launch_plan(ring32)
    assert [(b.rank, b.step, b.ring) for b in plan32] == [(b.rank, b.step, b.ring) for b in api.compass_launch_plan(ring)]


def test_fused_calls_refuse_bad_arguments_before_touching_the_gpu():
    lib = api.lib()
    pr = api.make_problem(OP_AG_GEMM, 2, 512, 1024, 1024)
    good = (C.c_void_p * 2)(0x1000, 0x2000)
    null = (C.c_void_p * 2)(0x1000, 0)
    odd = (C.c_void_p * 2)(0x1000, 0x2008)
    ws = C.c_void_p(0x10000)
    assert lib.compass_ag_gemm(None, good, good, good, ws, 256, None) == api.ERR_INVALID_ARG
    assert lib.compass_ag_gemm(C.byref(pr), None, good, good, ws, 256, None) == api.ERR_INVALID_ARG
    assert lib.compass_ag_gemm(C.byref(pr), good, null, good, ws, 256, None) == api.ERR_INVALID_ARG
    assert lib.compass_ag_gemm(C.byref(pr), good, good, odd, ws, 256, None) == api.ERR_ALIGNMENT
    assert lib.compass_ag_gemm(C.byref(pr), good, good, good, None, 256, None) == api.ERR_INVALID_ARG
    assert lib.compass_ag_gemm(C.byref(pr), good, good, good, C.c_void_p(0x10010), 256, None) == api.ERR_ALIGNMENT
    assert lib.compass_ag_gemm(C.byref(pr), good, good, good, ws, 255, None) == api.ERR_BUFFER_TOO_SMALL
    # the wrong entry point for the pattern
    assert lib.compass_gemm_rs(C.byref(pr), good, good, good, ws, 256, None) == api.ERR_INVALID_ARG
    dec = api.make_problem(OP_AG_GEMM, 2, 512, 1024, 1024, d=32)
    assert lib.compass_decomp(C.byref(dec), good, good, good, ws, 1 << 40, None, None) == api.ERR_UNSUPPORTED
    dec = api.make_problem(OP_AG_GEMM, 2, 512, 1024, 1024, d=2)
    assert lib.compass_decomp(C.byref(dec), good, good, good, ws, 1024, None, None) == api.ERR_BUFFER_TOO_SMALL
    need = C.c_size_t(0)
    assert lib.compass_fused_host(C.byref(pr), None, None, None, None, 0, C.byref(need), None, 0, None) == api.OK
    assert need.value == 2 * (256 * 1024 * 2 + 1024 * 1024 * 2 + 512 * 1024 * 2)
    assert api.status_string(api.ERR_TIMEOUT) == "device-side wait timed out"


@pytest.mark.parametrize("order", [api.ORDER_RANK_MAJOR, api.ORDER_STEP_MAJOR])
@pytest.mark.parametrize("P,rings", [(1, 2), (2, 2), (4, 2), (8, 2), (4, 1), (16, 2)])
def test_ag_launch_plan_keeps_each_ranks_schedule_order(P, rings, order):
    M, N, K = P * 512, 1024, 256
    pr = api.make_problem(OP_AG_GEMM, P, M, N, K, rings=rings, order=order)
    plan = api.compass_launch_plan(pr)
    table = oracle_schedule(OP_AG_GEMM, P, rings, M)
    assert len(plan) == len(table)
    m = M // P
    for r in range(P):
        mine = [b for b in plan if b.rank == r]
        want = table[table[:, 0] == r]
        assert [(b.step, b.ring, b.part) for b in mine] == [(int(e[1]), int(e[2]), int(e[3])) for e in want]
        for b, e in zip(mine, want):
            # the A rows are read from the shard of the chunk's owner: gather by address
            assert b.a_tensor == e[4] and b.a_row_begin == e[6] - e[4] * m and b.rows == e[7]
            assert b.out_tensor == r and b.out_row_begin == e[6]
    # how the ranks' sequences are merged, and tiles are consecutive
    if order == api.ORDER_STEP_MAJOR:
        assert [b.step for b in plan] == sorted(b.step for b in plan)
    else:
        assert [b.rank for b in plan] == sorted(b.rank for b in plan)
    tile_rows = 256 if M // P // rings >= 256 else 128
    first = 0
    for b in plan:
        assert b.first_tile == first and b.tile_count == math.ceil(b.rows / tile_rows) * math.ceil(N / 256)
        first += b.tile_count


@pytest.mark.parametrize("P,rings", [(2, 2), (4, 2), (8, 2), (4, 1)])
def test_rs_launch_plans(P, rings):
    M, N, K = P * 512, 1024, 256
    table = oracle_schedule(OP_GEMM_RS, P, rings, M)
    m = M // P
    seg = api.compass_launch_plan(api.make_problem(OP_GEMM_RS, P, M, N, K, rings=rings))
    assert len(seg) == rings * P
    for b in seg:
        chunk = b.part // rings
        assert b.out_tensor == chunk and b.a_row_begin == chunk * m + b.ring * (m // rings)
        assert b.out_row_begin == b.ring * (m // rings)
    ring = api.compass_launch_plan(api.make_problem(OP_GEMM_RS, P, M, N, K, rings=rings, rs_variant=api.RS_RING_RMW))
    assert len(ring) == len(table)
    for r in range(P):
        mine = [b for b in ring if b.rank == r]
        want = table[table[:, 0] == r]
        assert [(b.step, b.ring, b.part) for b in mine] == [(int(e[1]), int(e[2]), int(e[3])) for e in want]
        for b, e in zip(mine, want):
            assert b.a_tensor == r and b.a_row_begin == e[6] and b.out_tensor == e[4]
    # contributor s of a partition precedes contributor s+1 in the launch
    pos_of = {(b.part, b.step): i for i, b in enumerate(ring)}
    for (part, step), i in pos_of.items():
        if step > 0:
            assert pos_of[(part, step - 1)] < i
    # groups of G contributors: one block per (partition, group), named after the group's first contributor
    who = {(int(e[3]), int(e[1])): int(e[0]) for e in table}                # (part, step) -> rank
    for G in [g for g in (2, 4, 8) if P % g == 0]:
        grouped = api.compass_launch_plan(api.make_problem(OP_GEMM_RS, P, M, N, K, rings=rings, rs_variant=api.RS_RING_RMW,
                                                           ring_group=G))
        assert len(grouped) == len(table) // G
        assert sorted((b.part, b.step) for b in grouped) == sorted((part, s) for part in range(rings * P) for s in range(0, P, G))
        for i, b in enumerate(grouped):
            assert b.rank == who[(b.part, b.step)] and b.a_tensor == b.rank
            assert b.out_tensor == b.part // rings and b.rows == m // rings
        pos_of = {(b.part, b.step): i for i, b in enumerate(grouped)}
        for (part, step), i in pos_of.items():
            if step > 0:
                assert pos_of[(part, step - G)] < i
