"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.

Acceptance (every element of every rank's output):
    |gpu - ref| <= 1e-2 * max|ref| + 1e-3         (BF16 output, FP32 accumulate)
plus RMS error <= 2^-8 of the reference RMS (oracle.compare).  Schedules are
compared bit-exactly.  Small cases are checked element by element; the
full-size configurations on a row sample (rows next to every partition and
tile boundary plus 1 % random rows, full width)."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import operators as ops
from oracle.schedule import schedule as oracle_schedule
from paper_2609_10549_b200 import api
from paper_2609_10549_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def check_all(outs, refs, what):
    for r, (got, ref) in enumerate(zip(outs, refs)):
        rep = compare.check(got, ref)
        assert rep.ok, f"{what} rank {r}: {rep}"


def small(op, P, m, N, K, seed=1, dist=1.0):
    return wl.Workload(f"small-{op}-{P}-{m}-{N}-{K}", op, P=P, M=P * m, N=N, K=K,
                       a_dist=("normal", 1.0), b_dist=("normal", dist), seed=seed)


def test_library_was_loaded_and_counts_launches():
    before = api.kernel_launch_count()
    w = small(wl.OP_AG_GEMM, 1, 128, 256, 64)
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B)
    assert status == (api.OK, 0) and guards
    assert api.kernel_launch_count() == before + 1
    check_all(outs, ops.ag_gemm(A, B), w.name)


def test_kernel_clock_record_is_plausible():
    """CTA 0 records its cycles and nanoseconds: their ratio must be an SM clock a B200 can have."""
    w = small(wl.OP_AG_GEMM, 4, 512, 1024, 2048)
    A_bits, B_bits = wl.make_inputs(w)
    pr = api.make_problem(w.op, w.P, w.M, w.N, w.K)
    A, B = gu.device_inputs(A_bits, B_bits)
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr)
    assert api.compass_read_kernel_clock(ws) == (0, 0)
    api.compass_ag_gemm(pr, A, B, [o.view for o in outs], ws)
    cycles, ns = api.compass_read_kernel_clock(ws)
    assert cycles > 0 and ns > 0
    assert 300.0 < cycles / ns * 1e3 < 2500.0          # MHz
    assert api.compass_read_status(ws) == (api.OK, 0)


def test_config1_ag_gemm_full():
    w = wl.C1_AG
    A, B = wl.make_inputs(w)
    assert np.array_equal(api.compass_schedule(w.op, w.P, 2, w.M), oracle_schedule(w.op, w.P, 2, w.M))
    outs, status, guards = gu.run_fused(w, A, B)
    assert status == (api.OK, 0) and guards
    check_all(outs, ops.ag_gemm(A, B), w.name)


# (P, rows per rank, N, K, rings): several tiles, ragged tails in M, N and K,
# partitions smaller than a tile, K shorter than one k-block, odd P.
AG_SHAPES = [
    (1, 128, 256, 64, 2), (1, 256, 512, 128, 1), (2, 256, 256, 256, 2), (2, 144, 264, 72, 2),
    (3, 272, 520, 1376, 2), (4, 512, 768, 512, 2), (4, 384, 1024, 320, 1), (8, 80, 200, 8, 2),
    (5, 6, 8, 16, 2), (8, 256, 512, 192, 2), (16, 32, 64, 64, 2),
]


@pytest.mark.parametrize("P,m,N,K,rings", AG_SHAPES)
def test_ag_gemm_small_shapes(P, m, N, K, rings):
    w = small(wl.OP_AG_GEMM, P, m, N, K)
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rings=rings)
    assert status == (api.OK, 0) and guards
    check_all(outs, ops.ag_gemm(A, B, rings=rings), w.name)


RS_SHAPES = [
    (1, 128, 256, 64, 2), (2, 256, 256, 256, 2), (2, 144, 264, 72, 2), (3, 272, 520, 344, 2),
    (4, 512, 768, 512, 2), (4, 384, 1024, 320, 1), (8, 80, 200, 8, 2), (8, 256, 512, 1376, 2), (5, 6, 8, 16, 2),
]


@pytest.mark.parametrize("P,m,N,K,rings", RS_SHAPES)
def test_gemm_rs_small_shapes(P, m, N, K, rings):
    w = small(wl.OP_GEMM_RS, P, m, N, K, dist=0.05)
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rings=rings)
    assert status == (api.OK, 0) and guards
    check_all(outs, ops.gemm_rs(A, B, rings=rings), w.name)


# Enough 512-row partitions to fill whole waves of CTA pairs with 512x256 tiles and leave a
# tail of 256x256 tiles, with ragged N (2568 = 10 tiles + 8 columns) and a K tail; checked
# element by element.
@pytest.mark.parametrize("op,P,m,N,K,order", [
    (wl.OP_AG_GEMM, 4, 1024, 2568, 200, api.ORDER_RANK_MAJOR),
    (wl.OP_AG_GEMM, 4, 1024, 2568, 72, api.ORDER_STEP_MAJOR),
    (wl.OP_GEMM_RS, 8, 1024, 2568, 88, api.ORDER_RANK_MAJOR),
    (wl.OP_AG_GEMM, 2, 1536, 5128, 64, api.ORDER_RANK_MAJOR),      # 768-row partitions: 512-row tiles do not divide them
    # k-stage counts around the point where the two accumulators of a 512x256 tile start to be
    # issued skewed at the tile's ends (5, 6 and 7 stages, the last one partial; then a long loop)
    (wl.OP_AG_GEMM, 4, 1024, 2568, 320, api.ORDER_RANK_MAJOR),
    (wl.OP_AG_GEMM, 4, 1024, 2568, 384, api.ORDER_RANK_MAJOR),
    (wl.OP_AG_GEMM, 4, 1024, 2568, 424, api.ORDER_STEP_MAJOR),
    (wl.OP_AG_GEMM, 4, 1024, 2568, 1032, api.ORDER_RANK_MAJOR),
    (wl.OP_GEMM_RS, 4, 1024, 2568, 104, api.ORDER_RANK_MAJOR),     # 4 segments x 2 stages, every segment with a partial stage
])
def test_big_and_small_tiles_in_one_launch(op, P, m, N, K, order):
    w = small(op, P, m, N, K, dist=0.05)
    A_bits, B_bits = wl.make_inputs(w)
    pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, order=order)
    A, B = gu.device_inputs(A_bits, B_bits)
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr)
    (api.compass_ag_gemm if op == wl.OP_AG_GEMM else api.compass_gemm_rs)(pr, A, B, [o.view for o in outs], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    assert all(o.guards_intact() for o in outs)
    refs = ops.ag_gemm(A_bits, B_bits) if op == wl.OP_AG_GEMM else ops.gemm_rs(A_bits, B_bits)
    check_all([o.bits() for o in outs], refs, w.name)


@pytest.mark.parametrize("op", [wl.OP_AG_GEMM, wl.OP_GEMM_RS])
def test_integer_inputs_are_reproduced_exactly(op):
    """Small-integer inputs make every partial sum exact in FP32 and every
    result exactly representable in BF16 after at most one rounding, so a
    misplaced tile, row or k-slice shows up as an exact mismatch."""
    w = wl.Workload("ints", op, P=4, M=4 * 256, N=512, K=192)
    A, B = wl.make_structured_inputs(w, "index")
    outs, status, guards = gu.run_fused(w, A, B)
    assert status == (api.OK, 0) and guards
    refs = ops.ag_gemm(A, B) if op == wl.OP_AG_GEMM else ops.gemm_rs(A, B)
    for got, ref in zip(outs, refs):
        assert np.array_equal(ops.bf16_bits_to_f64(got), ops.f64_to_bf16_f64(ref))


def _sampled_ag(w, rings=2):
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rings=rings)
    assert status == (api.OK, 0) and guards
    rows = gu.sample_rows(w.M, w.P, rings)
    refs = ops.ag_gemm(A, B, rings=rings, rows=rows)
    for r in range(w.P):
        assert not np.any((outs[r] & 0x7F80) == 0x7F80), "NaN/Inf or unwritten output"
        rep = compare.check(outs[r][rows], refs[r])
        assert rep.ok, f"{w.name} rank {r}: {rep}"


def _sampled_rs(w, rings=2, rs_variant=api.RS_SEGMENTED_K):
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rings=rings, rs_variant=rs_variant)
    assert status == (api.OK, 0) and guards
    rows = gu.sample_rows(w.M, w.P, rings)
    found = ops.gemm_rs_rows(A, B, rows, rings=rings)
    assert sorted(found) == list(range(w.P))
    for c, (local, ref) in found.items():
        assert not np.any((outs[c] & 0x7F80) == 0x7F80), "NaN/Inf or unwritten output"
        rep = compare.check(outs[c][local], ref)
        assert rep.ok, f"{w.name} chunk {c}: {rep}"


def test_config2_ag_gemm_full_size_sampled():
    _sampled_ag(wl.C2_AG)


def test_config3_gemm_rs_full_size_sampled():
    _sampled_rs(wl.C3_RS)


def test_config4_gemm_rs_full_size_sampled():
    _sampled_rs(wl.C4_RS)


# The two operators of the benchmark step, in the configuration bench.py times, every element of every rank.
def test_config2_ag_gemm_every_element():
    w = wl.C2_AG
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B)
    assert status == (api.OK, 0) and guards
    for r in range(w.P):                                   # one rank at a time keeps the FP64 reference at 100 MB
        (ref,) = ops.ag_gemm(A, B, ranks=[r])
        rep = compare.check(outs[r], ref)
        assert rep.ok and rep.frac_within_1ulp > 0.999, f"{w.name} rank {r}: {rep}"


def test_config3_gemm_rs_every_element():
    w = wl.C3_RS
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B)
    assert status == (api.OK, 0) and guards
    for c in range(w.P):
        (ref,) = ops.gemm_rs(A, B, chunks=[c])
        rep = compare.check(outs[c], ref)
        assert rep.ok and rep.frac_within_1ulp > 0.999, f"{w.name} chunk {c}: {rep}"


def test_config5_ag_gemm_full_size_sampled():
    _sampled_ag(wl.C5_AG)


def test_config5_gemm_rs_full_size_sampled():
    _sampled_rs(wl.C5_RS)


@pytest.mark.parametrize("op,P,m,N,K,d", [
    (wl.OP_AG_GEMM, 2, 256, 256, 128, 1), (wl.OP_AG_GEMM, 2, 256, 256, 128, 2), (wl.OP_AG_GEMM, 4, 512, 520, 200, 4),
    (wl.OP_AG_GEMM, 4, 512, 256, 64, 16), (wl.OP_AG_GEMM, 3, 48, 64, 64, 8),
    (wl.OP_GEMM_RS, 2, 256, 256, 128, 1), (wl.OP_GEMM_RS, 2, 256, 256, 128, 2), (wl.OP_GEMM_RS, 4, 512, 520, 200, 4),
    (wl.OP_GEMM_RS, 4, 512, 256, 64, 16), (wl.OP_GEMM_RS, 3, 48, 64, 64, 8),
])
def test_interdecom_small_shapes(op, P, m, N, K, d):
    w = small(op, P, m, N, K, dist=0.1)
    A, B = wl.make_inputs(w)
    refs = ops.decomp_ag_gemm(A, B, d) if op == wl.OP_AG_GEMM else ops.decomp_gemm_rs(A, B, d)
    for copy_mode in ((api.COPY_KERNEL, api.COPY_ENGINES) if op == wl.OP_AG_GEMM else (api.COPY_KERNEL,)):
        outs, status, guards = gu.run_decomp(w, A, B, d, copy_mode=copy_mode)
        assert status == (api.OK, 0) and guards
        check_all(outs, refs, f"{w.name} d={d} copy_mode={copy_mode}")


@pytest.mark.parametrize("d", [1, 4, 16])
def test_config4_interdecom_full_size_sampled(d):
    for w in (wl.C4_AG, wl.C4_RS):
        A, B = wl.make_inputs(w)
        outs, status, guards = gu.run_decomp(w, A, B, d)
        assert status == (api.OK, 0) and guards
        rows = gu.sample_rows(w.M, w.P, 2, tile=max(1, w.m // d))
        if w.op == wl.OP_AG_GEMM:
            refs = ops.ag_gemm(A, B, rows=rows)
            for r in range(w.P):
                rep = compare.check(outs[r][rows], refs[r])
                assert rep.ok, f"{w.name} d={d} rank {r}: {rep}"
        else:
            for c, (local, ref) in ops.gemm_rs_rows(A, B, rows).items():
                rep = compare.check(outs[c][local], ref)
                assert rep.ok, f"{w.name} d={d} chunk {c}: {rep}"


@pytest.mark.parametrize("op", [wl.OP_AG_GEMM, wl.OP_GEMM_RS])
def test_host_buffer_entry_point(op):
    w = small(op, 2, 256, 264, 200, dist=0.1)
    A, B = wl.make_inputs(w)
    pr = gu.problem_of(w)
    hA = [torch.from_numpy(a.view(np.int16)).pin_memory() for a in A]
    hB = [torch.from_numpy(b.view(np.int16)).pin_memory() for b in B]
    hO = [torch.full(w.out_shape, gu.NAN_BITS, dtype=torch.int16).pin_memory() for _ in range(w.P)]
    staging = torch.empty(api.compass_fused_host_bytes(pr), dtype=torch.uint8, device="cuda")
    ws = api.alloc_workspace(pr)
    api.compass_fused_host(pr, hA, hB, hO, staging, ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    refs = ops.ag_gemm(A, B) if op == wl.OP_AG_GEMM else ops.gemm_rs(A, B)
    check_all([o.numpy().view(np.uint16) for o in hO], refs, w.name)


def test_repeated_calls_give_identical_bits():
    w = small(wl.OP_GEMM_RS, 4, 512, 768, 512, dist=0.05)
    A, B = wl.make_inputs(w)
    first, _, _ = gu.run_fused(w, A, B)
    second, _, _ = gu.run_fused(w, A, B)
    for x, y in zip(first, second):
        assert np.array_equal(x, y)


# ---- GEMM+ReduceScatter, ring read-modify-write variant --------------------------------------

def check_ring(outs, refs, what, P):
    """The running sum is rounded to BF16 once per contributor, so the RMS error
    may reach sqrt(P) roundings of 2^-9 relative each; the per-element
    acceptance rule is unchanged."""
    for r, (got, ref) in enumerate(zip(outs, refs)):
        rep = compare.check(got, ref)
        assert rep.violations == 0, f"{what} rank {r}: {rep}"
        assert rep.rms_rel <= 2.0 ** -9 * max(1.0, P ** 0.5), f"{what} rank {r}: {rep}"


@pytest.mark.parametrize("P,m,N,K,rings", RS_SHAPES)
def test_gemm_rs_ring_rmw_small_shapes(P, m, N, K, rings):
    w = small(wl.OP_GEMM_RS, P, m, N, K, dist=0.05)
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rings=rings, rs_variant=api.RS_RING_RMW)
    assert status == (api.OK, 0) and guards
    check_ring(outs, ops.gemm_rs(A, B, rings=rings), w.name, P)


def test_ring_rmw_integers_exact_and_counters_return_to_zero():
    w = wl.Workload("ints-ring", wl.OP_GEMM_RS, P=4, M=4 * 512, N=520, K=64)
    A_bits, B_bits = wl.make_structured_inputs(w, "index")       # every running sum is a small integer: no rounding
    pr = gu.problem_of(w, rs_variant=api.RS_RING_RMW)
    A, B = gu.device_inputs(A_bits, B_bits)
    ws = api.alloc_workspace(pr)
    ref = ops.gemm_rs(A_bits, B_bits)
    for _ in range(2):                                           # the second call reuses the counters
        outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
        api.compass_gemm_rs(pr, A, B, [o.view for o in outs], ws)
        assert api.compass_read_status(ws) == (api.OK, 0)
        for o, r in zip(outs, ref):
            assert np.array_equal(ops.bf16_bits_to_f64(o.bits()), r)
        assert int(ws[api.STATUS_BYTES:].view(torch.int32).abs().sum().item()) == 0


def test_config3_ring_rmw_full_size_sampled():
    w = wl.C3_RS
    A, B = wl.make_inputs(w)
    outs, status, guards = gu.run_fused(w, A, B, rs_variant=api.RS_RING_RMW)
    assert status == (api.OK, 0) and guards
    rows = gu.sample_rows(w.M, w.P, 2)
    for c, (local, ref) in ops.gemm_rs_rows(A, B, rows).items():
        rep = compare.check(outs[c][local], ref)
        assert rep.violations == 0 and rep.rms_rel <= 2.0 ** -9 * w.P ** 0.5, f"{w.name} chunk {c}: {rep}"


def test_bounded_wait_reports_timeout_and_the_context_survives():
    """A tile counter that no contributor will ever raise (the host plants a
    negative value) makes the ring epilogue's wait run out: the kernel must
    return with COMPASS_ERR_TIMEOUT in the status block, and the next call on
    a re-initialised workspace must work."""
    w = small(wl.OP_GEMM_RS, 2, 256, 256, 64, dist=0.05)
    A_bits, B_bits = wl.make_inputs(w)
    pr = gu.problem_of(w, rs_variant=api.RS_RING_RMW)
    A, B = gu.device_inputs(A_bits, B_bits)
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr)
    ws[api.STATUS_BYTES:].view(torch.int32).fill_(-1000)
    api.compass_set_wait_limit_us(20000)
    try:
        api.compass_gemm_rs(pr, A, B, [o.view for o in outs], ws)
        status, detail = api.compass_read_status(ws)
    finally:
        api.compass_set_wait_limit_us(0)
    assert status == api.ERR_TIMEOUT and detail in (3, 4, 6)      # a tile-counter wait or a wait behind it
    torch.cuda.synchronize()
    api.compass_workspace_init(ws)
    api.compass_gemm_rs(pr, A, B, [o.view for o in outs], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    check_ring([o.bits() for o in outs], ops.gemm_rs(A_bits, B_bits), w.name, w.P)


# ---- AllGather+GEMM driven by pushed partitions and readiness flags ----------------------------

def run_push(w, A_bits, B_bits, rings=2, calls=1):
    pr = gu.problem_of(w, rings=rings)
    A, B = gu.device_inputs(A_bits, B_bits)
    ws = torch.empty(api.compass_workspace_bytes(pr, api.WS_PUSH), dtype=torch.uint8, device="cuda")
    api.compass_workspace_init(ws)
    # poison the gather buffers: a tile that reads rows before they arrive produces NaN
    ws[api.STATUS_BYTES + 4096:].view(torch.int16).fill_(gu.NAN_BITS)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    results = []
    for _ in range(calls):
        outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
        api.compass_ag_gemm_push(pr, A, B, [o.view for o in outs], ws, torch.cuda.current_stream(), side)
        status = api.compass_read_status(ws)
        torch.cuda.synchronize()
        assert status == (api.OK, 0)
        assert all(o.guards_intact() for o in outs)
        results.append([o.bits() for o in outs])
    return results


@pytest.mark.parametrize("P,m,N,K,rings", [
    (1, 256, 256, 64, 2), (2, 256, 256, 256, 2), (2, 144, 264, 72, 2), (3, 272, 520, 344, 2), (4, 512, 768, 512, 2),
    (4, 384, 1024, 320, 1), (8, 256, 512, 192, 2), (4, 1024, 2568, 200, 2),
])
def test_ag_gemm_push_small_shapes(P, m, N, K, rings):
    w = small(wl.OP_AG_GEMM, P, m, N, K, dist=0.1)
    A, B = wl.make_inputs(w)
    (outs,) = run_push(w, A, B, rings=rings)
    check_all(outs, ops.ag_gemm(A, B, rings=rings), w.name)


def test_ag_gemm_push_repeated_calls_share_a_workspace():
    w = small(wl.OP_AG_GEMM, 4, 512, 520, 200, dist=0.1)
    A, B = wl.make_inputs(w)
    first, second, third = run_push(w, A, B, calls=3)
    ref = ops.ag_gemm(A, B)
    for outs in (first, second, third):
        check_all(outs, ref, w.name)


def test_config2_ag_gemm_push_full_size_sampled():
    w = wl.C2_AG
    A, B = wl.make_inputs(w)
    (outs,) = run_push(w, A, B)
    rows = gu.sample_rows(w.M, w.P, 2)
    refs = ops.ag_gemm(A, B, rows=rows)
    for r in range(w.P):
        assert not np.any((outs[r] & 0x7F80) == 0x7F80), "NaN/Inf or unwritten output"
        rep = compare.check(outs[r][rows], refs[r])
        assert rep.ok, f"{w.name} rank {r}: {rep}"


# ---- invariances: the same arithmetic in the same k order must give the same bits ------------------

def test_launch_order_push_and_decomposition_do_not_change_a_bit():
    """AllGather+GEMM sums every output element over k in the same order whatever the launch order,
    whether the A rows are read in place or from a pushed copy, and however many row slices
    InterDecom cuts: the BF16 outputs must be identical bit for bit."""
    w = small(wl.OP_AG_GEMM, 4, 1024, 776, 328, dist=0.1)
    A_bits, B_bits = wl.make_inputs(w)
    A, B = gu.device_inputs(A_bits, B_bits)

    def fused(order):
        pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, order=order)
        outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
        ws = api.alloc_workspace(pr)
        api.compass_ag_gemm(pr, A, B, [o.view for o in outs], ws)
        assert api.compass_read_status(ws) == (api.OK, 0)
        return [o.bits() for o in outs]

    base = fused(api.ORDER_RANK_MAJOR)
    others = {"step-major": fused(api.ORDER_STEP_MAJOR), "push": run_push(w, A_bits, B_bits)[0]}
    for d in (1, 2, 8):
        outs, status, guards = gu.run_decomp(w, A_bits, B_bits, d)
        assert status == (api.OK, 0) and guards
        others[f"decomp d={d}"] = outs
    for name, outs in others.items():
        for r in range(w.P):
            assert np.array_equal(outs[r], base[r]), f"{name}: rank {r} differs"


def test_single_ring_and_double_ring_agree_bitwise_for_ag_gemm():
    w = small(wl.OP_AG_GEMM, 4, 512, 520, 200, dist=0.1)
    A, B = wl.make_inputs(w)
    two, _, _ = gu.run_fused(w, A, B, rings=2)
    one, _, _ = gu.run_fused(w, A, B, rings=1)
    for x, y in zip(one, two):
        assert np.array_equal(x, y)


# ---- weights stored [K][N] (N contiguous): the layout the backward pass finds them in -----------------

def run_with_kn_weights(w, A_bits, B_bits, rings=2, rs_variant=api.RS_SEGMENTED_K, order=api.ORDER_RANK_MAJOR):
    pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, rings=rings, rs_variant=rs_variant, order=order, b_layout=api.B_KN)
    A = [api.to_device(a) for a in A_bits]
    B = [api.to_device(np.ascontiguousarray(b.T)) for b in B_bits]        # the same values, stored [K][N]
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr)
    (api.compass_ag_gemm if w.op == wl.OP_AG_GEMM else api.compass_gemm_rs)(pr, A, B, [o.view for o in outs], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    assert all(o.guards_intact() for o in outs)
    return [o.bits() for o in outs]


@pytest.mark.parametrize("op,P,m,N,K,rings", [
    (wl.OP_AG_GEMM, 1, 128, 256, 64, 2), (wl.OP_AG_GEMM, 2, 256, 256, 256, 2), (wl.OP_AG_GEMM, 2, 144, 264, 72, 2),
    (wl.OP_AG_GEMM, 3, 272, 520, 1376, 2), (wl.OP_AG_GEMM, 4, 384, 1024, 320, 1), (wl.OP_AG_GEMM, 8, 80, 200, 8, 2),
    (wl.OP_GEMM_RS, 2, 256, 256, 256, 2), (wl.OP_GEMM_RS, 3, 272, 520, 344, 2), (wl.OP_GEMM_RS, 8, 256, 512, 1376, 2),
    (wl.OP_GEMM_RS, 4, 384, 1024, 320, 1),
])
def test_kn_weights_small_shapes(op, P, m, N, K, rings):
    w = small(op, P, m, N, K)
    A, B = wl.make_inputs(w)
    outs = run_with_kn_weights(w, A, B, rings=rings)
    check_all(outs, ops.ag_gemm(A, B, rings=rings) if op == wl.OP_AG_GEMM else ops.gemm_rs(A, B, rings=rings), w.name)


@pytest.mark.parametrize("op,P,m,N,K,order", [
    (wl.OP_AG_GEMM, 4, 1024, 2568, 200, api.ORDER_RANK_MAJOR),      # 512x256 and 256x256 tiles, ragged N, K tail
    (wl.OP_AG_GEMM, 4, 1024, 2568, 424, api.ORDER_STEP_MAJOR),
    (wl.OP_GEMM_RS, 8, 1024, 2568, 88, api.ORDER_RANK_MAJOR),       # K segments with partial stages
])
def test_kn_weights_big_and_small_tiles(op, P, m, N, K, order):
    w = small(op, P, m, N, K, dist=0.05)
    A, B = wl.make_inputs(w)
    outs = run_with_kn_weights(w, A, B, order=order)
    check_all(outs, ops.ag_gemm(A, B) if op == wl.OP_AG_GEMM else ops.gemm_rs(A, B), w.name)


def test_kn_weights_give_the_same_bits_as_nk_weights():
    """The layout changes how the tile is fetched, not what is multiplied: bit-identical outputs."""
    for op, P, m, N, K in ((wl.OP_AG_GEMM, 4, 1024, 1032, 456), (wl.OP_GEMM_RS, 4, 512, 776, 200), (wl.OP_AG_GEMM, 2, 96, 264, 72)):
        w = small(op, P, m, N, K, dist=0.05)
        A, B = wl.make_inputs(w)
        kn = run_with_kn_weights(w, A, B)
        nk, status, guards = gu.run_fused(w, A, B)
        assert status == (api.OK, 0) and guards
        for x, y in zip(kn, nk):
            assert (x == y).all()


def test_kn_weights_ring_rmw_and_integer_inputs():
    w = small(wl.OP_GEMM_RS, 4, 512, 520, 344)
    A, B = wl.make_structured_inputs(w, "index")
    outs = run_with_kn_weights(w, A, B, rs_variant=api.RS_RING_RMW)
    refs = ops.gemm_rs(A, B)
    for r in range(w.P):
        assert (ops.bf16_bits_to_f64(outs[r]) == refs[r]).all()


def test_kn_weights_interdecom():
    w = small(wl.OP_AG_GEMM, 4, 512, 520, 200)
    A_bits, B_bits = wl.make_inputs(w)
    for d in (1, 4):
        pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, d=d, b_layout=api.B_KN)
        A = [api.to_device(a) for a in A_bits]
        B = [api.to_device(np.ascontiguousarray(b.T)) for b in B_bits]
        outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
        ws = api.alloc_workspace(pr, api.WS_DECOMP)
        api.compass_decomp(pr, A, B, [o.view for o in outs], ws, torch.cuda.current_stream(), torch.cuda.Stream())
        assert api.compass_read_status(ws) == (api.OK, 0)
        torch.cuda.synchronize()
        check_all([o.bits() for o in outs], ops.decomp_ag_gemm(A_bits, B_bits, d), f"{w.name} d={d}")


# ---- seeded sweep over random shapes and options ---------------------------------------------------------

def _random_cases(n, seed):
    """Shapes drawn so that all three kernels, ragged rows and columns, K tails, K segments, both rings,
    both launch orders, both reduce variants and both weight layouts occur."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        op = int(rng.integers(0, 2))
        P = int(rng.choice([1, 2, 3, 4, 5, 8]))
        rings = int(rng.choice([1, 2]))
        m = int(rng.choice([8, 40, 128, 136, 256, 264, 512, 520, 768, 1024])) * (1 if rng.random() < 0.7 else 2)
        if m % rings:
            continue
        N = int(rng.choice([8, 64, 200, 256, 264, 512, 776, 1032]))
        K = int(rng.choice([8, 16, 64, 72, 128, 200, 320, 384, 392, 456, 1024]))
        if P * m * N * K * P > 6e10:            # keep the FP64 oracle to about a second per case
            continue
        cases.append((op, P, m, N, K, rings, int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.integers(0, 2))))
    return cases


@pytest.mark.parametrize("op,P,m,N,K,rings,order,variant,layout", _random_cases(40, seed=20261125))
def test_random_shapes_and_options(op, P, m, N, K, rings, order, variant, layout):
    w = small(op, P, m, N, K, seed=P + m + N + K, dist=0.1)
    A_bits, B_bits = wl.make_inputs(w)
    rs_variant = api.RS_RING_RMW if (op == wl.OP_GEMM_RS and variant) else api.RS_SEGMENTED_K
    pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, rings=rings, rs_variant=rs_variant, order=order, b_layout=layout)
    A = [api.to_device(a) for a in A_bits]
    B = [api.to_device(np.ascontiguousarray(b.T) if layout == api.B_KN else b) for b in B_bits]
    outs = [gu.Guarded(*w.out_shape) for _ in range(w.P)]
    ws = api.alloc_workspace(pr)
    (api.compass_ag_gemm if op == wl.OP_AG_GEMM else api.compass_gemm_rs)(pr, A, B, [o.view for o in outs], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    assert all(o.guards_intact() for o in outs)
    refs = ops.ag_gemm(A_bits, B_bits, rings=rings) if op == wl.OP_AG_GEMM else ops.gemm_rs(A_bits, B_bits, rings=rings)
    for r, (o, ref) in enumerate(zip(outs, refs)):
        rep = compare.check(o.bits(), ref)
        limit = np.sqrt(P) * 2.0 ** -9 if rs_variant == api.RS_RING_RMW else compare.RMS_REL_LIMIT
        assert rep.violations == 0 and rep.rms_rel <= max(limit, compare.RMS_REL_LIMIT), f"rank {r}: {rep}"


# ---- CUDA graphs -------------------------------------------------------------------------------------------

@pytest.mark.parametrize("which", ["fused_ag", "fused_rs_rmw", "decomp", "push", "mlp"])
def test_entry_points_capture_into_cuda_graphs(which):
    """Every launch path can be captured into a CUDA graph; a replay computes on the CURRENT contents of the
    input buffers (checked by changing them in place between replays) and gives the bits of the eager call."""
    w = small(wl.OP_AG_GEMM if which != "fused_rs_rmw" else wl.OP_GEMM_RS, 4, 512, 520, 200, dist=0.05)
    side = torch.cuda.Stream()
    A_bits, B_bits = wl.make_inputs(w)
    A = [api.to_device(a) for a in A_bits]
    B = [api.to_device(b) for b in B_bits]
    if which == "mlp":
        mw = wl.MlpWorkload("graph-mlp", P=4, M=2048, hidden=200, ffn=528, activation=wl.ACT_SWIGLU, seed=2)
        X_bits, W0_bits, W1_bits = wl.make_mlp_inputs(mw)
        A = [api.to_device(a) for a in X_bits]
        W0, W1 = [api.to_device(a) for a in W0_bits], [api.to_device(a) for a in W1_bits]
        H = [torch.zeros((mw.M, mw.hc), dtype=torch.bfloat16, device="cuda") for _ in range(4)]
        outs = [torch.zeros((mw.m, mw.hidden), dtype=torch.bfloat16, device="cuda") for _ in range(4)]
        mp = api.make_mlp(4, mw.M, mw.hidden, mw.ffn, activation=api.ACT_SWIGLU)
        ws = api.alloc_mlp_workspace(mp)
        call = lambda: api.compass_mlp_block(mp, A, W0, H, W1, outs, ws, torch.cuda.current_stream())
    else:
        outs = [torch.zeros(w.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(w.P)]
        if which == "fused_ag":
            pr = api.make_problem(w.op, w.P, w.M, w.N, w.K)
            ws = api.alloc_workspace(pr)
            call = lambda: api.compass_ag_gemm(pr, A, B, outs, ws, torch.cuda.current_stream())
        elif which == "fused_rs_rmw":
            pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, rs_variant=api.RS_RING_RMW)
            ws = api.alloc_workspace(pr)
            call = lambda: api.compass_gemm_rs(pr, A, B, outs, ws, torch.cuda.current_stream())
        elif which == "decomp":
            pr = api.make_problem(w.op, w.P, w.M, w.N, w.K, d=4)
            ws = api.alloc_workspace(pr, api.WS_DECOMP)
            call = lambda: api.compass_decomp(pr, A, B, outs, ws, torch.cuda.current_stream(), side)
        else:
            pr = api.make_problem(w.op, w.P, w.M, w.N, w.K)
            ws = api.alloc_workspace(pr, api.WS_PUSH)
            call = lambda: api.compass_ag_gemm_push(pr, A, B, outs, ws, torch.cuda.current_stream(), side)

    def eager_bits():
        call()
        torch.cuda.synchronize()
        return [o.view(torch.int16).clone() for o in outs]

    first = eager_bits()                                    # also the warm-up the first launch on a device needs
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    for trial in range(3):
        if trial:                                            # new input values in the same buffers
            for t in A:
                t.mul_(-0.5 if trial == 1 else 1.25)
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        replayed = [o.view(torch.int16).clone() for o in outs]
        assert api.compass_read_status(ws) == (api.OK, 0)
        want = first if trial == 0 else eager_bits()
        for got, ref in zip(replayed, want):
            assert bool((got == ref).all()), f"{which}: replay {trial} differs from the eager call"
        assert any(bool((o != 0).any()) for o in replayed)
