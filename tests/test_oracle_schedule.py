"""Pins for the oracle's ring schedule (CPU only).

The closed form is checked against what the paper states (Section III-A/B),
against an independent token-passing enumeration, and against properties any
ring collective must have, so that a wrong sign, index or orientation fails.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import OP_AG_GEMM, OP_GEMM_RS
from oracle import ring_sim
from oracle.schedule import (CHUNK, PART, PEER, RANK, RING, ROW_BEGIN, ROW_COUNT, STEP,
                             ring_direction, schedule)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def paper_pins():
    pins = {}
    with open(os.path.join(GOLDEN, "paper_pins.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = [s.strip() for s in line.split("=")]
            pins[k] = Fraction(v)
    return pins


ALL_CASES = [(op, P, rings) for op in (OP_AG_GEMM, OP_GEMM_RS) for P in range(1, 17) for rings in (1, 2)]


@pytest.mark.parametrize("op,P,rings", ALL_CASES)
def test_closed_form_equals_token_passing(op, P, rings):
    M = P * rings * 5
    a = schedule(op, P, rings, M)
    b = ring_sim.simulate(op, P, rings, M)
    assert a.dtype == np.int32 and a.shape == (rings * P * P, 8)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("op,P,rings", ALL_CASES)
def test_every_rank_consumes_every_partition_exactly_once(op, P, rings):
    t = schedule(op, P, rings, P * rings * 4)
    for r in range(P):
        mine = t[t[:, RANK] == r]
        assert sorted(mine[:, PART].tolist()) == list(range(rings * P))
        # rows tile the whole tensor without overlap
        covered = np.zeros(P * rings * 4, dtype=int)
        for e in mine:
            covered[e[ROW_BEGIN]:e[ROW_BEGIN] + e[ROW_COUNT]] += 1
        assert (covered == 1).all()
        # order: step ascending, ring 0 before ring 1
        keys = [(int(e[STEP]), int(e[RING])) for e in mine]
        assert keys == sorted(keys) and len(set(keys)) == len(keys)


def test_paper_partition_count_and_steps():
    pins = paper_pins()
    t = schedule(OP_AG_GEMM, 4, 2, 4096)
    assert len(set(t[:, PART].tolist())) == pins["partitions_double_ring_P4"]
    t8 = schedule(OP_AG_GEMM, 8, 1, 4096)
    steps_with_transfers = {int(e[STEP]) for e in t8 if e[PEER] != e[RANK]}
    assert len(steps_with_transfers) == pins["transfer_steps_single_ring_P8"]
    # n_chunks = number of GPUs (Section V-B): P steps per rank
    assert set(t8[:, STEP].tolist()) == set(range(8))


@pytest.mark.parametrize("op", [OP_AG_GEMM, OP_GEMM_RS])
def test_paper_effective_bandwidth_factors(op):
    pins = paper_pins()
    f = lambda P, rings: ring_sim.effective_bandwidth_factor(schedule(op, P, rings, 64 * P), op, P, 64 * P)
    assert f(4, 2) == pins["bandwidth_factor_double_ring_P4"]
    assert f(4, 1) == pins["bandwidth_factor_single_ring_P4"]
    assert f(8, 1) == pins["bandwidth_factor_single_ring_P8"]
    assert f(4, 2) == 2 * f(4, 1)
    for P in range(2, 12):
        assert f(P, 1) == Fraction(P, P - 1)
        if P >= 3:                       # at P = 2 both rings share the one link pair
            assert f(P, 2) == Fraction(2 * P, P - 1)
    assert f(2, 2) == 2


@pytest.mark.parametrize("op,P,rings", [c for c in ALL_CASES if c[1] >= 2])
def test_one_partition_per_directed_link_per_step(op, P, rings):
    M = P * rings * 2
    t = schedule(op, P, rings, M)
    per_step = ring_sim.link_rows_per_step(t, op, P)
    busy = [s for s in per_step if s]
    assert len(busy) == P - 1
    shared = (P == 2 and rings == 2)      # forward and backward neighbour coincide
    for links in busy:
        # every rank sends exactly one partition per ring and step
        assert sum(links.values()) == P * rings * (M // P // rings)
        assert len(links) == (P if shared else P * rings)
        assert all(v == (2 if shared else 1) * (M // P // rings) for v in links.values())
        for (src, dst) in links:
            assert (dst - src) % P in (1, P - 1)


@pytest.mark.parametrize("P,rings", [(P, r) for P in range(1, 10) for r in (1, 2)])
def test_ag_local_first_rs_local_last_and_parity(P, rings):
    ag = schedule(OP_AG_GEMM, P, rings, P * rings)
    rs = schedule(OP_GEMM_RS, P, rings, P * rings)
    for e in ag:
        assert (e[PEER] == e[RANK]) == (e[STEP] == 0)
        if e[STEP] == 0:
            assert e[CHUNK] == e[RANK]
    for e in rs:
        assert (e[PEER] == e[RANK]) == (e[STEP] == P - 1)
        if e[STEP] == P - 1:
            assert e[CHUNK] == e[RANK]
    if rings == 2:
        for t in (ag, rs):
            for e in t:
                # backward ring carries even partitions, forward ring odd ones
                assert e[PART] % 2 == e[RING]
                assert ring_direction(2, int(e[RING])) == (-1 if e[RING] == 0 else 1)


@pytest.mark.parametrize("P,rings", [(P, r) for P in range(2, 10) for r in (1, 2)])
def test_ring_feasibility(P, rings):
    """AG: a rank can only forward what it obtained at the previous step.
    RS: what a rank emits at step s is what its downstream peer adds to at s+1."""
    ag = schedule(OP_AG_GEMM, P, rings, P * rings)
    rs = schedule(OP_GEMM_RS, P, rings, P * rings)
    lookup_ag = {(int(e[RANK]), int(e[STEP]), int(e[RING])): e for e in ag}
    lookup_rs = {(int(e[RANK]), int(e[STEP]), int(e[RING])): e for e in rs}
    for (r, s, g), e in lookup_ag.items():
        if s == 0:
            continue
        src = int(e[PEER])
        assert lookup_ag[(src, s - 1, g)][PART] == e[PART]
        # the sender is the upstream neighbour on that ring
        assert (r - src) % P == ring_direction(rings, g) % P
    for (r, s, g), e in lookup_rs.items():
        if s == P - 1:
            continue
        dst = int(e[PEER])
        assert lookup_rs[(dst, s + 1, g)][PART] == e[PART]
        assert (dst - r) % P == ring_direction(rings, g) % P


@pytest.mark.parametrize("P", range(1, 10))
def test_ag_rs_duality(P):
    """Reversing time and swapping ring directions maps one schedule onto the other."""
    ag = schedule(OP_AG_GEMM, P, 2, 2 * P)
    rs = schedule(OP_GEMM_RS, P, 2, 2 * P)
    look = {(int(e[RANK]), int(e[STEP]), int(e[RING])): int(e[CHUNK]) for e in ag}
    for e in rs:
        assert look[(int(e[RANK]), P - 1 - int(e[STEP]), 1 - int(e[RING]))] == int(e[CHUNK])


def test_row_ranges():
    t = schedule(OP_AG_GEMM, 4, 2, 4096)
    for e in t:
        assert e[ROW_COUNT] == 512
        assert e[ROW_BEGIN] == e[CHUNK] * 1024 + e[RING] * 512
        assert e[PART] == 2 * e[CHUNK] + e[RING]
    t1 = schedule(OP_GEMM_RS, 4, 1, 4096)
    for e in t1:
        assert e[ROW_COUNT] == 1024 and e[ROW_BEGIN] == e[CHUNK] * 1024 and e[PART] == e[CHUNK] and e[RING] == 0


def test_rejects_bad_shapes():
    for bad in [(OP_AG_GEMM, 0, 2, 8), (OP_AG_GEMM, 2, 3, 8), (OP_AG_GEMM, 3, 2, 8), (OP_AG_GEMM, 2, 2, 6), (7, 2, 2, 8)]:
        with pytest.raises(ValueError):
            schedule(*bad)


def test_golden_tables_unchanged():
    with open(os.path.join(GOLDEN, "schedule_tables.txt")) as f:
        lines = [l.split() for l in f if not l.startswith("#")]
    i = 0
    n_cases = 0
    while i < len(lines):
        assert lines[i][0] == "case"
        op, P, rings, M, count = map(int, lines[i][1:])
        rows = np.array([[int(v) for v in l] for l in lines[i + 1:i + 1 + count]], dtype=np.int32)
        assert np.array_equal(rows, schedule(op, P, rings, M))
        i += 1 + count
        n_cases += 1
    assert n_cases == 6
