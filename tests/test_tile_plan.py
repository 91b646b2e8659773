"""Host-side tile planning (compass_tile_plan; no GPU): how a launch is cut into 512x256, 256x256, 256x128 and
128x256 tiles.  Checked against hand-computed plans of the benchmark configurations, against conservation of the
tiled area, and against a brute-force search for the cheapest way to finish the last round over the CTA pairs."""
import math

import pytest
from hypothesis import given, settings, strategies as st

from paper_2609_10549_b200 import api

AG, RS = api.OP_AG_GEMM, api.OP_GEMM_RS
PAIRS = 74          # co-resident clusters of two CTAs on a B200 (148 SMs)


def plan(op, P, M, N, K, pairs=PAIRS, decomposed=False, **kw):
    t = api.compass_tile_plan(api.make_problem(op, P, M, N, K, **kw), decomposed=decomposed, cta_pairs=pairs)
    return {f: getattr(t, f) for f, _ in t._fields_}


def test_benchmark_configurations_by_hand():
    # C1: 8 entries of 128 rows; the two ring entries of a step share B_r: 4 groups x 4 column tiles
    c1 = plan(AG, 2, 512, 1024, 1024)
    assert (c1["cta_pairs"], c1["blocks_per_group"], c1["tiles_256x256"], c1["total_tiles"]) == (1, 2, 16, 16)
    # C2: 32 entries of 512 rows x 12 column tiles = 384 slots = 5 waves of 74 + 14; 14 slots end sooner as 56 tiles of
    # 256x128 (one round, 0.42) than as 28 of 256x256 (one round, 0.5)
    c2 = plan(AG, 4, 4096, 3072, 4096)
    assert (c2["tiles_512x256"], c2["tiles_256x256"], c2["tiles_256x128"]) == (370, 0, 56)
    # C3, segmented K: 16 partitions x 16 column tiles = 256 slots = 3 waves + 34: 68 tiles of 256x256 fill one round
    c3 = plan(RS, 8, 8192, 4096, 1376)
    assert (c3["blocks"], c3["tiles_512x256"], c3["tiles_256x256"], c3["tiles_256x128"]) == (16, 222, 68, 0)
    # C3, ring read-modify-write: 128 entries x 2 x 16 tiles of 256x256
    ring = plan(RS, 8, 8192, 4096, 1376, rs_variant=api.RS_RING_RMW)
    assert (ring["blocks"], ring["tiles_512x256"], ring["tiles_256x256"], ring["total_tiles"]) == (128, 0, 4096, 4096)
    # C4-RS: 128 slots = 1 wave + 54: one round of 256x256 (37 slots) and one of 256x128 (17 slots), 0.92 < 1.0
    c4 = plan(RS, 4, 4096, 4096, 1024)
    assert (c4["tiles_512x256"], c4["tiles_256x256"], c4["tiles_256x128"]) == (74, 74, 68)
    # C5-AG: 128 entries of 1024 rows x 28 column tiles = 7168 slots = 96 waves + 64 -> 128 tiles of 256x256
    c5 = plan(AG, 8, 16384, 7168, 8192)
    assert (c5["tiles_512x256"], c5["tiles_256x256"], c5["tiles_256x128"]) == (7104, 128, 0)


def test_which_small_blocks_are_paired():
    assert plan(AG, 8, 2048, 2048, 4096)["blocks_per_group"] == 2                       # 128-row partitions, two rings
    assert plan(AG, 8, 2048, 2048, 4096, order=api.ORDER_STEP_MAJOR)["blocks_per_group"] == 2
    seg = plan(RS, 8, 2048, 4096, 2048)                                                 # segmented K: no two partitions share B
    assert (seg["cta_pairs"], seg["tiles_128x256"], seg["total_tiles"]) == (0, 256, 256)
    assert plan(RS, 8, 2048, 4096, 2048, rs_variant=api.RS_RING_RMW)["blocks_per_group"] == 2
    assert plan(AG, 3, 384, 256, 64, rings=1)["blocks_per_group"] == 3                  # one ring, rank-major: a rank's 3 steps
    one = plan(AG, 3, 384, 256, 64, rings=1, order=api.ORDER_STEP_MAJOR)                # lockstep: neighbours are other ranks
    assert (one["cta_pairs"], one["blocks_per_group"]) == (0, 1)
    assert plan(AG, 4, 768, 256, 64)["blocks_per_group"] == 2                           # 96-row entries: padded to 128 rows, paired
    h192 = plan(AG, 4, 1536, 256, 64)                                                   # 192-row entries: a pair tile of their own each
    assert (h192["cta_pairs"], h192["blocks_per_group"], h192["tiles_256x256"]) == (1, 1, 32)
    d16 = plan(AG, 4, 4096, 3072, 4096, decomposed=True, d=16)                          # 64-row slices, a rank's 4 slices adjacent
    assert (d16["rows_per_block"], d16["blocks_per_group"], d16["tiles_256x256"]) == (64, 2, 96)
    d1 = plan(AG, 4, 4096, 3072, 4096, decomposed=True, d=1)
    assert (d1["blocks"], d1["rows_per_block"], d1["blocks_per_group"]) == (16, 1024, 1)


def test_without_clusters_everything_runs_on_single_ctas():
    t = plan(AG, 4, 4096, 3072, 4096, pairs=0)
    assert (t["cta_pairs"], t["tiles_128x256"], t["total_tiles"]) == (0, 32 * 4 * 12, 32 * 4 * 12)
    lib = api.lib()
    import ctypes as C
    out = api.TileCounts()
    pr = api.make_problem(AG, 4, 4096, 3072, 4096)
    assert lib.compass_tile_plan(C.byref(pr), 0, -1, C.byref(out)) == api.ERR_INVALID_ARG
    assert lib.compass_tile_plan(C.byref(pr), 0, 74, None) == api.ERR_INVALID_ARG
    assert lib.compass_tile_plan(C.byref(api.make_problem(AG, 3, 4096, 3072, 4096)), 0, 74, C.byref(out)) == api.ERR_SHAPE


def cheapest_remainder(slots, pairs):
    """Brute force over every split of the remaining slots into 256x256 tiles (2 per slot, 0.5 of a 512x256 tile's
    time per round) and 256x128 tiles (4 per slot, 0.42 per round): the minimal finishing time and, among the
    cheapest splits, the most slots given to 256x256 tiles."""
    best = None
    for small in range(slots, -1, -1):
        cost = 0.5 * math.ceil(2 * small / pairs) + 0.42 * math.ceil(4 * (slots - small) / pairs)
        if best is None or cost < best[0] - 1e-9:
            best = (cost, small)
    return best


@settings(max_examples=200, deadline=None)
@given(P=st.sampled_from([1, 2, 4, 8]), rows512=st.integers(1, 6), ntiles=st.integers(1, 40), pairs=st.sampled_from([8, 33, 66, 74]),
       op=st.sampled_from([AG, RS]))
def test_area_is_conserved_and_the_last_round_is_planned_optimally(P, rows512, ntiles, pairs, op):
    h = 512 * rows512                                  # rows per partition: whole 512-row slots
    M, N, K = P * 2 * h, 256 * ntiles, 64
    t = plan(op, P, M, N, K, pairs=pairs)
    assert t["cta_pairs"] == 1 and t["blocks_per_group"] == 1 and t["tiles_128x256"] == 0
    slots = t["blocks"] * rows512 * ntiles             # 512x256 slots of the launch
    assert t["blocks"] == (2 * P * P if op == AG else 2 * P)
    assert 4 * t["tiles_512x256"] + 2 * t["tiles_256x256"] + t["tiles_256x128"] == 4 * slots      # in units of 256x128
    assert t["tiles_512x256"] % pairs == 0 and t["tiles_512x256"] == (slots // pairs) * pairs
    assert t["total_tiles"] == t["tiles_512x256"] + t["tiles_256x256"] + t["tiles_256x128"]
    remaining = slots - t["tiles_512x256"]
    if t["tiles_512x256"] == 0:
        assert t["tiles_256x128"] == 0                 # nothing but a remainder: 256x256 tiles only
    else:
        cost, small = cheapest_remainder(remaining, pairs)
        assert t["tiles_256x256"] == 2 * small and t["tiles_256x128"] == 4 * (remaining - small)
