"""Pins for the oracle's operators (CPU only): brute force, textbook identities,
library routines and special cases, chosen so that a dropped term, a
transposed operand or a wrong row offset fails at least one of them."""
import numpy as np
import pytest
import torch

from oracle import OP_AG_GEMM, OP_GEMM_RS, compare
from oracle import operators as ops
from oracle.schedule import schedule
from paper_2609_10549_b200 import workloads as wl


def tiny(op, P, M, N, K, seed=3):
    w = wl.Workload("tiny", op, P=P, M=M, N=N, K=K, a_dist=("normal", 1.0), b_dist=("normal", 1.0), seed=seed)
    return w, *wl.make_inputs(w)


def bf16_value(bits: int) -> float:
    """Decode one BF16 pattern by the format's definition (sign, 8-bit
    exponent, 7-bit fraction), independent of any numpy view trick."""
    s = -1.0 if bits >> 15 else 1.0
    e = (bits >> 7) & 0xFF
    f = bits & 0x7F
    if e == 0:
        return s * (f / 128.0) * 2.0 ** -126
    assert e != 255
    return s * (1.0 + f / 128.0) * 2.0 ** (e - 127)


def brute_force_gemm(A_bits, B_bits):
    """Unsharded triple loop, pure Python."""
    M, K = A_bits.shape
    N = B_bits.shape[0]
    C = np.zeros((M, N))
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for k in range(K):
                acc += bf16_value(int(A_bits[i, k])) * bf16_value(int(B_bits[j, k]))
            C[i, j] = acc
    return C


def test_bf16_decode_matches_definition_and_torch():
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 1 << 16, size=4096, dtype=np.uint16)
    bits = bits[((bits >> 7) & 0xFF) != 255]                      # drop Inf/NaN patterns
    got = ops.bf16_bits_to_f64(bits)
    assert np.array_equal(got, np.array([bf16_value(int(b)) for b in bits]))
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got, t)


def test_input_rounding_matches_torch_bf16():
    x = np.random.default_rng(1).standard_normal(10000).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0e-39]          # ties and a subnormal
    bits = wl.f32_to_bf16_bits(x)
    t = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, t)


def test_bf16_rounding_helper_matches_torch():
    x = np.random.default_rng(2).standard_normal(5000) * 37.0
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ops.f64_to_bf16_f64(x), want)


@pytest.mark.parametrize("P,M,N,K", [(2, 8, 8, 8), (1, 4, 3, 7), (3, 12, 5, 1), (4, 16, 6, 9)])
@pytest.mark.parametrize("rings", [1, 2])
def test_ag_gemm_brute_force(P, M, N, K, rings):
    if (M // P) % rings:
        pytest.skip("rows per rank not divisible")
    w, A, B = tiny(OP_AG_GEMM, P, M, N, K)
    C = ops.ag_gemm(A, B, rings=rings)
    G = np.concatenate(A)
    for r in range(P):
        assert C[r].shape == (M, N)
        np.testing.assert_allclose(C[r], brute_force_gemm(G, B[r]), rtol=0, atol=1e-12)


@pytest.mark.parametrize("P,M,N,K", [(2, 8, 8, 8), (1, 4, 3, 7), (3, 12, 5, 1), (4, 16, 6, 9)])
@pytest.mark.parametrize("rings", [1, 2])
def test_gemm_rs_brute_force(P, M, N, K, rings):
    if (M // P) % rings:
        pytest.skip("rows per rank not divisible")
    w, A, B = tiny(OP_GEMM_RS, P, M, N, K)
    Out = ops.gemm_rs(A, B, rings=rings)
    total = sum(brute_force_gemm(A[q], B[q]) for q in range(P))
    m = M // P
    for c in range(P):
        assert Out[c].shape == (m, N)
        np.testing.assert_allclose(Out[c], total[c * m:(c + 1) * m], rtol=0, atol=1e-12)


def test_ag_gemm_equals_unsharded_library_gemm():
    w, A, B = tiny(OP_AG_GEMM, 4, 256, 96, 200)
    C = ops.ag_gemm(A, B)
    G = torch.from_numpy(np.concatenate(A).view(np.int16)).view(torch.bfloat16).to(torch.float64)
    for r in range(4):
        Br = torch.from_numpy(B[r].view(np.int16)).view(torch.bfloat16).to(torch.float64)
        np.testing.assert_allclose(C[r], (G @ Br.T).numpy(), rtol=1e-13, atol=1e-12)


def test_gemm_rs_equals_gemm_over_concatenated_k():
    """sum_q A_q B_q^T = [A_0|A_1|...] [B_0|B_1|...]^T : the row-parallel GEMM
    is the unsharded GEMM whose K dimension was cut into P slices."""
    P = 4
    w, A, B = tiny(OP_GEMM_RS, P, 128, 72, 40)
    Out = ops.gemm_rs(A, B)
    full = ops.unsharded_gemm(np.concatenate(A, axis=1), np.concatenate(B, axis=1))
    np.testing.assert_allclose(np.concatenate(Out), full, rtol=1e-13, atol=1e-12)


def test_one_hot_activation_selects_weight_columns():
    """A row that is one-hot at k makes the output row equal column k of B
    (stored as B[:, k]): catches transposed operands and row-offset mistakes."""
    P, m, K, N = 4, 8, 16, 5
    rng = np.random.default_rng(5)
    hot = rng.integers(0, K, size=(P, m))
    A = []
    for r in range(P):
        a = np.zeros((m, K), dtype=np.float32)
        a[np.arange(m), hot[r]] = 1.0
        A.append(wl.f32_to_bf16_bits(a))
    B = [wl.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32)) for _ in range(P)]
    C = ops.ag_gemm(A, B)
    for r in range(P):
        Bf = ops.bf16_bits_to_f64(B[r])
        for q in range(P):
            for i in range(m):
                assert np.array_equal(C[r][q * m + i], Bf[:, hot[q, i]])


def test_results_do_not_depend_on_rings_or_decomposition():
    w, A, B = tiny(OP_AG_GEMM, 4, 64, 24, 32)
    base = ops.ag_gemm(A, B, rings=2)
    for other in (ops.ag_gemm(A, B, rings=1), ops.decomp_ag_gemm(A, B, 1), ops.decomp_ag_gemm(A, B, 4),
                  ops.decomp_ag_gemm(A, B, 16)):
        for x, y in zip(base, other):
            assert np.array_equal(x, y)         # same terms, same k order: bit-identical
    w, A, B = tiny(OP_GEMM_RS, 4, 64, 24, 32)
    base = ops.gemm_rs(A, B, rings=2)
    for other in (ops.gemm_rs(A, B, rings=1), ops.decomp_gemm_rs(A, B, 1), ops.decomp_gemm_rs(A, B, 8)):
        for x, y in zip(base, other):
            np.testing.assert_allclose(x, y, rtol=1e-13, atol=1e-12)   # summation order differs


def test_gather_rejects_a_broken_table():
    w, A, B = tiny(OP_AG_GEMM, 4, 32, 4, 4)
    t = schedule(OP_AG_GEMM, 4, 2, 32).copy()
    t[3, 6] = t[2, 6]                          # two entries of rank 0 now cover the same rows
    with pytest.raises(AssertionError):
        ops.ag_gemm(A, B, table=t)
    t = schedule(OP_GEMM_RS, 4, 2, 32).copy()
    w, A, B = tiny(OP_GEMM_RS, 4, 32, 4, 4)
    t[0, 0], t[8, 0] = t[8, 0], t[0, 0]        # swap two ranks' entries: contributors no longer distinct
    with pytest.raises(AssertionError):
        ops.gemm_rs(A, B, table=t)


def test_sampled_rows_equal_full_rows():
    w, A, B = tiny(OP_AG_GEMM, 2, 32, 8, 16)
    full = ops.ag_gemm(A, B)
    rows = np.array([0, 7, 16, 31])
    part = ops.ag_gemm(A, B, rows=rows, ranks=[1])
    assert np.array_equal(part[0], full[1][rows])


def test_structured_inputs_are_exact_integers():
    w = wl.Workload("s", OP_AG_GEMM, P=2, M=16, N=8, K=32)
    A, B = wl.make_structured_inputs(w, "index")
    C = ops.ag_gemm(A, B)
    assert all(np.array_equal(c, np.round(c)) for c in C)


def test_acceptance_rule():
    ref = np.array([[1.0, -2.0], [0.5, 100.0]])
    exact = wl.f32_to_bf16_bits(ref.astype(np.float32))
    assert compare.check(exact, ref).ok
    tol = 1e-2 * 100.0 + 1e-3
    off = ref.copy(); off[0, 0] += 2 * tol
    rep = compare.check(wl.f32_to_bf16_bits(off.astype(np.float32)), ref)
    assert not rep.ok and rep.violations == 1 and rep.worst_index == (0, 0)
    nan = exact.copy(); nan[1, 0] = 0x7FC0
    assert compare.check(nan, ref).violations == 1
    # inside the per-element bound but systematically wrong: caught by the RMS rule
    drift = ref * 1.01
    rep = compare.check(wl.f32_to_bf16_bits(drift.astype(np.float32)), ref)
    assert rep.violations == 0 and not rep.ok


def test_sampled_reduce_scatter_rows_equal_full_rows():
    w, A, B = tiny(OP_GEMM_RS, 4, 64, 8, 16)
    full = ops.gemm_rs(A, B)
    rows = np.array([0, 7, 8, 15, 16, 40, 63])
    got = ops.gemm_rs_rows(A, B, rows)
    seen = 0
    for c, (local, vals) in got.items():
        assert np.array_equal(vals, full[c][local])
        seen += len(local)
    assert seen == len(rows)


# ---- the ring with BF16 messages: one rounding per contributor, so the ORDER of the contributors shows ----------

def scalar_shards(P, m, values):
    """K = 1, N = 1, every weight 1.0: partial of rank q for row i is values[q][i] itself."""
    A = [wl.f32_to_bf16_bits(np.asarray(values[q], dtype=np.float32).reshape(P * m, 1)) for q in range(P)]
    B = [wl.f32_to_bf16_bits(np.ones((1, 1), dtype=np.float32)) for _ in range(P)]
    return A, B


def test_fp32_to_bf16_rounding_matches_torch_and_ties_go_to_even():
    x = (np.random.default_rng(5).standard_normal(20000) * 41.0).astype(np.float32)
    x[:6] = [257.0, 259.0, 261.0, -257.0, 1.00390625, 1.01171875]                 # exact ties
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = ops.fp32_to_bf16_rne(x)
    assert np.array_equal(got, want)
    assert list(got[:4]) == [256.0, 260.0, 260.0, -256.0]                         # 8 significant bits: step 2 above 256


def test_bf16_hops_single_ring_order_is_owner_plus_one_first_owner_last():
    """Forward ring, P = 3, one row per chunk: the sum for chunk c starts at rank c+1 and ends at its owner c.
    256 + 1 is a tie and rounds to 256 (even), twice; 1 + 1 + 256 = 258 is exact.  So where the large term comes
    first the result is 256, where it comes last 258."""
    P = 3
    values = np.zeros((P, P))
    values[1][0], values[2][0], values[0][0] = 256.0, 1.0, 1.0      # chunk 0: ranks 1, 2, 0
    values[2][1], values[0][1], values[1][1] = 1.0, 1.0, 256.0      # chunk 1: ranks 2, 0, 1
    values[0][2], values[1][2], values[2][2] = 256.0, 3.0, 1.0      # chunk 2: ranks 0, 1, 2: 259 -> 260, 261 -> 260
    A, B = scalar_shards(P, 1, values)
    out = ops.gemm_rs(A, B, rings=1, bf16_hops=True)
    assert [float(o[0, 0]) for o in out] == [256.0, 258.0, 260.0]
    exact = ops.gemm_rs(A, B, rings=1)
    assert [float(o[0, 0]) for o in exact] == [258.0, 258.0, 260.0]


def test_bf16_hops_double_ring_halves_travel_in_opposite_directions():
    """P = 4, two rows per chunk.  Chunk 0's first row rides the backward ring (ranks 3, 2, 1, then the owner 0), its
    second row the forward ring (ranks 1, 2, 3, 0).  With rank 1 holding 256 and ranks 2, 3 holding 1:
    backward 1 + 1 = 2, + 256 = 258; forward 256 + 1 -> 256, + 1 -> 256."""
    P, m = 4, 2
    values = np.zeros((P, P * m))
    for row in (0, 1):
        values[1][row], values[2][row], values[3][row] = 256.0, 1.0, 1.0
    A, B = scalar_shards(P, m, values)
    out = ops.gemm_rs(A, B, rings=2, bf16_hops=True)
    assert float(out[0][0, 0]) == 258.0 and float(out[0][1, 0]) == 256.0
    sampled = ops.gemm_rs_rows(A, B, np.array([0, 1]), rings=2, bf16_hops=True)
    assert list(sampled[0][1][:, 0]) == [258.0, 256.0]


def test_bf16_hops_change_nothing_when_every_running_sum_is_a_bf16_value():
    w = wl.Workload("ints", OP_GEMM_RS, P=4, M=32, N=8, K=16)
    A, B = wl.make_structured_inputs(w, "index")
    exact = ops.gemm_rs(A, B)
    assert max(float(np.max(np.abs(e))) for e in exact) <= 256.0          # integers up to 256 are BF16 values
    for got, want in zip(ops.gemm_rs(A, B, bf16_hops=True), exact):
        assert np.array_equal(got, want)


@pytest.mark.parametrize("P", [1, 2, 5, 8])
def test_bf16_hops_error_bound(P):
    """Each hop rounds to nearest: at most half a BF16 step (8 significant bits: 2^-8 relative) of the sum after that
    hop, plus the FP32 rounding of the addition.  P = 1 is the correctly rounded product."""
    w, A, B = tiny(OP_GEMM_RS, P, P * 8, 16, 24, seed=11)
    exact = ops.gemm_rs(A, B)
    got = ops.gemm_rs(A, B, bf16_hops=True)
    prefix_max = np.zeros_like(np.concatenate(exact))
    table = schedule(OP_GEMM_RS, P, 2, w.M)
    Bf = [ops.bf16_bits_to_f64(b) for b in B]
    partial = [ops.bf16_bits_to_f64(A[q]) @ Bf[q].T for q in range(P)]
    for row in range(w.M):                                            # largest |prefix sum| along the row's ring
        order = [int(e[0]) for e in sorted((e for e in table if e[6] <= row < e[6] + e[7]), key=lambda e: int(e[1]))]
        run = np.zeros(w.N)
        for q in order:
            run = run + partial[q][row]
            prefix_max[row] = np.maximum(prefix_max[row], np.abs(run))
    err = np.abs(np.concatenate(got) - np.concatenate(exact))
    assert (err <= P * (2.0 ** -8 + 2.0 ** -23) * prefix_max * (1 + P * 2.0 ** -8)).all()
    if P == 1:
        want = torch.from_numpy(exact[0].astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
        assert np.array_equal(got[0], want)
    else:
        assert any(not np.array_equal(g, ops.f64_to_bf16_f64(e)) for g, e in zip(got, exact))   # the hops do show


def test_rule_for_a_bf16_ring_tells_the_order_of_the_contributors():
    """The hop-by-hop ring passes its own rule; the same sum reduced in the single ring's order (every partition
    forward) or rounded once at the end is the right sum, within every tolerance against the exact result, and still
    fails: too few elements are identical."""
    w, A, B = tiny(OP_GEMM_RS, 8, 8 * 16, 24, 40, seed=7)
    exact = ops.gemm_rs(A, B, rings=2)
    hops = ops.gemm_rs(A, B, rings=2, bf16_hops=True)
    other = ops.gemm_rs(A, B, rings=1, bf16_hops=True)
    to_bits = lambda x: wl.f32_to_bf16_bits(x.astype(np.float32))
    for c in range(8):
        assert compare.check_bf16_ring(to_bits(hops[c]), exact[c], hops[c], 8, 40).ok
        wrong = compare.check_bf16_ring(to_bits(other[c]), exact[c], hops[c], 8, 40)
        assert not wrong.ok and wrong.identical < 0.95 and wrong.exact.violations == 0
        once = compare.check_bf16_ring(to_bits(exact[c]), exact[c], hops[c], 8, 40)
        assert not once.ok and once.exact.ok


def test_bf16_hops_in_groups_round_once_per_group():
    """Forward ring, P = 4, one row per chunk; chunk 0's contributors are ranks 1, 2, 3, 0.  With 256, 1, 1, 1:
    hop by hop 256 + 1 -> 256 three times; in groups of two (256 + 1 = 257 -> 256, then 1 + 1 = 2 added: 258);
    in one group of four the exact 259 rounds to 260 (tie to even).  Groups of one are the plain hops, and without
    BF16 hops the grouping changes nothing."""
    P = 4
    values = np.zeros((P, P))
    values[1][0], values[2][0], values[3][0], values[0][0] = 256.0, 1.0, 1.0, 1.0
    A, B = scalar_shards(P, 1, values)
    got = {g: float(ops.gemm_rs(A, B, rings=1, bf16_hops=True, hop_group=g)[0][0, 0]) for g in (1, 2, 4)}
    assert got == {1: 256.0, 2: 258.0, 4: 260.0}
    assert float(ops.gemm_rs(A, B, rings=1, hop_group=2)[0][0, 0]) == 259.0
    w, A, B = tiny(OP_GEMM_RS, 8, 8 * 16, 24, 40, seed=9)
    for g in (2, 4, 8):
        grouped = ops.gemm_rs(A, B, bf16_hops=True, hop_group=g)
        rows = np.array([0, 5, 17, 40, 127])
        sampled = ops.gemm_rs_rows(A, B, rows, bf16_hops=True, hop_group=g)
        for c, (local, vals) in sampled.items():
            assert np.array_equal(vals, grouped[c][local])
    once = ops.gemm_rs(A, B, bf16_hops=True, hop_group=8)                      # one rounding of the FP32 sum
    exact = ops.gemm_rs(A, B)
    for o, e in zip(once, exact):
        assert np.array_equal(o, ops.fp32_to_bf16_rne(e.astype(np.float32)))
