"""GPU parity of the tensor-parallel MLP block (Section II-A, the two-layer MLP
figure): compass_mlp_block against oracle.mlp on the same seeded inputs.

Both the BF16 intermediate H (GEMM0 + activation) and the block's output are
checked with the acceptance rule of oracle.compare.  The oracle rounds the
exact FP64 activation once to BF16; the kernel rounds its FP32 value, so a few
elements of H differ by one BF16 step between the two sides -- far inside the
tolerance, and what the RMS limit on the output accounts for."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import mlp as omlp
from oracle import operators as ops
from paper_2609_10549_b200 import api
from paper_2609_10549_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

ACTS = [omlp.ACT_NONE, omlp.ACT_GELU_TANH, omlp.ACT_SWIGLU]


def make_inputs(P, m, hidden, ffn, act, seed=3):
    w = wl.MlpWorkload(f"mlp-{P}-{m}-{hidden}-{ffn}-{act}", P=P, M=P * m, hidden=hidden, ffn=ffn, activation=act, seed=seed)
    assert w.hc == omlp.hidden_columns(ffn, act)
    X, W0, W1 = wl.make_mlp_inputs(w)
    return X, W0, W1, w.hc


def run_block(P, m, hidden, ffn, act, X, W0, W1, hc, rings=2, rs_variant=api.RS_SEGMENTED_K, order=api.ORDER_RANK_MAJOR):
    mp = api.make_mlp(P, P * m, hidden, ffn, activation=act, rings=rings, rs_variant=rs_variant, order=order)
    dX, dW0, dW1 = [api.to_device(a) for a in X], [api.to_device(a) for a in W0], [api.to_device(a) for a in W1]
    H = [gu.Guarded(P * m, hc) for _ in range(P)]
    Out = [gu.Guarded(m, hidden) for _ in range(P)]
    ws = api.alloc_mlp_workspace(mp)
    before = api.kernel_launch_count()
    api.compass_mlp_block(mp, dX, dW0, [h.view for h in H], dW1, [o.view for o in Out], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    assert api.kernel_launch_count() == before + 2                       # two fused kernels, nothing else
    assert all(t.guards_intact() for t in H + Out)
    return [h.bits() for h in H], [o.bits() for o in Out]


def check_block(P, m, hidden, ffn, act, **kw):
    X, W0, W1, hc = make_inputs(P, m, hidden, ffn, act)
    H_gpu, Out_gpu = run_block(P, m, hidden, ffn, act, X, W0, W1, hc, **kw)
    Out_ref, H_ref_bits = omlp.mlp_block(X, W0, W1, act, rings=kw.get("rings", 2))
    C = ops.ag_gemm(X, W0, rings=kw.get("rings", 2))
    for r in range(P):
        rep = compare.check(H_gpu[r], omlp.activation(C[r], act))
        assert rep.ok, f"H rank {r}: {rep}"
        # the two sides' BF16 intermediates agree except for single-step rounding differences
        diff = np.abs(H_gpu[r].astype(np.int32) - H_ref_bits[r].astype(np.int32))
        same_sign = (H_gpu[r] >> 15) == (H_ref_bits[r] >> 15)
        assert (diff[same_sign] <= 1).mean() > 0.999
        rep = compare.check(Out_gpu[r], Out_ref[r])
        assert rep.ok, f"Out rank {r}: {rep}"


@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("P,m,hidden,ffn,rings", [
    (1, 128, 64, 256, 2), (2, 256, 256, 512, 2), (2, 144, 72, 272, 2), (4, 384, 320, 1024, 1), (8, 80, 200, 48, 2),
    (3, 272, 344, 528, 2),
])
def test_mlp_block_small_shapes(P, m, hidden, ffn, rings, act):
    check_block(P, m, hidden, ffn, act, rings=rings)


# 512-row partitions: the first kernel runs 512x256 and 256x256 tiles in one launch; ffn = 2576 leaves a
# ragged last column tile (16 columns, 8 after SwiGLU)
@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("order", [api.ORDER_RANK_MAJOR, api.ORDER_STEP_MAJOR])
def test_mlp_block_big_tiles_and_ragged_columns(act, order):
    check_block(4, 1024, 456, 2576, act, order=order)


@pytest.mark.parametrize("act", [omlp.ACT_GELU_TANH, omlp.ACT_SWIGLU])
def test_mlp_block_with_ring_rmw_reduction(act):
    X, W0, W1, hc = make_inputs(4, 512, 256, 768, act)
    H_gpu, Out_gpu = run_block(4, 512, 256, 768, act, X, W0, W1, hc, rs_variant=api.RS_RING_RMW)
    Out_ref, _ = omlp.mlp_block(X, W0, W1, act)
    for r in range(4):
        rep = compare.check(Out_gpu[r], Out_ref[r])
        # the running sum lives in the BF16 output rows: one rounding per contributor
        assert rep.violations == 0 and rep.rms_rel <= np.sqrt(4) * 2.0 ** -9, f"rank {r}: {rep}"


def test_mlp_block_with_ring_reduction_in_fp32_scratch():
    """The block's second kernel as the ring read-modify-write with the running sum in FP32 scratch (the block's
    workspace holds it): the single-rounding limits apply."""
    act = omlp.ACT_SWIGLU
    X, W0, W1, hc = make_inputs(4, 512, 256, 768, act)
    H_gpu, Out_gpu = run_block(4, 512, 256, 768, act, X, W0, W1, hc, rs_variant=api.RS_RING_RMW_F32)
    Out_ref, _ = omlp.mlp_block(X, W0, W1, act)
    for r in range(4):
        rep = compare.check(Out_gpu[r], Out_ref[r])
        assert rep.ok, f"rank {r}: {rep}"


def test_activation_special_values():
    """Accumulator values that stress the activations: zero and large magnitudes of either sign."""
    P, m, hidden, ffn = 1, 128, 16, 256
    X = [wl.f32_to_bf16_bits(np.eye(m, hidden, dtype=np.float32) * 64.0)]         # row i selects 64 * W0[:, i]
    rng = np.random.default_rng(0)
    w0 = rng.standard_normal((ffn, hidden)).astype(np.float32)
    w0[:, 0] = 0.0                                                                 # row 0: all zeros
    w0[:, 1] = 8.0                                                                 # row 1: +512 everywhere
    w0[:, 2] = -8.0                                                                # row 2: -512 everywhere
    w0[0::2, 3], w0[1::2, 3] = 8.0, -0.5                                            # row 3: gate +512, up -32
    w0[0::2, 4], w0[1::2, 4] = -8.0, 0.5                                            # row 4: gate -512
    W0 = [wl.f32_to_bf16_bits(w0)]
    for act in ACTS:
        hc = omlp.hidden_columns(ffn, act)
        W1 = [wl.f32_to_bf16_bits(np.eye(hidden, hc, dtype=np.float32))]
        H_gpu, _ = run_block(P, m, hidden, ffn, act, X, W0, W1, hc)
        ref = omlp.activation(ops.ag_gemm(X, W0)[0], act)
        got = ops.bf16_bits_to_f64(H_gpu[0])
        assert np.isfinite(got).all()
        assert (got[0] == 0.0).all()
        rep = compare.check(H_gpu[0], ref)
        assert rep.ok, f"act {act}: {rep}"
        if act == omlp.ACT_GELU_TANH:
            assert (got[1] == 512.0).all() and (got[2] == 0.0).all()
        if act == omlp.ACT_SWIGLU:
            assert (got[3] == 512.0 * -32.0).all() and (got[4] == 0.0).all()


def test_mlp_block_7b_shape_sampled():
    """LLaMA-7B MLP over 8 ranks: hidden 4096, 11008 / 8 = 1376 gate and up columns per rank (interleaved),
    8192 tokens; the second kernel is the GEMM+ReduceScatter of benchmark config 3."""
    w = wl.MLP_7B
    P, m, hidden, ffn, act, hc = w.P, w.m, w.hidden, w.ffn, w.activation, w.hc
    X, W0, W1 = wl.make_mlp_inputs(w)
    assert (act, hc, hidden, P * m) == (omlp.ACT_SWIGLU, wl.C3_RS.K, wl.C3_RS.N, wl.C3_RS.M)
    H_gpu, Out_gpu = run_block(P, m, hidden, ffn, act, X, W0, W1, hc)
    rows = gu.sample_rows(P * m, P, 2, tile=256, frac=0.002, seed=1)
    H_rows, found = omlp.mlp_block_rows(X, W0, W1, act, rows)
    C_rows = ops.ag_gemm(X, W0, rows=rows)
    for r in range(P):
        rep = compare.check(H_gpu[r][rows], omlp.activation(C_rows[r], act))
        assert rep.ok, f"H rank {r}: {rep}"
    seen = 0
    for c, (local, ref) in found.items():
        rep = compare.check(Out_gpu[c][local], ref)
        assert rep.ok, f"Out rank {c}: {rep}"
        seen += len(local)
    assert seen == len(rows)


def test_mlp_block_repeated_calls_are_bitwise_identical():
    P, m, hidden, ffn, act = 4, 512, 256, 1024, omlp.ACT_SWIGLU
    X, W0, W1, hc = make_inputs(P, m, hidden, ffn, act)
    a = run_block(P, m, hidden, ffn, act, X, W0, W1, hc)
    b = run_block(P, m, hidden, ffn, act, X, W0, W1, hc)
    for x, y in zip(a[0] + a[1], b[0] + b[1]):
        assert (x == y).all()


def test_backward_data_gradients_are_the_block_on_the_stored_weights():
    """dH_r = gather(dOut) * W1_r and dX = ReduceScatter(sum_q dH_q * W0_q): the block itself, called with
    the weights as stored ([hidden x hc] and [ffn x hidden]) and the [K][N] layout flag."""
    P, m, hidden, ffn = 4, 512, 264, 1040
    w = wl.MlpWorkload("mlp-bwd", P=P, M=P * m, hidden=hidden, ffn=ffn, activation=omlp.ACT_NONE, seed=5)
    dOut, W0, W1 = wl.make_mlp_inputs(w)                     # dOut_r [m x hidden], W0_r [ffn x hidden], W1_r [hidden x ffn]
    mp = api.make_mlp(P, P * m, hidden, ffn, activation=api.ACT_NONE, b_layout=api.B_KN)
    d_dOut, dW0, dW1 = [api.to_device(a) for a in dOut], [api.to_device(a) for a in W0], [api.to_device(a) for a in W1]
    dH = [gu.Guarded(P * m, ffn) for _ in range(P)]
    dX = [gu.Guarded(m, hidden) for _ in range(P)]
    ws = api.alloc_mlp_workspace(mp)
    api.compass_mlp_block(mp, d_dOut, dW1, [t.view for t in dH], dW0, [t.view for t in dX], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    assert all(t.guards_intact() for t in dH + dX)
    # oracle: the same chain with the weights written the way its GEMMs take them ([N][K])
    W1_t = [np.ascontiguousarray(a.T) for a in W1]            # [ffn x hidden]
    W0_t = [np.ascontiguousarray(a.T) for a in W0]            # [hidden x ffn]
    dX_ref, dH_ref_bits = omlp.mlp_block(dOut, W1_t, W0_t, omlp.ACT_NONE)
    C = ops.ag_gemm(dOut, W1_t)
    for r in range(P):
        rep = compare.check(dH[r].bits(), C[r])
        assert rep.ok, f"dH rank {r}: {rep}"
        rep = compare.check(dX[r].bits(), dX_ref[r])
        assert rep.ok, f"dX rank {r}: {rep}"


def test_mlp_block_kn_weights_match_nk_weights_bitwise():
    P, m, hidden, ffn, act = 4, 512, 256, 1056, omlp.ACT_SWIGLU
    X, W0, W1, hc = make_inputs(P, m, hidden, ffn, act)
    nk = run_block(P, m, hidden, ffn, act, X, W0, W1, hc)
    mp = api.make_mlp(P, P * m, hidden, ffn, activation=act, b_layout=api.B_KN)
    dX = [api.to_device(a) for a in X]
    dW0 = [api.to_device(np.ascontiguousarray(a.T)) for a in W0]
    dW1 = [api.to_device(np.ascontiguousarray(a.T)) for a in W1]
    H = [gu.Guarded(P * m, hc) for _ in range(P)]
    Out = [gu.Guarded(m, hidden) for _ in range(P)]
    ws = api.alloc_mlp_workspace(mp)
    api.compass_mlp_block(mp, dX, dW0, [h.view for h in H], dW1, [o.view for o in Out], ws)
    assert api.compass_read_status(ws) == (api.OK, 0)
    for got, want in zip([h.bits() for h in H] + [o.bits() for o in Out], nk[0] + nk[1]):
        assert (got == want).all()
