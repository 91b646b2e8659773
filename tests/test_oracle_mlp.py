"""Pins of the MLP-block oracle (Section II-A, the two-layer MLP figure):
library routines it does not call (torch's BF16 conversion, torch's GELU and
SiLU), closed forms, a brute-force triple loop without sharding, and the
unsharded definition of the block."""
import math

import numpy as np
import pytest
import torch

from oracle import mlp
from oracle import operators as ops
from paper_2609_10549_b200 import workloads as wl


def _bf16_bits(rng, shape, scale=1.0):
    return wl.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


# ---- rounding to BF16 ---------------------------------------------------------

def test_bf16_rounding_agrees_with_torch_on_float32_values():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(5000) * 1e-30).astype(np.float32),
        (rng.standard_normal(5000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 1.00390625, 1.01171875, 255.5, 3.3895314e38, 1e-40, -1e-40, 9.2e-41],
                 dtype=np.float32),
        # exact ties between neighbouring BF16 values: even significand wins
        (np.arange(128, 256, dtype=np.float32) + 0.5) * np.float32(2.0 ** -7),
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = mlp.f64_to_bf16_bits(x.astype(np.float64))
    assert (got == want).all()


def test_bf16_rounding_is_a_single_rounding():
    # 1 + 2^-8 is the tie between 1 and 1 + 2^-7; a hair above it must round up.  Rounding to
    # FP32 first would land on the tie and then go down to 1.0 (even significand).
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30, 1.0 + 2.0 ** -8 - 2.0 ** -30, 1.0 + 2.0 ** -8])
    assert mlp.f64_to_bf16_bits(x).tolist() == [0x3F81, 0x3F80, 0x3F80]
    assert mlp.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8])).tolist() == [0x3F82]      # tie, odd below: up


def test_bf16_rounding_roundtrip_and_monotone():
    bits = np.arange(0x0001, 0x7F80, 7, dtype=np.uint16)                 # positive finite BF16 values
    vals = ops.bf16_bits_to_f64(bits)
    assert (mlp.f64_to_bf16_bits(vals) == bits).all()
    assert (mlp.f64_to_bf16_bits(-vals) == (bits | 0x8000)).all()
    x = np.sort(np.random.default_rng(1).standard_normal(5000))
    r = ops.bf16_bits_to_f64(mlp.f64_to_bf16_bits(x))
    assert (np.diff(r) >= 0).all()
    assert (np.abs(r - x) <= np.abs(x) * 2.0 ** -8).all()                 # within half a unit in the last place


# ---- activations ----------------------------------------------------------------

def test_gelu_matches_torch_and_closed_forms():
    x = np.random.default_rng(2).standard_normal(10000) * 3.0
    want = torch.nn.functional.gelu(torch.from_numpy(x), approximate="tanh").numpy()
    assert np.allclose(mlp.activation(x, mlp.ACT_GELU_TANH), want, rtol=1e-13, atol=1e-15)
    assert mlp.activation(np.array([0.0]), mlp.ACT_GELU_TANH)[0] == 0.0
    assert mlp.activation(np.array([30.0]), mlp.ACT_GELU_TANH)[0] == 30.0
    assert abs(mlp.activation(np.array([-30.0]), mlp.ACT_GELU_TANH)[0]) < 1e-300
    one = 0.5 * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * 1.044715))
    assert mlp.activation(np.array([1.0]), mlp.ACT_GELU_TANH)[0] == pytest.approx(one, rel=1e-15)


def test_swiglu_matches_torch_and_takes_gate_from_even_columns():
    rng = np.random.default_rng(3)
    c = rng.standard_normal((50, 24)) * 4.0
    gate, up = torch.from_numpy(c[:, 0::2].copy()), torch.from_numpy(c[:, 1::2].copy())
    want = (torch.nn.functional.silu(gate) * up).numpy()
    got = mlp.activation(c, mlp.ACT_SWIGLU)
    assert got.shape == (50, 12)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-300)
    # gate = 0 kills the product, a large gate passes `up` times the gate, swapping the roles changes the result
    assert (mlp.activation(np.array([[0.0, 7.0]]), mlp.ACT_SWIGLU) == 0.0).all()
    assert mlp.activation(np.array([[40.0, 0.5]]), mlp.ACT_SWIGLU)[0, 0] == pytest.approx(20.0, rel=1e-15)
    assert mlp.activation(np.array([[0.5, 40.0]]), mlp.ACT_SWIGLU)[0, 0] == pytest.approx(0.5 / (1 + math.exp(-0.5)) * 40.0)
    assert mlp.activation(np.array([[-800.0, 1.0]]), mlp.ACT_SWIGLU)[0, 0] == 0.0       # exp overflows, the quotient is -0


def test_identity_activation_returns_its_argument():
    c = np.random.default_rng(4).standard_normal((3, 5))
    assert mlp.activation(c, mlp.ACT_NONE) is c
    with pytest.raises(ValueError):
        mlp.activation(c, 9)


# ---- the block --------------------------------------------------------------------

def _unsharded(X, W0, W1, act):
    """The block without sharding: one input, the ranks' weight slices put back together."""
    Xf = np.concatenate([ops.bf16_bits_to_f64(x) for x in X])
    H = []
    for w0 in W0:                                           # column-parallel: every rank owns output columns
        c = Xf @ ops.bf16_bits_to_f64(w0).T
        H.append(ops.bf16_bits_to_f64(mlp.f64_to_bf16_bits(mlp.activation(c, act))))
    Hf = np.concatenate(H, axis=1)
    W1f = np.concatenate([ops.bf16_bits_to_f64(w1) for w1 in W1], axis=1)      # row-parallel: slices of K
    return Hf @ W1f.T


@pytest.mark.parametrize("act", [mlp.ACT_NONE, mlp.ACT_GELU_TANH, mlp.ACT_SWIGLU])
@pytest.mark.parametrize("P,m,hidden,ffn,rings", [(1, 4, 8, 8, 2), (2, 6, 16, 12, 2), (4, 4, 8, 16, 1), (3, 2, 24, 8, 2)])
def test_block_equals_the_unsharded_mlp(P, m, hidden, ffn, rings, act):
    rng = np.random.default_rng(10 * P + act)
    hc = mlp.hidden_columns(ffn, act)
    X = [_bf16_bits(rng, (m, hidden)) for _ in range(P)]
    W0 = [_bf16_bits(rng, (ffn, hidden), 0.3) for _ in range(P)]
    W1 = [_bf16_bits(rng, (hidden, hc), 0.3) for _ in range(P)]
    Out, H = mlp.mlp_block(X, W0, W1, act, rings=rings)
    assert all(h.shape == (P * m, hc) and h.dtype == np.uint16 for h in H)
    want = _unsharded(X, W0, W1, act)
    got = np.concatenate(Out)
    assert got.shape == (P * m, hidden)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)          # only the order of the FP64 sums differs


def test_block_against_a_triple_loop():
    """P = 2, every product written out: catches a transposed weight or a swapped gate/up pair."""
    rng = np.random.default_rng(5)
    P, m, hidden, ffn = 2, 2, 4, 4
    X = [_bf16_bits(rng, (m, hidden)) for _ in range(P)]
    W0 = [_bf16_bits(rng, (ffn, hidden)) for _ in range(P)]
    W1 = [_bf16_bits(rng, (hidden, ffn // 2)) for _ in range(P)]
    Out, _ = mlp.mlp_block(X, W0, W1, mlp.ACT_SWIGLU)
    x = [ops.bf16_bits_to_f64(a) for a in X]
    w0 = [ops.bf16_bits_to_f64(a) for a in W0]
    w1 = [ops.bf16_bits_to_f64(a) for a in W1]
    for row in range(P * m):
        xr = x[row // m][row % m]
        for n in range(hidden):
            total = 0.0
            for q in range(P):
                for j in range(ffn // 2):
                    gate = sum(xr[k] * w0[q][2 * j][k] for k in range(hidden))
                    up = sum(xr[k] * w0[q][2 * j + 1][k] for k in range(hidden))
                    h = gate / (1.0 + math.exp(-gate)) * up
                    h = float(ops.bf16_bits_to_f64(mlp.f64_to_bf16_bits(np.array([h])))[0])
                    total += h * w1[q][n][j]
            assert Out[row // m][row % m, n] == pytest.approx(total, rel=1e-12, abs=1e-12)


def test_identity_block_with_one_hot_weights_routes_the_input():
    """W0 = W1 = identity and no activation: the block is AllGather followed by ReduceScatter of P equal
    copies... of disjoint column slices, i.e. every rank gets its own rows back."""
    P, m, hidden = 4, 4, 8
    rng = np.random.default_rng(6)
    X = [_bf16_bits(rng, (m, hidden)) for _ in range(P)]
    eye = np.eye(hidden, dtype=np.float32)
    per = hidden // P
    W0 = [wl.f32_to_bf16_bits(eye[r * per:(r + 1) * per]) for r in range(P)]            # rank r keeps columns of its slice
    W1 = [wl.f32_to_bf16_bits(eye[:, r * per:(r + 1) * per].copy()) for r in range(P)]  # and puts them back in place
    Out, H = mlp.mlp_block(X, W0, W1, mlp.ACT_NONE)
    for r in range(P):
        assert (Out[r] == ops.bf16_bits_to_f64(X[r])).all()
        assert (H[r] == np.concatenate(X)[:, r * per:(r + 1) * per]).all()


def test_sampled_rows_agree_with_the_full_block():
    rng = np.random.default_rng(7)
    P, m, hidden, ffn = 4, 8, 16, 24
    X = [_bf16_bits(rng, (m, hidden)) for _ in range(P)]
    W0 = [_bf16_bits(rng, (ffn, hidden), 0.3) for _ in range(P)]
    W1 = [_bf16_bits(rng, (hidden, ffn), 0.3) for _ in range(P)]
    Out, H = mlp.mlp_block(X, W0, W1, mlp.ACT_GELU_TANH)
    rows = np.array([0, 3, 4, 9, 17, 30, 31])
    H_rows, found = mlp.mlp_block_rows(X, W0, W1, mlp.ACT_GELU_TANH, rows)
    for r in range(P):
        assert (H_rows[r] == H[r][rows]).all()
    seen = 0
    for c, (local, vals) in found.items():
        assert np.allclose(vals, Out[c][local], rtol=1e-12, atol=1e-12)
        seen += len(local)
    assert seen == len(rows)
