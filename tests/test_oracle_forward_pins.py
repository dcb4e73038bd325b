"""Pins for the oracle's forward pass (Eq. 2 then Eq. 3) and its bf16 rounding (no GPU)."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import ACT_GELU_TANH, ACT_RELU, ACT_SILU

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "mlp_forward_handworked.json")


def _cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"])
def test_handworked_forward(case):
    Z, H = oracle.mlp_forward(np.array(case["X"], dtype=np.float32), case["Wg"], case["Wu"], case["Wd"],
                              case["act"], False, want_h=True)
    rel = case.get("rel", 0.0)
    np.testing.assert_allclose(H, np.array(case["H"], dtype=np.float64), rtol=rel, atol=0.0)
    np.testing.assert_allclose(Z, np.array(case["Z"], dtype=np.float64), rtol=rel, atol=0.0)


# --------------------------------------------------------------------------- bf16 rounding

def test_round_bf16_hand_picked():
    # 8 significant bits: spacing in [1, 2) is 2^-7
    assert oracle.round_bf16(1.0) == 1.0
    assert oracle.round_bf16(1.0 + 2.0 ** -8) == 1.0                      # tie -> even mantissa (1.0)
    assert oracle.round_bf16(1.0 + 3.0 * 2.0 ** -8) == 1.0 + 2.0 ** -6    # tie -> even mantissa (1 + 2/128)
    assert oracle.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -30) == 1.0 + 2.0 ** -7   # just above the tie
    assert oracle.round_bf16(-(1.0 + 2.0 ** -8 + 2.0 ** -30)) == -(1.0 + 2.0 ** -7)
    assert oracle.round_bf16(255.5) == 256.0                              # carries into the next binade
    assert oracle.round_bf16(0.0) == 0.0
    assert oracle.round_bf16(2.0 ** -133) == 2.0 ** -133                   # smallest subnormal
    assert oracle.round_bf16(2.0 ** -134) == 0.0                           # tie between 0 and 2^-133 -> even (0)
    assert oracle.round_bf16(3.0 * 2.0 ** -134) == 2.0 ** -132             # tie -> even


def test_round_bf16_matches_torch_conversion():
    # float32 inputs: torch's float32 -> bfloat16 conversion is round-to-nearest-even on the same value
    rng = np.random.default_rng(11)
    v = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-30, 30, 4000),
                        rng.standard_normal(500) * 1e-39,                 # subnormal range
                        np.ldexp(1.0 + np.arange(256) / 128.0 + 1.0 / 256.0, rng.integers(-20, 20, 256))])   # exact ties
    v32 = v.astype(np.float32)
    want = torch.from_numpy(v32).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.round_bf16(float(x)) for x in v32])
    finite = np.isfinite(want)
    np.testing.assert_array_equal(got[finite], want[finite])


# --------------------------------------------------------------------------- Eq. 2 + Eq. 3

@pytest.mark.parametrize("kind", [ACT_SILU, ACT_GELU_TANH, ACT_RELU])
def test_forward_is_matmul_composition(kind):
    # the same layer through numpy's float64 matmul and torch's float64 activations
    rng = np.random.default_rng(5 + kind)
    T, d, I = 7, 12, 20
    X = rng.standard_normal((T, d)).astype(np.float32)
    Wg = rng.standard_normal((I, d)).astype(np.float32)
    Wu = rng.standard_normal((I, d)).astype(np.float32)
    Wd = rng.standard_normal((d, I)).astype(np.float32)
    G = torch.from_numpy(X.astype(np.float64) @ Wg.astype(np.float64).T)
    U = X.astype(np.float64) @ Wu.astype(np.float64).T
    if kind == ACT_SILU:
        A = torch.nn.functional.silu(G)
    elif kind == ACT_GELU_TANH:
        A = torch.nn.functional.gelu(G, approximate="tanh")
    else:
        A = torch.relu(G)
    H_ref = A.numpy() * U
    Z_ref = H_ref @ Wd.astype(np.float64).T
    Z, H = oracle.mlp_forward(X, Wg, Wu, Wd, kind, False, want_h=True)
    np.testing.assert_allclose(H, H_ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(Z, Z_ref, rtol=1e-11, atol=1e-12)


def test_forward_identity_down_projection_returns_h():
    # Wd = identity (d = I): Eq. 3 returns y unchanged, and y is what calib_sumsq sums the squares of
    rng = np.random.default_rng(9)
    T, n = 5, 9
    X = rng.standard_normal((T, n)).astype(np.float32)
    Wg = rng.standard_normal((n, n)).astype(np.float32)
    Wu = rng.standard_normal((n, n)).astype(np.float32)
    Z, H = oracle.mlp_forward(X, Wg, Wu, np.eye(n, dtype=np.float32), ACT_SILU, False, want_h=True)
    np.testing.assert_array_equal(Z, H)
    np.testing.assert_allclose((H * H).sum(axis=0), oracle.calib_sumsq(X, Wg, Wu, ACT_SILU), rtol=1e-13)
    for t in range(T):
        np.testing.assert_allclose(H[t], oracle.glu_row(X[t], Wg, Wu, ACT_SILU), rtol=1e-14, atol=0)


def test_forward_one_hot_down_rows_pick_neurons():
    # a down-projection row that is one-hot at neuron j (times c) outputs c * y_j: catches a transposed Wd
    rng = np.random.default_rng(10)
    T, d, I = 4, 3, 6
    X = rng.standard_normal((T, d)).astype(np.float32)
    Wg = rng.standard_normal((I, d)).astype(np.float32)
    Wu = rng.standard_normal((I, d)).astype(np.float32)
    Wd = np.zeros((d, I), dtype=np.float32)
    Wd[0, 4] = 2.0
    Wd[1, 0] = -1.0
    Wd[2, 5] = 0.5
    Z, H = oracle.mlp_forward(X, Wg, Wu, Wd, ACT_GELU_TANH, False, want_h=True)
    np.testing.assert_array_equal(Z[:, 0], 2.0 * H[:, 4])
    np.testing.assert_array_equal(Z[:, 1], -H[:, 0])
    np.testing.assert_array_equal(Z[:, 2], 0.5 * H[:, 5])


def test_forward_linear_in_wd_and_masking_equals_dropping():
    rng = np.random.default_rng(12)
    T, d, I = 6, 8, 16
    X = rng.standard_normal((T, d)).astype(np.float32)
    Wg = rng.standard_normal((I, d)).astype(np.float32)
    Wu = rng.standard_normal((I, d)).astype(np.float32)
    Wa = rng.integers(-4, 5, (d, I)).astype(np.float32)
    Wb = rng.integers(-4, 5, (d, I)).astype(np.float32)
    Za = oracle.mlp_forward(X, Wg, Wu, Wa, ACT_SILU, False)
    Zb = oracle.mlp_forward(X, Wg, Wu, Wb, ACT_SILU, False)
    Zs = oracle.mlp_forward(X, Wg, Wu, Wa + Wb, ACT_SILU, False)
    np.testing.assert_allclose(Zs, Za + Zb, rtol=1e-12, atol=1e-12)
    # zeroing column j of Wd (pruning every weight that reads neuron j) = removing neuron j from the layer
    keep = np.ones(I, dtype=bool)
    keep[[3, 7, 8]] = False
    Wm = Wa.copy()
    Wm[:, ~keep] = 0.0
    Zm = oracle.mlp_forward(X, Wg, Wu, Wm, ACT_SILU, False)
    Zd = oracle.mlp_forward(X, Wg[keep], Wu[keep], Wa[:, keep], ACT_SILU, False)
    np.testing.assert_allclose(Zm, Zd, rtol=1e-12, atol=1e-12)


def test_forward_h_round_rounds_only_the_intermediate():
    rng = np.random.default_rng(13)
    T, d, I = 5, 10, 12
    X = rng.standard_normal((T, d)).astype(np.float32)
    Wg = rng.standard_normal((I, d)).astype(np.float32)
    Wu = rng.standard_normal((I, d)).astype(np.float32)
    Wd = rng.standard_normal((d, I)).astype(np.float32)
    _, H = oracle.mlp_forward(X, Wg, Wu, Wd, ACT_SILU, False, want_h=True)
    Zr, Hr = oracle.mlp_forward(X, Wg, Wu, Wd, ACT_SILU, True, want_h=True)
    want_h = torch.from_numpy(H.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    # (double -> float32 -> bf16 can differ from double -> bf16 only at a double-rounding tie: none in 60 values)
    np.testing.assert_array_equal(Hr, want_h)
    np.testing.assert_allclose(Zr, Hr @ Wd.astype(np.float64).T, rtol=1e-12, atol=1e-12)
