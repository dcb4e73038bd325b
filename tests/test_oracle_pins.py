"""Pins for the fp64 CPU oracle (no GPU): each check ties an oracle function to something
other than itself -- closed forms, hand-worked fixtures, exact-rational brute force,
a library routine on a special case, or an invariant the paper's definitions imply."""
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import ACT_GELU_TANH, ACT_RELU, ACT_SILU, AXIS_COLS, AXIS_ROWS

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "nm_handworked.json")


# --------------------------------------------------------------------------- activations

@pytest.mark.parametrize("kind", [ACT_SILU, ACT_GELU_TANH, ACT_RELU])
def test_act_zero_and_limits(kind):
    assert oracle.act(kind, 0.0) == 0.0
    assert oracle.act(kind, 40.0) == pytest.approx(40.0, rel=1e-15)
    assert abs(oracle.act(kind, -40.0)) < 1e-15


@pytest.mark.parametrize("kind", [ACT_SILU, ACT_GELU_TANH, ACT_RELU])
def test_act_odd_part_identity(kind):
    # x*s(x) with s(x)+s(-x)=1 (sigmoid, 0.5(1+tanh), step): act(x) - act(-x) = x
    for x in np.linspace(0.01, 12.0, 57):
        assert oracle.act(kind, x) - oracle.act(kind, -x) == pytest.approx(x, rel=1e-13)


def test_act_known_values():
    # silu(1) = 1/(1+e^-1); silu(ln 3) = ln3 * 3/4
    assert oracle.act(ACT_SILU, 1.0) == pytest.approx(1.0 / (1.0 + math.exp(-1.0)), rel=1e-15)
    assert oracle.act(ACT_SILU, math.log(3.0)) == pytest.approx(math.log(3.0) * 0.75, rel=1e-14)
    # tanh-GeLU at 1: 0.5*(1+tanh(sqrt(2/pi)*1.044715))
    ref = 0.5 * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * 1.044715))
    assert oracle.act(ACT_GELU_TANH, 1.0) == pytest.approx(ref, rel=1e-15)
    assert oracle.act(ACT_RELU, -3.0) == 0.0 and oracle.act(ACT_RELU, 3.0) == 3.0


def test_act_matches_torch_functional_fp64():
    xs = torch.linspace(-9.0, 9.0, 181, dtype=torch.float64)
    silu = torch.nn.functional.silu(xs)
    gelu = torch.nn.functional.gelu(xs, approximate="tanh")
    for x, s, g in zip(xs.tolist(), silu.tolist(), gelu.tolist()):
        assert oracle.act(ACT_SILU, x) == pytest.approx(s, rel=1e-13, abs=1e-15)
        assert oracle.act(ACT_GELU_TANH, x) == pytest.approx(g, rel=1e-12, abs=1e-15)


# --------------------------------------------------------------------------- stage (a)

def _rand_layer(rng, T, d, I, scale=0.2):
    X = rng.standard_normal((T, d)).astype(np.float32)
    Wg = (rng.standard_normal((I, d)) * scale).astype(np.float32)
    Wu = (rng.standard_normal((I, d)) * scale).astype(np.float32)
    return X, Wg, Wu


@pytest.mark.parametrize("kind", [ACT_SILU, ACT_GELU_TANH])
def test_sumsq_matches_matmul_definition(kind):
    """Eq. 2 through a library matmul: H = act(X Wg^T) * (X Wu^T), sumsq = column sums of H^2.
    Wg and Wu get different values and a non-square shape so a swapped or transposed operand shows."""
    rng = np.random.default_rng(1)
    X, Wg, Wu = _rand_layer(rng, T=37, d=24, I=19)
    Xt, Wgt, Wut = (torch.from_numpy(a).double() for a in (X, Wg, Wu))
    G, U = Xt @ Wgt.T, Xt @ Wut.T
    A = torch.nn.functional.silu(G) if kind == ACT_SILU else torch.nn.functional.gelu(G, approximate="tanh")
    ref = ((A * U) ** 2).sum(0).numpy()
    got = oracle.calib_sumsq(X, Wg, Wu, kind)
    np.testing.assert_allclose(got, ref, rtol=1e-12)
    # swapping gate and up must change the answer (the activation sits on the gate branch only)
    swapped = oracle.calib_sumsq(X, Wu, Wg, kind)
    assert np.max(np.abs(swapped - ref) / ref) > 1e-3


def test_sumsq_one_hot_closed_form():
    """X = one-hot rows e_k, Wu all ones (u == 1): H[t,i] = silu(Wg[i,k_t]); sumsq in closed form."""
    d, I = 5, 3
    Wg = np.array([[0.0, 1.0, -1.0, 2.0, math.log(3.0)],
                   [1.0, 1.0, 1.0, 1.0, 1.0],
                   [0.0, 0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    Wu = np.ones((I, d), dtype=np.float32)
    ks = [0, 1, 1, 3, 4, 2]
    X = np.zeros((len(ks), d), dtype=np.float32)
    for t, k in enumerate(ks):
        X[t, k] = 1.0
    silu = lambda v: v / (1.0 + math.exp(-v))
    ref = [sum(silu(float(Wg[i, k])) ** 2 for k in ks) for i in range(I)]
    got = oracle.calib_sumsq(X, Wg, Wu, ACT_SILU)
    np.testing.assert_allclose(got, ref, rtol=1e-14, atol=0)
    assert got[2] == 0.0


def test_sumsq_zero_input_and_accumulation():
    rng = np.random.default_rng(2)
    X, Wg, Wu = _rand_layer(rng, T=30, d=16, I=8)
    assert np.all(oracle.calib_sumsq(np.zeros_like(X), Wg, Wu, ACT_SILU) == 0.0)
    full = oracle.calib_sumsq(X, Wg, Wu, ACT_SILU)
    acc = np.zeros(8, dtype=np.float64)
    for a, b in [(0, 7), (7, 8), (8, 30)]:
        oracle.calib_sumsq(X[a:b], Wg, Wu, ACT_SILU, acc)
    np.testing.assert_allclose(acc, full, rtol=1e-14)
    both = oracle.calib_sumsq(np.concatenate([X, X]), Wg, Wu, ACT_SILU)
    np.testing.assert_allclose(both, 2.0 * full, rtol=1e-14)


def test_sumsq_power_of_two_scaling_is_exact():
    rng = np.random.default_rng(3)
    X, Wg, Wu = _rand_layer(rng, T=21, d=12, I=6)
    a = oracle.calib_sumsq(X, Wg, Wu, ACT_GELU_TANH)
    b = oracle.calib_sumsq(X, Wg, 2.0 * Wu, ACT_GELU_TANH)
    assert np.array_equal(b, 4.0 * a)
    na, nb = oracle.norm_from_sumsq(a), oracle.norm_from_sumsq(b)
    assert np.array_equal(nb, 2.0 * na)


def test_glu_row_matches_sumsq():
    rng = np.random.default_rng(4)
    X, Wg, Wu = _rand_layer(rng, T=9, d=10, I=7)
    H = np.stack([oracle.glu_row(X[t], Wg, Wu, ACT_SILU) for t in range(9)])
    np.testing.assert_allclose((H ** 2).sum(0), oracle.calib_sumsq(X, Wg, Wu, ACT_SILU), rtol=1e-14)


def test_norm_is_correctly_rounded_sqrt():
    s = np.array([0.0, 4.0, 2.0, 1e-30, 3.5e20], dtype=np.float64)
    n = oracle.norm_from_sumsq(s)
    assert n.dtype == np.float32
    assert np.array_equal(n, np.sqrt(s).astype(np.float32))
    assert n[1] == 2.0 and n[0] == 0.0


def test_feature_sumsq_matches_numpy_and_known_vector():
    rng = np.random.default_rng(31)
    X = rng.standard_normal((29, 13)).astype(np.float32)
    ref = (X.astype(np.float64) ** 2).sum(0)
    np.testing.assert_allclose(oracle.feature_sumsq(X), ref, rtol=1e-14)
    acc = oracle.feature_sumsq(X[:10])
    oracle.feature_sumsq(X[10:], acc)
    np.testing.assert_allclose(acc, ref, rtol=1e-14)
    K = np.array([[3.0, 0.0], [4.0, 2.0]], dtype=np.float32)          # columns (3,4) and (0,2): 25 and 4
    assert oracle.feature_sumsq(K).tolist() == [25.0, 4.0]


def test_wanda_eq1_through_score_nm():
    """Eq. 1 on an attention-style projection: |W_ij| * ||X_j||_2 compared per output row."""
    rng = np.random.default_rng(32)
    X = rng.standard_normal((40, 16)).astype(np.float32)
    W = (rng.standard_normal((12, 16)) * 0.02).astype(np.float32)
    norm = oracle.norm_from_sumsq(oracle.feature_sumsq(X))
    mask, _ = oracle.score_nm(W, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)
    score = np.abs(W.astype(np.float64)) * np.linalg.norm(X.astype(np.float64), axis=0).astype(np.float32).astype(np.float64)[None, :]
    ref = np.zeros_like(mask)
    for r in range(12):
        for c0 in range(0, 16, 4):
            ref[r, c0 + np.argsort(-score[r, c0:c0 + 4], kind="stable")[:2]] = 1
    assert np.array_equal(mask, ref)


# --------------------------------------------------------------------------- scale recipe

def test_scale_special_exponents():
    assert oracle.scale(0.0, 0.0) == 1.0            # 0^0 := 1
    assert oracle.scale(123.5, 0.0) == 1.0
    assert oracle.scale(123.5, 1.0) == 123.5
    assert oracle.scale(16.0, 0.5) == 4.0
    assert oracle.scale(16.0, 0.25) == 2.0
    assert oracle.scale(16.0, 0.75) == 8.0
    assert oracle.scale(0.0, 0.5) == 0.0


def test_scale_rounding_against_rationals():
    """float32(sqrt(n)) must be the float nearest to the real sqrt: check s_lo^2 <= n <= s_hi^2
    for the midpoints to the neighbouring floats, in exact rational arithmetic."""
    rng = np.random.default_rng(5)
    for n in np.abs(rng.standard_normal(200)).astype(np.float32) * 37.0:
        s = np.float32(oracle.scale(float(n), 0.5))
        lo = (Fraction(float(s)) + Fraction(float(np.nextafter(s, np.float32(0))))) / 2
        hi = (Fraction(float(s)) + Fraction(float(np.nextafter(s, np.float32(np.inf))))) / 2
        assert lo * lo <= Fraction(float(n)) <= hi * hi


def test_scale_generic_alpha_matches_pow():
    for n in [0.3, 1.0, 7.25, 1234.5]:
        got = oracle.scale(n, 0.3)
        ref = float(np.float32(float(np.float32(n)) ** float(np.float32(0.3))))
        assert got == pytest.approx(ref, rel=2e-7)


# --------------------------------------------------------------------------- N:M selection

def _py_scale(norm32, alpha):
    """Independent restatement of the norm^alpha rounding recipe with numpy IEEE ops."""
    n = np.float64(np.float32(norm32))
    if alpha == 0.0:
        return Fraction(1)
    if alpha == 1.0:
        return Fraction(float(n))
    if alpha == 0.5:
        return Fraction(float(np.float32(np.sqrt(n))))
    if alpha == 0.25:
        return Fraction(float(np.float32(np.sqrt(np.sqrt(n)))))
    if alpha == 0.75:
        return Fraction(float(np.float32(np.sqrt(n) * np.sqrt(np.sqrt(n)))))
    raise AssertionError


def _is_rounded_sqrt(x: float, r: float) -> bool:
    """r is the double nearest to sqrt(x): (r - ulp/2)^2 <= x <= (r + ulp/2)^2, in exact rationals."""
    import math
    half = Fraction(math.ulp(r)) / 2
    lo, hi = Fraction(r) - half, Fraction(r) + half
    return lo >= 0 and lo * lo <= Fraction(x) <= hi * hi


def _is_rounded_f32(d: float, f: float) -> bool:
    """f (a float32 value) is a float32 nearest to the double d."""
    f32 = np.float32(f)
    up, dn = np.nextafter(f32, np.float32(np.inf)), np.nextafter(f32, np.float32(-np.inf))
    err = abs(Fraction(float(f32)) - Fraction(d))
    return err <= abs(Fraction(float(up)) - Fraction(d)) and err <= abs(Fraction(float(dn)) - Fraction(d))


@pytest.mark.parametrize("alpha", [0.25, 0.75, 0.5])
def test_scale_roots_on_random_norms_bit_for_bit_and_by_exact_brackets(alpha):
    """The norm^alpha recipe at 1/4 and 3/4 (and 1/2) where the roots are NOT exact: the oracle's value equals the
    numpy restatement bit for bit, and every step of the stated route -- square root(s) correctly rounded in double,
    their product rounded in double, one rounding to float -- is confirmed by exact-rational brackets, so another
    rounding route (a float sqrt, pow, a fused product) would be caught."""
    import math
    rng = np.random.default_rng(int(alpha * 100))
    norms = np.concatenate([rng.uniform(1e-3, 1e3, 300), rng.lognormal(0.0, 6.0, 300), [1e-30, 3.0e38, 2.0, 3.0, 0.1]]).astype(np.float32)
    differ_from_float_route = 0
    for n in norms:
        got = oracle.scale(float(n), alpha)
        assert Fraction(got) == _py_scale(n, alpha), (float(n), alpha)
        x = float(n)
        r1 = math.sqrt(x)
        assert _is_rounded_sqrt(x, r1)
        if alpha == 0.5:
            d = r1
        else:
            r2 = math.sqrt(r1)
            assert _is_rounded_sqrt(r1, r2)
            if alpha == 0.25:
                d = r2
            else:
                d = r1 * r2                                   # one rounding in double: check it as a nearest double
                exact = Fraction(r1) * Fraction(r2)
                assert abs(Fraction(d) - exact) <= Fraction(math.ulp(d)) / 2
        assert _is_rounded_f32(d, got) and np.float32(got) == np.float32(d)
        # the same exponent evaluated all in float32 differs for a fair share of inputs: the pin can tell them apart
        f = np.float32(n)
        alt = {0.5: np.sqrt(f), 0.25: np.sqrt(np.sqrt(f)), 0.75: np.float32(np.sqrt(f) * np.sqrt(np.sqrt(f)))}[alpha]
        differ_from_float_route += int(np.float32(alt) != np.float32(got))
    if alpha != 0.5:
        assert differ_from_float_route > 0


def _brute_force_group(scores, n_keep):
    """The unique subset whose every member precedes every non-member in
    (score desc, index asc); also returns the max-sum / lexicographically smallest subset."""
    m = len(scores)
    valid = []
    best = None
    for S in itertools.combinations(range(m), n_keep):
        rest = [b for b in range(m) if b not in S]
        ok = all(scores[a] > scores[b] or (scores[a] == scores[b] and a < b) for a in S for b in rest)
        if ok:
            valid.append(S)
        key = (-sum(scores[a] for a in S), S)
        if best is None or key < best:
            best = key
    assert len(valid) == 1
    assert best[1] == valid[0]
    return set(valid[0])


def _brute_force_mask(W, norm, norm_axis, alpha, n_keep, m, group_axis):
    rows, cols = W.shape
    mask = np.zeros((rows, cols), dtype=np.uint8)
    sc = [[abs(Fraction(float(W[r, c]))) * _py_scale(norm[r if norm_axis == AXIS_ROWS else c], alpha)
           for c in range(cols)] for r in range(rows)]
    if group_axis == AXIS_COLS:
        for r in range(rows):
            for c0 in range(0, cols, m):
                for p in _brute_force_group([sc[r][c0 + p] for p in range(m)], n_keep):
                    mask[r, c0 + p] = 1
    else:
        for c in range(cols):
            for r0 in range(0, rows, m):
                for p in _brute_force_group([sc[r0 + p][c] for p in range(m)], n_keep):
                    mask[r0 + p, c] = 1
    return mask


@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (1, 4), (3, 4), (5, 8)])
@pytest.mark.parametrize("norm_axis,group_axis", [(AXIS_ROWS, AXIS_ROWS), (AXIS_COLS, AXIS_COLS),
                                                  (AXIS_ROWS, AXIS_COLS), (AXIS_COLS, AXIS_ROWS)])
@pytest.mark.parametrize("alpha", [0.0, 0.25, 0.5, 0.75, 1.0])
def test_score_nm_vs_exact_brute_force(n_keep, m, norm_axis, group_axis, alpha):
    rng = np.random.default_rng(100 * m + 10 * n_keep + int(alpha * 4))
    rows, cols = 16, 16
    # few distinct magnitudes and norms -> many exact ties, signed zeros included
    W = rng.choice(np.array([0.0, -0.0, 0.25, -0.25, 0.5, 1.0, -1.0, 2.0, 3.0], dtype=np.float32), (rows, cols))
    norm = rng.choice(np.array([0.0, 1.0, 4.0, 16.0, 2.0, 9.0], dtype=np.float32),
                      rows if norm_axis == AXIS_ROWS else cols)
    mask, pruned = oracle.score_nm(W, norm, norm_axis, alpha, n_keep, m, group_axis)
    ref = _brute_force_mask(W, norm, norm_axis, alpha, n_keep, m, group_axis)
    assert np.array_equal(mask, ref)
    # survivors keep their exact value, pruned entries are +0
    assert np.array_equal(pruned[ref == 1].view(np.uint32), W[ref == 1].view(np.uint32))
    assert np.all(pruned[ref == 0].view(np.uint32) == 0)


@pytest.mark.parametrize("seed", range(4))
def test_score_nm_random_floats_vs_brute_force(seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((8, 16)) * 0.02).astype(np.float32)
    norm_r = np.abs(rng.standard_normal(8)).astype(np.float32) * 30
    norm_c = np.abs(rng.standard_normal(16)).astype(np.float32) * 30
    for (na, ga, nv) in [(AXIS_ROWS, AXIS_ROWS, norm_r), (AXIS_COLS, AXIS_COLS, norm_c)]:
        for (n_keep, m) in [(2, 4), (4, 8)]:
            mask, _ = oracle.score_nm(W, nv, na, 0.5, n_keep, m, ga)
            assert np.array_equal(mask, _brute_force_mask(W, nv, na, 0.5, n_keep, m, ga))


def _mask_from_strings(rows):
    return np.array([[int(ch) for ch in r] for r in rows], dtype=np.uint8)


def _golden_cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
def test_golden_handworked(case):
    W = np.array(case["W"], dtype=np.float32)
    norm = np.array(case["norm"], dtype=np.float32)
    mask, pruned = oracle.score_nm(W, norm, case["norm_axis"], case["alpha"], case["n_keep"], case["m"],
                                   case["group_axis"])
    want = _mask_from_strings(case["mask"])
    assert np.array_equal(mask, want), case["why"]
    assert np.array_equal(pruned, np.where(want == 1, W, np.float32(0.0)))
    if "meta_words" in case:
        values, meta = oracle.compress_nm(W, mask, case["n_keep"], case["m"], case["group_axis"])
        want_meta = np.array([[int(w, 16) for w in line] for line in case["meta_words"]], dtype=np.uint32)
        assert np.array_equal(meta, want_meta), case["meta_why"]
        assert np.array_equal(values.view(np.uint32), np.array(case["values"], dtype=np.float32).view(np.uint32))


@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8)])
def test_exactly_n_survivors_per_group(n_keep, m):
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((64, 96)) * 0.02).astype(np.float32)
    norm = np.abs(rng.standard_normal(96)).astype(np.float32)
    mask, _ = oracle.score_nm(W, norm, AXIS_COLS, 1.0, n_keep, m, AXIS_COLS)
    assert np.all(mask.reshape(64, 96 // m, m).sum(-1) == n_keep)
    norm = np.abs(rng.standard_normal(64)).astype(np.float32)
    mask, _ = oracle.score_nm(W, norm, AXIS_ROWS, 0.5, n_keep, m, AXIS_ROWS)
    assert np.all(mask.reshape(64 // m, m, 96).sum(1) == n_keep)


def test_shape_not_divisible_is_rejected():
    W = np.ones((6, 6), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.score_nm(W, np.ones(6, dtype=np.float32), AXIS_COLS, 1.0, 2, 4, AXIS_COLS)


# --------------------------------------------------------------------------- Eq. 5 == Wanda (Eq. 1) with X := H

def test_down_score_reduces_to_wanda_on_intermediate_activations():
    """Independent route: H by library matmul, ||H_j||_2 by numpy, Eq. 1 score |W_ij| * ||X_j||,
    per-row 2:4 by a stable argsort.  Must give the oracle's down-projection mask when the oracle
    is fed the norms it computed itself from the same calibration data."""
    rng = np.random.default_rng(11)
    T, d, I = 48, 16, 32
    X, Wg, Wu = _rand_layer(rng, T, d, I, scale=0.3)
    Wd = (rng.standard_normal((d, I)) * 0.02).astype(np.float32)
    norm = oracle.norm_from_sumsq(oracle.calib_sumsq(X, Wg, Wu, ACT_SILU))
    mask, _ = oracle.score_nm(Wd, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)

    Xt, Wgt, Wut = (torch.from_numpy(a).double() for a in (X, Wg, Wu))
    H = (torch.nn.functional.silu(Xt @ Wgt.T) * (Xt @ Wut.T)).numpy()
    feat_norm = np.linalg.norm(H, axis=0).astype(np.float32).astype(np.float64)   # ||X_j||_2 of Eq. 1
    score = np.abs(Wd.astype(np.float64)) * feat_norm[None, :]
    wanda = np.zeros_like(mask)
    for r in range(d):
        for c0 in range(0, I, 4):
            order = np.argsort(-score[r, c0:c0 + 4], kind="stable")
            wanda[r, c0 + order[:2]] = 1
    assert np.array_equal(mask, wanda)


# --------------------------------------------------------------------------- Eq. 4 special cases and invariances

def _magnitude_nm(W, n_keep, m, group_axis):
    A = np.abs(W.astype(np.float64))
    mask = np.zeros(W.shape, dtype=np.uint8)
    if group_axis == AXIS_COLS:
        for r in range(W.shape[0]):
            for c0 in range(0, W.shape[1], m):
                mask[r, c0 + np.argsort(-A[r, c0:c0 + m], kind="stable")[:n_keep]] = 1
    else:
        for c in range(W.shape[1]):
            for r0 in range(0, W.shape[0], m):
                mask[r0 + np.argsort(-A[r0:r0 + m, c], kind="stable")[:n_keep], c] = 1
    return mask


def test_alpha_zero_and_equal_norms_reduce_to_magnitude():
    rng = np.random.default_rng(13)
    W = (rng.standard_normal((32, 24)) * 0.02).astype(np.float32)
    norm = np.abs(rng.standard_normal(32)).astype(np.float32) * 10
    ref = _magnitude_nm(W, 2, 4, AXIS_ROWS)
    m0, _ = oracle.score_nm(W, norm, AXIS_ROWS, 0.0, 2, 4, AXIS_ROWS)
    assert np.array_equal(m0, ref)
    for a in (0.25, 0.5, 1.0):
        me, _ = oracle.score_nm(W, np.full(32, 7.5, dtype=np.float32), AXIS_ROWS, a, 2, 4, AXIS_ROWS)
        assert np.array_equal(me, ref)
    # and alpha actually matters when norms differ
    mh, _ = oracle.score_nm(W, norm, AXIS_ROWS, 0.5, 2, 4, AXIS_ROWS)
    assert not np.array_equal(mh, ref)


def test_uniform_rescaling_of_norms_changes_nothing():
    rng = np.random.default_rng(14)
    W = (rng.standard_normal((32, 24)) * 0.02).astype(np.float32)
    norm = (np.abs(rng.standard_normal(32)) * 10 + 0.1).astype(np.float32)
    base, _ = oracle.score_nm(W, norm, AXIS_ROWS, 0.5, 2, 4, AXIS_ROWS)
    for c in (4.0, 0.0625):   # even powers of two: sqrt stays exact, so the invariance is bitwise
        other, _ = oracle.score_nm(W, norm * np.float32(c), AXIS_ROWS, 0.5, 2, 4, AXIS_ROWS)
        assert np.array_equal(base, other)


def test_literal_rowwise_gate_mode_is_independent_of_norms():
    rng = np.random.default_rng(15)
    W = (rng.standard_normal((16, 32)) * 0.02).astype(np.float32)
    a, _ = oracle.score_nm(W, np.abs(rng.standard_normal(16)).astype(np.float32) + 0.1, AXIS_ROWS, 0.5, 2, 4, AXIS_COLS)
    b, _ = oracle.score_nm(W, np.abs(rng.standard_normal(16)).astype(np.float32) + 0.1, AXIS_ROWS, 1.0, 2, 4, AXIS_COLS)
    assert np.array_equal(a, b)
    assert np.array_equal(a, _magnitude_nm(W, 2, 4, AXIS_COLS))


def test_paper_grouping_reacts_to_one_neuron_norm():
    """Groups of gate/up must mix different neurons: raising one neuron's norm changes the mask
    under the input-balanced grouping."""
    rng = np.random.default_rng(16)
    W = (rng.standard_normal((16, 32)) * 0.02).astype(np.float32)
    norm = np.ones(16, dtype=np.float32)
    a, _ = oracle.score_nm(W, norm, AXIS_ROWS, 0.5, 2, 4, AXIS_ROWS)
    norm2 = norm.copy()
    norm2[5] = 1e4
    b, _ = oracle.score_nm(W, norm2, AXIS_ROWS, 0.5, 2, 4, AXIS_ROWS)
    assert b[5].all()                       # neuron 5 now wins every group it is in
    assert not np.array_equal(a, b)


# --------------------------------------------------------------------------- dependency invariants (unstructured)

def test_unstructured_keep_counts_and_floor_rule():
    rng = np.random.default_rng(17)
    W = (rng.standard_normal((40, 12)) * 0.02).astype(np.float32)
    norm = np.abs(rng.standard_normal(40)).astype(np.float32) + 0.1
    for s in (0.5, 0.33, 0.0, 0.9):
        mk = oracle.select_unstructured(W, norm, AXIS_ROWS, 0.5, s, AXIS_ROWS)      # input-balanced
        assert np.all(mk.sum(0) == 40 - math.floor(s * 40))
        mk = oracle.select_unstructured(W.T.copy(), norm, AXIS_COLS, 1.0, s, AXIS_COLS)  # output-balanced
        assert np.all(mk.sum(1) == 40 - math.floor(s * 40))


def test_unstructured_matches_argsort_definition():
    rng = np.random.default_rng(18)
    W = (rng.standard_normal((24, 10)) * 0.02).astype(np.float32)
    norm = np.abs(rng.standard_normal(24)).astype(np.float32) + 0.1
    mk = oracle.select_unstructured(W, norm, AXIS_ROWS, 1.0, 0.5, AXIS_ROWS)
    score = np.abs(W.astype(np.float64)) * norm.astype(np.float64)[:, None]
    ref = np.zeros_like(mk)
    for c in range(10):
        ref[np.argsort(-score[:, c], kind="stable")[:12], c] = 1
    assert np.array_equal(mk, ref)


def test_raising_a_neuron_norm_never_loses_it_weights():
    rng = np.random.default_rng(19)
    W = (rng.standard_normal((48, 20)) * 0.02).astype(np.float32)
    norm = (np.abs(rng.standard_normal(48)) + 0.1).astype(np.float32)
    base = oracle.select_unstructured(W, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
    for i in (0, 7, 31):
        for c in (1.5, 4.0, 100.0):
            n2 = norm.copy()
            n2[i] *= np.float32(c)
            mk = oracle.select_unstructured(W, n2, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
            assert np.all(mk[i] >= base[i])          # kept set of neuron i only grows


def test_dominating_neuron_keeps_superset():
    rng = np.random.default_rng(20)
    W = (rng.standard_normal((32, 16)) * 0.02).astype(np.float32)
    W[3] = np.abs(W[9]) * np.float32(1.25)           # |W[3,:]| >= |W[9,:]| element-wise
    norm = (np.abs(rng.standard_normal(32)) + 0.1).astype(np.float32)
    norm[3] = norm[9] * np.float32(2.0)
    mk = oracle.select_unstructured(W, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
    assert np.all(mk[3] >= mk[9])


def test_constant_magnitude_keep_count_monotone_in_norm():
    """With equal |w| everywhere, a neuron with a larger norm keeps at least as many gate/up weights."""
    rng = np.random.default_rng(21)
    W = (rng.choice([-1.0, 1.0], (64, 24)) * 0.02).astype(np.float32)
    norm = (np.abs(rng.standard_normal(64)) * 5 + 0.01).astype(np.float32)
    mk = oracle.select_unstructured(W, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
    kept = mk.sum(1)
    order = np.argsort(norm, kind="stable")
    assert np.all(np.diff(kept[order]) >= 0)
    # Wanda-style output-balanced selection keeps the same count for every neuron instead
    out_bal = oracle.select_unstructured(W, np.ones(24, dtype=np.float32), AXIS_COLS, 1.0, 0.5, AXIS_COLS)
    assert len(set(out_bal.sum(1).tolist())) == 1


# --------------------------------------------------------------------------- packing and compression

def test_pack_mask_bit_layout():
    rng = np.random.default_rng(22)
    mask = rng.integers(0, 2, (5, 70)).astype(np.uint8)
    bits = oracle.pack_mask(mask)
    assert bits.shape == (5, 3)
    for r in range(5):
        for c in range(70):
            assert ((int(bits[r, c // 32]) >> (c % 32)) & 1) == mask[r, c]
        assert int(bits[r, 2]) >> (70 - 64) == 0     # padding bits stay clear


def _decompress(values, meta, rows, cols, n_keep, m, group_axis):
    out = np.zeros((rows, cols), dtype=np.float32)
    two_four = (n_keep == 2 and m == 4)
    bpg = 4 if two_four else m
    fpw = 32 // bpg
    lines = rows if group_axis == AXIS_COLS else rows // m
    fields = cols // m if group_axis == AXIS_COLS else cols
    nfields = 0
    for l in range(lines):
        for f in range(fields):
            field = (int(meta[l, f // fpw]) >> (bpg * (f % fpw))) & ((1 << bpg) - 1)
            if two_four:
                pos = [field & 3, field >> 2]
                assert pos[0] < pos[1]
            else:
                pos = [p for p in range(m) if (field >> p) & 1]
                assert len(pos) == n_keep
            nfields += 1
            for q, p in enumerate(pos):
                if group_axis == AXIS_COLS:
                    out[l, f * m + p] = values[l, f * n_keep + q]
                else:
                    out[l * m + p, f] = values[l * n_keep + q, f]
    assert nfields == rows * cols // m
    return out


@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (1, 4)])
@pytest.mark.parametrize("group_axis", [AXIS_ROWS, AXIS_COLS])
def test_compress_round_trip(n_keep, m, group_axis):
    rng = np.random.default_rng(23)
    rows, cols = 24, 40
    W = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    W[W == 0] = 0.01
    norm = (np.abs(rng.standard_normal(rows if group_axis == AXIS_ROWS else cols)) + 0.1).astype(np.float32)
    mask, pruned = oracle.score_nm(W, norm, group_axis, 0.5, n_keep, m, group_axis)
    values, meta = oracle.compress_nm(W, mask, n_keep, m, group_axis)
    assert values.shape == oracle.values_shape(rows, cols, n_keep, m, group_axis)
    back = _decompress(values, meta, rows, cols, n_keep, m, group_axis)
    assert np.array_equal(back.view(np.uint32), pruned.view(np.uint32))


def test_compress_rejects_non_nm_mask():
    W = np.ones((4, 8), dtype=np.float32)
    mask = np.ones((4, 8), dtype=np.uint8)
    with pytest.raises(ValueError):
        oracle.compress_nm(W, mask, 2, 4, AXIS_COLS)


# --------------------------------------------------------------------------- a planted mistake must be caught

def test_pins_catch_a_transposed_norm_axis():
    """Feeding the down projection the wrong norm axis (a plausible indexing slip) must not
    reproduce the Wanda route's mask -- i.e. the pin above has teeth."""
    rng = np.random.default_rng(24)
    Wd = (rng.standard_normal((16, 16)) * 0.02).astype(np.float32)
    norm = (np.abs(rng.standard_normal(16)) * 3 + 0.1).astype(np.float32)
    good, _ = oracle.score_nm(Wd, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)
    bad, _ = oracle.score_nm(Wd, norm, AXIS_ROWS, 1.0, 2, 4, AXIS_COLS)
    assert not np.array_equal(good, bad)
