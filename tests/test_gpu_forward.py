"""Forward pass of the (pruned) layer, Eq. 2 then Eq. 3, through the C ABI against the fp64 oracle.

Tolerances, from the arithmetic.  bf16 path: the two dot products of Eq. 2 are accumulated in fp32 over d exact
products, so |dg| <= d 2^-24 Gabs with Gabs = sum_k |x_k| |wg_k| (likewise u); the activations' slopes are at most
about 1.1, so |dh| <= 2.2 d 2^-24 Gabs Uabs before rounding, and rounding to bf16 adds 2^-9 |h| (one more 2^-9 |h|
is allowed for values the fp32 error pushes across a rounding boundary).  Eq. 3 then sees the kernel's own H:
|dz| <= |dH| |Wd|^T (measured dH) + I 2^-24 |H| |Wd|^T (fp32 accumulation) + 2^-8 |z| (final rounding).
fp32 path: the same with 2^-23 in place of the bf16 rounding terms."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bits_of, to_np32
from paper_2405_01943_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _h_from_workspace(ws: torch.Tensor, T: int, I: int, dtype: torch.dtype) -> torch.Tensor:
    unit = 8 if dtype == torch.bfloat16 else 4
    ldh = (I + unit - 1) // unit * unit
    elt = 2 if dtype == torch.bfloat16 else 4
    return ws[256:256 + T * ldh * elt].view(dtype).view(T, ldh)[:, :I]


def _check_forward(cfg, X, Wg, Wu, Wd, act_name, rows=None):
    """Runs the layer on the GPU (one pass) and compares H and Z with the oracle on `rows` (default: all tokens)."""
    act = binding.ACT_BY_NAME[act_name]
    T, d = X.shape
    I = Wg.shape[0]
    bf16 = X.dtype == torch.bfloat16
    ws = binding.mlp_forward_workspace(binding.mlp_forward_workspace_bytes(T, d, I, X.dtype)[1], DEV)
    Z = binding.mlp_forward(X, Wg, Wu, Wd, act, workspace=ws)
    binding.calib_status(ws)
    H = _h_from_workspace(ws, T, I, X.dtype)
    if rows is None:
        rows = np.arange(T)
    rt = torch.from_numpy(rows).to(DEV)
    Xs, Wg32, Wu32, Wd32 = to_np32(X[rt]), to_np32(Wg), to_np32(Wu), to_np32(Wd)
    Z_ref, H_ref = oracle.mlp_forward(Xs, Wg32, Wu32, Wd32, act, bf16, want_h=True)
    _, H_exact = oracle.mlp_forward(Xs, Wg32, Wu32, Wd32, act, False, want_h=True)
    H_gpu = to_np32(H[rt]).astype(np.float64)
    Z_gpu = to_np32(Z[rt]).astype(np.float64)

    Gabs = np.abs(Xs).astype(np.float64) @ np.abs(Wg32).astype(np.float64).T
    Uabs = np.abs(Xs).astype(np.float64) @ np.abs(Wu32).astype(np.float64).T
    rnd = 2.0 ** -8 if bf16 else 2.0 ** -22
    tol_h = rnd * np.abs(H_exact) + 2.2 * d * 2.0 ** -24 * Gabs * Uabs + 1e-30
    dH = np.abs(H_gpu - H_exact)
    assert np.all(dH <= tol_h), f"H off by up to {np.max(dH / tol_h):.2f} tolerances"
    if bf16:
        # almost every element rounds to the very bf16 value the oracle rounds to
        assert np.mean(H_gpu == H_ref) > 0.97
    dHr = np.abs(H_gpu - H_ref)
    Wabs = np.abs(Wd32).astype(np.float64)
    tol_z = dHr @ Wabs.T + I * 2.0 ** -24 * (np.abs(H_gpu) @ Wabs.T) + (2.0 ** -8 if bf16 else 2.0 ** -23) * np.abs(Z_ref) + 1e-30
    dZ = np.abs(Z_gpu - Z_ref)
    assert np.all(dZ <= tol_z), f"Z off by up to {np.max(dZ / tol_z):.2f} tolerances"
    # and the tolerance is not what makes it pass: typical error is a small fraction of the output's scale
    scale = np.sqrt(np.mean(Z_ref ** 2)) + 1e-30
    assert np.sqrt(np.mean(dZ ** 2)) <= (6e-3 if bf16 else 2e-5) * scale
    return Z, ws


@pytest.mark.parametrize("name,d,I,T", [
    ("llama2_7b", 256, 688, 1500),      # ragged T and I, one 256-row block of Wd
    ("gemma_7b", 328, 344, 700),        # k tails in both contractions, a half-empty second block of Wd
    ("relullama_7b", 512, 1376, 300),   # ReGLU, two blocks of Wd
    ("llama2_7b", 64, 40, 37),          # smaller than one tile in every direction
])
def test_forward_bf16_matches_oracle(name, d, I, T):
    cfg = synth.scaled(synth.CONFIGS[name], d=d, I=I, T=T)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    _check_forward(cfg, X, Wg, Wu, Wd, cfg.act)


def test_forward_f32_matches_oracle():
    cfg = synth.CONFIGS["tiny"]
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    assert X.dtype == torch.float32
    _check_forward(cfg, X, Wg, Wu, Wd, cfg.act)


def test_forward_of_the_pruned_layer():
    """The use the entry point exists for: prune with DaSS (2:4), then run the pruned layer."""
    cfg = synth.scaled(synth.CONFIGS["llama2_7b"], d=256, I=688, T=1200)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    sumsq = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(cfg.T, cfg.d, cfg.I, X.dtype, DEV)
    binding.calib_accumulate(X, Wg, Wu, binding.ACT_SILU, sumsq, ws)
    norm = binding.norm_finalize(sumsq)
    pruned = []
    for W, na, alpha, ga in ((Wg, binding.AXIS_ROWS, 0.5, binding.AXIS_ROWS), (Wu, binding.AXIS_ROWS, 0.5, binding.AXIS_ROWS),
                             (Wd, binding.AXIS_COLS, 1.0, binding.AXIS_COLS)):
        _, Wp = binding.score_nm(W, norm, na, alpha, 2, 4, ga)
        pruned.append(Wp[:, :W.shape[1]].contiguous())
    assert all(float((Wp == 0).float().mean()) >= 0.5 for Wp in pruned)
    Zp, _ = _check_forward(cfg, X, pruned[0], pruned[1], pruned[2], "silu")
    Zd, _ = _check_forward(cfg, X, Wg, Wu, Wd, "silu")
    # pruning half of the weights changes the output, but not beyond recognition
    zp, zd = to_np32(Zp).astype(np.float64), to_np32(Zd).astype(np.float64)
    rel = np.linalg.norm(zp - zd) / np.linalg.norm(zd)
    assert 0.05 < rel < 1.0


@pytest.mark.parametrize("name,T", [("llama2_70b", 32768), ("gemma_7b", 8192 + 77)])
def test_forward_full_size_sampled_tokens(name, T):
    """Full-size layers in the launch configuration the benchmark times (70B shape, 32768 tokens, one pass); the
    oracle redoes sampled token rows: the first and last lane of both CTAs of a pair, tile borders, the ragged end."""
    cfg = synth.scaled(synth.CONFIGS[name], T=T)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    rows = np.array([0, 127, 128, 255, 256, 4095, 4096, T // 2 + 33, T - 257, T - 1])
    _check_forward(cfg, X, Wg, Wu, Wd, cfg.act, rows=rows)


def test_forward_chunked_equals_one_pass():
    cfg = synth.scaled(synth.CONFIGS["llama2_7b"], d=256, I=688, T=1500)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    lo, full = binding.mlp_forward_workspace_bytes(cfg.T, cfg.d, cfg.I, X.dtype)
    assert lo < full
    Z_full = binding.mlp_forward(X, Wg, Wu, Wd, binding.ACT_SILU, workspace=binding.mlp_forward_workspace(full, DEV))
    for nbytes in (lo, lo + 3 * 256 * 688 * 2 + 100):           # 256-token chunks; 1024-token chunks
        ws = binding.mlp_forward_workspace(nbytes, DEV)
        Z = binding.mlp_forward(X, Wg, Wu, Wd, binding.ACT_SILU, workspace=ws)
        binding.calib_status(ws)
        assert np.array_equal(bits_of(Z), bits_of(Z_full))


def test_forward_pitched_operands_and_output():
    cfg = synth.scaled(synth.CONFIGS["llama2_7b"], d=192, I=264, T=520)
    X0 = synth.make_x(cfg, DEV)
    Wg0, Wu0, Wd0 = synth.make_weights(cfg, DEV)

    def pitched(t, pad):
        buf = torch.full((t.shape[0], t.shape[1] + pad), 7.0, dtype=t.dtype, device=DEV)
        buf[:, :t.shape[1]] = t
        return buf[:, :t.shape[1]]

    X, Wg, Wu, Wd = pitched(X0, 8), pitched(Wg0, 16), pitched(Wu0, 16), pitched(Wd0, 24)
    Zbuf = torch.full((cfg.T, cfg.d + 5), 3.0, dtype=X.dtype, device=DEV)
    Z = binding.mlp_forward(X, Wg, Wu, Wd, binding.ACT_SILU, Z=Zbuf[:, :cfg.d])
    Z_ref = binding.mlp_forward(X0, Wg0, Wu0, Wd0, binding.ACT_SILU)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(Z.contiguous()), bits_of(Z_ref))
    assert bool((Zbuf[:, cfg.d:] == 3.0).all())                 # nothing written past the row


def test_forward_argument_errors():
    cfg = synth.scaled(synth.CONFIGS["llama2_7b"], d=64, I=40, T=37)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    lo, _ = binding.mlp_forward_workspace_bytes(cfg.T, cfg.d, cfg.I, X.dtype)
    with pytest.raises(binding.DassError) as e:
        binding.mlp_forward(X, Wg, Wu, Wd, binding.ACT_SILU, workspace=binding.mlp_forward_workspace(lo - 1, DEV))
    assert e.value.code == 6
    with pytest.raises(binding.DassError) as e:
        binding.mlp_forward(X, Wg, Wu, Wd, 9)
    assert e.value.code == 4
    with pytest.raises(ValueError):
        binding.mlp_forward(X, Wg, Wu, Wd.t().contiguous(), binding.ACT_SILU)
