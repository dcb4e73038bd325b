"""GPU parity of stage (a): dass_calib_accumulate (+ dass_norm_finalize) against the fp64 oracle.
Tolerances: neuron norms within 1e-5 relative for fp32 inputs and 2e-3 for bf16 inputs."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_np32
from paper_2405_01943_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}
ACTS = [("silu", oracle.ACT_SILU, binding.ACT_SILU), ("gelu_tanh", oracle.ACT_GELU_TANH, binding.ACT_GELU_TANH),
        ("relu", oracle.ACT_RELU, binding.ACT_RELU)]


def gpu_sumsq(X, Wg, Wu, act, batches=None):
    T, d = X.shape
    I = Wg.shape[0]
    sumsq = torch.zeros(I, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(T, d, I, X.dtype, DEV)
    for (a, b) in (batches or [(0, T)]):
        binding.calib_accumulate(X[a:b], Wg, Wu, act, sumsq, ws)
    binding.calib_status(ws)
    return sumsq


def rel_err_of_norm(sumsq_gpu, sumsq_ref):
    n_gpu = np.sqrt(sumsq_gpu.cpu().numpy())
    n_ref = np.sqrt(sumsq_ref)
    return np.abs(n_gpu - n_ref) / np.maximum(n_ref, 1e-300)


def _layer(T, d, I, dtype, seed, ldx=None, ldw=None, outliers=True):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    ldx, ldw = ldx or d, ldw or d
    Xb = torch.zeros((T, ldx), dtype=dtype, device=DEV)
    x = torch.randn((T, d), generator=g, device=DEV)
    if outliers and d >= 8:
        x[:, torch.randperm(d, generator=g, device=DEV)[: max(1, d // 64)]] *= 20.0
    Xb[:, :d] = x.to(dtype)
    Wgb = torch.zeros((I, ldw), dtype=dtype, device=DEV)
    Wub = torch.zeros((I, ldw), dtype=dtype, device=DEV)
    Wgb[:, :d] = (torch.randn((I, d), generator=g, device=DEV) * 0.02).to(dtype)
    Wub[:, :d] = (torch.randn((I, d), generator=g, device=DEV) * 0.02).to(dtype)
    return Xb[:, :d], Wgb[:, :d], Wub[:, :d]


def test_tiny_config_full_fp32():
    """The small fp32 SwiGLU case in full: every neuron's norm within 1e-5 of the oracle."""
    cfg = synth.CONFIGS["tiny"]
    X = synth.make_x(cfg, DEV)
    Wg, Wu, _ = synth.make_weights(cfg, DEV)
    ref = oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oracle.ACT_SILU)
    got = gpu_sumsq(X, Wg, Wu, binding.ACT_SILU)
    assert rel_err_of_norm(got, ref).max() <= TOL[torch.float32]
    norm = binding.norm_finalize(got)
    torch.cuda.synchronize()
    assert np.array_equal(norm.cpu().numpy(), oracle.norm_from_sumsq(got.cpu().numpy()))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("name,oact,gact", ACTS, ids=[a[0] for a in ACTS])
@pytest.mark.parametrize("T,d,I,ldx,ldw", [
    (128, 256, 688, 256, 256),      # the tiny config's shape; I is not a multiple of the 128-neuron tile
    (300, 200, 136, 208, 216),      # ragged in every dimension, padded pitches
    (1, 8, 1, 8, 8),                # degenerate
    (1030, 96, 520, 96, 96),        # several token tiles with a tail
])
def test_small_shapes(dtype, name, oact, gact, T, d, I, ldx, ldw):
    X, Wg, Wu = _layer(T, d, I, dtype, seed=T + d + I, ldx=ldx, ldw=ldw)
    ref = oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oact)
    got = gpu_sumsq(X, Wg, Wu, gact)
    err = rel_err_of_norm(got, ref)
    live = np.sqrt(ref) > 1e-12
    assert err[live].max() <= TOL[dtype]
    assert np.all(got.cpu().numpy()[~live] <= 1e-20)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_batched_accumulation_and_determinism(dtype):
    X, Wg, Wu = _layer(700, 128, 264, dtype, seed=3)
    whole = gpu_sumsq(X, Wg, Wu, binding.ACT_SILU)
    again = gpu_sumsq(X, Wg, Wu, binding.ACT_SILU)
    assert torch.equal(whole, again)                                  # fixed reduction order
    pieces = gpu_sumsq(X, Wg, Wu, binding.ACT_SILU, batches=[(0, 256), (256, 264), (264, 700)])
    ref = oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oracle.ACT_SILU)
    assert rel_err_of_norm(pieces, ref).max() <= TOL[dtype]
    np.testing.assert_allclose(pieces.cpu().numpy(), whole.cpu().numpy(), rtol=1e-5)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_zero_input_gives_zero(dtype):
    X, Wg, Wu = _layer(130, 64, 136, dtype, seed=4)
    got = gpu_sumsq(torch.zeros_like(X), Wg, Wu, binding.ACT_GELU_TANH)
    assert torch.all(got == 0)


def test_power_of_two_scaling_exact_bf16_and_f32():
    for dtype in (torch.float32, torch.bfloat16):
        X, Wg, Wu = _layer(200, 64, 136, dtype, seed=5)
        a = gpu_sumsq(X, Wg, Wu, binding.ACT_SILU)
        b = gpu_sumsq(X, Wg, (Wu.float() * 2).to(dtype), binding.ACT_SILU)
        assert torch.equal(b, 4.0 * a)
