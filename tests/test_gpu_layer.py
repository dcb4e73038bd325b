"""LayerPruner (the sequence of C-ABI calls for one layer) against the oracle: the neuron norms within the
tolerance of their dtype, and -- stage (b) being exact given a norm vector -- every mask word, pruned weight,
compressed value and metadata word bit for bit when the oracle is fed the norms the GPU produced."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_stage_b_equal, bits_like, bits_of, oracle_stage_b, to_np32, u32
from paper_2405_01943_b200 import synth
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS
from paper_2405_01943_b200.layer import LayerPruner

pytestmark = pytest.mark.gpu
DEV = "cuda"
ORACLE_ACT = {"silu": oracle.ACT_SILU, "gelu_tanh": oracle.ACT_GELU_TANH, "relu": oracle.ACT_RELU}


def _layer(name, **scale):
    cfg = synth.scaled(synth.CONFIGS[name], **scale) if scale else synth.CONFIGS[name]
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    return cfg, X, Wg, Wu, Wd


@pytest.mark.parametrize("name,scale,tol", [("tiny", {}, 1e-5), ("mistral_7b", dict(d=256, I=688, T=900), 2e-3),
                                            ("gemma_7b", dict(d=192, I=1024, T=520), 2e-3)])
def test_prune_nm_matches_oracle(name, scale, tol):
    cfg, X, Wg, Wu, Wd = _layer(name, **scale)
    pruner = LayerPruner(cfg.T, cfg.d, cfg.I, X.dtype, act=cfg.act, n_keep=cfg.n_keep, m=cfg.m, device=DEV)
    out = pruner.prune(X, Wg, Wu, Wd, alpha=0.5)
    pruner.check()
    ref_norm = oracle.norm_from_sumsq(oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), ORACLE_ACT[cfg.act]))
    norm = to_np32(pruner.norm)
    assert np.max(np.abs(norm - ref_norm) / ref_norm) <= tol
    for pname, W, axis, alpha in (("gate", Wg, AXIS_ROWS, 0.5), ("up", Wu, AXIS_ROWS, 0.5), ("down", Wd, AXIS_COLS, 1.0)):
        ref = oracle_stage_b(W, norm, axis, alpha, cfg.n_keep, cfg.m, axis)
        o = out[pname]
        got = dict(words=u32(o["mask"]), pruned_bits=bits_of(o["pruned"]), values_bits=bits_of(o["values"]), meta=u32(o["meta"]))
        assert_stage_b_equal(got, ref)
        assert np.array_equal(got["values_bits"], ref["values_bits"]) and np.array_equal(got["meta"], ref["meta"])


def test_prune_unstructured_and_batched_calibration():
    cfg, X, Wg, Wu, Wd = _layer("llama2_7b", d=256, I=688, T=1100)
    pruner = LayerPruner(cfg.T, cfg.d, cfg.I, X.dtype, act=cfg.act, device=DEV, compressed=False)
    out = pruner.prune(X, Wg, Wu, Wd, alpha=0.5, sparsity=0.6)
    norm_one_call = to_np32(pruner.norm).copy()
    for pname, W, axis, alpha in (("gate", Wg, AXIS_ROWS, 0.5), ("down", Wd, AXIS_COLS, 1.0)):
        want = oracle.select_unstructured(to_np32(W), norm_one_call, axis, alpha, 0.6, axis)
        assert np.array_equal(u32(out[pname]["mask"]), oracle.pack_mask(want))
        want_pruned = np.where(want == 1, to_np32(W), np.float32(0.0))
        assert np.array_equal(bits_of(out[pname]["pruned"]), bits_like(want_pruned, W.dtype))
    # the sums carry over between calls: three uneven batches give the same norms up to fp64 rounding of the sums
    pruner.reset()
    for t0, t1 in ((0, 300), (300, 301), (301, cfg.T)):
        pruner.accumulate(X[t0:t1], Wg, Wu)
    pruner.finalize()
    pruner.check()
    assert np.max(np.abs(to_np32(pruner.norm) - norm_one_call) / norm_one_call) <= 1e-6


def test_prune_unstructured_with_long_lines_through_the_layer_calls():
    """A layer whose comparison lines have 4608 elements (the streaming selection kernels): calibration, then the
    paper's 50 % unstructured setting on all three matrices, against the oracle fed the GPU's norms; then the same
    weights through forward_pruned()."""
    cfg, X, Wg, Wu, Wd = _layer("llama2_7b", d=384, I=4608, T=300)
    pruner = LayerPruner(cfg.T, cfg.d, cfg.I, X.dtype, act=cfg.act, device=DEV, compressed=False)
    out = pruner.prune(X, Wg, Wu, Wd, alpha=0.5, sparsity=0.5)
    pruner.check()
    ref_norm = oracle.norm_from_sumsq(oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), ORACLE_ACT[cfg.act]))
    norm = to_np32(pruner.norm)
    assert np.max(np.abs(norm - ref_norm) / ref_norm) <= 2e-3
    for pname, W, axis, alpha in (("gate", Wg, AXIS_ROWS, 0.5), ("up", Wu, AXIS_ROWS, 0.5), ("down", Wd, AXIS_COLS, 1.0)):
        want = oracle.select_unstructured(to_np32(W), norm, axis, alpha, 0.5, axis)
        assert np.array_equal(u32(out[pname]["mask"]), oracle.pack_mask(want)), pname
        assert np.array_equal(bits_of(out[pname]["pruned"]), bits_like(np.where(want == 1, to_np32(W), np.float32(0.0)), W.dtype)), pname
    Z = pruner.forward_pruned(X)
    pruner.check()
    Z_ref, _ = oracle.mlp_forward(to_np32(X), to_np32(out["gate"]["pruned"]), to_np32(out["up"]["pruned"]),
                                  to_np32(out["down"]["pruned"]), ORACLE_ACT[cfg.act], True, want_h=True)
    z = to_np32(Z).astype(np.float64)
    err = np.sqrt(np.mean((z - Z_ref) ** 2)) / (np.sqrt(np.mean(Z_ref ** 2)) + 1e-30)
    assert err <= 6e-3                                          # the bound test_gpu_forward.py derives for bf16


def test_forward_of_the_pruned_layer_matches_oracle_forward_of_the_same_weights():
    """prune() then forward_pruned(): the oracle's forward pass of the very weights the GPU pruned (bf16 rounding
    of the intermediate on both sides), in one pass and in token chunks."""
    cfg, X, Wg, Wu, Wd = _layer("llama2_7b", d=256, I=688, T=700)
    pruner = LayerPruner(cfg.T, cfg.d, cfg.I, X.dtype, act=cfg.act, device=DEV, compressed=False)
    out = pruner.prune(X, Wg, Wu, Wd, alpha=0.5)
    Z = pruner.forward_pruned(X)
    pruner.check()
    Zc = pruner.forward_pruned(X, workspace_bytes=1)            # smallest workspace: 256-token chunks
    assert np.array_equal(bits_of(Z), bits_of(Zc))
    Z_ref, _ = oracle.mlp_forward(to_np32(X), to_np32(out["gate"]["pruned"]), to_np32(out["up"]["pruned"]),
                                  to_np32(out["down"]["pruned"]), ORACLE_ACT[cfg.act], True, want_h=True)
    z = to_np32(Z).astype(np.float64)
    err = np.sqrt(np.mean((z - Z_ref) ** 2)) / (np.sqrt(np.mean(Z_ref ** 2)) + 1e-30)
    assert err <= 6e-3                                          # the bound test_gpu_forward.py derives for bf16
    assert float((out["gate"]["pruned"] == 0).float().mean()) >= 0.5
