"""Parity at the full sizes of the large layer shapes (LLaMA2-7B / 13B / 70B, Mistral-7B, Gemma-7B),
in the launch configuration the benchmark times (whole 262144-token calibration batch in one call).

The oracle cannot redo 10^13..10^14 flops, so stage (a) is checked on outputs it can compute one by one:
 (i)  sampled neurons (strided through every part of the matrix plus the largest-norm ones) over ALL tokens;
 (ii) all neurons on a token prefix (a separate GPU call).
Stage (b) is checked in full: every mask word, pruned weight, compressed value and metadata word of the
gate and down matrices, bit for bit, with the oracle's norm vector.  Finally the end-to-end rule: masks from
GPU norms may differ from masks from oracle norms only in groups whose oracle score gap is below 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_stage_b_equal, gpu_stage_b, oracle_stage_b, to_np32, u32, unpack_mask
from paper_2405_01943_b200 import binding, synth
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAMES = ["llama2_7b", "llama2_13b", "mistral_7b", "gemma_7b", "llama2_70b"]
ORACLE_ACT = {"silu": oracle.ACT_SILU, "gelu_tanh": oracle.ACT_GELU_TANH}
T_PREFIX = {"llama2_70b": 1024}         # tokens of the all-neuron prefix; 2048 for the other shapes
N_SAMPLED = 64


@pytest.fixture(scope="module", params=NAMES)
def layer(request):
    cfg = synth.CONFIGS[request.param]
    X = synth.make_x(cfg, DEV)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV, layer=0)
    yield cfg, X, Wg, Wu, Wd
    del X, Wg, Wu, Wd
    torch.cuda.empty_cache()


def _gpu_sumsq(cfg, X, Wg, Wu):
    sumsq = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(X.shape[0], cfg.d, cfg.I, X.dtype, DEV)
    binding.calib_accumulate(X, Wg, Wu, binding.ACT_BY_NAME[cfg.act], sumsq, ws)
    binding.calib_status(ws)
    return sumsq


def test_stage_a_sampled_neurons_over_all_tokens(layer):
    cfg, X, Wg, Wu, _ = layer
    got = _gpu_sumsq(cfg, X, Wg, Wu).cpu().numpy()
    assert np.all(np.isfinite(got)) and np.all(got > 0)
    top = np.argsort(-got)[: N_SAMPLED // 4]
    strided = np.linspace(0, cfg.I - 1, N_SAMPLED - len(top)).astype(np.int64)    # includes first and last neuron
    idx = np.unique(np.concatenate([top, strided]))
    sel = torch.from_numpy(idx).to(DEV)
    wg, wu = to_np32(Wg[sel]), to_np32(Wu[sel])
    ref = np.zeros(len(idx), dtype=np.float64)
    step = 32768
    for t0 in range(0, cfg.T, step):                       # the oracle accumulates batch by batch
        oracle.calib_sumsq(to_np32(X[t0:t0 + step]), wg, wu, ORACLE_ACT[cfg.act], ref)
    rel = np.abs(np.sqrt(got[idx]) - np.sqrt(ref)) / np.sqrt(ref)
    assert rel.max() <= 2e-3, f"{cfg.name}: sampled-neuron norm error {rel.max():.3e}"


def _group_gaps(Wn, scale, na, ga, n_keep, m, diff):
    """Oracle score gap (s_(n_keep) - s_(n_keep+1)) / s_(n_keep) of every group that holds a differing mask bit."""
    r, c = diff[:, 0], diff[:, 1]
    if ga == AXIS_COLS:
        keys = np.unique(np.stack([r, c // m], 1), axis=0)
        rr = np.repeat(keys[:, :1], m, 1)
        cc = keys[:, 1:2] * m + np.arange(m)[None, :]
    else:
        keys = np.unique(np.stack([r // m, c], 1), axis=0)
        rr = keys[:, :1] * m + np.arange(m)[None, :]
        cc = np.repeat(keys[:, 1:2], m, 1)
    score = np.abs(Wn[rr, cc].astype(np.float64)) * (scale[cc] if na == AXIS_COLS else scale[rr])
    srt = -np.sort(-score, axis=1)
    top, nxt = srt[:, n_keep - 1], srt[:, n_keep]
    return keys, (top - nxt) / np.where(top > 0, top, 1.0)


def test_stage_a_all_neurons_on_a_token_prefix_then_end_to_end_masks(layer):
    cfg, X, Wg, Wu, Wd = layer
    Xp = X[:T_PREFIX.get(cfg.name, 2048)]
    sumsq = _gpu_sumsq(cfg, Xp, Wg, Wu)
    ref = oracle.calib_sumsq(to_np32(Xp), to_np32(Wg), to_np32(Wu), ORACLE_ACT[cfg.act])
    rel = np.abs(np.sqrt(sumsq.cpu().numpy()) - np.sqrt(ref)) / np.sqrt(ref)
    assert rel.max() <= 2e-3, f"{cfg.name}: prefix norm error {rel.max():.3e}"

    # end to end over the WHOLE down and gate projections: masks from the GPU's norms against the oracle's masks from
    # the oracle's norms may differ only in groups whose oracle score gap is below 1e-3 (and such groups are rare)
    norm_gpu = binding.norm_finalize(sumsq)
    norm_ref = oracle.norm_from_sumsq(ref)
    for W, na, alpha, ga in ((Wd, AXIS_COLS, 1.0, AXIS_COLS), (Wg, AXIS_ROWS, 0.5, AXIS_ROWS)):
        mask_gpu, _, _, _ = binding.prune_nm(W, norm_gpu, na, alpha, cfg.n_keep, cfg.m, ga, want_pruned=False, want_compressed=False)
        binding.prune_status()
        got = unpack_mask(u32(mask_gpu), W.shape[1])
        Wn = to_np32(W)
        want, _ = oracle.score_nm(Wn, norm_ref, na, alpha, cfg.n_keep, cfg.m, ga, want_pruned=False)
        diff = np.argwhere(got != want)
        n_groups = got.size // cfg.m
        if len(diff):
            scale = np.array([oracle.scale(float(v), alpha) for v in norm_ref], dtype=np.float64)
            keys, gaps = _group_gaps(Wn, scale, na, ga, cfg.n_keep, cfg.m, diff)
            print(f"{cfg.name} {'down' if ga == AXIS_COLS else 'gate'}: {len(keys)} of {n_groups} groups differ, "
                  f"largest oracle gap {gaps.max():.3e}")
            worst = int(np.argmax(gaps))
            assert gaps.max() < 1e-3, f"{cfg.name}: group {tuple(keys[worst])} differs although the oracle gap is {gaps.max():.3e}"
            assert len(keys) <= 1e-3 * n_groups                            # and such near-ties are rare
        del got, want, Wn


def test_stage_b_full_matrices_bit_exact(layer):
    cfg, X, Wg, Wu, Wd = layer
    gen = torch.Generator(device=DEV)
    gen.manual_seed(cfg.seed + 77)
    # a norm vector with the spread real intermediate norms have (a few neurons far above the rest)
    norm = (torch.randn(cfg.I, generator=gen, device=DEV).abs() * 40 + 0.5)
    norm[torch.randperm(cfg.I, generator=gen, device=DEV)[: cfg.I // 100]] *= 30
    norm = norm.float().contiguous()
    norm32 = to_np32(norm)
    for alpha in cfg.alphas:
        ref = oracle_stage_b(Wg, norm32, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS)
        assert_stage_b_equal(gpu_stage_b(Wg, norm, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS), ref)
        del ref
    ref = oracle_stage_b(Wd, norm32, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS)
    got = gpu_stage_b(Wd, norm, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS)
    assert_stage_b_equal(got, ref)
    mk = unpack_mask(got["words"], cfg.I)
    assert np.all(mk.reshape(cfg.d, cfg.I // cfg.m, cfg.m).sum(-1) == cfg.n_keep)


@pytest.mark.parametrize("layer_id", [39, 79])
def test_70b_stream_other_layers_sampled_neurons(layer_id):
    """The 80-layer stream draws every layer from its own seed: check two more of them (middle and last)
    on sampled neurons over all tokens, as for layer 0 above."""
    cfg = synth.CONFIGS["llama2_70b"]
    X = synth.make_x(cfg, DEV)
    Wg, Wu, _ = synth.make_weights(cfg, DEV, layer=layer_id)
    got = _gpu_sumsq(cfg, X, Wg, Wu).cpu().numpy()
    idx = np.unique(np.concatenate([np.argsort(-got)[:4], np.linspace(0, cfg.I - 1, 12).astype(np.int64)]))
    sel = torch.from_numpy(idx).to(DEV)
    wg, wu = to_np32(Wg[sel]), to_np32(Wu[sel])
    ref = np.zeros(len(idx), dtype=np.float64)
    for t0 in range(0, cfg.T, 32768):
        oracle.calib_sumsq(to_np32(X[t0:t0 + 32768]), wg, wu, ORACLE_ACT[cfg.act], ref)
    rel = np.abs(np.sqrt(got[idx]) - np.sqrt(ref)) / np.sqrt(ref)
    assert rel.max() <= 2e-3, f"layer {layer_id}: sampled-neuron norm error {rel.max():.3e}"


@pytest.mark.parametrize("name,T", [("llama2_70b", 32768), ("llama2_7b", 8192 + 300), ("gemma_7b", 16384), ("llama2_13b", 2048)])
def test_stage_a_short_batches_sampled_neurons(name, T):
    """Short calibration batches of the full-width layers: the tensor-core kernels pick shorter bands of token tiles
    for them (other item counts, other partial-sum layouts than the full 262144-token call), and two such batches
    accumulate.  Sampled neurons over all tokens against the oracle."""
    cfg = synth.scaled(synth.CONFIGS[name], T=T)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, _ = synth.make_weights(cfg, DEV)
    sumsq = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(T, cfg.d, cfg.I, X.dtype, DEV)
    act = binding.ACT_BY_NAME[cfg.act]
    binding.calib_accumulate(X, Wg, Wu, act, sumsq, ws)
    once = sumsq.clone()
    binding.calib_accumulate(X, Wg, Wu, act, sumsq, ws)            # a second batch (the same tokens) adds the same sums
    binding.calib_status(ws)
    got = once.cpu().numpy()
    assert np.array_equal(sumsq.cpu().numpy(), 2.0 * got)          # doubling is exact: the kernel is deterministic
    idx = np.unique(np.concatenate([np.argsort(-got)[:8], np.linspace(0, cfg.I - 1, 24).astype(np.int64)]))
    sel = torch.from_numpy(idx).to(DEV)
    ref = oracle.calib_sumsq(to_np32(X), to_np32(Wg[sel]), to_np32(Wu[sel]), ORACLE_ACT[cfg.act])
    rel = np.abs(np.sqrt(got[idx]) - np.sqrt(ref)) / np.sqrt(ref)
    assert rel.max() <= 2e-3, f"{name} T={T}: sampled-neuron norm error {rel.max():.3e}"


def test_workspace_sized_for_more_tokens_serves_shorter_batches():
    """A workspace obtained for a long batch is accepted for shorter ones even where the short batch alone would have
    asked for more room (finer partial sums): the call then falls back to coarser bands; results agree to rounding."""
    cfg = synth.scaled(synth.CONFIGS["llama2_70b"], T=65536)
    X = synth.make_x(cfg, DEV)
    Wg, Wu, _ = synth.make_weights(cfg, DEV)
    act = binding.ACT_BY_NAME[cfg.act]
    big = binding.calib_workspace_bytes(cfg.T, cfg.d, cfg.I, X.dtype)
    sizes = {T: binding.calib_workspace_bytes(T, cfg.d, cfg.I, X.dtype) for T in (49152, 32768, 300)}
    assert max(sizes.values()) > big                      # the case this test is about exists at these shapes
    ws_big = binding.calib_workspace(cfg.T, cfg.d, cfg.I, X.dtype, DEV)
    for T in sizes:
        a = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
        b_ = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
        binding.calib_accumulate(X[:T], Wg, Wu, act, a, ws_big)
        binding.calib_status(ws_big)
        ws_own = binding.calib_workspace(T, cfg.d, cfg.I, X.dtype, DEV)
        binding.calib_accumulate(X[:T], Wg, Wu, act, b_, ws_own)
        binding.calib_status(ws_own)
        a, b_ = a.cpu().numpy(), b_.cpu().numpy()
        assert np.all(a > 0) and np.max(np.abs(a - b_) / b_) <= 1e-12
