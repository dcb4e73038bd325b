"""GPU parity of stage (b): dass_score_nm and dass_compress_nm against the fp64 oracle, bit for bit,
with the oracle's norm vector fed to the GPU (so no floating-point slack is involved)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_stage_b_equal, bits_of, gpu_stage_b, oracle_stage_b, to_np32, u32, unpack_mask
from paper_2405_01943_b200 import binding, synth
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _padded(rows, cols, ld, dtype, gen, sigma=0.02, ties=False):
    base = torch.full((rows, ld), 7.0, dtype=dtype, device=DEV)      # poison in the padding
    if ties:
        vals = torch.tensor([0.0, -0.0, 0.25, -0.25, 0.5, 1.0, -1.0, 2.0], device=DEV)
        w = vals[torch.randint(0, len(vals), (rows, cols), generator=gen, device=DEV)]
    else:
        w = torch.randn((rows, cols), generator=gen, device=DEV) * sigma
    base[:, :cols] = w.to(dtype)
    return base, base[:, :cols]


def _norm(n, gen, ties=False):
    if ties:
        vals = torch.tensor([0.0, 1.0, 4.0, 16.0, 2.0, 9.0], device=DEV)
        return vals[torch.randint(0, len(vals), (n,), generator=gen, device=DEV)].contiguous()
    return (torch.randn(n, generator=gen, device=DEV).abs() * 30 + 0.01).float().contiguous()


SHAPES = [  # rows, cols, ld  (several 32x256 tiles plus ragged edges in both directions)
    (40, 688, 688), (72, 344, 352), (8, 8, 8), (264, 1032, 1040), (96, 24, 24),
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (1, 4), (3, 4), (5, 8)])
@pytest.mark.parametrize("norm_axis,group_axis", [(AXIS_ROWS, AXIS_ROWS), (AXIS_COLS, AXIS_COLS),
                                                  (AXIS_ROWS, AXIS_COLS), (AXIS_COLS, AXIS_ROWS)])
def test_random_shapes_bit_exact(dtype, n_keep, m, norm_axis, group_axis):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1000 * m + 100 * n_keep + 10 * norm_axis + group_axis)
    for (rows, cols, ld) in SHAPES:
        for alpha, ties in [(0.5, False), (1.0, True), (0.0, False), (0.25, True), (0.75, False)]:
            base, W = _padded(rows, cols, ld, dtype, gen, ties=ties)
            norm = _norm(rows if norm_axis == AXIS_ROWS else cols, gen, ties=ties)
            ref = oracle_stage_b(W, to_np32(norm), norm_axis, alpha, n_keep, m, group_axis)
            got = gpu_stage_b(W, norm, norm_axis, alpha, n_keep, m, group_axis)
            assert_stage_b_equal(got, ref)
            # exactly n_keep survivors in every group (Section 3, N:M)
            mk = unpack_mask(got["words"], cols)
            if group_axis == AXIS_COLS:
                assert np.all(mk.reshape(rows, cols // m, m).sum(-1) == n_keep)
            else:
                assert np.all(mk.reshape(rows // m, m, cols).sum(1) == n_keep)


@pytest.mark.parametrize("n_keep", [1, 2, 3])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_row_groups_of_four_with_an_odd_number_of_groups(dtype, n_keep):
    """Row counts that are a multiple of 4 but not of 8 (the row-group kernels take 8 rows at a time, so the last
    group of 4 stands alone), down to a single group, with ragged column counts."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(4242 + n_keep)
    for rows, cols, ld in [(4, 8, 8), (12, 40, 40), (44, 344, 352), (36, 1032, 1040), (100, 24, 24)]:
        for ties in (False, True):
            base, W = _padded(rows, cols, ld, dtype, gen, ties=ties)
            norm = _norm(rows, gen, ties=ties)
            ref = oracle_stage_b(W, to_np32(norm), AXIS_ROWS, 0.5, n_keep, 4, AXIS_ROWS)
            assert_stage_b_equal(gpu_stage_b(W, norm, AXIS_ROWS, 0.5, n_keep, 4, AXIS_ROWS), ref)
            assert torch.all(base[:, cols:] == 7.0)                # the padding of the input is never touched


def test_generic_alpha_uses_pow():
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    base, W = _padded(64, 512, 512, torch.bfloat16, gen)
    norm = _norm(64, gen)
    ref = oracle_stage_b(W, to_np32(norm), AXIS_ROWS, 0.3, 2, 4, AXIS_ROWS)
    got = gpu_stage_b(W, norm, AXIS_ROWS, 0.3, 2, 4, AXIS_ROWS)
    # pow() may differ in the last place between host and device libraries: allow a handful of
    # near-tie groups to differ, nothing more
    diff = (unpack_mask(got["words"], 512) != ref["mask"]).sum()
    assert diff <= 8


def test_outputs_do_not_touch_padding_and_padding_bits_are_zero():
    gen = torch.Generator(device=DEV)
    gen.manual_seed(6)
    rows, cols, ld = 40, 344, 352
    base, W = _padded(rows, cols, ld, torch.bfloat16, gen)
    norm = _norm(cols, gen)
    pruned_base = torch.full((rows, ld), -3.0, dtype=torch.bfloat16, device=DEV)
    mask = torch.full((rows, binding.mask_words_per_row(cols)), -1, dtype=torch.int32, device=DEV)
    binding.score_nm(W, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS, mask_bits=mask, W_pruned=pruned_base[:, :cols])
    torch.cuda.synchronize()
    assert torch.all(pruned_base[:, cols:] == -3.0)
    words = u32(mask)
    assert np.all(words[:, -1] >> (cols - 32 * (words.shape[1] - 1)) == 0)


@pytest.mark.parametrize("group_axis", [AXIS_ROWS, AXIS_COLS])
def test_in_place_and_single_output_calls(group_axis):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(7)
    base, W = _padded(64, 768, 768, torch.bfloat16, gen)
    norm = _norm(64 if group_axis == AXIS_ROWS else 768, gen)
    ref = oracle_stage_b(W, to_np32(norm), group_axis, 0.5, 2, 4, group_axis)
    mask_only, none = binding.score_nm(W, norm, group_axis, 0.5, 2, 4, group_axis, want_pruned=False)
    assert none is None
    none, pruned_only = binding.score_nm(W, norm, group_axis, 0.5, 2, 4, group_axis, want_mask=False)
    assert none is None
    Wc = W.clone()
    binding.score_nm(Wc, norm, group_axis, 0.5, 2, 4, group_axis, want_mask=False, W_pruned=Wc)   # in place
    torch.cuda.synchronize()
    assert np.array_equal(u32(mask_only), ref["words"])
    assert np.array_equal(bits_of(pruned_only), ref["pruned_bits"])
    assert np.array_equal(bits_of(Wc), ref["pruned_bits"])


def test_tiny_config_all_three_projections():
    """The small SwiGLU case in full: gate/up by Eq. 4 (input-balanced 2:4), down by Eq. 5."""
    cfg = synth.CONFIGS["tiny"]
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    X = synth.make_x(cfg, DEV)
    norm32 = oracle.norm_from_sumsq(oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oracle.ACT_SILU))
    norm = torch.from_numpy(norm32).to(DEV)
    for W in (Wg, Wu):
        for alpha in (0.0, 0.5, 1.0):
            ref = oracle_stage_b(W, norm32, AXIS_ROWS, alpha, 2, 4, AXIS_ROWS)
            assert_stage_b_equal(gpu_stage_b(W, norm, AXIS_ROWS, alpha, 2, 4, AXIS_ROWS), ref)
        ref = oracle_stage_b(W, norm32, AXIS_ROWS, 0.5, 2, 4, AXIS_COLS)          # literal row-wise reading
        assert_stage_b_equal(gpu_stage_b(W, norm, AXIS_ROWS, 0.5, 2, 4, AXIS_COLS), ref)
    ref = oracle_stage_b(Wd, norm32, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)
    assert_stage_b_equal(gpu_stage_b(Wd, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS), ref)


@pytest.mark.parametrize("name", ["llama2_7b", "mistral_7b", "gemma_7b", "llama2_70b"])
def test_scaled_down_configs(name):
    """Each large layer's recipe (row amplification, heavy tails, its n:m) at 1/16 of the size."""
    big = synth.CONFIGS[name]
    cfg = synth.scaled(big, d=big.d // 16, I=big.I // 16, T=256)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(cfg.seed)
    norm = (torch.randn(cfg.I, generator=gen, device=DEV).abs() * 40 + 0.5).float()
    norm32 = to_np32(norm)
    for alpha in cfg.alphas:
        for W in (Wg, Wu):
            ref = oracle_stage_b(W, norm32, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS)
            assert_stage_b_equal(gpu_stage_b(W, norm, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS), ref)
    ref = oracle_stage_b(Wd, norm32, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS)
    assert_stage_b_equal(gpu_stage_b(Wd, norm, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS), ref)


def test_norm_finalize_bit_exact():
    s = torch.tensor([0.0, 4.0, 2.0, 1e-30, 3.5e20, 123456.789], dtype=torch.float64, device=DEV)
    n = binding.norm_finalize(s)
    torch.cuda.synchronize()
    assert np.array_equal(n.cpu().numpy(), oracle.norm_from_sumsq(s.cpu().numpy()))
