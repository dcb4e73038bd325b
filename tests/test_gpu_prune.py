"""GPU parity of dass_prune_nm (stage (b) in one pass: score, N:M selection, mask, pruned copy, compressed values and
metadata from a single read of W) against the fp64 oracle, bit for bit, with the oracle's norm vector fed to the GPU."""
import numpy as np
import pytest
import torch

from helpers import assert_stage_b_equal, bits_of, oracle_stage_b, to_np32, u32, unpack_mask
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


def gpu_prune(W, norm, norm_axis, alpha, n_keep, m, group_axis, **kw):
    mask, pruned, values, meta = binding.prune_nm(W, norm, norm_axis, alpha, n_keep, m, group_axis, **kw)
    binding.prune_status()                   # waits for the stream; raises if a bounded wait ran out
    cols = W.shape[1]
    return dict(words=u32(mask), pruned_bits=bits_of(pruned[:, :cols]), values_bits=bits_of(values), meta=u32(meta))


SHAPES = [  # rows, cols, ld  (several 8 x 256 units plus ragged edges in both directions)
    (40, 688, 688), (72, 344, 352), (8, 8, 8), (264, 1032, 1040), (96, 24, 24), (44, 520, 520),
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (1, 4), (3, 4), (5, 8)])
@pytest.mark.parametrize("norm_axis,group_axis", [(AXIS_ROWS, AXIS_ROWS), (AXIS_COLS, AXIS_COLS),
                                                  (AXIS_ROWS, AXIS_COLS), (AXIS_COLS, AXIS_ROWS)])
def test_random_shapes_bit_exact(dtype, n_keep, m, norm_axis, group_axis):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(7000 + 1000 * m + 100 * n_keep + 10 * norm_axis + group_axis)
    for (rows, cols, ld) in SHAPES:
        if group_axis == AXIS_ROWS and rows % m:
            continue
        for alpha, ties in [(0.5, False), (1.0, True), (0.0, False), (0.25, True), (0.75, False)]:
            base, W = _padded(rows, cols, ld, dtype, gen, ties=ties)
            norm = _norm(rows if norm_axis == AXIS_ROWS else cols, gen, ties=ties)
            ref = oracle_stage_b(W, to_np32(norm), norm_axis, alpha, n_keep, m, group_axis)
            got = gpu_prune(W, norm, norm_axis, alpha, n_keep, m, group_axis)
            assert_stage_b_equal(got, ref)
            mk = unpack_mask(got["words"], cols)                   # exactly n_keep survivors in every group
            if group_axis == AXIS_COLS:
                assert np.all(mk.reshape(rows, cols // m, m).sum(-1) == n_keep)
            else:
                assert np.all(mk.reshape(rows // m, m, cols).sum(1) == n_keep)
            assert torch.all(base[:, cols:] == 7.0)                # the padding of the input is never touched


@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (3, 4)])
@pytest.mark.parametrize("group_axis", [AXIS_ROWS, AXIS_COLS])
def test_same_bits_as_the_two_pass_route(n_keep, m, group_axis):
    """dass_prune_nm against dass_score_nm followed by dass_compress_nm on a few thousand units."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(99 + m + group_axis)
    rows, cols = 1048, 2568
    base, W = _padded(rows, cols, cols, torch.bfloat16, gen)
    norm = _norm(rows if group_axis == AXIS_ROWS else cols, gen)
    mask, pruned = binding.score_nm(W, norm, group_axis, 0.5, n_keep, m, group_axis)
    values, meta = binding.compress_nm(W, mask, n_keep, m, group_axis)
    got = gpu_prune(W, norm, group_axis, 0.5, n_keep, m, group_axis)
    assert np.array_equal(got["words"], u32(mask)) and np.array_equal(got["pruned_bits"], bits_of(pruned))
    assert np.array_equal(got["values_bits"], bits_of(values)) and np.array_equal(got["meta"], u32(meta))


@pytest.mark.parametrize("group_axis", [AXIS_ROWS, AXIS_COLS])
@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8), (1, 4)])
def test_any_subset_of_outputs_and_in_place(group_axis, n_keep, m):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(17 + m)
    base, W = _padded(64, 776, 776, torch.bfloat16, gen)
    norm = _norm(64 if group_axis == AXIS_ROWS else 776, gen)
    ref = oracle_stage_b(W, to_np32(norm), group_axis, 0.5, n_keep, m, group_axis)
    args = (W, norm, group_axis, 0.5, n_keep, m, group_axis)
    mask, none1, none2, none3 = binding.prune_nm(*args, want_pruned=False, want_compressed=False)
    assert none1 is None and none2 is None and none3 is None
    none0, pruned, none2, none3 = binding.prune_nm(*args, want_mask=False, want_compressed=False)
    assert none0 is None and none2 is None
    none0, none1, values, meta = binding.prune_nm(*args, want_mask=False, want_pruned=False)
    assert none0 is None and none1 is None
    Wc = W.clone()
    _, _, values2, meta2 = binding.prune_nm(Wc, *args[1:], want_mask=False, W_pruned=Wc)       # in place, with values
    torch.cuda.synchronize()
    assert np.array_equal(u32(mask), ref["words"])
    assert np.array_equal(bits_of(pruned), ref["pruned_bits"]) and np.array_equal(bits_of(Wc), ref["pruned_bits"])
    for v, t in ((values, meta), (values2, meta2)):
        assert np.array_equal(bits_of(v), ref["values_bits"]) and np.array_equal(u32(t), ref["meta"])


def test_values_whose_rows_are_not_vector_aligned():
    """cols not a multiple of 8: the value rows of a row-group matrix start at odd 4-byte offsets."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(23)
    for n_keep, m in ((2, 4), (4, 8)):
        for rows, cols, ld in ((16, 260, 264), (24, 12, 16), (8, 508, 512)):
            base, W = _padded(rows, cols, ld, torch.bfloat16, gen)
            for axis in (AXIS_ROWS, AXIS_COLS):
                if axis == AXIS_COLS and cols % m:
                    continue
                norm = _norm(rows if axis == AXIS_ROWS else cols, gen)
                ref = oracle_stage_b(W, to_np32(norm), axis, 0.5, n_keep, m, axis)
                assert_stage_b_equal(gpu_prune(W, norm, axis, 0.5, n_keep, m, axis), ref)


@pytest.mark.parametrize("name", ["llama2_7b", "mistral_7b", "gemma_7b", "llama2_70b"])
def test_scaled_down_configs(name):
    """Each large layer's recipe (row amplification, heavy tails, its n:m) at 1/16 of the size."""
    big = synth.CONFIGS[name]
    cfg = synth.scaled(big, d=big.d // 16, I=big.I // 16, T=256)
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(cfg.seed)
    norm = (torch.randn(cfg.I, generator=gen, device=DEV).abs() * 40 + 0.5).float()
    norm[::97] = 0.0                                               # dead neurons
    norm32 = to_np32(norm)
    for alpha in cfg.alphas:
        for W in (Wg, Wu):
            ref = oracle_stage_b(W, norm32, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS)
            assert_stage_b_equal(gpu_prune(W, norm, AXIS_ROWS, alpha, cfg.n_keep, cfg.m, AXIS_ROWS), ref)
    ref = oracle_stage_b(Wd, norm32, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS)
    assert_stage_b_equal(gpu_prune(Wd, norm, AXIS_COLS, 1.0, cfg.n_keep, cfg.m, AXIS_COLS), ref)


def test_outputs_stay_inside_their_buffers():
    from test_gpu_guard_bands import guarded, intact
    rows, cols = 72, 344
    for dtype in (torch.bfloat16, torch.float32):
        for group_axis in (AXIS_ROWS, AXIS_COLS):
            for n_keep, m in ((2, 4), (4, 8), (3, 4)):
                W = (torch.randn((rows, cols), device=DEV) * 0.02).to(dtype)
                norm = (torch.rand(rows if group_axis == AXIS_ROWS else cols, device=DEV) * 10 + 0.1).float()
                mbuf, mask = guarded((rows, binding.mask_words_per_row(cols)), torch.int32, 0x5A5A5A5A)
                pbuf, pruned = guarded((rows, cols), dtype, 7.0)
                vshape, mshape = binding.compress_shapes(rows, cols, n_keep, m, group_axis)
                vbuf, values = guarded(vshape, dtype, 7.0)
                tbuf, meta = guarded(mshape, torch.int32, 0x5A5A5A5A)
                binding.prune_nm(W, norm, group_axis, 0.5, n_keep, m, group_axis, mask_bits=mask, W_pruned=pruned,
                                 values=values, meta=meta)
                torch.cuda.synchronize()
                assert intact(mbuf, mask.numel(), 0x5A5A5A5A) and intact(pbuf, pruned.numel(), 7.0)
                assert intact(vbuf, values.numel(), 7.0) and intact(tbuf, meta.numel(), 0x5A5A5A5A)
                words = u32(mask)
                assert np.all(words[:, -1] >> (cols - 32 * (words.shape[1] - 1)) == 0)      # padding bits are zero
