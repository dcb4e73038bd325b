"""GPU parity of dass_select_unstructured (Section 3, "Pruning Granularity": prune the floor(s*L) lowest scores
of every comparison line) against the oracle, bit for bit, given the oracle's norm vector."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bits_like, bits_of, to_np32, u32, unpack_mask
from paper_2405_01943_b200 import binding, synth
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _check(W, norm, norm_axis, alpha, s, compare_axis):
    mask_bits, pruned = binding.select_unstructured(W, norm, norm_axis, alpha, s, compare_axis)
    torch.cuda.synchronize()
    rows, cols = W.shape
    Wn = to_np32(W)
    want = oracle.select_unstructured(Wn, to_np32(norm), norm_axis, alpha, s, compare_axis)
    assert np.array_equal(u32(mask_bits), oracle.pack_mask(want)), "mask words differ"
    want_pruned = np.where(want == 1, Wn, np.float32(0.0))
    assert np.array_equal(bits_of(pruned[:, :cols]), bits_like(want_pruned, W.dtype)), "pruned weights differ"
    L = rows if compare_axis == AXIS_ROWS else cols
    kept = unpack_mask(u32(mask_bits), cols).sum(0 if compare_axis == AXIS_ROWS else 1)
    assert np.all(kept == L - int(np.floor(s * L)))


def _mat(rows, cols, ld, dtype, gen, ties=False):
    base = torch.full((rows, ld), 7.0, dtype=dtype, device=DEV)
    if ties:
        vals = torch.tensor([0.0, -0.0, 0.25, -0.25, 0.5, 1.0, -1.0, 2.0], device=DEV)
        w = vals[torch.randint(0, len(vals), (rows, cols), generator=gen, device=DEV)]
    else:
        w = torch.randn((rows, cols), generator=gen, device=DEV) * 0.02
    base[:, :cols] = w.to(dtype)
    return base[:, :cols]


def _norm(n, gen, ties=False):
    if ties:
        vals = torch.tensor([0.0, 1.0, 4.0, 16.0, 2.0, 9.0], device=DEV)
        return vals[torch.randint(0, len(vals), (n,), generator=gen, device=DEV)].contiguous()
    return (torch.randn(n, generator=gen, device=DEV).abs() * 30 + 0.01).float().contiguous()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("norm_axis,compare_axis", [(AXIS_ROWS, AXIS_ROWS), (AXIS_COLS, AXIS_COLS),
                                                    (AXIS_ROWS, AXIS_COLS), (AXIS_COLS, AXIS_ROWS)])
@pytest.mark.parametrize("ties", [False, True], ids=["random", "ties"])
def test_small_shapes_bit_exact(dtype, norm_axis, compare_axis, ties):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(17 + 2 * norm_axis + compare_axis)
    for rows, cols, ld in [(40, 688, 688), (73, 344, 352), (1, 8, 8), (300, 1031, 1032), (9, 3, 8), (688, 256, 256)]:
        for s, alpha in [(0.5, 0.5), (0.33, 1.0), (0.0, 0.0), (0.9, 0.25)]:
            W = _mat(rows, cols, ld, dtype, gen, ties)
            norm = _norm(rows if norm_axis == AXIS_ROWS else cols, gen, ties)
            _check(W, norm, norm_axis, alpha, s, compare_axis)


def test_tiny_config_input_and_output_balanced():
    cfg = synth.CONFIGS["tiny"]
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    X = synth.make_x(cfg, DEV)
    norm32 = oracle.norm_from_sumsq(oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oracle.ACT_SILU))
    norm = torch.from_numpy(norm32).to(DEV)
    for W in (Wg, Wu):
        _check(W, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)        # Eq. 4, input-balanced
    _check(Wd, norm, AXIS_COLS, 1.0, 0.5, AXIS_COLS)            # Eq. 5, output-balanced


def test_full_size_70b_sampled_lines():
    """Full 70B-shaped matrices on the GPU; the oracle redoes a sample of the lines (lines are independent)."""
    cfg = synth.CONFIGS["llama2_70b"]
    Wg, _, Wd = synth.make_weights(cfg, DEV)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    norm = (torch.randn(cfg.I, generator=gen, device=DEV).abs() * 40 + 0.5).float().contiguous()
    norm32 = to_np32(norm)
    # gate: lines are columns
    mask_bits, _ = binding.select_unstructured(Wg, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS, want_pruned=False)
    torch.cuda.synchronize()
    got = unpack_mask(u32(mask_bits), cfg.d)
    assert np.all(got.sum(0) == cfg.I - cfg.I // 2)
    cols = np.array([0, 1, 31, 32, 4095, 8190, 8191])
    want = oracle.select_unstructured(to_np32(Wg[:, torch.from_numpy(cols).to(DEV)]), norm32, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
    assert np.array_equal(got[:, cols], want)
    del mask_bits
    # down: lines are rows
    mask_bits, pruned = binding.select_unstructured(Wd, norm, AXIS_COLS, 1.0, 0.5, AXIS_COLS)
    torch.cuda.synchronize()
    got = unpack_mask(u32(mask_bits), cfg.I)
    assert np.all(got.sum(1) == cfg.I - cfg.I // 2)
    rws = np.array([0, 1, 2, 4097, 8190, 8191])
    sub = Wd[torch.from_numpy(rws).to(DEV)]
    want = oracle.select_unstructured(to_np32(sub), norm32, AXIS_COLS, 1.0, 0.5, AXIS_COLS)
    assert np.array_equal(got[rws], want)
    want_pruned = np.where(want == 1, to_np32(sub), np.float32(0.0))
    assert np.array_equal(bits_of(pruned[torch.from_numpy(rws).to(DEV)]), bits_like(want_pruned, Wd.dtype))


def test_argument_errors():
    lib = binding.load()
    F = 0x10000
    f = lib.dass_select_unstructured
    assert f(None, 8, 64, 64, 0, F, 1, 1.0, 0.5, 1, F, F, F, 1 << 20, None) == 1
    assert f(F, 8, 64, 64, 0, F, 1, 1.0, 1.0, 1, F, F, F, 1 << 20, None) == 2      # sparsity must be < 1
    assert f(F, 8, 64, 64, 0, F, 1, 1.0, -0.1, 1, F, F, F, 1 << 20, None) == 2
    assert f(F, 8, 64, 68, 0, F, 1, 1.0, 0.5, 1, F, F, F, 1 << 20, None) == 3
    assert f(F, 8, 64, 64, 0, F, 1, 1.0, 0.5, 1, F, F, None, 0, None) == 6
    assert f(F, 8, 200000, 200000, 0, F, 1, 1.0, 0.5, 1, F, F, F, 1 << 26, None) == 5   # a line does not fit in shared memory
