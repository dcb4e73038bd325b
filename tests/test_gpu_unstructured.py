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


# ---------------------------------------------------------------- lines long enough for the streaming kernels
# (4096 elements and more: sampled bracket, one histogram sweep, the cut's bin ranked at the end; lines those
# kernels cannot decide go to the radix select)
def _long_case(kind, rows, cols, dtype, gen, line_axis):
    """A matrix whose comparison lines run along `line_axis` (0: columns are the lines, 1: rows are)."""
    L = rows if line_axis == 0 else cols
    n_lines = cols if line_axis == 0 else rows
    w = torch.randn((rows, cols), generator=gen, device=DEV) * 0.02
    lines = torch.arange(n_lines, device=DEV)
    along = torch.arange(L, device=DEV)

    def put(sel_lines, values):                      # values: [L, len(sel_lines)] along the line
        if line_axis == 0:
            w[:, sel_lines] = values
        else:
            w[sel_lines, :] = values.t()

    if kind == "ties":                               # a handful of magnitudes: the cut's bin overflows everywhere
        vals = torch.tensor([0.0, -0.0, 0.25, -0.25, 0.5, 1.0, -1.0, 2.0], device=DEV)
        w = vals[torch.randint(0, len(vals), (rows, cols), generator=gen, device=DEV)]
    elif kind == "mixed":                            # every third line tied, the others random
        sel = lines[::3]
        vals = torch.tensor([0.125, -0.125, 0.5, 3.0], device=DEV)
        put(sel, vals[torch.randint(0, len(vals), (L, len(sel)), generator=gen, device=DEV)])
    elif kind == "zeros":                            # two thirds of every other line are zero: the cut sits at zero
        sel = lines[::2]
        v = torch.randn((L, len(sel)), generator=gen, device=DEV) * 0.02
        v[torch.rand((L, len(sel)), generator=gen, device=DEV) < 0.66] = 0.0
        put(sel, v)
    elif kind == "outliers":                         # a few huge and a few tiny magnitudes in every line
        big = torch.randint(0, L, (16,), generator=gen, device=DEV)
        tiny = torch.randint(0, L, (64,), generator=gen, device=DEV)
        if line_axis == 0:
            w[big, :] *= 1e6
            w[tiny, :] *= 1e-12
        else:
            w[:, big] *= 1e6
            w[:, tiny] *= 1e-12
    elif kind == "spread":                           # magnitudes over 24 octaves: the window must follow the quantile
        e = torch.randint(-12, 12, (rows, cols), generator=gen, device=DEV).float()
        w = w * torch.exp2(e)
    ld = (cols + 7) // 8 * 8
    base = torch.full((rows, ld), 7.0, dtype=dtype, device=DEV)
    base[:, :cols] = w.to(dtype)
    return base[:, :cols]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("line_axis", [0, 1], ids=["column-lines", "row-lines"])
@pytest.mark.parametrize("kind", ["random", "ties", "mixed", "zeros", "outliers", "spread"])
def test_long_lines_bit_exact(dtype, line_axis, kind):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(101 + 7 * line_axis + len(kind))
    compare_axis = AXIS_ROWS if line_axis == 0 else AXIS_COLS
    # ragged everywhere: 4099 / 4233 elements per line, 27 / 21 lines (not multiples of 8 or 32)
    rows, cols = (4099, 27) if line_axis == 0 else (21, 4233)
    for norm_axis in (AXIS_ROWS, AXIS_COLS):         # the scale varies along the line, or is one number per line
        for s, alpha in [(0.5, 0.5), (0.07, 1.0), (0.97, 1.0), (0.0, 0.5), (0.5, 0.0)]:
            W = _long_case(kind, rows, cols, dtype, gen, line_axis)
            norm = _norm(rows if norm_axis == AXIS_ROWS else cols, gen, ties=(kind == "ties"))
            _check(W, norm, norm_axis, alpha, s, compare_axis)
    binding.prune_status()                           # raises if a bounded wait ran out or the passes disagreed


@pytest.mark.parametrize("line_axis", [0, 1], ids=["column-lines", "row-lines"])
def test_long_lines_in_place(line_axis):
    """W_pruned may be W itself: the streaming passes read every element before they overwrite it, and the elements
    of the cut's bin are put back from what was set aside."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(55 + line_axis)
    compare_axis = AXIS_ROWS if line_axis == 0 else AXIS_COLS
    rows, cols = (8200, 40) if line_axis == 0 else (24, 8200)
    norm_axis = compare_axis
    for kind in ("random", "mixed"):
        W = _long_case(kind, rows, cols, torch.bfloat16, gen, line_axis)
        norm = _norm(rows if norm_axis == AXIS_ROWS else cols, gen)
        Wn = to_np32(W)
        want = oracle.select_unstructured(Wn, to_np32(norm), norm_axis, 1.0, 0.5, compare_axis)
        mask_bits, pruned = binding.select_unstructured(W, norm, norm_axis, 1.0, 0.5, compare_axis, W_pruned=W)
        torch.cuda.synchronize()
        assert pruned.data_ptr() == W.data_ptr()
        assert np.array_equal(u32(mask_bits), oracle.pack_mask(want))
        assert np.array_equal(bits_of(W), bits_like(np.where(want == 1, Wn, np.float32(0.0)), W.dtype))
    binding.prune_status()


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


def test_column_lines_at_and_beyond_the_streaming_limit():
    """Columns of 2^18 rows still take the streaming kernels (128 stages of the bulk-copy ring per strip); one row more
    and the radix select decides them.  Both against the oracle, every element; 11 columns (a ragged last strip)."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(77)
    for rows in (1 << 18, (1 << 18) + 1):
        cols = 11
        W = _long_case("random", rows, cols, torch.bfloat16, gen, 0)
        norm = _norm(rows, gen)
        _check(W, norm, AXIS_ROWS, 0.5, 0.5, AXIS_ROWS)
    binding.prune_status()


def test_full_matrices_7b_shape_every_line():
    """Whole LLaMA2-7B-shaped matrices against the oracle, every line and every element: gate with columns as the
    lines (Eq. 4, alpha = 0.5, and alpha = 0 where equal magnitudes tie in every column), down with rows as the lines
    (Eq. 5).  Masks, pruned copies and the count of survivors per line."""
    cfg = synth.CONFIGS["llama2_7b"]
    Wg, _, Wd = synth.make_weights(cfg, DEV)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(9)
    norm = (torch.randn(cfg.I, generator=gen, device=DEV).abs() * 40 + 0.5).float().contiguous()
    norm32 = to_np32(norm)
    for W, axis, alpha, s in ((Wg, AXIS_ROWS, 0.5, 0.5), (Wg, AXIS_ROWS, 0.0, 0.5), (Wd, AXIS_COLS, 1.0, 0.5)):
        mask_bits, pruned = binding.select_unstructured(W, norm, axis, alpha, s, axis)
        binding.prune_status()
        Wn = to_np32(W)
        want = oracle.select_unstructured(Wn, norm32, axis, alpha, s, axis)
        assert np.array_equal(u32(mask_bits), oracle.pack_mask(want)), "mask words differ"
        assert np.array_equal(bits_of(pruned), bits_like(np.where(want == 1, Wn, np.float32(0.0)), W.dtype)), "pruned weights differ"
        L = W.shape[0] if axis == AXIS_ROWS else W.shape[1]
        assert np.all(want.sum(0 if axis == AXIS_ROWS else 1) == L - int(np.floor(s * L)))


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
