"""The checked-access build of the library (libdass_check.so: every global load and store of the kernels tested
against the buffers the call was given) run over ragged small cases of every entry point: no access may fall outside.
It stands in for a memory sanitizer.  A control shows that the checker does see an access outside a registered range:
the test hook registers the buffers a few kilobytes short, the accesses to that (perfectly valid) tail are skipped and
counted, nothing faults."""
import numpy as np
import pytest
import torch

from helpers import bits_of, oracle_stage_b, to_np32, u32
from paper_2405_01943_b200 import binding, build
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def check_lib():
    path = build.build_bounds_check()
    with binding.library(path):
        assert binding.bounds_report()["violations"] == 0
        yield
    torch.cuda.synchronize()


def _clean():
    rep = binding.bounds_report()
    assert rep["violations"] == 0, f"access outside the call's buffers: {rep}"


def _rand(shape, dtype, scale=0.02):
    return (torch.randn(shape, device=DEV) * scale).to(dtype)


def test_regular_library_has_no_checker():
    n = binding.load().dass_bounds_shrink_next(16)
    assert n == 5                                                   # DASS_ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_calibration_and_finalize(check_lib, dtype):
    for T, d, I in ((1030, 200, 392), (130, 72, 136), (300, 256, 688)):
        X, Wg, Wu = _rand((T, d), dtype, 1.0), _rand((I, d), dtype), _rand((I, d), dtype)
        sumsq = torch.zeros(I, dtype=torch.float64, device=DEV)
        ws = binding.calib_workspace(T, d, I, dtype, DEV)
        for act in (binding.ACT_SILU, binding.ACT_GELU_TANH, binding.ACT_RELU):
            binding.calib_accumulate(X, Wg, Wu, act, sumsq, ws)
            binding.calib_status(ws)
        norm = binding.norm_finalize(sumsq)
        addr = binding.calib_accumulate_static(X, Wg, Wu, binding.ACT_SILU, sumsq)
        binding.calib_status_at(addr)
        assert bool(torch.all(norm > 0))
        _clean()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("axis", [AXIS_ROWS, AXIS_COLS])
def test_stage_b_entry_points(check_lib, dtype, axis):
    for rows, cols, ld in ((72, 344, 352), (8, 8, 8), (264, 1032, 1040), (44, 520, 520)):
        base = torch.full((rows, ld), 7.0, dtype=dtype, device=DEV)
        base[:, :cols] = _rand((rows, cols), dtype)
        W = base[:, :cols]
        for n_keep, m in ((2, 4), (4, 8), (3, 4), (5, 8)):
            if axis == AXIS_ROWS and rows % m:
                continue
            for norm_axis in (AXIS_ROWS, AXIS_COLS):
                norm = (torch.rand(rows if norm_axis == AXIS_ROWS else cols, device=DEV) * 10 + 0.1).float()
                mask, pruned = binding.score_nm(W, norm, norm_axis, 0.5, n_keep, m, axis)
                values, meta = binding.compress_nm(W, mask, n_keep, m, axis)
                m2, p2, v2, t2 = binding.prune_nm(W, norm, norm_axis, 0.5, n_keep, m, axis)
                binding.prune_status()
                _clean()
                assert np.array_equal(u32(mask), u32(m2)) and np.array_equal(bits_of(values), bits_of(v2))
                assert np.array_equal(u32(meta), u32(t2)) and np.array_equal(bits_of(pruned[:, :cols]), bits_of(p2[:, :cols]))
    # and the results of the checking build are the oracle's
    ref = oracle_stage_b(W, to_np32(norm), AXIS_COLS, 0.5, 5, 8, axis) if (axis == AXIS_COLS or rows % 8 == 0) else None
    if ref is not None:
        assert np.array_equal(u32(m2), ref["words"]) and np.array_equal(bits_of(v2), ref["values_bits"])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_unstructured_selection_and_feature_norms(check_lib, dtype):
    for rows, cols in ((72, 344), (4104, 264), (40, 4200)):       # short lines, long column lines and long row lines (streaming kernels)
        W = _rand((rows, cols), dtype)
        for axis in (AXIS_ROWS, AXIS_COLS):
            norm = (torch.rand(rows if axis == AXIS_ROWS else cols, device=DEV) * 10 + 0.1).float()
            for sparsity in (0.5, 0.0, 0.73):
                binding.select_unstructured(W, norm, axis, 0.5, sparsity, axis)
            binding.select_unstructured(W, norm, axis, 0.0, 0.5, axis)          # ties everywhere
            binding.prune_status()
            _clean()
    X = _rand((1030, 200), dtype, 1.0)
    binding.feature_sumsq(X)
    _clean()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_forward_pass(check_lib, dtype):
    T, d, I = 530, 200, 392
    X, Wg, Wu, Wd = _rand((T, d), dtype, 1.0), _rand((I, d), dtype), _rand((I, d), dtype), _rand((d, I), dtype)
    ws_small = binding.mlp_forward_workspace(binding.mlp_forward_workspace_bytes(T, d, I, dtype)[0], DEV)
    for ws in (None, ws_small):
        binding.mlp_forward(X, Wg, Wu, Wd, binding.ACT_SILU, workspace=ws)
        _clean()


def test_control_a_shortened_range_is_caught_and_skipped(check_lib):
    rows, cols = 72, 344
    W = _rand((rows, cols), torch.bfloat16)
    norm = (torch.rand(cols, device=DEV) * 10 + 0.1).float()
    mask = torch.full((rows, binding.mask_words_per_row(cols)), -1, dtype=torch.int32, device=DEV)
    pruned = torch.full((rows, cols), 7.0, dtype=torch.bfloat16, device=DEV)
    binding.bounds_shrink_next(2048)            # every buffer of the next call is registered 2 KB short
    binding.score_nm(W, norm, AXIS_COLS, 1.0, 3, 4, AXIS_COLS, mask_bits=mask, W_pruned=pruned)
    rep = binding.bounds_report()
    assert rep["violations"] > 0 and rep["first_line"] > 0 and rep["first_bytes"] in (2, 4, 16)
    # the skipped stores never happened: the tails of the outputs still hold their fill values
    assert bool(torch.all(pruned.view(-1)[-512:] == 7.0)) and bool(torch.all(mask.view(-1)[-64:] == -1))
    # the hook applies to one call only
    binding.score_nm(W, norm, AXIS_COLS, 1.0, 3, 4, AXIS_COLS, mask_bits=mask, W_pruned=pruned)
    _clean()
    ref = oracle_stage_b(W, to_np32(norm), AXIS_COLS, 1.0, 3, 4, AXIS_COLS)
    assert np.array_equal(u32(mask), ref["words"]) and np.array_equal(bits_of(pruned), ref["pruned_bits"])
