"""Host-side checks of the C ABI that need no GPU: the library loads, exports everything the header
declares, and rejects bad arguments with the documented codes before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2405_01943_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dass.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dass_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert "dass_calib_accumulate" in names and "dass_score_nm" in names and "dass_compress_nm" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in dass.h but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings_and_version(lib):
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(c) for c in range(10)}
    assert len(seen) == 10
    assert binding.status_string(1234) == "unknown status"
    assert binding.version() >= 100


def test_workspace_query_validation(lib):
    out = ctypes.c_size_t(0)
    assert lib.dass_calib_workspace_bytes(128, 256, 688, binding.F32, ctypes.byref(out)) == 0
    assert out.value >= 256 + 688 * 8
    assert lib.dass_calib_workspace_bytes(128, 256, 688, binding.F32, None) == 1          # NULL
    assert lib.dass_calib_workspace_bytes(0, 256, 688, binding.F32, ctypes.byref(out)) == 2  # SHAPE
    assert lib.dass_calib_workspace_bytes(128, 256, 688, 7, ctypes.byref(out)) == 4        # DTYPE
    assert lib.dass_calib_workspace_bytes(262144, 8192, 28672, binding.BF16, ctypes.byref(out)) == 0
    assert out.value < (1 << 30)


def test_select_workspace_query(lib):
    """The selection's scratch holds a result per column, the rounded scale vector, the list of rows left to the exact
    kernel and, per column, a counter and the slots of the elements ranked last."""
    out = ctypes.c_size_t(0)
    f = lib.dass_select_workspace_bytes
    assert f(8192, 28672, binding.AXIS_COLS, None) == 1                                   # NULL
    assert f(0, 64, binding.AXIS_COLS, ctypes.byref(out)) == 2                            # SHAPE
    assert f(64, 64, 5, ctypes.byref(out)) == 4                                           # bad axis
    sizes = {}
    for rows, cols, axis in ((8192, 28672, binding.AXIS_COLS), (28672, 8192, binding.AXIS_ROWS), (1, 8, binding.AXIS_ROWS)):
        assert f(rows, cols, axis, ctypes.byref(out)) == 0
        sizes[(rows, cols)] = out.value
        n_norm = rows if axis == binding.AXIS_ROWS else cols
        floor = 24 * cols + 4 * n_norm + 4 * rows + 4 * cols      # results, scale, row list, per-column counters
        assert out.value >= floor
        assert out.value <= floor + 4096 + cols * 3 * 4 * 256     # the ranked slots: a few hundred 12-byte entries per column at most
    assert sizes[(8192, 28672)] > sizes[(28672, 8192)] > sizes[(1, 8)]


def test_calib_workspace_of_short_batches_stays_within_the_static_scratch(lib):
    """The band length of the tensor-core calibration depends on (T, I, d): shorter bands for short batches mean
    more partial sums.  Whatever it picks, a problem that bands of 16 token tiles (256 tokens each) would have kept
    within the fixed scratch of dass_calib_accumulate_static must still fit there, the full-size call keeps bands
    of 16, and no choice needs more partial rows than one per token tile."""
    limit = 16 << 20
    out = ctypes.c_size_t(0)
    for d, I in ((4096, 11008), (5120, 13824), (4096, 14336), (3072, 24576), (8192, 28672), (256, 688), (8192, 57344)):
        for T in (1, 255, 256, 2048, 8192, 16384, 32768, 65536, 98304, 100000, 131072, 262144, 300000):
            assert lib.dass_calib_workspace_bytes(T, d, I, binding.BF16, ctypes.byref(out)) == 0
            token_tiles = -(-T // 256)
            with_16 = 256 + (-(-token_tiles // 16)) * I * 8
            assert with_16 <= out.value <= 256 + token_tiles * I * 8
            if with_16 <= limit:
                assert out.value <= limit, (T, d, I, out.value)
    assert lib.dass_calib_workspace_bytes(262144, 8192, 28672, binding.BF16, ctypes.byref(out)) == 0
    assert out.value == 256 + 64 * 28672 * 8


FAKE = 0x10000  # a 16-byte aligned non-NULL address; validation must fail before it is ever dereferenced


def test_score_nm_argument_errors(lib):
    f = lib.dass_score_nm
    ok_args = dict(W=FAKE, rows=8, cols=64, ld=64, dt=binding.BF16, norm=FAKE, na=1, alpha=1.0, n=2, m=4, ga=1,
                   mask=FAKE, wp=FAKE, st=None)

    def call(**kw):
        a = dict(ok_args, **kw)
        return f(a["W"], a["rows"], a["cols"], a["ld"], a["dt"], a["norm"], a["na"], a["alpha"], a["n"], a["m"],
                 a["ga"], a["mask"], a["wp"], a["st"])

    assert call(W=None) == 1
    assert call(norm=None) == 1
    assert call(mask=None, wp=None) == 1
    assert call(rows=0) == 2
    assert call(cols=62) == 2              # not a multiple of m along the group axis
    assert call(ld=32) == 2                # ld < cols
    assert call(n=4) == 2 and call(n=0) == 2
    assert call(m=16, n=2) == 5            # valid pattern without a kernel
    assert call(m=1, n=0) == 2
    assert call(ld=68) == 3                # bf16 pitch must be a multiple of 8
    assert call(W=FAKE + 2) == 3
    assert call(dt=9) == 4 and call(na=3) == 4 and call(ga=-1) == 4
    assert call(alpha=-0.5) == 5 and call(alpha=float("nan")) == 5 and call(alpha=float("inf")) == 5
    assert call(ga=0, rows=6) == 2         # rows not a multiple of m for row groups


def test_prune_nm_argument_errors(lib):
    f = lib.dass_prune_nm
    ok_args = dict(W=FAKE, rows=8, cols=64, ld=64, dt=binding.BF16, norm=FAKE, na=1, alpha=1.0, n=2, m=4, ga=1,
                   mask=FAKE, wp=FAKE, values=FAKE, meta=FAKE, st=None)

    def call(**kw):
        a = dict(ok_args, **kw)
        return f(a["W"], a["rows"], a["cols"], a["ld"], a["dt"], a["norm"], a["na"], a["alpha"], a["n"], a["m"],
                 a["ga"], a["mask"], a["wp"], a["values"], a["meta"], a["st"])

    assert call(W=None) == 1 and call(norm=None) == 1
    assert call(mask=None, wp=None, values=None, meta=None) == 1      # no output at all
    assert call(values=None) == 1 and call(meta=None) == 1           # the compressed form is both or neither
    assert call(rows=0) == 2 and call(cols=62) == 2 and call(ld=32) == 2
    assert call(n=4) == 2 and call(n=0) == 2 and call(ga=0, rows=6) == 2
    assert call(m=16, n=2) == 5
    assert call(ld=68) == 3 and call(W=FAKE + 2) == 3 and call(wp=FAKE + 4) == 3
    assert call(meta=FAKE + 2) == 3 and call(values=FAKE + 1) == 3 and call(mask=FAKE + 1) == 3
    assert call(dt=9) == 4 and call(na=3) == 4 and call(ga=-1) == 4
    assert call(alpha=-0.5) == 5 and call(alpha=float("nan")) == 5


def test_compress_nm_argument_errors(lib):
    f = lib.dass_compress_nm
    assert f(None, FAKE, 8, 64, 64, 0, 2, 4, 1, FAKE, FAKE, None) == 1
    assert f(FAKE, None, 8, 64, 64, 0, 2, 4, 1, FAKE, FAKE, None) == 1
    assert f(FAKE, FAKE, 8, 64, 64, 0, 2, 4, 1, None, FAKE, None) == 1
    assert f(FAKE, FAKE, 8, 64, 64, 0, 2, 4, 1, FAKE, None, None) == 1
    assert f(FAKE, FAKE, 8, 60, 64, 0, 4, 8, 1, FAKE, FAKE, None) == 2
    assert f(FAKE, FAKE, 8, 64, 60, 0, 2, 4, 1, FAKE, FAKE, None) == 2
    assert f(FAKE, FAKE, 8, 64, 64, 0, 2, 4, 1, FAKE, FAKE + 2, None) == 3


def test_calib_argument_errors(lib):
    f = lib.dass_calib_accumulate
    ok = [FAKE, 128, 256, FAKE, FAKE, 688, 256, 256, binding.F32, 0, FAKE, FAKE, 1 << 20, None]

    def call(idx=None, val=None):
        a = list(ok)
        if idx is not None:
            a[idx] = val
        return f(*a)

    assert call(0, None) == 1 and call(3, None) == 1 and call(4, None) == 1 and call(10, None) == 1
    assert call(1, 0) == 2 and call(5, 0) == 2 and call(6, 0) == 2
    assert call(2, 128) == 2                       # ldx < d
    assert call(2, 258) == 3                       # f32 pitch must be a multiple of 4
    assert call(8, 5) == 4 and call(9, 9) == 4
    assert call(11, None) == 6 and call(12, 16) == 6
    assert call(11, FAKE + 8) == 3                 # workspace not 256-byte aligned
    assert lib.dass_norm_finalize(None, 4, FAKE, None) == 1
    assert lib.dass_norm_finalize(FAKE, 0, FAKE, None) == 2
    assert lib.dass_calib_status(None, None) == 1


def test_binding_refuses_cpu_tensors():
    import torch
    W = torch.zeros((8, 64), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        binding.score_nm(W, torch.ones(64), binding.AXIS_COLS, 1.0, 2, 4, binding.AXIS_COLS)
