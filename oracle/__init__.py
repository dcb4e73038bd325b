"""DaSS fp64 CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin numpy/ctypes marshalling over ``dass_oracle.c`` (plain C, fp64, written
from the paper's equations).  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library and its
Python binding never do, and nothing here imports them.

Arrays are numpy ``float32`` (bf16 tensors widen to float32 exactly); all
arithmetic inside the C code is fp64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

ACT_SILU, ACT_GELU_TANH, ACT_RELU = 0, 1, 2
AXIS_ROWS, AXIS_COLS = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dass_oracle.c")
_LIB = os.path.join(_HERE, "libdass_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved). Returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                   "-ffp-contract=off", "-fno-fast-math", "-D_GNU_SOURCE",
                   _SRC, "-o", tmp, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, f32p, f64p = ctypes.c_int64, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double)
        u8p, u32p = ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_uint32)
        lib.dass_oracle_act.restype = ctypes.c_double
        lib.dass_oracle_act.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.dass_oracle_calib_sumsq.restype = None
        lib.dass_oracle_calib_sumsq.argtypes = [f32p, i64, i64, f32p, f32p, i64, i64, i64, ctypes.c_int, f64p]
        lib.dass_oracle_feature_sumsq.restype = None
        lib.dass_oracle_feature_sumsq.argtypes = [f32p, i64, i64, i64, f64p]
        lib.dass_oracle_glu_row.restype = None
        lib.dass_oracle_glu_row.argtypes = [f32p, f32p, f32p, i64, i64, i64, ctypes.c_int, f64p]
        lib.dass_oracle_round_bf16.restype = ctypes.c_double
        lib.dass_oracle_round_bf16.argtypes = [ctypes.c_double]
        lib.dass_oracle_mlp_forward.restype = None
        lib.dass_oracle_mlp_forward.argtypes = [f32p, i64, i64, f32p, f32p, i64, i64, i64, f32p, i64,
                                                ctypes.c_int, ctypes.c_int, f64p, f64p]
        lib.dass_oracle_norm.restype = None
        lib.dass_oracle_norm.argtypes = [f64p, i64, f32p]
        lib.dass_oracle_scale.restype = ctypes.c_float
        lib.dass_oracle_scale.argtypes = [ctypes.c_float, ctypes.c_float]
        lib.dass_oracle_score_nm.restype = ctypes.c_int
        lib.dass_oracle_score_nm.argtypes = [f32p, i64, i64, i64, f32p, ctypes.c_int, ctypes.c_float,
                                             ctypes.c_int, ctypes.c_int, ctypes.c_int, u8p, f32p]
        lib.dass_oracle_select_unstructured.restype = ctypes.c_int
        lib.dass_oracle_select_unstructured.argtypes = [f32p, i64, i64, i64, f32p, ctypes.c_int, ctypes.c_float,
                                                        ctypes.c_double, ctypes.c_int, u8p]
        lib.dass_oracle_pack_mask.restype = None
        lib.dass_oracle_pack_mask.argtypes = [u8p, i64, i64, u32p]
        lib.dass_oracle_compress_nm.restype = ctypes.c_int
        lib.dass_oracle_compress_nm.argtypes = [f32p, u8p, i64, i64, i64, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, f32p, u32p]
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the usable cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def act(kind: int, g: float) -> float:
    """sigma of Eq. 2: SiLU, tanh-GeLU or ReLU, in fp64."""
    return float(_load().dass_oracle_act(int(kind), float(g)))


def calib_sumsq(X, Wg, Wu, act_kind: int, sumsq=None) -> np.ndarray:
    """sumsq[i] (+)= sum_t (act(x_t.Wg_i) * (x_t.Wu_i))^2  (Eq. 2, then the squared l2 norm)."""
    X, Wg, Wu = _f32(X), _f32(Wg), _f32(Wu)
    T, d = X.shape
    I, d2 = Wg.shape
    assert d2 == d and Wu.shape == Wg.shape
    if sumsq is None:
        sumsq = np.zeros(I, dtype=np.float64)
    assert sumsq.dtype == np.float64 and sumsq.shape == (I,) and sumsq.flags.c_contiguous
    _load().dass_oracle_calib_sumsq(_p(X, ctypes.c_float), T, d, _p(Wg, ctypes.c_float), _p(Wu, ctypes.c_float),
                                    I, d, d, int(act_kind), _p(sumsq, ctypes.c_double))
    return sumsq


def feature_sumsq(X, sumsq=None) -> np.ndarray:
    """sumsq[j] (+)= sum_t X[t,j]^2: the squared input-feature norms of Eq. 1."""
    X = _f32(X)
    T, d = X.shape
    if sumsq is None:
        sumsq = np.zeros(d, dtype=np.float64)
    assert sumsq.dtype == np.float64 and sumsq.shape == (d,) and sumsq.flags.c_contiguous
    _load().dass_oracle_feature_sumsq(_p(X, ctypes.c_float), T, d, d, _p(sumsq, ctypes.c_double))
    return sumsq


def glu_row(x, Wg, Wu, act_kind: int) -> np.ndarray:
    """H[t,:] of Eq. 2 for one token, fp64."""
    x, Wg, Wu = _f32(x), _f32(Wg), _f32(Wu)
    I, d = Wg.shape
    h = np.zeros(I, dtype=np.float64)
    _load().dass_oracle_glu_row(_p(x, ctypes.c_float), _p(Wg, ctypes.c_float), _p(Wu, ctypes.c_float),
                                I, d, d, int(act_kind), _p(h, ctypes.c_double))
    return h


def round_bf16(v: float) -> float:
    """v rounded to the nearest bf16 value, ties to even."""
    return float(_load().dass_oracle_round_bf16(float(v)))


def mlp_forward(X, Wg, Wu, Wd, act_kind: int, h_round: bool, want_h: bool = False):
    """Eq. 2 then Eq. 3 for every token: z = (act(x Wg^T) * (x Wu^T)) Wd^T.

    ``h_round`` rounds the intermediate activation to bf16 before Eq. 3.  Returns Z [T x d] (fp64), or
    (Z, H) with H [T x I] as Eq. 3 used it."""
    X, Wg, Wu, Wd = _f32(X), _f32(Wg), _f32(Wu), _f32(Wd)
    T, d = X.shape
    I, d2 = Wg.shape
    assert d2 == d and Wu.shape == Wg.shape and Wd.shape == (d, I)
    Z = np.zeros((T, d), dtype=np.float64)
    H = np.zeros((T, I), dtype=np.float64) if want_h else None
    _load().dass_oracle_mlp_forward(_p(X, ctypes.c_float), T, d, _p(Wg, ctypes.c_float), _p(Wu, ctypes.c_float),
                                    I, d, d, _p(Wd, ctypes.c_float), I, int(act_kind), int(bool(h_round)),
                                    _p(Z, ctypes.c_double), _p(H, ctypes.c_double) if want_h else None)
    return (Z, H) if want_h else Z


def norm_from_sumsq(sumsq) -> np.ndarray:
    """norm[i] = float32(sqrt(sumsq[i]))."""
    sumsq = np.ascontiguousarray(sumsq, dtype=np.float64)
    out = np.zeros(sumsq.shape[0], dtype=np.float32)
    _load().dass_oracle_norm(_p(sumsq, ctypes.c_double), sumsq.shape[0], _p(out, ctypes.c_float))
    return out


def scale(norm: float, alpha: float) -> float:
    """float32(norm ** alpha) by the exact recipe (Eq. 4's factor)."""
    return float(_load().dass_oracle_scale(float(np.float32(norm)), float(np.float32(alpha))))


def score_nm(W, norm, norm_axis: int, alpha: float, n_keep: int, m: int, group_axis: int,
             want_pruned: bool = True):
    """Eq. 4 / Eq. 5 score and N:M selection. Returns (mask uint8 [rows x cols], W_pruned or None)."""
    W, norm = _f32(W), _f32(norm)
    rows, cols = W.shape
    assert norm.shape[0] == (rows if norm_axis == AXIS_ROWS else cols)
    mask = np.zeros((rows, cols), dtype=np.uint8)
    pruned = np.zeros((rows, cols), dtype=np.float32) if want_pruned else None
    rc = _load().dass_oracle_score_nm(_p(W, ctypes.c_float), rows, cols, cols, _p(norm, ctypes.c_float),
                                      int(norm_axis), float(alpha), int(n_keep), int(m), int(group_axis),
                                      _p(mask, ctypes.c_uint8),
                                      _p(pruned, ctypes.c_float) if want_pruned else None)
    if rc != 0:
        raise ValueError("oracle score_nm: unsupported shape / n:m")
    return mask, pruned


def select_unstructured(W, norm, norm_axis: int, alpha: float, sparsity: float, compare_axis: int) -> np.ndarray:
    """Unstructured selection: prune the floor(s*size) lowest scores of each comparison line."""
    W, norm = _f32(W), _f32(norm)
    rows, cols = W.shape
    mask = np.zeros((rows, cols), dtype=np.uint8)
    rc = _load().dass_oracle_select_unstructured(_p(W, ctypes.c_float), rows, cols, cols, _p(norm, ctypes.c_float),
                                                 int(norm_axis), float(alpha), float(sparsity), int(compare_axis),
                                                 _p(mask, ctypes.c_uint8))
    if rc != 0:
        raise ValueError("oracle select_unstructured: bad sparsity")
    return mask


def pack_mask(mask) -> np.ndarray:
    """One bit per weight, LSB = lowest column, rows padded to whole uint32 words."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    rows, cols = mask.shape
    bits = np.zeros((rows, (cols + 31) // 32), dtype=np.uint32)
    _load().dass_oracle_pack_mask(_p(mask, ctypes.c_uint8), rows, cols, _p(bits, ctypes.c_uint32))
    return bits


def meta_shape(rows: int, cols: int, n_keep: int, m: int, group_axis: int):
    """(lines, words per line) of the metadata array."""
    bpg = 4 if (n_keep == 2 and m == 4) else m
    fpw = 32 // bpg
    if group_axis == AXIS_COLS:
        return rows, (cols // m + fpw - 1) // fpw
    return rows // m, (cols + fpw - 1) // fpw


def values_shape(rows: int, cols: int, n_keep: int, m: int, group_axis: int):
    if group_axis == AXIS_COLS:
        return rows, cols * n_keep // m
    return rows * n_keep // m, cols


def compress_nm(W, mask, n_keep: int, m: int, group_axis: int):
    """Values (survivors in index order) and per-group metadata. Returns (values f32, meta u32)."""
    W = _f32(W)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    rows, cols = W.shape
    values = np.zeros(values_shape(rows, cols, n_keep, m, group_axis), dtype=np.float32)
    meta = np.zeros(meta_shape(rows, cols, n_keep, m, group_axis), dtype=np.uint32)
    rc = _load().dass_oracle_compress_nm(_p(W, ctypes.c_float), _p(mask, ctypes.c_uint8), rows, cols, cols,
                                         int(n_keep), int(m), int(group_axis),
                                         _p(values, ctypes.c_float), _p(meta, ctypes.c_uint32))
    if rc != 0:
        raise ValueError("oracle compress_nm: mask is not n:m or m does not divide 32")
    return values, meta
