"""ctypes binding over libdass.so -- argument marshalling only.

Every function here has the name of the C entry point it forwards to (minus the ``dass_`` prefix
where that reads better) and does nothing but check tensor devices/dtypes, allocate requested
outputs with torch, and pass raw pointers, sizes and the current CUDA stream across the C ABI
(``include/dass.h``).  There is no CPU or PyTorch fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdass.so")

OK = 0
BF16, F32 = 0, 1
ACT_SILU, ACT_GELU_TANH, ACT_RELU = 0, 1, 2
AXIS_ROWS, AXIS_COLS = 0, 1
ACT_BY_NAME = {"silu": ACT_SILU, "gelu_tanh": ACT_GELU_TANH, "relu": ACT_RELU}

EXPORTS = (
    "dass_calib_workspace_bytes", "dass_calib_accumulate", "dass_calib_accumulate_static", "dass_calib_status",
    "dass_norm_finalize",
    "dass_score_nm", "dass_compress_nm", "dass_prune_nm", "dass_prune_status", "dass_select_workspace_bytes", "dass_select_unstructured",
    "dass_selftest_wait_timeout", "dass_feature_workspace_bytes", "dass_feature_sumsq",
    "dass_mlp_forward_workspace_bytes", "dass_mlp_forward",
    "dass_bounds_report", "dass_bounds_shrink_next",
    "dass_status_string", "dass_version",
)


class DassError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (dass_status {int(code)})")


_lib = None


def load() -> ctypes.CDLL:
    """Loads libdass.so (built in-tree by ``python -m paper_2405_01943_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2405_01943_b200.build` "
                           "(there is no fallback implementation)")
    _lib = _declare(ctypes.CDLL(LIB_PATH))
    return _lib


class library:
    """Context manager that routes every call of this module through another build of the library (the
    checked-access build, ``libdass_check.so``) and switches back on exit."""

    def __init__(self, path: str):
        self.path = path

    def __enter__(self):
        global _lib
        self._saved = _lib
        _lib = _declare(ctypes.CDLL(self.path))
        return _lib

    def __exit__(self, *exc):
        global _lib
        _lib = self._saved
        return False


def _declare(lib: ctypes.CDLL) -> ctypes.CDLL:
    i64, vp, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t
    lib.dass_calib_workspace_bytes.restype = ctypes.c_int
    lib.dass_calib_workspace_bytes.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.POINTER(sz)]
    lib.dass_calib_accumulate.restype = ctypes.c_int
    lib.dass_calib_accumulate.argtypes = [vp, i64, i64, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int,
                                          vp, vp, sz, vp]
    lib.dass_calib_accumulate_static.restype = ctypes.c_int
    lib.dass_calib_accumulate_static.argtypes = [vp, i64, i64, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int,
                                                 vp, ctypes.POINTER(ctypes.c_void_p), vp]
    lib.dass_calib_status.restype = ctypes.c_int
    lib.dass_calib_status.argtypes = [vp, vp]
    lib.dass_norm_finalize.restype = ctypes.c_int
    lib.dass_norm_finalize.argtypes = [vp, i64, vp, vp]
    lib.dass_score_nm.restype = ctypes.c_int
    lib.dass_score_nm.argtypes = [vp, i64, i64, i64, ctypes.c_int, vp, ctypes.c_int, ctypes.c_float,
                                  ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp]
    lib.dass_compress_nm.restype = ctypes.c_int
    lib.dass_compress_nm.argtypes = [vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                     ctypes.c_int, vp, vp, vp]
    lib.dass_prune_nm.restype = ctypes.c_int
    lib.dass_prune_nm.argtypes = [vp, i64, i64, i64, ctypes.c_int, vp, ctypes.c_int, ctypes.c_float,
                                  ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp]
    lib.dass_prune_status.restype = ctypes.c_int
    lib.dass_prune_status.argtypes = [vp]
    lib.dass_select_workspace_bytes.restype = ctypes.c_int
    lib.dass_select_workspace_bytes.argtypes = [i64, i64, ctypes.c_int, ctypes.POINTER(sz)]
    lib.dass_select_unstructured.restype = ctypes.c_int
    lib.dass_select_unstructured.argtypes = [vp, i64, i64, i64, ctypes.c_int, vp, ctypes.c_int, ctypes.c_float,
                                             ctypes.c_double, ctypes.c_int, vp, vp, vp, sz, vp]
    lib.dass_selftest_wait_timeout.restype = ctypes.c_int
    lib.dass_selftest_wait_timeout.argtypes = [vp, i64, vp]
    lib.dass_feature_workspace_bytes.restype = ctypes.c_int
    lib.dass_feature_workspace_bytes.argtypes = [i64, i64, ctypes.POINTER(sz)]
    lib.dass_feature_sumsq.restype = ctypes.c_int
    lib.dass_feature_sumsq.argtypes = [vp, i64, i64, i64, ctypes.c_int, vp, vp, sz, vp]
    lib.dass_mlp_forward_workspace_bytes.restype = ctypes.c_int
    lib.dass_mlp_forward_workspace_bytes.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.dass_mlp_forward.restype = ctypes.c_int
    lib.dass_mlp_forward.argtypes = [vp, i64, i64, vp, vp, i64, i64, i64, vp, i64, ctypes.c_int, ctypes.c_int,
                                     vp, i64, vp, sz, vp]
    lib.dass_status_string.restype = ctypes.c_char_p
    lib.dass_status_string.argtypes = [ctypes.c_int]
    lib.dass_version.restype = ctypes.c_int
    lib.dass_version.argtypes = []
    lib.dass_bounds_report.restype = ctypes.c_int
    lib.dass_bounds_report.argtypes = [ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_ulonglong),
                                       ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int), vp]
    lib.dass_bounds_shrink_next.restype = ctypes.c_int
    lib.dass_bounds_shrink_next.argtypes = [sz]
    return lib


def status_string(code: int) -> str:
    return load().dass_status_string(int(code)).decode()


def version() -> int:
    return int(load().dass_version())


def _check(code: int, where: str) -> None:
    if code != OK:
        raise DassError(code, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes bfloat16 or float32")


def _matrix(t: torch.Tensor, name: str) -> Tuple[int, int, int]:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name} must be a 2-D row-major tensor (unit stride along columns)")
    return t.shape[0], t.shape[1], t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


# ----------------------------------------------------------------------------- stage (a)

def calib_workspace_bytes(T: int, d: int, I: int, dtype: torch.dtype) -> int:
    out = ctypes.c_size_t(0)
    code = load().dass_calib_workspace_bytes(int(T), int(d), int(I), BF16 if dtype == torch.bfloat16 else F32,
                                             ctypes.byref(out))
    _check(code, "dass_calib_workspace_bytes")
    return int(out.value)


def calib_workspace(T: int, d: int, I: int, dtype: torch.dtype, device="cuda") -> torch.Tensor:
    """A uint8 tensor large (and aligned) enough to serve as workspace of calib_accumulate."""
    n = calib_workspace_bytes(T, d, I, dtype)
    buf = torch.empty(n + 256, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 256
    return buf[off:off + n]


def calib_accumulate(X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, act: int, sumsq: torch.Tensor,
                     workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """sumsq[i] += sum_t (act(X Wg^T) * (X Wu^T))[t, i]^2 on the given (or current) stream."""
    T, d, ldx = _matrix(X, "X")
    I, d2, ldw = _matrix(Wg, "Wg")
    I3, d3, ldw3 = _matrix(Wu, "Wu")
    if (d2, I3, d3, ldw3) != (d, I, d, ldw) or Wg.dtype != X.dtype or Wu.dtype != X.dtype:
        raise ValueError("X [T x d], Wg [I x d], Wu [I x d] must agree in d, I, dtype and row pitch")
    if sumsq.dtype != torch.float64 or not sumsq.is_cuda or sumsq.numel() != I or not sumsq.is_contiguous():
        raise ValueError("sumsq must be a contiguous CUDA float64 tensor of I elements")
    if not workspace.is_cuda or workspace.dtype != torch.uint8:
        raise ValueError("workspace must be a CUDA uint8 tensor (see calib_workspace)")
    code = load().dass_calib_accumulate(X.data_ptr(), T, ldx, Wg.data_ptr(), Wu.data_ptr(), I, d, ldw,
                                        _dtype_code(X), int(act), sumsq.data_ptr(),
                                        workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(code, "dass_calib_accumulate")


STATIC_SCRATCH_BYTES = 16 << 20


def calib_accumulate_static(X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, act: int, sumsq: torch.Tensor,
                            stream: Optional[torch.cuda.Stream] = None) -> int:
    """calib_accumulate for callers that must not allocate: the scratch is a fixed array inside the
    library (at most STATIC_SCRATCH_BYTES, shared by all calls on the device -- do not overlap calls).
    Returns the scratch's device address, which calib_status_at() accepts."""
    T, d, ldx = _matrix(X, "X")
    I, d2, ldw = _matrix(Wg, "Wg")
    I3, d3, ldw3 = _matrix(Wu, "Wu")
    if (d2, I3, d3, ldw3) != (d, I, d, ldw) or Wg.dtype != X.dtype or Wu.dtype != X.dtype:
        raise ValueError("X [T x d], Wg [I x d], Wu [I x d] must agree in d, I, dtype and row pitch")
    if sumsq.dtype != torch.float64 or not sumsq.is_cuda or sumsq.numel() != I or not sumsq.is_contiguous():
        raise ValueError("sumsq must be a contiguous CUDA float64 tensor of I elements")
    addr = ctypes.c_void_p(0)
    code = load().dass_calib_accumulate_static(X.data_ptr(), T, ldx, Wg.data_ptr(), Wu.data_ptr(), I, d, ldw,
                                               _dtype_code(X), int(act), sumsq.data_ptr(), ctypes.byref(addr),
                                               _stream(stream))
    _check(code, "dass_calib_accumulate_static")
    return int(addr.value)


def calib_status_at(address: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """calib_status for a raw device address (the one calib_accumulate_static returned)."""
    _check(load().dass_calib_status(int(address), _stream(stream)), "dass_calib_status")


def calib_status(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Waits for the stream and raises if the last calibration kernel reported a timed-out wait."""
    _check(load().dass_calib_status(workspace.data_ptr(), _stream(stream)), "dass_calib_status")


def norm_finalize(sumsq: torch.Tensor, norm: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """norm = float32(sqrt(sumsq))."""
    if norm is None:
        norm = torch.empty(sumsq.numel(), dtype=torch.float32, device=sumsq.device)
    code = load().dass_norm_finalize(sumsq.data_ptr(), sumsq.numel(), norm.data_ptr(), _stream(stream))
    _check(code, "dass_norm_finalize")
    return norm


# ----------------------------------------------------------------------------- stage (b)

def mask_words_per_row(cols: int) -> int:
    return (cols + 31) // 32


def score_nm(W: torch.Tensor, norm: torch.Tensor, norm_axis: int, alpha: float, n_keep: int, m: int,
             group_axis: int, mask_bits: Optional[torch.Tensor] = None, W_pruned: Optional[torch.Tensor] = None,
             want_mask: bool = True, want_pruned: bool = True,
             stream: Optional[torch.cuda.Stream] = None):
    """Eq. 4 / Eq. 5 score + N:M selection. Returns (mask_bits or None, W_pruned or None)."""
    rows, cols, ld = _matrix(W, "W")
    if norm.dtype != torch.float32 or not norm.is_cuda or not norm.is_contiguous():
        raise ValueError("norm must be a contiguous CUDA float32 tensor")
    if norm.numel() != (rows if norm_axis == AXIS_ROWS else cols):
        raise ValueError("norm has the wrong length for norm_axis")
    if mask_bits is None and want_mask:
        mask_bits = torch.empty((rows, mask_words_per_row(cols)), dtype=torch.int32, device=W.device)
    if W_pruned is None and want_pruned:
        W_pruned = torch.empty_strided((rows, cols), (ld, 1), dtype=W.dtype, device=W.device)
    if W_pruned is not None:
        prow, pcol, pld = _matrix(W_pruned, "W_pruned")
        if (prow, pcol, pld) != (rows, cols, ld) or W_pruned.dtype != W.dtype:
            raise ValueError("W_pruned must have W's shape, dtype and row pitch")
    code = load().dass_score_nm(W.data_ptr(), rows, cols, ld, _dtype_code(W), norm.data_ptr(), int(norm_axis),
                                float(alpha), int(n_keep), int(m), int(group_axis),
                                _ptr(mask_bits), _ptr(W_pruned), _stream(stream))
    _check(code, "dass_score_nm")
    return mask_bits, W_pruned


def compress_shapes(rows: int, cols: int, n_keep: int, m: int, group_axis: int):
    """((value rows, value cols), (meta lines, meta words per line))."""
    bits = 4 if (n_keep == 2 and m == 4) else m
    fpw = 32 // bits
    if group_axis == AXIS_COLS:
        return (rows, cols // m * n_keep), (rows, (cols // m + fpw - 1) // fpw)
    return (rows // m * n_keep, cols), (rows // m, (cols + fpw - 1) // fpw)


def compress_nm(W: torch.Tensor, mask_bits: torch.Tensor, n_keep: int, m: int, group_axis: int,
                values: Optional[torch.Tensor] = None, meta: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None):
    """Compressed values + metadata of W under mask_bits. Returns (values, meta)."""
    rows, cols, ld = _matrix(W, "W")
    vshape, mshape = compress_shapes(rows, cols, n_keep, m, group_axis)
    if values is None:
        values = torch.empty(vshape, dtype=W.dtype, device=W.device)
    if meta is None:
        meta = torch.empty(mshape, dtype=torch.int32, device=W.device)
    if tuple(values.shape) != vshape or not values.is_contiguous() or values.dtype != W.dtype:
        raise ValueError(f"values must be a contiguous {vshape} tensor of W's dtype")
    if tuple(meta.shape) != mshape or not meta.is_contiguous() or meta.dtype != torch.int32:
        raise ValueError(f"meta must be a contiguous int32 {mshape} tensor")
    if mask_bits.dtype != torch.int32 or not mask_bits.is_contiguous() or \
            tuple(mask_bits.shape) != (rows, mask_words_per_row(cols)):
        raise ValueError("mask_bits must be the contiguous int32 [rows x ceil(cols/32)] tensor score_nm produced")
    code = load().dass_compress_nm(W.data_ptr(), mask_bits.data_ptr(), rows, cols, ld, _dtype_code(W),
                                   int(n_keep), int(m), int(group_axis), values.data_ptr(), meta.data_ptr(),
                                   _stream(stream))
    _check(code, "dass_compress_nm")
    return values, meta


def prune_nm(W: torch.Tensor, norm: torch.Tensor, norm_axis: int, alpha: float, n_keep: int, m: int,
             group_axis: int, mask_bits: Optional[torch.Tensor] = None, W_pruned: Optional[torch.Tensor] = None,
             values: Optional[torch.Tensor] = None, meta: Optional[torch.Tensor] = None,
             want_mask: bool = True, want_pruned: bool = True, want_compressed: bool = True,
             stream: Optional[torch.cuda.Stream] = None):
    """score_nm and compress_nm of the same selection in one pass over W.
    Returns (mask_bits or None, W_pruned or None, values or None, meta or None)."""
    rows, cols, ld = _matrix(W, "W")
    if norm.dtype != torch.float32 or not norm.is_cuda or not norm.is_contiguous():
        raise ValueError("norm must be a contiguous CUDA float32 tensor")
    if norm.numel() != (rows if norm_axis == AXIS_ROWS else cols):
        raise ValueError("norm has the wrong length for norm_axis")
    if mask_bits is None and want_mask:
        mask_bits = torch.empty((rows, mask_words_per_row(cols)), dtype=torch.int32, device=W.device)
    if W_pruned is None and want_pruned:
        W_pruned = torch.empty_strided((rows, cols), (ld, 1), dtype=W.dtype, device=W.device)
    if W_pruned is not None:
        prow, pcol, pld = _matrix(W_pruned, "W_pruned")
        if (prow, pcol, pld) != (rows, cols, ld) or W_pruned.dtype != W.dtype:
            raise ValueError("W_pruned must have W's shape, dtype and row pitch")
    if mask_bits is not None and (mask_bits.dtype != torch.int32 or not mask_bits.is_contiguous() or
                                  tuple(mask_bits.shape) != (rows, mask_words_per_row(cols))):
        raise ValueError("mask_bits must be a contiguous int32 [rows x ceil(cols/32)] tensor")
    if want_compressed or values is not None or meta is not None:
        vshape, mshape = compress_shapes(rows, cols, n_keep, m, group_axis)
        if values is None:
            values = torch.empty(vshape, dtype=W.dtype, device=W.device)
        if meta is None:
            meta = torch.empty(mshape, dtype=torch.int32, device=W.device)
        if tuple(values.shape) != vshape or not values.is_contiguous() or values.dtype != W.dtype:
            raise ValueError(f"values must be a contiguous {vshape} tensor of W's dtype")
        if tuple(meta.shape) != mshape or not meta.is_contiguous() or meta.dtype != torch.int32:
            raise ValueError(f"meta must be a contiguous int32 {mshape} tensor")
    code = load().dass_prune_nm(W.data_ptr(), rows, cols, ld, _dtype_code(W), norm.data_ptr(), int(norm_axis),
                                float(alpha), int(n_keep), int(m), int(group_axis),
                                _ptr(mask_bits), _ptr(W_pruned), _ptr(values), _ptr(meta), _stream(stream))
    _check(code, "dass_prune_nm")
    return mask_bits, W_pruned, values, meta


def prune_status(stream: Optional[torch.cuda.Stream] = None) -> None:
    """Waits for the stream and raises if, since the last query, a bounded wait inside a prune_nm or
    select_unstructured kernel ran out or the passes of a select_unstructured call disagreed."""
    _check(load().dass_prune_status(_stream(stream)), "dass_prune_status")


def bounds_report(stream: Optional[torch.cuda.Stream] = None) -> dict:
    """Checked-access build only: accesses outside the registered buffers since the last report (and clears it)."""
    n, addr, nbytes, line = ctypes.c_int(0), ctypes.c_ulonglong(0), ctypes.c_int(0), ctypes.c_int(0)
    _check(load().dass_bounds_report(ctypes.byref(n), ctypes.byref(addr), ctypes.byref(nbytes), ctypes.byref(line),
                                     _stream(stream)), "dass_bounds_report")
    return {"violations": n.value, "first_address": addr.value, "first_bytes": nbytes.value, "first_line": line.value}


def bounds_shrink_next(nbytes: int) -> None:
    """Checked-access build only (test hook): the next call registers every buffer `nbytes` shorter."""
    _check(load().dass_bounds_shrink_next(int(nbytes)), "dass_bounds_shrink_next")


def select_workspace(rows: int, cols: int, norm_axis: int, device="cuda") -> torch.Tensor:
    """A 16-byte aligned uint8 CUDA tensor of the size dass_select_unstructured needs."""
    need = ctypes.c_size_t(0)
    _check(load().dass_select_workspace_bytes(int(rows), int(cols), int(norm_axis), ctypes.byref(need)),
           "dass_select_workspace_bytes")
    buf = torch.empty(need.value + 16, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 16
    return buf[off:off + need.value]


def select_unstructured(W: torch.Tensor, norm: torch.Tensor, norm_axis: int, alpha: float, sparsity: float,
                        compare_axis: int, mask_bits: Optional[torch.Tensor] = None,
                        W_pruned: Optional[torch.Tensor] = None, want_mask: bool = True, want_pruned: bool = True,
                        workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Unstructured selection at `sparsity` inside every column (compare_axis = ROWS) or row (COLS).
    Returns (mask_bits or None, W_pruned or None)."""
    rows, cols, ld = _matrix(W, "W")
    if norm.dtype != torch.float32 or not norm.is_cuda or not norm.is_contiguous():
        raise ValueError("norm must be a contiguous CUDA float32 tensor")
    if norm.numel() != (rows if norm_axis == AXIS_ROWS else cols):
        raise ValueError("norm has the wrong length for norm_axis")
    if mask_bits is None and want_mask:
        mask_bits = torch.empty((rows, mask_words_per_row(cols)), dtype=torch.int32, device=W.device)
    if W_pruned is None and want_pruned:
        W_pruned = torch.empty_strided((rows, cols), (ld, 1), dtype=W.dtype, device=W.device)
    if workspace is None:
        workspace = select_workspace(rows, cols, norm_axis, W.device)
    code = load().dass_select_unstructured(W.data_ptr(), rows, cols, ld, _dtype_code(W), norm.data_ptr(), int(norm_axis),
                                           float(alpha), float(sparsity), int(compare_axis), _ptr(mask_bits),
                                           _ptr(W_pruned), workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(code, "dass_select_unstructured")
    return mask_bits, W_pruned


def selftest_wait_timeout(status_word: torch.Tensor, limit_us: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launches the bounded-wait self-test; read the outcome with calib_status(status_word)."""
    if not status_word.is_cuda or status_word.dtype != torch.int32 or status_word.numel() < 1:
        raise ValueError("status_word must be a CUDA int32 tensor")
    _check(load().dass_selftest_wait_timeout(status_word.data_ptr(), int(limit_us), _stream(stream)),
           "dass_selftest_wait_timeout")


def feature_sumsq(X: torch.Tensor, sumsq: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """sumsq[j] += sum_t X[t,j]^2 (Eq. 1's squared input-feature norms). Returns sumsq (float64 [d])."""
    T, d, ldx = _matrix(X, "X")
    if sumsq is None:
        sumsq = torch.zeros(d, dtype=torch.float64, device=X.device)
    if sumsq.dtype != torch.float64 or not sumsq.is_cuda or sumsq.numel() != d or not sumsq.is_contiguous():
        raise ValueError("sumsq must be a contiguous CUDA float64 tensor of d elements")
    need = ctypes.c_size_t(0)
    _check(load().dass_feature_workspace_bytes(T, d, ctypes.byref(need)), "dass_feature_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need.value + 16, dtype=torch.uint8, device=X.device)
        off = (-workspace.data_ptr()) % 16
        workspace = workspace[off:off + need.value]
    code = load().dass_feature_sumsq(X.data_ptr(), T, d, ldx, _dtype_code(X), sumsq.data_ptr(), workspace.data_ptr(),
                                     workspace.numel(), _stream(stream))
    _check(code, "dass_feature_sumsq")
    return sumsq


# ----------------------------------------------------------------------------- forward pass (Eq. 2, Eq. 3)

def mlp_forward_workspace_bytes(T: int, d: int, I: int, dtype: torch.dtype) -> Tuple[int, int]:
    """(smallest accepted, one-pass) workspace sizes of mlp_forward."""
    lo, full = ctypes.c_size_t(0), ctypes.c_size_t(0)
    code = load().dass_mlp_forward_workspace_bytes(int(T), int(d), int(I), BF16 if dtype == torch.bfloat16 else F32,
                                                   ctypes.byref(lo), ctypes.byref(full))
    _check(code, "dass_mlp_forward_workspace_bytes")
    return int(lo.value), int(full.value)


def mlp_forward_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned uint8 CUDA tensor of nbytes."""
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 256
    return buf[off:off + nbytes]


def mlp_forward(X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor, act: int,
                Z: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Z = (act(X Wg^T) * (X Wu^T)) Wd^T in X's dtype, with the weights as given (pruned = zeros in place).

    Without ``workspace`` a one-pass workspace is allocated; a smaller one makes the call process the
    tokens in chunks.  The workspace's status word is read by calib_status(workspace)."""
    T, d, ldx = _matrix(X, "X")
    I, d2, ldw = _matrix(Wg, "Wg")
    I3, d3, ldw3 = _matrix(Wu, "Wu")
    d4, I4, ldd = _matrix(Wd, "Wd")
    if (d2, I3, d3, ldw3) != (d, I, d, ldw) or (d4, I4) != (d, I):
        raise ValueError("X [T x d], Wg / Wu [I x d] (same pitch) and Wd [d x I] must agree in d and I")
    if not (Wg.dtype == Wu.dtype == Wd.dtype == X.dtype):
        raise ValueError("X, Wg, Wu, Wd must have one dtype")
    if Z is None:
        Z = torch.empty((T, d), dtype=X.dtype, device=X.device)
    Tz, dz, ldz = _matrix(Z, "Z")
    if (Tz, dz) != (T, d) or Z.dtype != X.dtype:
        raise ValueError("Z must be [T x d] in X's dtype")
    if workspace is None:
        workspace = mlp_forward_workspace(mlp_forward_workspace_bytes(T, d, I, X.dtype)[1], X.device)
    if not workspace.is_cuda or workspace.dtype != torch.uint8:
        raise ValueError("workspace must be a CUDA uint8 tensor (see mlp_forward_workspace)")
    code = load().dass_mlp_forward(X.data_ptr(), T, ldx, Wg.data_ptr(), Wu.data_ptr(), I, d, ldw,
                                   Wd.data_ptr(), ldd, _dtype_code(X), int(act), Z.data_ptr(), ldz,
                                   workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(code, "dass_mlp_forward")
    return Z
