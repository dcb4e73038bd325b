"""Glue shared by the GPU parity tests: move tensors between the CUDA library's world (torch, device)
and the oracle's (numpy, float32 views of the same stored values) and compare bit patterns."""
import numpy as np
import torch

import oracle
from paper_2405_01943_b200 import binding


def to_np32(t: torch.Tensor) -> np.ndarray:
    """Stored values widened to float32 exactly (bf16 -> f32 is lossless)."""
    return t.detach().float().cpu().contiguous().numpy()


def bits_of(t: torch.Tensor) -> np.ndarray:
    """Raw element bits as an unsigned numpy array (16-bit for bf16, 32-bit for f32)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.view(torch.int32).numpy().view(np.uint32)


def bits_like(a32: np.ndarray, dtype: torch.dtype) -> np.ndarray:
    """Bits of the float32 array `a32` (holding values representable in dtype) stored as dtype."""
    return bits_of(torch.from_numpy(np.ascontiguousarray(a32)).to(dtype))


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy().view(np.uint32)


def unpack_mask(bits: np.ndarray, cols: int) -> np.ndarray:
    """[rows x words] uint32 -> [rows x cols] uint8."""
    rows = bits.shape[0]
    b = np.unpackbits(bits.view(np.uint8).reshape(rows, -1), axis=1, bitorder="little")
    return b[:, :cols]


def oracle_stage_b(W: torch.Tensor, norm32: np.ndarray, norm_axis, alpha, n_keep, m, group_axis):
    """Oracle mask words, pruned bits, values bits and metadata for a device matrix W."""
    Wn = to_np32(W)
    mask, pruned = oracle.score_nm(Wn, norm32, norm_axis, alpha, n_keep, m, group_axis)
    words = oracle.pack_mask(mask)
    values, meta = oracle.compress_nm(Wn, mask, n_keep, m, group_axis)
    return dict(mask=mask, words=words, pruned_bits=bits_like(pruned, W.dtype),
                values_bits=bits_like(values, W.dtype), meta=meta)


def gpu_stage_b(W: torch.Tensor, norm: torch.Tensor, norm_axis, alpha, n_keep, m, group_axis):
    mask_bits, pruned = binding.score_nm(W, norm, norm_axis, alpha, n_keep, m, group_axis)
    values, meta = binding.compress_nm(W, mask_bits, n_keep, m, group_axis)
    torch.cuda.synchronize()
    rows, cols = W.shape
    return dict(words=u32(mask_bits), pruned_bits=bits_of(pruned[:, :cols]), values_bits=bits_of(values),
                meta=u32(meta))


def assert_stage_b_equal(gpu: dict, ref: dict):
    assert np.array_equal(gpu["words"], ref["words"]), "mask words differ"
    assert np.array_equal(gpu["pruned_bits"], ref["pruned_bits"]), "pruned weights differ"
    assert np.array_equal(gpu["values_bits"], ref["values_bits"]), "compressed values differ"
    assert np.array_equal(gpu["meta"], ref["meta"]), "metadata differs"
