"""Out-of-bounds writes show up as damaged guard bands: every output buffer sits between two sentinel regions that
must come back untouched (ragged shapes, so that partial tiles and tails are exercised)."""
import pytest
import torch

from paper_2405_01943_b200 import binding
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 4096      # elements on each side


def guarded(shape, dtype, fill):
    n = 1
    for s in shape:
        n *= s
    n_al = (n + 63) // 64 * 64
    buf = torch.full((GUARD + n_al + GUARD,), fill, dtype=dtype, device=DEV)
    return buf, buf[GUARD:GUARD + n].view(shape)


def intact(buf, n, fill):
    n_al = (n + 63) // 64 * 64
    return bool(torch.all(buf[:GUARD] == fill)) and bool(torch.all(buf[GUARD + n_al:] == fill))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("group_axis", [AXIS_ROWS, AXIS_COLS])
@pytest.mark.parametrize("n_keep,m", [(2, 4), (4, 8)])
def test_stage_b_outputs_stay_inside_their_buffers(dtype, group_axis, n_keep, m):
    rows, cols = 72, 344                       # not multiples of the 32 x 256 tile
    W = (torch.randn((rows, cols), device=DEV) * 0.02).to(dtype)
    norm = (torch.rand(rows if group_axis == AXIS_ROWS else cols, device=DEV) * 10 + 0.1).float()
    mbuf, mask = guarded((rows, binding.mask_words_per_row(cols)), torch.int32, 0x5A5A5A5A)
    pbuf, pruned = guarded((rows, cols), dtype, 7.0)
    binding.score_nm(W, norm, group_axis, 0.5, n_keep, m, group_axis, mask_bits=mask, W_pruned=pruned)
    vshape, mshape = binding.compress_shapes(rows, cols, n_keep, m, group_axis)
    vbuf, values = guarded(vshape, dtype, 7.0)
    tbuf, meta = guarded(mshape, torch.int32, 0x5A5A5A5A)
    binding.compress_nm(W, mask, n_keep, m, group_axis, values=values, meta=meta)
    ubuf, umask = guarded((rows, binding.mask_words_per_row(cols)), torch.int32, 0x5A5A5A5A)
    qbuf, upruned = guarded((rows, cols), dtype, 7.0)
    binding.select_unstructured(W, norm, group_axis, 0.5, 0.5, group_axis, mask_bits=umask, W_pruned=upruned)
    torch.cuda.synchronize()
    assert intact(mbuf, mask.numel(), 0x5A5A5A5A) and intact(pbuf, pruned.numel(), 7.0)
    assert intact(vbuf, values.numel(), 7.0) and intact(tbuf, meta.numel(), 0x5A5A5A5A)
    assert intact(ubuf, umask.numel(), 0x5A5A5A5A) and intact(qbuf, upruned.numel(), 7.0)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_calibration_outputs_stay_inside_their_buffers(dtype):
    T, d, I = 1030, 200, 392                   # ragged in tokens, k and neurons
    X = torch.randn((T, d), device=DEV).to(dtype)
    Wg = (torch.randn((I, d), device=DEV) * 0.02).to(dtype)
    Wu = (torch.randn((I, d), device=DEV) * 0.02).to(dtype)
    sbuf, sumsq = guarded((I,), torch.float64, -1.0)
    sumsq.zero_()
    nbytes = binding.calib_workspace_bytes(T, d, I, dtype)
    wbuf = torch.full((GUARD + nbytes + GUARD + 256,), 0x5A, dtype=torch.uint8, device=DEV)
    off = GUARD + ((-(wbuf.data_ptr() + GUARD)) % 256)
    ws = wbuf[off:off + nbytes]
    binding.calib_accumulate(X, Wg, Wu, binding.ACT_SILU, sumsq, ws)
    binding.calib_status(ws)
    nbuf, norm = guarded((I,), torch.float32, -1.0)
    binding.norm_finalize(sumsq, norm)
    torch.cuda.synchronize()
    assert intact(sbuf, I, -1.0) and intact(nbuf, I, -1.0)
    assert bool(torch.all(wbuf[:off] == 0x5A)) and bool(torch.all(wbuf[off + nbytes:] == 0x5A))
    assert bool(torch.all(sumsq > 0))
