"""Eq. 1 (Wanda) on the GPU: input-feature norms from dass_feature_sumsq, then N:M per output row through
dass_score_nm -- the route the paper uses for the attention projections."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_stage_b_equal, gpu_stage_b, oracle_stage_b, to_np32
from paper_2405_01943_b200 import binding
from paper_2405_01943_b200.binding import AXIS_COLS

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype,tol", [(torch.bfloat16, 1e-6), (torch.float32, 1e-6)], ids=["bf16", "f32"])
@pytest.mark.parametrize("T,d,ld", [(1, 8, 8), (300, 200, 208), (5000, 1031, 1032), (70000, 520, 520)])
def test_feature_sumsq_matches_oracle(dtype, tol, T, d, ld):
    g = torch.Generator(device=DEV)
    g.manual_seed(T + d)
    base = torch.zeros((T, ld), dtype=dtype, device=DEV)
    base[:, :d] = (torch.randn((T, d), generator=g, device=DEV) * 3).to(dtype)
    X = base[:, :d]
    got = binding.feature_sumsq(X)
    again = binding.feature_sumsq(X)
    half = binding.feature_sumsq(X[: T // 2]) if T > 1 else None
    torch.cuda.synchronize()
    ref = oracle.feature_sumsq(to_np32(X))
    np.testing.assert_allclose(got.cpu().numpy(), ref, rtol=tol)
    assert torch.equal(got, again)                                  # fixed reduction order
    if half is not None:
        binding.feature_sumsq(X[T // 2:], sumsq=half)               # accumulates over batches
        np.testing.assert_allclose(half.cpu().numpy(), ref, rtol=tol)


def test_wanda_nm_on_an_attention_shaped_projection():
    g = torch.Generator(device=DEV)
    g.manual_seed(9)
    X = torch.randn((4096, 1024), generator=g, device=DEV).to(torch.bfloat16)
    X[:, :10] *= 20
    W = (torch.randn((512, 1024), generator=g, device=DEV) * 0.02).to(torch.bfloat16)      # a [out x in] projection
    norm_ref = oracle.norm_from_sumsq(oracle.feature_sumsq(to_np32(X)))
    norm_gpu = binding.norm_finalize(binding.feature_sumsq(X))
    torch.cuda.synchronize()
    np.testing.assert_allclose(norm_gpu.cpu().numpy(), norm_ref, rtol=1e-6)
    norm = torch.from_numpy(norm_ref).to(DEV)
    ref = oracle_stage_b(W, norm_ref, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)
    assert_stage_b_equal(gpu_stage_b(W, norm, AXIS_COLS, 1.0, 2, 4, AXIS_COLS), ref)
