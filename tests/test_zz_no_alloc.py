"""dass_calib_accumulate_static -- the calibration entry point for callers that cannot allocate device
memory (allocator callbacks, memory-planned regions, plugins that own only the tensors they are given,
fixed-budget processes).  It must give what the regular, workspace-taking entry point gives, call after
call, although all its calls share one fixed scratch array that still holds the previous call's data.

Collected last on purpose (file name): a failure here cannot hide the other tests from a -x run."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_01943_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}


def _layer(T, d, I, dtype, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    X = torch.randn((T, d), generator=g, device=DEV)
    X[:, :2] *= 20.0
    Wg = torch.randn((I, d), generator=g, device=DEV) * 0.02
    Wu = torch.randn((I, d), generator=g, device=DEV) * 0.02
    return X.to(dtype), Wg.to(dtype), Wu.to(dtype)


def _regular(X, Wg, Wu, act):
    sumsq = torch.zeros(Wg.shape[0], dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(X.shape[0], X.shape[1], Wg.shape[0], X.dtype, DEV)
    binding.calib_accumulate(X, Wg, Wu, act, sumsq, ws)
    binding.calib_status(ws)
    return sumsq


def _static(X, Wg, Wu, act):
    sumsq = torch.zeros(Wg.shape[0], dtype=torch.float64, device=DEV)
    addr = binding.calib_accumulate_static(X, Wg, Wu, act, sumsq)
    binding.calib_status_at(addr)
    return sumsq


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(dtype):
    # two different problems back to back: the second call finds the first one's partial sums in the scratch
    a = _layer(1500, 192, 520, dtype, seed=11)
    b = _layer(700, 128, 264, dtype, seed=12)
    for (X, Wg, Wu), act, oact in ((a, binding.ACT_SILU, oracle.ACT_SILU), (b, binding.ACT_GELU_TANH, oracle.ACT_GELU_TANH)):
        want = _regular(X, Wg, Wu, act).cpu().numpy()
        got = _static(X, Wg, Wu, act).cpu().numpy()
        rel = np.abs(np.sqrt(got) - np.sqrt(want)) / np.sqrt(want)
        assert rel.max() <= TOL[dtype]
        # and against the fp64 oracle, not only against the library's other entry point
        f32 = lambda t: t.float().cpu().numpy()
        ref = oracle.calib_sumsq(f32(X), f32(Wg), f32(Wu), oact)
        rel = np.abs(np.sqrt(got) - np.sqrt(ref)) / np.sqrt(ref)
        assert rel.max() <= TOL[dtype]
    # and the very same call twice: equal to itself and to the regular path
    X, Wg, Wu = a
    first, second = _static(X, Wg, Wu, binding.ACT_SILU), _static(X, Wg, Wu, binding.ACT_SILU)
    want = _regular(X, Wg, Wu, binding.ACT_SILU)
    for got in (first, second):
        rel = (got.sqrt() - want.sqrt()).abs() / want.sqrt()
        assert float(rel.max()) <= TOL[dtype]


def test_static_scratch_refuses_oversized_problems():
    # 262144 tokens x 65536 neurons would need 64 bands x 65536 x 8 bytes = 32 MiB of partial sums
    T, d, I = 262144, 64, 65536
    assert binding.calib_workspace_bytes(T, d, I, torch.bfloat16) > binding.STATIC_SCRATCH_BYTES
    X = torch.zeros((8, d), dtype=torch.bfloat16, device=DEV)      # never read: the call must refuse first
    sumsq = torch.zeros(I, dtype=torch.float64, device=DEV)
    lib = binding.load()
    code = lib.dass_calib_accumulate_static(X.data_ptr(), T, d, X.data_ptr(), X.data_ptr(), I, d, d,
                                            binding.BF16, binding.ACT_SILU, sumsq.data_ptr(), None, None)
    assert code == 6   # DASS_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.all(sumsq == 0)
