"""Failure detection without faulting the GPU: a bounded device-side wait that nothing ever satisfies must run
out, be reported as DASS_ERR_TIMEOUT through the status word, and leave the context fully usable."""
import time

import pytest
import torch

from paper_2405_01943_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_bounded_wait_runs_out_and_context_survives():
    word = torch.zeros(64, dtype=torch.int32, device=DEV)
    t0 = time.time()
    binding.selftest_wait_timeout(word, 20000)                 # 20 ms
    with pytest.raises(binding.DassError) as err:
        binding.calib_status(word)                             # waits for the stream, then reads the word
    assert err.value.code == 8                                 # DASS_ERR_TIMEOUT
    assert time.time() - t0 < 5.0
    # the context is intact: a real calibration runs and reports OK through the same mechanism
    X = torch.randn((300, 128), device=DEV).to(torch.bfloat16)
    Wg = (torch.randn((264, 128), device=DEV) * 0.02).to(torch.bfloat16)
    Wu = (torch.randn((264, 128), device=DEV) * 0.02).to(torch.bfloat16)
    sumsq = torch.zeros(264, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(300, 128, 264, torch.bfloat16, DEV)
    binding.calib_accumulate(X, Wg, Wu, binding.ACT_SILU, sumsq, ws)
    binding.calib_status(ws)
    assert torch.all(sumsq > 0)


def test_selftest_argument_errors():
    lib = binding.load()
    assert lib.dass_selftest_wait_timeout(None, 10, None) == 1
    assert lib.dass_selftest_wait_timeout(0x10000, 0, None) == 2
    assert lib.dass_selftest_wait_timeout(0x10000, 2000000, None) == 2
    assert lib.dass_selftest_wait_timeout(0x10002, 10, None) == 3
