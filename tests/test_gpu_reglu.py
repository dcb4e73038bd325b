"""ReGLU (the ReLU variant of Eq. 2, used by the ReluLLaMA models in the paper): dead neurons -- a gate that never
fires on the calibration set -- get an exactly zero norm, and their weights lose every comparison (Eq. 4, Eq. 5)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_stage_b_equal, gpu_stage_b, oracle_stage_b, to_np32
from paper_2405_01943_b200 import binding, synth
from paper_2405_01943_b200.binding import AXIS_COLS, AXIS_ROWS

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_dead_neurons_have_zero_norm_and_lose_their_weights():
    cfg = synth.scaled(synth.CONFIGS["relullama_7b"], d=256, I=688, T=1500)
    X = synth.make_x(cfg, DEV).abs()                            # non-negative inputs ...
    Wg, Wu, Wd = synth.make_weights(cfg, DEV)
    dead = torch.arange(0, cfg.I, 7, device=DEV)
    Wg[dead] = -Wg[dead].abs()                                  # ... and all-negative gate rows: relu(g) == 0 always
    sumsq = torch.zeros(cfg.I, dtype=torch.float64, device=DEV)
    ws = binding.calib_workspace(cfg.T, cfg.d, cfg.I, X.dtype, DEV)
    binding.calib_accumulate(X, Wg, Wu, binding.ACT_RELU, sumsq, ws)
    binding.calib_status(ws)
    norm = binding.norm_finalize(sumsq)
    torch.cuda.synchronize()
    ref = oracle.calib_sumsq(to_np32(X), to_np32(Wg), to_np32(Wu), oracle.ACT_RELU)
    got = sumsq.cpu().numpy()
    assert np.all(got[dead.cpu().numpy()] == 0.0) and np.all(ref[dead.cpu().numpy()] == 0.0)
    live = ref > 0
    assert np.max(np.abs(np.sqrt(got[live]) - np.sqrt(ref[live])) / np.sqrt(ref[live])) <= 2e-3

    # stage (b) with the oracle's norms (zeros included): bit-exact, and no weight of a dead neuron survives a group
    # in which enough live neurons compete
    norm_ref = oracle.norm_from_sumsq(ref)
    nref = torch.from_numpy(norm_ref).to(DEV)
    for W, na, alpha, ga in ((Wg, AXIS_ROWS, 0.5, AXIS_ROWS), (Wd, AXIS_COLS, 1.0, AXIS_COLS)):
        r = oracle_stage_b(W, norm_ref, na, alpha, 2, 4, ga)
        assert_stage_b_equal(gpu_stage_b(W, nref, na, alpha, 2, 4, ga), r)
    mask_d = oracle.score_nm(to_np32(Wd), norm_ref, AXIS_COLS, 1.0, 2, 4, AXIS_COLS)[0]
    assert mask_d[:, dead.cpu().numpy()].sum() == 0             # every group of 4 holds at most one dead neuron (stride 7)
    assert float(norm.cpu()[dead.cpu()].abs().max()) == 0.0
