"""One GLU MLP layer through the DaSS path: the sequence of C-ABI calls a user makes, and nothing else.

    pruner = LayerPruner(T, d, I, dtype, act="silu", n_keep=2, m=4)          # buffers allocated once
    out = pruner.prune(X, Wg, Wu, Wd, alpha=0.5)                               # all work runs in the CUDA library

Section 3 of the paper: the norm of every intermediate neuron over the calibration tokens (Eq. 2, then
"Incorporating Dependency into Weight Importance"), Eq. 4 on gate / up with input-balanced comparison, Eq. 5 on
down with output-balanced comparison, N:M ("Extension to N:M Sparsity") or unstructured ("Pruning Granularity").
"""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as b

_PROJECTIONS = ("gate", "up", "down")


class LayerPruner:
    """Holds the output and scratch buffers of one layer shape, so that pruning a stack of layers allocates once."""

    def __init__(self, T: int, d: int, I: int, dtype: torch.dtype, act: str = "silu", n_keep: int = 2, m: int = 4,
                 device="cuda", compressed: bool = True, overlap_projections: bool = True):
        self.T, self.d, self.I, self.dtype = int(T), int(d), int(I), dtype
        self.act = b.ACT_BY_NAME[act]
        self.n_keep, self.m, self.device = int(n_keep), int(m), torch.device(device)
        self.sumsq = torch.zeros(I, dtype=torch.float64, device=self.device)
        self.norm = torch.empty(I, dtype=torch.float32, device=self.device)
        self.calib_ws = b.calib_workspace(T, d, I, dtype, self.device)
        # (rows, cols, the axis the neuron index runs along = the axis of a comparison line)
        self.geometry = {"gate": (I, d, b.AXIS_ROWS), "up": (I, d, b.AXIS_ROWS), "down": (d, I, b.AXIS_COLS)}
        self.out: Dict[str, Dict[str, torch.Tensor]] = {}
        for name, (rows, cols, axis) in self.geometry.items():
            o = dict(mask=torch.empty((rows, b.mask_words_per_row(cols)), dtype=torch.int32, device=self.device),
                     pruned=torch.empty((rows, cols), dtype=dtype, device=self.device))
            if compressed:
                vshape, mshape = b.compress_shapes(rows, cols, n_keep, m, axis)
                o["values"] = torch.empty(vshape, dtype=dtype, device=self.device)
                o["meta"] = torch.empty(mshape, dtype=torch.int32, device=self.device)
            self.out[name] = o
        self.compressed = compressed
        # The three projections are independent once the norms exist: up and down are launched on two side streams, so
        # that one kernel's last CTAs drain while the next one's first CTAs start (the tail of a 40-200 us launch).
        self._side = [torch.cuda.Stream(device=self.device) for _ in range(2)] if overlap_projections else None
        self._select_ws: Optional[Dict[str, torch.Tensor]] = None
        self._forward_ws: Optional[torch.Tensor] = None

    # ------------------------------------------------------------------ stage (a)
    def reset(self) -> None:
        self.sumsq.zero_()

    def accumulate(self, X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor) -> None:
        """Adds a batch of calibration tokens to the per-neuron sums (any number of calls after reset())."""
        b.calib_accumulate(X, Wg, Wu, self.act, self.sumsq, self.calib_ws)

    def finalize(self) -> torch.Tensor:
        return b.norm_finalize(self.sumsq, self.norm)

    def check(self) -> None:
        """Raises if a bounded device-side wait of the calibration kernel or of a stage-(b) kernel gave up, or the passes
        of an unstructured selection disagreed (synchronises the stream)."""
        b.calib_status(self.calib_ws)
        b.prune_status()

    # ------------------------------------------------------------------ stage (b)
    def score_nm(self, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor, alpha: float = 0.5) -> None:
        for name, W in zip(_PROJECTIONS, (Wg, Wu, Wd)):
            _, _, axis = self.geometry[name]
            o = self.out[name]
            b.score_nm(W, self.norm, axis, alpha if name != "down" else 1.0, self.n_keep, self.m, axis,
                       mask_bits=o["mask"], W_pruned=o["pruned"])

    def prune_nm(self, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor, alpha: float = 0.5) -> None:
        """score_nm and compress_nm in one pass per projection: each weight is read once for all of its outputs."""
        cur = torch.cuda.current_stream(self.device)
        fork = None
        if self._side is not None:
            fork = torch.cuda.Event()
            fork.record(cur)                         # everything the projections read (the norms, the weights) is ordered before it
        for i, (name, W) in enumerate(zip(_PROJECTIONS, (Wg, Wu, Wd))):
            _, _, axis = self.geometry[name]
            o = self.out[name]
            stream = cur if (fork is None or i == 0) else self._side[i - 1]
            if stream is not cur:
                stream.wait_event(fork)
            b.prune_nm(W, self.norm, axis, alpha if name != "down" else 1.0, self.n_keep, self.m, axis,
                       mask_bits=o["mask"], W_pruned=o["pruned"], values=o.get("values"), meta=o.get("meta"),
                       want_compressed=self.compressed, stream=stream)
            if stream is not cur:
                join = torch.cuda.Event()
                join.record(stream)
                cur.wait_event(join)                 # later work on the caller's stream sees all three projections done

    def compress_nm(self, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor) -> None:
        for name, W in zip(_PROJECTIONS, (Wg, Wu, Wd)):
            _, _, axis = self.geometry[name]
            o = self.out[name]
            b.compress_nm(W, o["mask"], self.n_keep, self.m, axis, values=o["values"], meta=o["meta"])

    def select_unstructured(self, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor, sparsity: float,
                            alpha: float = 0.5) -> None:
        if self._select_ws is None:
            self._select_ws = {name: b.select_workspace(rows, cols, axis, self.device)
                               for name, (rows, cols, axis) in self.geometry.items()}
        for name, W in zip(_PROJECTIONS, (Wg, Wu, Wd)):
            _, _, axis = self.geometry[name]
            o = self.out[name]
            b.select_unstructured(W, self.norm, axis, alpha if name != "down" else 1.0, sparsity, axis,
                                  mask_bits=o["mask"], W_pruned=o["pruned"], workspace=self._select_ws[name])

    # ------------------------------------------------------------------ the whole layer
    def prune(self, X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor, alpha: float = 0.5,
              sparsity: Optional[float] = None) -> Dict[str, Dict[str, torch.Tensor]]:
        """Calibrates on X and prunes the three projections: N:M (and the compressed form) by default,
        unstructured at `sparsity` when that is given.  Returns the output buffers (reused by the next call)."""
        self.reset()
        self.accumulate(X, Wg, Wu)
        self.finalize()
        if sparsity is None:
            self.prune_nm(Wg, Wu, Wd, alpha)
        else:
            self.select_unstructured(Wg, Wu, Wd, sparsity, alpha)
        return self.out

    # ------------------------------------------------------------------ the pruned layer's output
    def forward_pruned(self, X: torch.Tensor, Z: Optional[torch.Tensor] = None,
                       workspace_bytes: Optional[int] = None) -> torch.Tensor:
        """Z = (act(X Wg'^T) * (X Wu'^T)) Wd'^T (Eq. 2 then Eq. 3) with the pruned copies the last prune() /
        score_nm() / select_unstructured() wrote, e.g. to feed the next layer's calibration.  `workspace_bytes`
        bounds the scratch that holds the intermediate activations (default: all tokens in one pass)."""
        return self.forward_with(X, self.out["gate"]["pruned"], self.out["up"]["pruned"], self.out["down"]["pruned"],
                                 Z=Z, workspace_bytes=workspace_bytes)

    def forward_with(self, X: torch.Tensor, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor,
                     Z: Optional[torch.Tensor] = None, workspace_bytes: Optional[int] = None) -> torch.Tensor:
        """The layer's output for the weights given (e.g. the dense weights of a layer that is left unpruned)."""
        T = X.shape[0]
        lo, full = b.mlp_forward_workspace_bytes(T, self.d, self.I, self.dtype)
        nbytes = full if workspace_bytes is None else max(lo, min(full, int(workspace_bytes)))
        if self._forward_ws is None or self._forward_ws.numel() != nbytes:
            self._forward_ws = b.mlp_forward_workspace(nbytes, self.device)
        return b.mlp_forward(X, Wg, Wu, Wd, self.act, Z=Z, workspace=self._forward_ws)
