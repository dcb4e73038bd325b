"""A stack of GLU MLP layers through the DaSS path, layer by layer, on one GPU.

    stream = LayerStream(pruner, source, n_layers, skip=skip_consecutive(10, 20))
    for res in stream.run(X):
        ...   # res.norm, res.out[...] are valid until the next iteration

The paper prunes whole models layer by layer (its "Pruning speed" table is the total over all MLP layers: 32 for the
7B models, 80 for LLaMA2-70B, model-configuration table in the appendix) and, for its MMLU runs, leaves a quarter of
the layers dense -- 20 consecutive layers of LLaMA2-70B starting at index 10 (appendix, "MMLU Results").  Here the next
layer's weights are brought to the device on a second CUDA stream while the current layer runs through the C-ABI calls,
into one of two device weight sets, and a `skip(layer) -> bool` predicate names the layers that stay dense: they are
still calibrated (their norms are reported, and with `chain=True` their output still feeds the next layer) but nothing
of theirs is pruned.  All arithmetic runs in the CUDA library; this module only sequences calls, copies and events.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Dict, Iterator, Optional, Sequence, Tuple, Union

import torch

from .layer import LayerPruner

Weights = Tuple[torch.Tensor, torch.Tensor, torch.Tensor]          # Wg [I x d], Wu [I x d], Wd [d x I]
Producer = Callable[[int, Weights], None]                           # fills the three device tensors for layer l


def skip_consecutive(start: int, count: int) -> Callable[[int], bool]:
    """Predicate for `count` consecutive dense layers from index `start` (the paper: start 10, a quarter of the layers)."""
    lo, hi = int(start), int(start) + int(count)
    return lambda layer: lo <= int(layer) < hi


@dataclass
class LayerResult:
    layer: int
    skipped: bool
    norm: torch.Tensor                                   # ||y_i||_2 of this layer's intermediate neurons (device)
    weights: Weights                                     # the layer's input weights (device; the stream's buffer)
    out: Optional[Dict[str, Dict[str, torch.Tensor]]]    # LayerPruner outputs, None for a skipped layer
    Z: Optional[torch.Tensor] = None                     # with chain=True: the layer's output on X (pruned unless skipped)


class LayerStream:
    """Prunes `n_layers` layers of one shape with one LayerPruner.

    source: either a sequence of (Wg, Wu, Wd) triples -- CUDA tensors are used where they are, CPU tensors (pinned for
            an asynchronous copy) are uploaded -- or a callable producer(layer, (Wg, Wu, Wd)) that fills the given device
            tensors on the current CUDA stream (e.g. a checkpoint reader or a synthetic generator).
    skip:   layers for which it returns True are calibrated but not pruned.
    chain:  feed each layer's output (Eq. 2 then Eq. 3 with the pruned weights, or the dense ones for a skipped
            layer) to the next layer as its calibration input, instead of reusing X for every layer.
    """

    def __init__(self, pruner: LayerPruner, source: Union[Sequence[Weights], Producer], n_layers: int,
                 skip: Optional[Callable[[int], bool]] = None, alpha: float = 0.5, sparsity: Optional[float] = None,
                 chain: bool = False):
        self.pruner, self.source, self.n = pruner, source, int(n_layers)
        self.skip = skip if skip is not None else (lambda layer: False)
        self.alpha, self.sparsity, self.chain = alpha, sparsity, chain
        self._side = torch.cuda.Stream(device=pruner.device)
        self._bufs = None
        if callable(source) or any(not w.is_cuda for w in source[0]):
            p = pruner
            self._bufs = [tuple(torch.empty(shape, dtype=p.dtype, device=p.device)
                                for shape in ((p.I, p.d), (p.I, p.d), (p.d, p.I))) for _ in range(2)]

    # -- the side stream: bring layer l to the device (slot l % 2) once the slot's previous user is done with it
    def _fetch(self, layer: int, free_event: Optional[torch.cuda.Event]) -> Tuple[Weights, Optional[torch.cuda.Event]]:
        if self._bufs is None:
            return self.source[layer], None                       # already on the device
        dst = self._bufs[layer % 2]
        with torch.cuda.stream(self._side):
            if free_event is not None:
                self._side.wait_event(free_event)
            if callable(self.source):
                self.source(layer, dst)
            else:
                for d, s in zip(dst, self.source[layer]):
                    d.copy_(s, non_blocking=True)
            ready = torch.cuda.Event()
            ready.record(self._side)
        return dst, ready

    def run(self, X: torch.Tensor) -> Iterator[LayerResult]:
        p = self.pruner
        comp = torch.cuda.current_stream(p.device)
        self._side.wait_stream(comp)
        free = [None, None]                                        # recorded when a slot's layer has been worked through
        nxt = self._fetch(0, None) if self.n > 0 else None
        Xl = X
        for layer in range(self.n):
            weights, ready = nxt
            if layer >= 1:
                # whatever the caller enqueued on the compute stream for the previous layer is covered by this event
                free[(layer - 1) % 2] = torch.cuda.Event()
                free[(layer - 1) % 2].record(comp)
            if layer + 1 < self.n:
                nxt = self._fetch(layer + 1, free[(layer + 1) % 2])
            if ready is not None:
                comp.wait_event(ready)
            Wg, Wu, Wd = weights
            skipped = bool(self.skip(layer))
            p.reset()
            p.accumulate(Xl, Wg, Wu)
            p.finalize()
            if not skipped:
                if self.sparsity is None:
                    p.prune_nm(Wg, Wu, Wd, self.alpha)
                else:
                    p.select_unstructured(Wg, Wu, Wd, self.sparsity, self.alpha)
            Z = None
            if self.chain:
                Z = p.forward_with(Xl, Wg, Wu, Wd) if skipped else p.forward_pruned(Xl)
            yield LayerResult(layer, skipped, p.norm, weights, None if skipped else p.out, Z)
            if self.chain:
                Xl = Z
        comp.wait_stream(self._side)
