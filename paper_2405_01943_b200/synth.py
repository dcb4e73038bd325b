"""Seeded synthetic inputs shaped like the paper's MLP layers and calibration set.

This module holds input generation only -- none of the method's arithmetic --
so that both the CUDA library's tests/benchmark and the CPU oracle's tests can
draw the very same tensors from it.

Shapes follow the paper's model-configuration table (LLaMA2-7B/70B, Mistral-7B,
Gemma-7B: hidden / intermediate sizes) and its calibration set of 128 sequences
of 2048 tokens.  Values are stand-ins for trained checkpoints and real text:
Gaussian weights with a few amplified rows (or heavy-tailed entries) so that
intermediate-neuron norms are far from uniform, and Gaussian activations with
a few amplified "outlier" feature channels.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    d: int                 # d_hidden
    I: int                 # d_int
    T: int                 # calibration tokens (sequences x sequence length)
    dtype: str             # "bf16" | "f32"
    act: str               # "silu" | "gelu_tanh"
    n_keep: int
    m: int
    sigma: float           # weight standard deviation
    row_frac: float = 0.0  # fraction of rows of each matrix amplified ...
    row_scale: float = 1.0  # ... by this factor
    t_frac: float = 0.0    # per-entry probability of a Student-t(3) replacement
    outlier_frac: float = 0.0   # fraction of X's feature channels amplified x20 ...
    outlier_count: int = 0      # ... or an absolute count (takes precedence when > 0)
    outlier_scale: float = 20.0
    seed: int = 0
    layers: int = 1
    alphas: Tuple[float, ...] = (0.5,)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


CONFIGS = {
    "tiny": LayerConfig("tiny", d=256, I=688, T=128, dtype="f32", act="silu", n_keep=2, m=4,
                        sigma=0.02, outlier_count=4, seed=0),
    "llama2_7b": LayerConfig("llama2_7b", d=4096, I=11008, T=128 * 2048, dtype="bf16", act="silu",
                             n_keep=2, m=4, sigma=0.02, row_frac=0.005, row_scale=4.0,
                             outlier_frac=0.01, seed=1, layers=32),
    "llama2_13b": LayerConfig("llama2_13b", d=5120, I=13824, T=128 * 2048, dtype="bf16", act="silu",
                              n_keep=2, m=4, sigma=0.02, row_frac=0.005, row_scale=4.0,
                              outlier_frac=0.01, seed=6, layers=40),
    "relullama_7b": LayerConfig("relullama_7b", d=4096, I=11008, T=128 * 2048, dtype="bf16", act="relu",
                                n_keep=2, m=4, sigma=0.02, row_frac=0.005, row_scale=4.0,
                                outlier_frac=0.01, seed=5, layers=32),
    "mistral_7b": LayerConfig("mistral_7b", d=4096, I=14336, T=128 * 2048, dtype="bf16", act="silu",
                              n_keep=4, m=8, sigma=0.02, row_frac=0.005, row_scale=4.0,
                              outlier_frac=0.01, seed=2, layers=32, alphas=(0.0, 0.5, 1.0)),
    "gemma_7b": LayerConfig("gemma_7b", d=3072, I=24576, T=128 * 2048, dtype="bf16", act="gelu_tanh",
                            n_keep=2, m=4, sigma=0.02, outlier_frac=0.01, seed=3, layers=28),
    "llama2_70b": LayerConfig("llama2_70b", d=8192, I=28672, T=128 * 2048, dtype="bf16", act="silu",
                              n_keep=2, m=4, sigma=0.015, t_frac=0.001, outlier_frac=0.01,
                              seed=4, layers=80),
}


def scaled(cfg: LayerConfig, **overrides) -> LayerConfig:
    """Same recipe, other sizes (tests shrink d / I / T to what a CPU check finishes quickly)."""
    return replace(cfg, **overrides)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _n_outliers(cfg: LayerConfig) -> int:
    if cfg.outlier_count > 0:
        return min(cfg.outlier_count, cfg.d)
    return int(math.ceil(cfg.outlier_frac * cfg.d)) if cfg.outlier_frac > 0 else 0


def outlier_channels(cfg: LayerConfig) -> torch.Tensor:
    """Indices of the amplified feature channels of X (seeded choice, CPU tensor)."""
    k = _n_outliers(cfg)
    perm = torch.randperm(cfg.d, generator=_gen("cpu", cfg.seed * 7919 + 17))
    return perm[:k].sort().values


def make_x(cfg: LayerConfig, device="cpu", T: Optional[int] = None, chunk: int = 16384) -> torch.Tensor:
    """Calibration activations X[T x d] ~ N(0,1), outlier channels x20, in cfg's dtype."""
    T = cfg.T if T is None else int(T)
    dev = torch.device(device)
    g = _gen(dev, cfg.seed * 1_000_003 + 1)
    colscale = torch.ones(cfg.d, dtype=torch.float32, device=dev)
    ch = outlier_channels(cfg).to(dev)
    if ch.numel():
        colscale[ch] = cfg.outlier_scale
    out = torch.empty((T, cfg.d), dtype=cfg.torch_dtype, device=dev)
    for t0 in range(0, T, chunk):
        t1 = min(T, t0 + chunk)
        blk = torch.randn((t1 - t0, cfg.d), generator=g, dtype=torch.float32, device=dev)
        blk.mul_(colscale)
        out[t0:t1] = blk.to(cfg.torch_dtype)
    return out


def _make_matrix(cfg: LayerConfig, rows: int, cols: int, g: torch.Generator, dev) -> torch.Tensor:
    w = torch.randn((rows, cols), generator=g, dtype=torch.float32, device=dev)
    w.mul_(cfg.sigma)
    if cfg.t_frac > 0:
        # heavy tail: a Bernoulli(t_frac) subset of entries becomes sigma * t_3,
        # t_3 = Z / sqrt((Z1^2 + Z2^2 + Z3^2) / 3)
        pick = torch.rand((rows, cols), generator=g, dtype=torch.float32, device=dev) < cfg.t_frac
        z = torch.randn((rows, cols), generator=g, dtype=torch.float32, device=dev)
        chi = torch.zeros((rows, cols), dtype=torch.float32, device=dev)
        for _ in range(3):
            chi.add_(torch.randn((rows, cols), generator=g, dtype=torch.float32, device=dev).square_())
        t3 = z / (chi / 3.0).sqrt_()
        w = torch.where(pick, cfg.sigma * t3, w)
        del pick, z, chi, t3
    if cfg.row_frac > 0:
        k = int(math.ceil(cfg.row_frac * rows))
        cpu_g = _gen("cpu", int(g.initial_seed()) + rows)
        idx = torch.randperm(rows, generator=cpu_g)[:k].to(dev)
        w[idx] *= cfg.row_scale
    return w.to(cfg.torch_dtype)


def make_weights(cfg: LayerConfig, device="cpu", layer: int = 0):
    """(Wg [I x d], Wu [I x d], Wd [d x I]) for one layer; layers differ only by seed."""
    dev = torch.device(device)
    base = (cfg.seed * 1_000_003 + 1000 + int(layer)) * 3
    wg = _make_matrix(cfg, cfg.I, cfg.d, _gen(dev, base + 0), dev)
    wu = _make_matrix(cfg, cfg.I, cfg.d, _gen(dev, base + 1), dev)
    wd = _make_matrix(cfg, cfg.d, cfg.I, _gen(dev, base + 2), dev)
    return wg, wu, wd


def checksum(t: torch.Tensor, chunk: int = 1 << 26) -> int:
    """Order-dependent 64-bit checksum of a tensor's raw bytes (for run-to-run comparison):
    sum of byte[i] * (i % 65521 + 1) modulo 2^64, evaluated in chunks so that large tensors need little scratch."""
    raw = t.contiguous().view(-1).view(torch.uint8)
    n = raw.numel()
    total = 0
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        weights = (torch.arange(lo, hi, device=raw.device, dtype=torch.int64) % 65521) + 1
        total = (total + int((raw[lo:hi].to(torch.int64) * weights).sum().item())) & 0xFFFFFFFFFFFFFFFF
    return total
