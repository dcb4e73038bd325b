#!/usr/bin/env python
"""Throughput of the DaSS hot path on B200: one step = one MLP layer through the whole path
(fused GLU calibration norms -> norm finalize -> one-pass N:M scoring + selection + compression of
gate / up / down) on synthetic inputs shaped like the paper's models and its 128 x 2048-token calibration set.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config llama2_70b] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample of
the same workload instead.  `--gpus N` means N ranks: started under torch.distributed.run the script checks that
WORLD_SIZE is N, started plainly with N > 1 it launches the N ranks itself.  Every rank prunes its own independent
layers -- the path has no cross-GPU exchange -- and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_01943_b200 import synth  # noqa: E402

METRIC = "calib tokens/s (fused GLU-norm pass + N:M scoring + compression, per layer step)"
UNIT = "tokens/s"
KERNEL_LAUNCHES_PER_STEP = 7    # status clear, calib GEMM, partial reduce, finalize, 3 x one-pass prune
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}     # data-sheet figures (HBM3e, dense bf16), for context
PER_CONFIG = ("tiny", "llama2_7b", "mistral_7b", "gemma_7b")   # reported beside the headline shape


# --------------------------------------------------------------------------- small helpers

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def stage_b_bytes(cfg, compress=True):
    """Algorithmic bytes of stage (b) for the three projections of one layer: (score pass, compress pass, one pass)."""
    esz = 2 if cfg.dtype == "bf16" else 4
    elems = 3 * cfg.d * cfg.I
    score = elems * (esz + esz + 0.125)                                   # read W, write pruned + mask bit
    frac = cfg.n_keep / cfg.m
    meta_bits = 4 / 4 if (cfg.n_keep == 2 and cfg.m == 4) else 1.0        # field bits per weight
    comp = elems * (esz + 0.125 + esz * frac + meta_bits / 8.0) if compress else 0.0
    fused = elems * (esz + esz + 0.125 + esz * frac + meta_bits / 8.0)    # one read of W for all four outputs
    return score, comp, fused


def _git_blob_sha(path):
    """The id git gives the file's content: ties a stored counter to the kernel source it was captured from."""
    try:
        data = open(os.path.join(ROOT, path), "rb").read()
    except OSError:
        return None
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch, from ncu captures summarised under profiles/.
# Each entry names its summary and the git blob ids of the kernel sources it was captured from; when a source has
# changed since, the number is withheld (reported as null) instead of going stale.
NCU_DRAM_BYTES = {
    "llama2_70b": {
        "calib": {"bytes": 4 * (29.607549696e9 + 15.025152e6), "profile": "profiles/calib_tc2_kernel_llama2_70b_T65536_dram.md",
                  "sources": {"paper_2405_01943_b200/csrc/calib_tc2.cu": "729748d82f305308578b4f36418f5fcceedbd567"},
                  "how": "one launch at T = 65536 (one group of 16 interleaved bands) x 4: the full launch repeats that group four times"},
        "prune": {"bytes": (1176.3 + 1176.6 + 1178.0) * 1e6, "profile": "profiles/prune_bf16_kernels_llama2_70b_matrices.md",
                  "sources": {"paper_2405_01943_b200/csrc/prune_nm_bf16.cu": "589f5434a8fb3dc0205c8543aba82e894d24f928",
                              "paper_2405_01943_b200/csrc/stream_units.cuh": "09bbd579b7cb40f0fd99356d6d5c9bcdee68fc45"},
                  "how": "the three launches of one step (gate, up, down) on the full-size matrices"},
    },
}


def ncu_traffic(cfg_name, key):
    rec = NCU_DRAM_BYTES.get(cfg_name, {}).get(key)
    if rec is None:
        return None, None
    changed = [src for src, blob in rec["sources"].items() if _git_blob_sha(src) != blob]
    if changed:
        return None, {"withheld": f"{', '.join(changed)} changed since {rec['profile']} was captured"}
    return rec["bytes"], {"profile": rec["profile"], "sources": rec["sources"], "how": rec["how"]}


def roofline_b(kernel, algorithmic_bytes, in_step_ms, isolated_ms, peaks, peak_src, traffic, provenance):
    """HBM roofline entry of the stage-(b) launches of one step (three matrices).  The headline fraction is the one
    measured where the kernels run, inside the step right after the power-capped GEMM; the same launches timed
    alone are reported beside it."""
    gbs = algorithmic_bytes / (in_step_ms * 1e-3) / 1e9
    out = {"bound": "hbm", "kernel": kernel, "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
           "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal": gbs / NOMINAL["hbm_gbs"], "peak_source": peak_src,
           "timed": "inside the step", "ms": in_step_ms,
           "algorithmic_bytes_per_step": algorithmic_bytes, "traffic": traffic, "traffic_provenance": provenance}
    if isolated_ms:
        alone = algorithmic_bytes / (isolated_ms * 1e-3) / 1e9
        out.update({"alone_gbs": alone, "alone_frac": alone / peaks["hbm_gbs"], "alone_ms": isolated_ms,
                    "alone_timed": "the same launches back to back after the step loop"})
    return out


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(mhz)}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def max_over_ranks(value: float, world: int, device) -> float:
    """Max of a per-rank scalar (the slowest rank defines the step time)."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def layer_ids_for_rank(rank: int, world: int, steps: int, warmup: int):
    """Independent layers handed to a rank: each rank prunes its own layers, nothing is exchanged."""
    per_rank = steps + warmup
    return [rank * per_rank + i for i in range(per_rank)]


def aggregate_value(tokens_per_step: int, steps: int, world: int, seconds_max: float) -> float:
    return tokens_per_step * steps * world / seconds_max


# --------------------------------------------------------------------------- the GPU arm

class LayerPath:
    """One step = the library's public per-layer API (paper_2405_01943_b200.layer.LayerPruner: device buffers
    and the sequence of C-ABI calls), with CUDA events between the stages."""

    def __init__(self, cfg, device, binding):
        from paper_2405_01943_b200.layer import LayerPruner
        self.cfg, self.dev, self.b = cfg, device, binding
        self.pruner = LayerPruner(cfg.T, cfg.d, cfg.I, cfg.torch_dtype, act=cfg.act, n_keep=cfg.n_keep, m=cfg.m,
                                  device=device)
        self.act = self.pruner.act
        self.sumsq, self.norm, self.ws, self.out = self.pruner.sumsq, self.pruner.norm, self.pruner.calib_ws, self.pruner.out
        self.ev = {k: [] for k in ("calib", "prune")}

    def step(self, X, Wg, Wu, Wd, alpha, record=False, before_stage_b=None, x_chunks=None):
        """x_chunks: [(first token, last token + 1, event or None)]: the calibration is then accumulated chunk by
        chunk (the sums carry over between calls), each call waiting for its chunk's event on the current stream."""
        pr = self.pruner
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)] if record else None
        pr.reset()
        if record:
            e[0].record()
        if x_chunks is None:
            pr.accumulate(X, Wg, Wu)
        else:
            for t0, t1, ready in x_chunks:
                if ready is not None:
                    torch.cuda.current_stream().wait_event(ready)
                pr.accumulate(X[t0:t1], Wg, Wu)
        if record:
            e[1].record()
        if before_stage_b is not None:
            before_stage_b()
        pr.finalize()
        pr.prune_nm(Wg, Wu, Wd, alpha)
        if record:
            e[2].record()
            self.ev["calib"].append((e[0], e[1]))
            self.ev["prune"].append((e[1], e[2]))

    def mean_ms(self, key):
        v = [a.elapsed_time(b) for a, b in self.ev[key]]
        return sum(v) / len(v) if v else None

    def check(self):
        self.b.calib_status(self.ws)
        self.b.prune_status()


class PinnedArena:
    """One pinned host allocation carved into tensors, so that the end-to-end legs of several shapes pay for page
    locking once."""

    def __init__(self, nbytes):
        self.buf = torch.empty(int(nbytes), dtype=torch.uint8, pin_memory=True)
        self.off = 0

    def reset(self):
        self.off = 0

    def take(self, like):
        n = like.numel() * like.element_size()
        start = (self.off + 255) // 256 * 256
        if start + n > self.buf.numel():
            raise RuntimeError("pinned arena too small")
        self.off = start + n
        return self.buf[start:start + n].view(like.dtype).view(like.shape)


def e2e_bytes(cfg):
    esz = 2 if cfg.dtype == "bf16" else 4
    up = (cfg.T * cfg.d + 3 * cfg.d * cfg.I) * esz
    down = cfg.I * 4 + 3 * cfg.d * cfg.I * (0.125 + esz * cfg.n_keep / cfg.m + 0.125) + 4096
    return int(up + down) + (1 << 20)


def timed_steps(path, X, pool, alpha, steps, warmup, world, device, rank, local_rank):
    """W untimed steps, then K timed ones between barriers; the clock of this GPU is sampled meanwhile."""
    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        path.step(X, *pool[i % len(pool)], alpha)
    path.check()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(steps):
        path.step(X, *pool[(warmup + i) % len(pool)], alpha, record=True)
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    path.check()
    seconds = max_over_ranks(t0.elapsed_time(t1) / 1e3, world, device)
    return seconds, clocks


def calib_roofline(cfg, calib_ms, peaks, peak_src, traffic, provenance):
    flops = 4.0 * cfg.T * cfg.d * cfg.I
    tf = flops / (calib_ms * 1e-3) / 1e12
    out = {"bound": "tensor", "kernel": "calib_tc2_kernel", "achieved": tf, "peak": peaks["bf16_tflops_sustained"],
           "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops_sustained"], "frac_of_burst_peak": tf / peaks["bf16_tflops"],
           "frac_of_nominal": tf / NOMINAL["bf16_tflops"], "peak_source": peak_src,
           "peak_note": "frac is against the cuBLAS bf16 rate this pool sustains under its power cap (the kernel runs "
                        "inside a seconds-long step); burst and data-sheet fractions beside it",
           "algorithmic_flops_per_launch": flops, "traffic": traffic, "traffic_provenance": provenance}
    if cfg.dtype != "bf16":
        out.update({"bound": "alu", "kernel": "calib_simt_kernel", "peak": None, "frac": None, "frac_of_burst_peak": None,
                    "frac_of_nominal": None, "peak_note": "fp32 FMA correctness path of the tiny configuration; no roofline claim"})
    return out


def run_ours(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the DaSS path has no CPU fallback (use --impl reference for the oracle)")
    from paper_2405_01943_b200 import binding, build
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    if os.environ.get("DASS_NO_BUILD") != "1" and local_rank == 0 and build.is_stale():
        build.build()                    # one rank per node builds; the others wait at the barrier below
    if world > 1:
        dist.barrier()
    binding.load()

    cfg = synth.CONFIGS[args.config]
    if args.tokens:
        cfg = synth.scaled(cfg, T=args.tokens)
    alpha = 0.5
    peaks, peak_src = load_peaks()
    extra = [n for n in PER_CONFIG if n != args.config] if (args.per_config and not args.tokens) else []
    arena = None
    if args.e2e_steps > 0:
        arena = PinnedArena(max(e2e_bytes(c) for c in [cfg] + [synth.CONFIGS[n] for n in extra]))

    X = synth.make_x(cfg, device)
    pool = [synth.make_weights(cfg, device, layer=l) for l in layer_ids_for_rank(rank, world, args.pool, 0)]
    path = LayerPath(cfg, device, binding)
    seconds, clocks = timed_steps(path, X, pool, alpha, args.steps, args.warmup, world, device, rank, local_rank)
    value = aggregate_value(cfg.T, args.steps, world, seconds)

    # per-kernel durations measured live inside the timed region
    calib_ms, prune_ms = path.mean_ms("calib"), path.mean_ms("prune")
    sb, cb, fb = stage_b_bytes(cfg)

    # stage (b) alone: the same launches back to back, away from the power-capped GEMM
    iso = isolated_stage_b(path, pool, alpha, iters=args.iso_iters) if args.iso_iters > 0 else None
    unstructured = unstructured_leg(path, pool, alpha, args.unstructured_iters, peaks) if args.unstructured_iters > 0 else None
    forward = None
    if args.forward_iters > 0 and cfg.dtype == "bf16":
        forward = forward_leg(path, X, pool[0], args.forward_tokens, args.forward_iters, peaks)

    # end to end: pinned host inputs -> device -> path -> results back to the host, every step
    e2e = run_e2e(cfg, path, X, pool[0], alpha, args.e2e_steps, world, device, arena) if args.e2e_steps > 0 else None

    # the whole stack of layers through the layer stream: distinct weights per layer, produced on a second stream
    stream = None
    n_stream = args.stream_layers if args.stream_layers >= 0 else (cfg.layers if not args.tokens else 0)
    if n_stream > 0:
        stream = stream_leg(cfg, path, X, alpha, n_stream, rank, world, device)

    out = None
    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = cpu_baseline(cfg, X, pool[0], budget_s=args.cpu_seconds)
        checks = {n: synth.checksum(t) for n, t in zip(("X", "Wg", "Wu", "Wd"), (X,) + tuple(pool[0]))}
    del X, pool, path
    torch.cuda.empty_cache()

    per_config = []
    for name in extra:
        entry = config_entry(name, args, alpha, peaks, peak_src, world, device, rank, local_rank, binding, arena)
        if rank == 0:
            per_config.append(entry)

    if rank == 0:
        t_calib, prov_calib = (None, None) if args.tokens else ncu_traffic(cfg.name, "calib")
        t_prune, prov_prune = ncu_traffic(cfg.name, "prune")
        headline = {"config": cfg.name, "n_m": f"{cfg.n_keep}:{cfg.m}", "ms_per_step": seconds * 1e3 / args.steps,
                    "tokens_per_s": value, "calib_ms": calib_ms, "prune_ms": prune_ms,
                    "calib_tflops": 4.0 * cfg.T * cfg.d * cfg.I / (calib_ms * 1e-3) / 1e12,
                    "calib_frac_sustained": 4.0 * cfg.T * cfg.d * cfg.I / (calib_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                    "calib_frac_burst": 4.0 * cfg.T * cfg.d * cfg.I / (calib_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "prune_in_step_frac": fb / (prune_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "prune_alone_frac": (fb / (iso["prune"] * 1e-3) / 1e9 / peaks["hbm_gbs"]) if iso else None,
                    "e2e_tokens_per_s": e2e["value"] if e2e else None, "clocks": clocks}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": seconds * 1e3 / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": f"{cfg.name}-shaped {cfg.act} layer, d={cfg.d}, I={cfg.I}, T={cfg.T} calibration tokens, "
                                   f"{cfg.n_keep}:{cfg.m} on gate/up (Eq. 4, alpha={alpha}, input-balanced) and down (Eq. 5); "
                                   "mask + pruned weights + compressed values/metadata",
                       "layers_per_rank": args.steps, "weight_sets_cycled": args.pool, "input_checksums": checks,
                       "l2": "inputs exceed L2 (X and each weight set are far larger than 126 MB); no flush",
                       "parallelism": "independent layers per GPU, no collective" if world > 1 else "single GPU"},
            "stage_ms": {"calib": calib_ms, "prune_x3": prune_ms},
            "score_gbs": fb / (prune_ms * 1e-3) / 1e9,
            "roofline": calib_roofline(cfg, calib_ms, peaks, peak_src, t_calib, prov_calib),
            "roofline_prune": roofline_b("prune_rows_bf16_kernel x2 (gate, up) + prune_cols_bf16_kernel (down): score, N:M "
                                         "selection, mask, pruned copy, values and metadata from one read of W",
                                         fb, prune_ms, iso and iso["prune"], peaks, peak_src, t_prune, prov_prune),
            "two_pass_alone": None if not iso else {
                "note": "dass_score_nm then dass_compress_nm on the same matrices, timed alone: what the one-pass call replaces",
                "score_ms": iso["score"], "compress_ms": iso["compress"],
                "score_gbs": sb / (iso["score"] * 1e-3) / 1e9, "compress_gbs": cb / (iso["compress"] * 1e-3) / 1e9},
            "unstructured": unstructured, "forward": forward, "stream": stream,
            "per_config": [headline] + per_config,
            "e2e": e2e, "gpu_launches": KERNEL_LAUNCHES_PER_STEP * args.steps, "clocks": clocks,
            "cpu_baseline": cpu,
        }
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    return out


def config_entry(name, args, alpha, peaks, peak_src, world, device, rank, local_rank, binding, arena):
    """The same step on another of the paper's shapes: its own inputs, its own timed loop (long enough for the clock
    sampler to see it), its own stage-(b)-alone and end-to-end timings."""
    cfg = synth.CONFIGS[name]
    X = synth.make_x(cfg, device)
    pool = [synth.make_weights(cfg, device, layer=l) for l in layer_ids_for_rank(rank, world, 2, 0)]
    path = LayerPath(cfg, device, binding)
    for i in range(2):
        path.step(X, *pool[i % 2], alpha)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    path.step(X, *pool[0], alpha)
    b.record()
    torch.cuda.synchronize()
    est_ms = max(a.elapsed_time(b), 0.02)
    steps = int(min(20000, max(4, math.ceil(args.per_config_seconds * 1e3 / est_ms))))
    seconds, clocks = timed_steps(path, X, pool, alpha, steps, 3, world, device, rank, local_rank)
    calib_ms, prune_ms = path.mean_ms("calib"), path.mean_ms("prune")
    _, _, fb = stage_b_bytes(cfg)
    iso = isolated_stage_b(path, pool, alpha, iters=20, two_pass=False)
    e2e = None
    if args.e2e_steps > 0:
        e2e = run_e2e(cfg, path, X, pool[0], alpha, max(3, min(args.e2e_steps, 6)), world, device, arena)
    flops = 4.0 * cfg.T * cfg.d * cfg.I
    tf = flops / (calib_ms * 1e-3) / 1e12
    bf16 = cfg.dtype == "bf16"
    entry = {"config": cfg.name, "n_m": f"{cfg.n_keep}:{cfg.m}", "dtype": cfg.dtype, "steps": steps,
             "ms_per_step": seconds * 1e3 / steps, "tokens_per_s": aggregate_value(cfg.T, steps, world, seconds),
             "calib_ms": calib_ms, "prune_ms": prune_ms, "calib_tflops": tf,
             "calib_frac_sustained": tf / peaks["bf16_tflops_sustained"] if bf16 else None,
             "calib_frac_burst": tf / peaks["bf16_tflops"] if bf16 else None,
             "prune_in_step_frac": fb / (prune_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
             "prune_alone_frac": fb / (iso["prune"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
             "e2e_tokens_per_s": e2e["value"] if e2e else None,
             "e2e_bytes_per_step": (e2e["h2d_bytes_per_step"], e2e["d2h_bytes_per_step"]) if e2e else None,
             "clocks": clocks}
    if not bf16:
        entry["note"] = "fp32 correctness configuration: a step is a handful of launch-bound kernels, no roofline claim"
    del X, pool, path
    torch.cuda.empty_cache()
    return entry


def isolated_stage_b(path, pool, alpha, iters, two_pass=True):
    """Mean ms of the three one-pass launches (and, for context, of the two-pass route), timed alone."""
    legs = [("prune", lambda ws: path.pruner.prune_nm(*ws, alpha))]
    if two_pass:
        legs += [("score", lambda ws: path.pruner.score_nm(*ws, alpha)), ("compress", lambda ws: path.pruner.compress_nm(*ws))]
    out = {}
    time.sleep(0.5)                      # let the clocks recover from the power-capped GEMM
    for key, fn in legs:
        for i in range(3):
            fn(pool[i % len(pool)])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(pool[i % len(pool)])
        e1.record()
        torch.cuda.synchronize()
        out[key] = e0.elapsed_time(e1) / iters
    return out


def unstructured_leg(path, pool, alpha, iters, peaks, sparsity=0.5):
    """The paper's unstructured setting on the same three matrices, timed alone: per input column of gate / up
    (input-balanced) and per output row of down (output-balanced) the floor(s * L) lowest scores are pruned."""
    cfg = path.cfg

    def timed(a):
        for i in range(3):
            path.pruner.select_unstructured(*pool[i % len(pool)], sparsity, a)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            path.pruner.select_unstructured(*pool[i % len(pool)], sparsity, a)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    ms = timed(alpha)
    ms_a0 = timed(0.0)                   # alpha = 0: equal rounded products everywhere, the selection's worst case
    nbytes, _, _ = stage_b_bytes(cfg, compress=False)
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"sparsity": sparsity, "ms_x3": ms, "achieved": gbs, "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
            "frac_of_nominal": gbs / NOMINAL["hbm_gbs"],
            "alpha0_ms_x3": ms_a0, "alpha0_frac": nbytes / (ms_a0 * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "kernels": "select_cols_kernel + select_emit_stream_kernel + select_fix_cols_kernel (gate, up), "
                       "select_rows_stream_kernel + select_rows_kernel for the rows it leaves (down)",
            "algorithmic_bytes_per_step": nbytes, "timed": "alone, back to back, after the step loop"}


def forward_leg(path, X, weights, tokens, iters, peaks):
    """Forward pass of the layer (Eq. 2 then Eq. 3) with the weights as they are, on a prefix of the calibration
    tokens, timed alone: two tensor-core launches (GLU projection writing H in bf16, down projection)."""
    b, cfg = path.b, path.cfg
    n = min(tokens, cfg.T)
    Xs = X[:n]
    Wg, Wu, Wd = weights
    ws = b.mlp_forward_workspace(b.mlp_forward_workspace_bytes(n, cfg.d, cfg.I, Xs.dtype)[1], path.dev)
    Z = torch.empty((n, cfg.d), dtype=Xs.dtype, device=path.dev)
    for _ in range(2):
        b.mlp_forward(Xs, Wg, Wu, Wd, path.act, Z=Z, workspace=ws)
    b.calib_status(ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        b.mlp_forward(Xs, Wg, Wu, Wd, path.act, Z=Z, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    b.calib_status(ws)
    ms = e0.elapsed_time(e1) / iters
    flops = 6.0 * n * cfg.d * cfg.I
    tf = flops / (ms * 1e-3) / 1e12
    return {"tokens": n, "ms": ms, "tokens_per_s": n / (ms * 1e-3), "achieved": tf, "unit": "TFLOP/s",
            "frac": tf / peaks["bf16_tflops_sustained"], "frac_of_burst_peak": tf / peaks["bf16_tflops"],
            "frac_of_nominal": tf / NOMINAL["bf16_tflops"],
            "kernels": "mlp_forward_tc_kernel<GLU> + mlp_forward_tc_kernel<PLAIN>",
            "algorithmic_flops": flops, "timed": "alone, back to back, after the step loop"}


def stream_leg(cfg, path, X, alpha, n_layers, rank, world, device):
    """All MLP layers of the model, one after another, through paper_2405_01943_b200.stream.LayerStream: every layer
    has its own weights, produced on a second CUDA stream into the other of two device weight sets while the current
    layer runs (X is reused: feeding a layer the previous layer's output needs the attention blocks in between)."""
    from paper_2405_01943_b200.stream import LayerStream
    first = rank * n_layers                                # every rank streams its own layers

    def produce(layer, dst):
        for d_, s_ in zip(dst, synth.make_weights(cfg, device, layer=first + layer)):
            d_.copy_(s_)

    stream = LayerStream(path.pruner, produce, n_layers, alpha=alpha)
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in stream.run(X):
        pass
    b.record()
    torch.cuda.synchronize()
    path.check()
    seconds = max_over_ranks(a.elapsed_time(b) / 1e3, world, device)
    return {"layers": n_layers, "seconds": seconds, "ms_per_layer": seconds * 1e3 / n_layers,
            "tokens_per_s": aggregate_value(cfg.T, n_layers, world, seconds),
            "weights": "a distinct synthetic layer per index (seeded), generated on a second stream into two device "
                       "weight sets while the previous layer runs; generation is inside the timed region",
            "paper_context": "the paper's pruning pass alone took 20.70 s for LLaMA2-70B's 80 MLP layers on 8 A100 "
                             "(table 'Pruning speed'; its calibration forward is not included)"}


def run_e2e(cfg, path, X, weights, alpha, steps, world, device, arena):
    """Same step driven from pinned host memory: every step's inputs (X and the three weight matrices) are
    copied host -> device and its results (norms, masks, values, metadata) device -> host, all inside the
    timed region.  Copies run on a second stream into double-buffered device inputs, so the upload of step
    i+1 overlaps the kernels of step i, as a user streaming layers through the library would do."""
    Wg, Wu, Wd = weights
    arena.reset()
    host_in = [arena.take(t).copy_(t) for t in (X, Wg, Wu, Wd)]
    dev_in = [[torch.empty_like(t) for t in (X, Wg, Wu, Wd)] for _ in range(2)]
    outs = [path.norm] + [path.out[n][k] for n in ("gate", "up", "down") for k in ("mask", "values", "meta")]
    host_out = [arena.take(t) for t in outs]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)
    comp = torch.cuda.current_stream()
    copy = torch.cuda.Stream()

    FIRST_CHUNKS = 4          # the very first upload has no step to hide behind: its X goes up in chunks

    def run(n):
        uploaded = [torch.cuda.Event() for _ in range(2)]
        computed = [torch.cuda.Event() for _ in range(2)]
        downloaded = torch.cuda.Event()
        have_download = False

        def upload(slot, after=None):
            with torch.cuda.stream(copy):
                if after is not None:
                    copy.wait_event(after)             # the slot's previous step must be done with it
                for h, dv in zip(host_in, dev_in[slot]):
                    dv.copy_(h, non_blocking=True)
                uploaded[slot].record(copy)

        def upload_first(slot):
            """Weights first, then X in chunks, an event per chunk: the calibration of chunk c runs while chunk
            c + 1 is still on its way (the per-neuron sums accumulate across calls)."""
            chunks = []
            with torch.cuda.stream(copy):
                for h, dv in list(zip(host_in, dev_in[slot]))[1:]:
                    dv.copy_(h, non_blocking=True)
                T = host_in[0].shape[0]
                step_t = -(-T // FIRST_CHUNKS)
                for t0 in range(0, T, step_t):
                    t1 = min(T, t0 + step_t)
                    dev_in[slot][0][t0:t1].copy_(host_in[0][t0:t1], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(copy)
                    chunks.append((t0, t1, ev))
                uploaded[slot].record(copy)
            return chunks

        copy.wait_stream(comp)
        first_chunks = upload_first(0)
        for i in range(n):
            slot = i % 2
            if i > 0:
                comp.wait_event(uploaded[slot])
            wait_dl = (lambda: comp.wait_event(downloaded)) if have_download else None
            path.step(*dev_in[slot], alpha, before_stage_b=wait_dl,             # outputs are reused: wait for their download
                      x_chunks=first_chunks if i == 0 else None)
            computed[slot].record(comp)
            if i + 1 < n:
                upload(1 - slot, after=computed[1 - slot] if i >= 1 else None)
            with torch.cuda.stream(copy):
                copy.wait_event(computed[slot])
                for o, h in zip(outs, host_out):
                    h.copy_(o, non_blocking=True)
                downloaded.record(copy)
            have_download = True
        comp.wait_stream(copy)

    run(1)
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    run(steps)
    b.record()
    torch.cuda.synchronize()
    path.check()
    seconds = max_over_ranks(a.elapsed_time(b) / 1e3, world, device)
    return {"value": aggregate_value(cfg.T, steps, world, seconds), "unit": UNIT, "steps": steps,
            "ms_per_step": seconds * 1e3 / steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "overlap": "uploads of step i+1 and downloads of step i run on a copy stream beside the kernels; the first "
                       "step's X goes up in 4 chunks and is calibrated chunk by chunk"}


# --------------------------------------------------------------------------- the oracle legs

def _oracle_sample_rate(Xs, Wg32, Wu32, act_code):
    import oracle
    t = time.perf_counter()
    oracle.calib_sumsq(Xs, Wg32, Wu32, act_code)
    return time.perf_counter() - t


def cpu_baseline(cfg, X, weights, budget_s=15.0):
    """The fp64 oracle, as it stands, on this host's cores over a bounded token sample."""
    import numpy as np
    import oracle
    act_code = {"silu": oracle.ACT_SILU, "gelu_tanh": oracle.ACT_GELU_TANH, "relu": oracle.ACT_RELU}[cfg.act]
    Wg32 = weights[0].float().cpu().numpy()
    Wu32 = weights[1].float().cpu().numpy()
    probe = 4
    Xp = X[:probe].float().cpu().numpy()
    dt = _oracle_sample_rate(Xp, Wg32, Wu32, act_code)
    n = int(max(probe, min(cfg.T, budget_s / (dt / probe))))
    Xs = X[:n].float().cpu().numpy()
    dt = _oracle_sample_rate(Xs, Wg32, Wu32, act_code)
    return {"value": n / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"stage (a) of the fp64 C oracle on the first {n} of {cfg.T} tokens x all {cfg.I} neurons "
                      f"({dt:.1f} s); stage (b) is O(d*I) and adds < 1% to a full CPU step"}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return None
    import oracle
    cfg = synth.CONFIGS[args.config]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    act_code = {"silu": oracle.ACT_SILU, "gelu_tanh": oracle.ACT_GELU_TANH, "relu": oracle.ACT_RELU}[cfg.act]
    Wg, Wu, _ = synth.make_weights(cfg, dev, layer=0)
    Wg32, Wu32 = Wg.float().cpu().numpy(), Wu.float().cpu().numpy()
    n = args.ref_tokens
    X = synth.make_x(cfg, dev, T=n * (args.steps + args.warmup)).float().cpu().numpy()
    for i in range(args.warmup):
        _oracle_sample_rate(X[i * n:(i + 1) * n], Wg32, Wu32, act_code)
    t = time.perf_counter()
    for i in range(args.warmup, args.warmup + args.steps):
        _oracle_sample_rate(X[i * n:(i + 1) * n], Wg32, Wu32, act_code)
    seconds = time.perf_counter() - t
    value = n * args.steps / seconds
    cores = oracle.num_threads()
    sample = (f"each step = stage (a) of the fp64 C oracle on {n} tokens x all {cfg.I} neurons of the "
              f"{cfg.name}-shaped layer (of {cfg.T} tokens per full step)")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": seconds * 1e3 / args.steps, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{cfg.name}-shaped {cfg.act} layer, d={cfg.d}, I={cfg.I}; {sample}"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)
    return out


def free_port():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def launch_ranks(n, argv):
    """`--gpus N` without a launcher around it: start the N ranks here (one process per GPU, torch.distributed.run on
    this node, rendezvous on 127.0.0.1) and hand back their exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def launch_check(args):
    """What `--gpus N` resolved to, without any GPU work (gloo on a box without GPUs): every rank reports its
    (rank, world size); rank 0 prints them.  Used by the host tests of the launcher."""
    import torch.distributed as dist
    rank, _, world = dist_env()
    if world > 1:
        dist.init_process_group("gloo" if not torch.cuda.is_available() else "nccl")
        seen = [None] * world
        dist.all_gather_object(seen, (rank, world))
        dist.destroy_process_group()
    else:
        seen = [(rank, world)]
    if rank == 0:
        print(json.dumps({"launch_check": True, "gpus": args.gpus, "ranks": seen}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama2_70b", choices=sorted(synth.CONFIGS))
    ap.add_argument("--tokens", type=int, default=0, help="override the number of calibration tokens (debugging)")
    ap.add_argument("--pool", type=int, default=3, help="distinct synthetic layers cycled through the steps")
    ap.add_argument("--e2e-steps", type=int, default=12)
    ap.add_argument("--iso-iters", type=int, default=20, help="iterations of the stage-(b)-only timing loop (0 = skip)")
    ap.add_argument("--unstructured-iters", type=int, default=10,
                    help="iterations of the unstructured-selection timing loop on the same matrices (0 = skip)")
    ap.add_argument("--forward-iters", type=int, default=5, help="iterations of the forward-pass timing loop (0 = skip)")
    ap.add_argument("--forward-tokens", type=int, default=32768, help="tokens of the forward-pass timing loop")
    ap.add_argument("--stream-layers", type=int, default=-1,
                    help="layers of the layer-stream leg (-1 = all MLP layers of the model, 0 = skip)")
    ap.add_argument("--per-config", type=int, default=1, help="1 = also run the paper's other shapes (0 = skip)")
    ap.add_argument("--per-config-seconds", type=float, default=2.4, help="timed seconds per extra shape")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-tokens", type=int, default=64, help="tokens per step of the reference (oracle) arm")
    ap.add_argument("--launch-check", action="store_true", help="only report the ranks --gpus resolved to")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if "WORLD_SIZE" in os.environ:
        if int(os.environ["WORLD_SIZE"]) != args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={os.environ['WORLD_SIZE']} ranks")
    elif args.gpus > 1:
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.launch_check:
        launch_check(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
