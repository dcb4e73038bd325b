#!/usr/bin/env python
"""Throughput of the DaSS hot path on B200: one step = one MLP layer through the whole path
(fused GLU calibration norms -> norm finalize -> N:M scoring of gate / up / down -> compression)
on synthetic inputs shaped like the paper's models and its 128 x 2048-token calibration set.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config llama2_70b] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample of
the same workload instead.  With N > 1 (launched by torch.distributed.run) every rank prunes its own
independent layers -- the path has no cross-GPU exchange -- and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
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
KERNEL_LAUNCHES_PER_STEP = 10   # status clear, calib GEMM, partial reduce, finalize, 3 x score, 3 x compress
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


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
    """Algorithmic bytes of stage (b) for the three projections of one layer."""
    esz = 2 if cfg.dtype == "bf16" else 4
    elems = 3 * cfg.d * cfg.I
    score = elems * (esz + esz + 0.125)                                   # read W, write pruned + mask bit
    frac = cfg.n_keep / cfg.m
    meta_bits = 4 / 4 if (cfg.n_keep == 2 and cfg.m == 4) else 1.0        # field bits per weight
    comp = elems * (esz + 0.125 + esz * frac + meta_bits / 8.0) if compress else 0.0
    return score, comp


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from one ncu capture of this very
# command on the default workload; see profiles/.  None where the kernel changed after the capture.
NCU_DRAM_BYTES = {"llama2_70b": {"calib": 122.00e9 + 20.8e6,                                  # one launch, T = 262144
                                 "score": (2 * (470.4 + 443.6) + 471.4 + 454.4) * 1e6,         # gate + up + down
                                 "compress": (2 * (499.1 + 206.7) + 499.2 + 214.1) * 1e6}}


def roofline_b(kernel, algorithmic_bytes, in_step_ms, isolated_ms, peaks, peak_src, traffic):
    """HBM roofline entry of a group of stage-(b) launches (bytes are per step: three matrices)."""
    ms = isolated_ms if isolated_ms else in_step_ms
    gbs = algorithmic_bytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": gbs / peaks["hbm_gbs"], "peak_source": peak_src,
            "timed": "alone, back to back, after the step loop" if isolated_ms else "inside the step",
            "in_step_gbs": algorithmic_bytes / (in_step_ms * 1e-3) / 1e9,
            "algorithmic_bytes_per_step": algorithmic_bytes, "traffic": traffic}


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
        self.ev = {k: [] for k in ("calib", "score", "compress")}

    def step(self, X, Wg, Wu, Wd, alpha, record=False, before_stage_b=None, x_chunks=None):
        """x_chunks: [(first token, last token + 1, event or None)]: the calibration is then accumulated chunk by
        chunk (the sums carry over between calls), each call waiting for its chunk's event on the current stream."""
        pr = self.pruner
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record else None
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
        pr.score_nm(Wg, Wu, Wd, alpha)
        if record:
            e[2].record()
        pr.compress_nm(Wg, Wu, Wd)
        if record:
            e[3].record()
            self.ev["calib"].append((e[0], e[1]))
            self.ev["score"].append((e[1], e[2]))
            self.ev["compress"].append((e[2], e[3]))

    def mean_ms(self, key):
        v = [a.elapsed_time(b) for a, b in self.ev[key]]
        return sum(v) / len(v) if v else None


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

    X = synth.make_x(cfg, device)
    pool = [synth.make_weights(cfg, device, layer=l) for l in layer_ids_for_rank(rank, world, args.pool, 0)]
    path = LayerPath(cfg, device, binding)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        path.step(X, *pool[i % len(pool)], alpha)
    binding.calib_status(path.ws)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        path.step(X, *pool[(args.warmup + i) % len(pool)], alpha, record=True)
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    binding.calib_status(path.ws)
    seconds = max_over_ranks(t0.elapsed_time(t1) / 1e3, world, device)
    value = aggregate_value(cfg.T, args.steps, world, seconds)

    # per-kernel durations measured live inside the timed region
    calib_ms, score_ms, comp_ms = path.mean_ms("calib"), path.mean_ms("score"), path.mean_ms("compress")
    flops = 4.0 * cfg.T * cfg.d * cfg.I
    achieved_tf = flops / (calib_ms * 1e-3) / 1e12
    sb, cb = stage_b_bytes(cfg)
    score_gbs, comp_gbs = sb / (score_ms * 1e-3) / 1e9, cb / (comp_ms * 1e-3) / 1e9

    # stage (b) alone: the same launches back to back, away from the power-capped GEMM, so that the
    # bandwidth-bound kernels are measured at the clocks they get by themselves
    iso = isolated_stage_b(path, pool, alpha, iters=args.iso_iters) if args.iso_iters > 0 else None

    unstructured = unstructured_leg(path, pool, alpha, args.unstructured_iters, peaks) if args.unstructured_iters > 0 else None

    forward = None
    if args.forward_iters > 0 and cfg.dtype == "bf16":
        forward = forward_leg(path, X, pool[0], args.forward_tokens, args.forward_iters, peaks)

    # end to end: pinned host inputs -> device -> path -> results back to the host, every step
    e2e = None
    if args.e2e_steps > 0:
        e2e = run_e2e(cfg, path, X, pool[0], alpha, args.e2e_steps, world, device)

    out = None
    traffic = NCU_DRAM_BYTES.get(cfg.name, {}) if not args.tokens else {}
    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = cpu_baseline(cfg, X, pool[0], budget_s=args.cpu_seconds)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": seconds * 1e3 / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": f"{cfg.name}-shaped {cfg.act} layer, d={cfg.d}, I={cfg.I}, T={cfg.T} calibration tokens, "
                                   f"{cfg.n_keep}:{cfg.m} on gate/up (Eq. 4, alpha={alpha}, input-balanced) and down (Eq. 5); "
                                   "mask + pruned weights + compressed values/metadata",
                       "layers_per_rank": args.steps, "weight_sets_cycled": len(pool),
                       "input_checksums": {n: synth.checksum(t) for n, t in zip(("X", "Wg", "Wu", "Wd"), (X,) + tuple(pool[0]))},
                       "l2": "inputs exceed L2 (X and each weight set are far larger than 126 MB); no flush",
                       "parallelism": "independent layers per GPU, no collective" if world > 1 else "single GPU"},
            "stage_ms": {"calib": calib_ms, "score_x3": score_ms, "compress_x3": comp_ms},
            "score_gbs": score_gbs, "compress_gbs": comp_gbs,
            "roofline": {"bound": "tensor", "kernel": "calib_tc2_kernel", "achieved": achieved_tf,
                         "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": achieved_tf / peaks["bf16_tflops_sustained"],
                         "frac_of_burst_peak": achieved_tf / peaks["bf16_tflops"], "peak_source": peak_src,
                         "algorithmic_flops_per_launch": flops, "traffic": traffic.get("calib")},
            "roofline_score": roofline_b("score_{rows,cols}_bf16_kernel x3 (gate, up, down)", sb, score_ms, iso and iso["score"],
                                         peaks, peak_src, traffic.get("score")),
            "roofline_compress": roofline_b("compress_rows_bf16_kernel x2 (gate, up) + compress_cols_bf16_kernel (down)", cb, comp_ms, iso and iso["compress"],
                                            peaks, peak_src, traffic.get("compress")),
            "unstructured": unstructured, "forward": forward,
            "e2e": e2e, "gpu_launches": KERNEL_LAUNCHES_PER_STEP * args.steps, "clocks": clocks,
            "cpu_baseline": cpu,
        }
        if cfg.dtype != "bf16":
            out["roofline"]["bound"] = "alu"
            out["roofline"]["kernel"] = "calib_simt_kernel"
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    return out


def isolated_stage_b(path, pool, alpha, iters):
    """Mean ms of the three scoring launches and of the three compression launches, timed alone."""
    def score(ws):
        path.pruner.score_nm(*ws, alpha)

    def compress(ws):
        path.pruner.compress_nm(*ws)

    out = {}
    time.sleep(0.5)                      # let the clocks recover from the power-capped GEMM
    for key, fn in (("score", score), ("compress", compress)):
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

    def run(ws):
        path.pruner.select_unstructured(*ws, sparsity, alpha)

    for i in range(3):
        run(pool[i % len(pool)])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        run(pool[i % len(pool)])
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    nbytes, _ = stage_b_bytes(cfg, compress=False)
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"sparsity": sparsity, "ms_x3": ms, "achieved": gbs, "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
            "kernels": "select_cols_kernel + select_emit_cols_kernel (gate, up), select_rows_kernel (down)",
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
            "kernels": "mlp_forward_tc_kernel<GLU> + mlp_forward_tc_kernel<PLAIN>",
            "algorithmic_flops": flops, "timed": "alone, back to back, after the step loop"}


def run_e2e(cfg, path, X, weights, alpha, steps, world, device):
    """Same step driven from pinned host memory: every step's inputs (X and the three weight matrices) are
    copied host -> device and its results (norms, masks, values, metadata) device -> host, all inside the
    timed region.  Copies run on a second stream into double-buffered device inputs, so the upload of step
    i+1 overlaps the kernels of step i, as a user streaming layers through the library would do."""
    Wg, Wu, Wd = weights
    host_in = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in (X, Wg, Wu, Wd)]
    dev_in = [[torch.empty_like(t) for t in (X, Wg, Wu, Wd)] for _ in range(2)]
    outs = [path.norm] + [path.out[n][k] for n in ("gate", "up", "down") for k in ("mask", "values", "meta")]
    host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
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
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-tokens", type=int, default=64, help="tokens per step of the reference (oracle) arm")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
