"""Host logic of the N > 1 benchmark path, run as two gloo ranks on the CPU: every rank gets its own
independent layers (the path has no cross-GPU exchange), the step time is the max over ranks, and the
reported value is the aggregate over all ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        ids = bench.layer_ids_for_rank(rank, world, steps=4, warmup=3)
        gathered = [None] * world
        dist.all_gather_object(gathered, ids)
        flat = [i for ids_r in gathered for i in ids_r]
        assert len(flat) == len(set(flat)) == world * 7          # disjoint layers, none shared
        my_seconds = 1.0 + 0.5 * rank                              # rank 1 is the slow one
        slowest = bench.max_over_ranks(my_seconds, world, torch.device("cpu"))
        assert slowest == 1.0 + 0.5 * (world - 1)
        value = bench.aggregate_value(tokens_per_step=1000, steps=4, world=world, seconds_max=slowest)
        if rank == 0:
            out.put(value)
    finally:
        dist.destroy_process_group()


def test_two_rank_timing_and_sharding():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert out.get(timeout=5) == 1000 * 4 * 2 / 1.5


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(2.5, 1, torch.device("cpu")) == 2.5
    assert bench.layer_ids_for_rank(0, 1, 8, 3) == list(range(11))
    assert bench.aggregate_value(10, 2, 1, 4.0) == 5.0


def _bench(*flags, env=None):
    import json
    import subprocess
    e = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                         cwd=ROOT, env=e, timeout=600)
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    return res.returncode, lines


def test_gpus_flag_alone_starts_that_many_ranks():
    """`bench.py --gpus 2` with no launcher around it starts two ranks itself (gloo here, no GPU work), and both
    see WORLD_SIZE == 2."""
    rc, lines = _bench("--gpus", "2", "--launch-check")
    assert rc == 0 and len(lines) == 1
    assert lines[0]["gpus"] == 2 and sorted(map(tuple, lines[0]["ranks"])) == [(0, 2), (1, 2)]
    rc, lines = _bench("--launch-check")
    assert rc == 0 and lines[0]["ranks"] == [[0, 1]]


def test_gpus_flag_must_agree_with_the_launcher():
    rc, lines = _bench("--gpus", "2", "--launch-check", env={"WORLD_SIZE": "3", "RANK": "0", "LOCAL_RANK": "0"})
    assert rc != 0 and lines == []
    rc, lines = _bench("--gpus", "0", "--launch-check")
    assert rc != 0
