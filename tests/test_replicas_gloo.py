"""The N-GPU protocol of the benchmark (replicas only, no data-path collective) on two gloo ranks on CPU:
barrier, maximum over ranks of the per-rank times, whole-job throughput from the slowest rank."""
import os
import socket

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_12399_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world() == (rank, world)
        replicas.barrier()
        local = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
        got = replicas.max_over_ranks(local)
        replicas.barrier()
        out.put((rank, got, replicas.aggregate_throughput(1000, got[0], world)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_maximum_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [15.0, 3.0]                           # both ranks see the same maxima
        assert value == pytest.approx(2 * 1000 / 15e-3)     # two replicas, the slowest rank's time


def test_single_process_is_identity():
    assert replicas.world() == (0, 1)
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.aggregate_throughput(10, 2.0, 1) == pytest.approx(5000.0)


def test_bench_starts_its_own_ranks_and_aggregates_over_them():
    """`python bench.py --gpus 2` (no launcher around it) starts two ranks itself; the timing protocol takes the
    slowest rank's time (rank r reports r + 1 ms here) and the value counts both replicas' units.  CPU only."""
    import json
    import subprocess
    import sys
    from pathlib import Path

    root = Path(__file__).resolve().parent.parent
    r = subprocess.run([sys.executable, str(root / "bench.py"), "--gpus", "2", "--rank-plumbing-only"], capture_output=True,
                       text=True, timeout=300, env={k: v for k, v in __import__("os").environ.items()
                                                    if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")})
    assert r.returncode == 0, r.stdout + r.stderr
    line = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 2.0
    assert line["value"] == 2 * 1000 / 2.0e-3
