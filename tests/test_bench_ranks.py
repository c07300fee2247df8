"""Host logic of a multi-rank bench run, on CPU with the gloo backend (world size 2): the ranks are independent
replicas, the whole-job rate is all ranks' frames over the slowest rank's time, and only rank 0 runs the
reference arm."""
import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_seconds = 0.001 * (1 + rank)          # rank 1 is twice as slow
    slowest = bench.max_over_ranks(local_seconds, device="cpu")
    rate = bench.whole_job_rate(640.0, local_seconds, world, device="cpu")
    dist.barrier()
    out.put((rank, slowest, rate))
    dist.destroy_process_group()


def test_whole_job_rate_uses_the_slowest_rank():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate in got:
        assert abs(slowest - 0.002) < 1e-12
        assert abs(rate - 2 * 640.0 / 0.002) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, device="cpu") == 0.5
    assert bench.whole_job_rate(100.0, 0.5, 1, device="cpu") == 200.0
