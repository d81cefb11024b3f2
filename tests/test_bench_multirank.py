"""The benchmark's multi-rank plumbing on CPU: two gloo ranks, max-over-ranks timing, whole-job throughput.
The optimizer step itself needs no exchange between data-parallel replicas, so this is all the N > 1 path adds."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    seconds = 1.0 + rank                      # rank 1 is the slow one
    smax = bench.max_over_ranks(seconds, "cpu")
    value = bench.job_throughput(1000.0, world, smax)
    dist.barrier()
    out.put((rank, smax, value))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_max_time_and_aggregate_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, smax, value in res:
        assert smax == 2.0                    # the slowest rank's time on every rank
        assert value == pytest.approx(2 * 1000.0 / 2.0)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, "cpu") == 3.5
    assert bench.job_throughput(10.0, 1, 2.0) == 5.0
