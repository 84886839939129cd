"""The N > 1 path of the benchmark on CPU: independent replicas, one process each, meeting only to take the
slowest replica's time (gloo, world size 2).  The data path has no collective to test: sequences are independent."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    local_ms = [12.0, 20.0][rank]                       # rank 1 is the slower replica
    ms = bench.max_over_ranks(local_ms, dist, "cpu")
    value = bench.job_value(world, 4, 26, ms / 10)      # 10 steps
    out.put((rank, ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_throughput():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 20.0
        assert value == pytest.approx(2 * 4 * 26 / 2.0e-3)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, None, "cpu") == 7.5
    assert bench.job_value(1, 1, 8, 5.0) == pytest.approx(1600.0)
