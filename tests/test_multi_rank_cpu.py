"""The N > 1 path of the benchmark is batch-sharded replicas with no data-path collective: the only exchange is
the max-over-ranks of the timings.  Exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 5.0 - rank]                       # rank 0: (1, 5), rank 1: (2, 4)
    got = bench.max_over_ranks(mine, world, "cpu")
    dist.barrier()
    out.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [2.0, 5.0]


def test_job_throughput_is_the_sum_over_replicas():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.job_throughput(64, 20, 1, 0.5) == 64 * 20 / 0.5
    assert bench.job_throughput(64, 20, 8, 0.5) == 8 * bench.job_throughput(64, 20, 1, 0.5)
    assert bench.max_over_ranks([3.0], 1) == [3.0]
