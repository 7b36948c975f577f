"""Host logic of the multi-process benchmark path, on CPU with gloo and two ranks: the path has no
collective on its data (each rank runs its own batch); only the timing is reduced (max) and the
processed images summed."""
import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    r, wsize = bench.init_dist("gloo")
    assert (r, wsize) == (rank, world)
    bench.barrier()
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 256 * 7)
    q.put((rank, ms, units))
    import torch.distributed as dist
    dist.destroy_process_group()


def test_aggregate_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, units in got:
        assert ms == 15.0            # max over ranks
        assert units == 2 * 256 * 7  # whole-job images


def test_aggregate_single_process():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(3.0, 10) == (3.0, 10.0)
    assert bench.dist_env()[1] >= 1
