"""The N > 1 path of bench.py is "independent replicas": no data-path collective, only the timing is
combined (max over ranks) and the units are summed.  Checked here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    val = bench.aggregate_value(world, 1000, 4, ms * 1e-3)
    dist.barrier()
    if rank == 0:
        out.put((ms, val))
    dist.destroy_process_group()


def test_two_rank_replica_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    ms, val = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert ms == 15.0                                   # the slowest rank's time
    assert abs(val - 2 * 1000 * 4 / 0.015) < 1e-6       # both ranks' units over that time


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.aggregate_value(1, 10, 2, 0.5) == 40.0
