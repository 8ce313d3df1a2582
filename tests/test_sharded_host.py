"""Host logic of the row-sharded path: the row partition, the entry selection and the sum-exchange (two
gloo ranks on CPU tensors; the kernels themselves need a GPU and are covered by the gpu tests)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_00977_b200 import sharded as S


def test_row_blocks_partition_the_rows():
    for m in (1, 7, 100, 2_000_000):
        for world in (1, 2, 3, 8):
            blocks = [S.row_block(m, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == m
            assert all(a[1] == b[0] for a, b in zip(blocks, blocks[1:]))
            sizes = [b - a for a, b in blocks]
            assert max(sizes) - min(sizes) <= 1


def test_shard_coo_keeps_order_and_renumbers():
    rows = torch.tensor([5, 0, 3, 9, 4, 3], dtype=torch.int32)
    cols = torch.tensor([1, 2, 3, 4, 5, 6], dtype=torch.int32)
    vals = torch.arange(6, dtype=torch.float32)
    r, c, v = S.shard_coo(rows, cols, vals, 3, 6)
    assert r.tolist() == [2, 0, 1, 0] and c.tolist() == [1, 3, 5, 6] and v.tolist() == [0.0, 2.0, 4.0, 5.0]
    assert r.dtype == torch.int32


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank's partial G_Q and its column counts; the exchange must give every rank the sums
    gq = torch.full((6,), float(rank + 1))
    cnt = torch.tensor([rank, 2, 0], dtype=torch.int32)
    S.all_reduce_sum(gq, dist)
    S.all_reduce_sum(cnt, dist)
    dist.barrier()
    out.put((rank, gq.tolist(), cnt.tolist()))
    dist.destroy_process_group()


def test_two_rank_sum_exchange():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(2)]
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for _, gq, cnt in got:
        assert gq == [3.0] * 6 and cnt == [1, 4, 0]


def test_no_process_group_is_identity():
    t = torch.tensor([1.0, 2.0])
    assert S.all_reduce_sum(t).tolist() == [1.0, 2.0]
    assert S.all_reduce_sum(t, dist).tolist() == [1.0, 2.0]     # module given, group not initialised


def test_minibatch_split_is_a_seeded_partition():
    from paper_2608_00977_b200.minibatch import split_batches
    a = split_batches(1003, 7, 5, "cpu")
    b = split_batches(1003, 7, 5, "cpu")
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    assert sorted(torch.cat(a).tolist()) == list(range(1003))
    assert max(len(x) for x in a) - min(len(x) for x in a) <= 1
    assert not torch.equal(torch.cat(a), torch.cat(split_batches(1003, 7, 6, "cpu")))
    assert len(split_batches(10, 1, 0, "cpu")) == 1 and len(split_batches(0, 3, 0, "cpu")) == 3
