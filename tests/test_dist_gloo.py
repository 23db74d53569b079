"""The N > 1 plumbing on CPU: two gloo ranks, row sharding without overlap, max-over-ranks timing."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2608_06912_b200 import dist as D


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = D.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    cpu = torch.device("cpu")
    D.barrier()
    slow = D.max_over_ranks(10.0 + rank, cpu)          # the slower rank sets the step time
    total = D.sum_over_ranks(float(rank + 1), cpu)
    lo, hi = D.row_shard(65537, rank, world)
    covered = D.sum_over_ranks(float(hi - lo), cpu)
    out.put((rank, slow, total, lo, hi, covered))
    D.barrier()
    D.finalize()


def test_two_gloo_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [x[1] for x in res] == [11.0, 11.0]
    assert [x[2] for x in res] == [3.0, 3.0]
    assert res[0][3] == 0 and res[0][4] == res[1][3] and res[1][4] == 65537
    assert res[0][5] == 65537.0


def test_row_shard_partitions_exactly():
    for rows in (1, 2, 7, 8, 65536, 65537):
        for world in (1, 2, 3, 8):
            edges = [D.row_shard(rows, r, world) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == rows
            assert all(edges[i][1] == edges[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in edges]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_is_a_noop():
    assert D.env_world() == (0, 0, 1) or "WORLD_SIZE" in os.environ
    assert D.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    D.barrier()
