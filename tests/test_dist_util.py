"""World-size-2 gloo test of the benchmark's multi-process plumbing (CPU only)."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2609_34420_b200 import dist_util
    dist_util.init_process_group("gloo")
    dev = torch.device("cpu")
    dist_util.barrier(dev)
    ms, units = dist_util.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1), dev)
    q.put((rank, ms, units, dist_util.shard_seed(7, rank)))
    dist_util.barrier(dev)
    torch.distributed.destroy_process_group()


def test_two_rank_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]          # max over ranks
    assert [r[2] for r in res] == [300.0, 300.0]        # sum over ranks
    assert res[0][3] != res[1][3]                       # different batch per rank


def test_single_process_is_identity():
    from paper_2609_34420_b200 import dist_util
    assert dist_util.aggregate(3.5, 9.0, torch.device("cpu")) == (3.5, 9.0)
