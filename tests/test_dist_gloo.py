"""World-size-2 run of the multi-GPU plumbing on CPU (gloo): work units are sharded with
no data-path collective; ranks only meet at a barrier and at the max / sum of a scalar."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_1709_04060_b200 import dist as qdist
    r, w = qdist.init("gloo")
    units = list(range(16))
    mine = qdist.shard(units, r, w)
    qdist.barrier()
    slowest = qdist.max_over_ranks(10.0 + r)
    total = qdist.sum_over_ranks(float(len(mine)))
    qdist.barrier()
    q.put((r, w, mine, slowest, total))
    qdist.finalize()


def test_two_ranks_shard_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1] and all(g[1] == 2 for g in got)
    assert got[0][2] + got[1][2] == list(range(16))          # disjoint, complete, ordered
    assert all(g[3] == 11.0 for g in got)                     # max over ranks
    assert all(g[4] == 16.0 for g in got)                     # every unit counted once


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_1709_04060_b200 import dist as qdist
    assert qdist.max_over_ranks(3.5) == 3.5
    assert qdist.shard([1, 2, 3], 0, 1) == [1, 2, 3]
