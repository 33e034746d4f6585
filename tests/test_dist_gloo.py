"""The N > 1 host logic on CPU: two gloo ranks line up, shard the units and reduce the timing."""
import os
import socket

import torch.multiprocessing as mp

from paper_2602_03203_b200 import workloads as wl
from paper_2602_03203_b200.dist import Ranks, shard


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r = Ranks(backend="gloo")
    segs = wl.segment_list(wl.shrink(wl.config(4), num_layers=2, batch=3))
    mine = shard(segs, r.rank, r.world)
    r.barrier()
    slowest = r.max(10.0 + rank)               # "time" of this rank
    total = r.sum(float(len(mine)))
    out.put((rank, slowest, total, mine[0], mine[-1], len(segs)))
    r.close()


def test_two_gloo_ranks_shard_and_reduce():
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, m0, t0, first0, last0, n), (r1, m1, t1, first1, last1, _) = res
    assert m0 == m1 == 11.0                       # max over ranks
    assert t0 == t1 == float(n)                   # the shards cover every segment exactly once
    assert first0 == (0, 0, 0) and last1 == (1, 2, 3) and last0 < first1


def test_shard_is_a_partition():
    items = list(range(17))
    for world in (1, 2, 3, 8):
        parts = [shard(items, r, world) for r in range(world)]
        assert sum(parts, []) == items
        assert max(map(len, parts)) - min(map(len, parts)) <= 1
