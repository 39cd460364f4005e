"""World-size-2 check (gloo, CPU) of the replica logic bench.py uses for N > 1 GPUs."""
import os
import socket

import torch.multiprocessing as mp

from paper_2203_16487_b200 import replicas


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [replicas.batch_index(s, rank, world, 7) for s in range(5)]
    toks, ms = replicas.reduce_job(100.0 * (rank + 1), 10.0 + rank)
    q.put((rank, mine, toks, ms))
    dist.destroy_process_group()


def test_two_ranks_take_disjoint_batches_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    [p.start() for p in ps]
    res = sorted(q.get(timeout=120) for _ in range(world))
    [p.join(60) for p in ps]
    assert all(p.exitcode == 0 for p in ps)
    (r0, b0, t0, m0), (r1, b1, t1, m1) = res
    assert b0 == [0, 2, 4, 6, 1] and b1 == [1, 3, 5, 0, 2]
    assert not set(b0[:3]) & set(b1[:3])
    assert t0 == t1 == 300.0 and m0 == m1 == 11.0


def test_single_process_is_identity():
    assert replicas.reduce_job(5.0, 2.0) == (5.0, 2.0)
    assert replicas.batch_index(3, 0, 1, 4) == 3
