"""Replica plumbing with two gloo ranks on CPU: sharding helper, barrier, max/sum reductions."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2608_16491_b200 import replicas
    assert replicas.init("gloo") == world
    assert replicas.world() == (rank, rank, world)
    b, e = replicas.shard(10_001, rank, world)
    replicas.barrier()
    # every rank times its own replica; the job's time is the slowest rank's
    elapsed = 1.0 + rank
    t_max = replicas.max_over_ranks(elapsed)
    done = replicas.sum_over_ranks(e - b)
    out.put((rank, b, e, t_max, done))
    replicas.barrier()
    dist.destroy_process_group()


def test_two_rank_reductions_and_sharding():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, b0, e0, t0, d0), (r1, b1, e1, t1, d1) = res
    assert (b0, e0, b1, e1) == (0, 5001, 5001, 10_001)     # contiguous, covers the batch once
    assert t0 == t1 == 2.0                                  # max over ranks
    assert d0 == d1 == 10_001                               # units summed over ranks


def test_shard_covers_every_query_once():
    from paper_2608_16491_b200 import replicas
    for nq in (0, 1, 7, 10_000):
        for world in (1, 2, 3, 8):
            blocks = [replicas.shard(nq, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == nq
            assert all(a[1] == b[0] for a, b in zip(blocks, blocks[1:]))
            sizes = [e - b for b, e in blocks]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_is_a_no_op():
    from paper_2608_16491_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(2) == 2.0
    replicas.barrier()
