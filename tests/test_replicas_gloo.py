"""The N > 1 mode on CPU: two gloo ranks shard a stream, agree on the max time and on the totals."""
import os
import zlib
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import zlib
    sys.path.insert(0, ROOT)
    from paper_2306_17266_b200 import replicas, workload as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfgs = wl.markov_stream(101, seed=4)
    mine = replicas.shard_stream(cfgs, rank, world)
    keys = [zlib.crc32(c.key()) for c in mine]
    n = torch.tensor([len(mine)])
    dist.all_reduce(n)
    ms = torch.tensor([10.0 + 5.0 * rank])
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    gathered = [None] * world
    dist.all_gather_object(gathered, keys)
    dist.barrier()
    if rank == 0:
        all_keys = [k for part in gathered for k in part]
        ref = [zlib.crc32(c.key()) for c in cfgs]
        out.put((int(n.item()), float(ms.item()), all_keys == ref,
                 replicas.aggregate_throughput([len(p) for p in gathered], [10.0, 15.0])))
    dist.destroy_process_group()


def test_two_ranks_shard_the_stream_and_agree():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    total, max_ms, in_order, qps = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert total == 101 and max_ms == 15.0 and in_order
    assert abs(qps - 101 / 0.015) < 1e-6


def test_shard_bounds_partition():
    sys.path.insert(0, ROOT)
    from paper_2306_17266_b200 import replicas
    for n in (0, 1, 7, 100, 101):
        for world in (1, 2, 3, 8):
            spans = [replicas.shard_bounds(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    assert replicas.rotated_stream(list(range(10)), 1, 4, stride=3) == [3, 4, 5, 6]
