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


def _mean_hit_ratio(encs, q=4):
    """Appendix A.4 hit ratio of a shard served with the intersection policy (window q), from the checker's formulas."""
    import numpy as np
    import oracle
    G, hits = None, []
    for t, e in enumerate(encs):
        hits.append(0.0 if G is None else oracle.hit_ratio(e, G))
        if (t + 1) % q == 0:
            G = encs[t - q + 1]
            for f in encs[t - q + 2:t + 1]:
                G = oracle.intersect(G, f)
    return float(np.mean(hits))


def test_affinity_shards_partition_and_raise_the_hit_ratio():
    # i.i.d. uniform configs have no temporal locality: contiguous shards see unrelated SubNets back to back.  Shards
    # built from the encodings are a partition of equal sizes, keep the stream order inside a shard, and give every
    # replica a strictly higher analytic hit ratio than its contiguous shard.
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    from paper_2306_17266_b200 import replicas, workload as wl
    net = oracle.Net(wl.RESNET, wl.make_blob(wl.RESNET, seed=0, bf16_weights=True))
    cfgs = wl.uniform_stream(wl.RESNET, 400, seed=2)
    encs = [net.encode(c) for c in cfgs]
    vec = np.stack([e[:, :2].reshape(-1) for e in encs])
    assert replicas.affinity_shards(vec, 1) == [list(range(400))]
    for world in (2, 8):
        shards = replicas.affinity_shards(vec, world)
        assert sorted(q for s in shards for q in s) == list(range(400))
        assert max(len(s) for s in shards) - min(len(s) for s in shards) <= 1
        assert all(s == sorted(s) for s in shards)
        assert shards == replicas.affinity_shards(vec, world)          # deterministic: every rank computes the same
        for r in range(world):
            b, e = replicas.shard_bounds(400, r, world)
            plain = _mean_hit_ratio(encs[b:e])
            near = _mean_hit_ratio([encs[q] for q in shards[r]])
            assert near > plain, (world, r, near, plain)


def _affinity_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2306_17266_b200 import replicas, workload as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfgs = wl.uniform_stream(wl.RESNET, 64 * world, seed=2)
    # (a rank of the benchmark takes the encodings from its SuperNet handle; here a plain feature vector of the config)
    vec = np.array([[c.depth[s] for s in range(4)] + [c.width[s] for s in range(5)] + [c.expand[s][b] for s in range(4) for b in range(6)] for c in cfgs])
    mine = replicas.affinity_shards(vec, world)[rank]
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    dist.barrier()
    if rank == 0:
        out.put(sorted(q for part in gathered for q in part) == list(range(64 * world)) and all(len(p) == 64 for p in gathered))
    dist.destroy_process_group()


def test_ranks_agree_on_the_affinity_partition():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 30500 + os.getpid() % 1000
    procs = [ctx.Process(target=_affinity_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
