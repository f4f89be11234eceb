"""Host-side logic of the multi-GPU mode: replicas that each serve a shard of the query stream.

Queries are independent (paper Section 2.1: a stream of queries, each answered by one SubNet), so the
only multi-GPU structure is data parallelism over queries with one SuperNet replica per GPU.  There is
no data-path collective; torch.distributed is used for the barrier and for the max of the timings.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def shard_bounds(n_queries: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous shard [begin, end) of a stream of n_queries for `rank`; shards differ by at most one."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("bad rank / world size")
    base, extra = divmod(n_queries, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_stream(items: Sequence, rank: int, world: int) -> List:
    """Contiguous shards keep consecutive queries together, which preserves the temporal locality the
    SubGraph cache lives on (paper Section 2.2)."""
    b, e = shard_bounds(len(items), rank, world)
    return list(items[b:e])


def affinity_shards(encodings, world: int) -> List[List[int]]:
    """Partition of the queries 0..n-1 into `world` shards of equal size (they differ by at most one) such that
    queries whose SubNets are close in the vector encoding of paper Section 3.3 (the (K_i, C_i) entries of every
    layer) land on the same replica.  Each replica's SubGraph cache then sees SubNets with a larger common
    SubGraph: the multi-GPU form of the temporal locality of Section 2.2.  Inside a shard the queries keep their
    stream order.

    Recursive bisection, deterministic (every rank computes the same partition without talking to the others): the
    queries of a group are ordered by their projection on the group's direction of largest variance (power
    iteration from the all-ones vector) and cut in proportion to the replicas on either side.  `encodings` is an
    (n, d) array-like; world == 1 returns the stream as it is."""
    x = np.asarray(encodings, dtype=np.float64)
    if world <= 0:
        raise ValueError("bad world size")
    n = x.shape[0]
    x = x.reshape(n, -1)

    def split(idx: List[int], parts: int) -> List[List[int]]:
        if parts == 1:
            return [sorted(idx)]
        c = x[idx] - x[idx].mean(axis=0) if idx else x[idx]
        v = np.ones(c.shape[1])
        for _ in range(30):
            w = c.T @ (c @ v)
            norm = np.linalg.norm(w)
            if norm == 0:
                break
            v = w / norm
        order = [idx[i] for i in np.argsort(c @ v, kind="stable")]
        left = parts // 2
        # sizes: the first n % world shards overall get one more query; here simply in proportion, rounded down
        cut = len(order) * left // parts
        return split(order[:cut], left) + split(order[cut:], parts - left)

    return split(list(range(n)), world)


def rotated_stream(items: Sequence, rank: int, n: int, stride: int = 131) -> List:
    """Weak-scaling stream of a replica: n queries of the same distribution, starting at a
    rank-dependent offset of the base stream."""
    m = len(items)
    return [items[(i + stride * rank) % m] for i in range(n)]


def aggregate_throughput(queries_per_rank: Sequence[int], ms_per_rank: Sequence[float]) -> float:
    """Whole-job queries/s: all queries served divided by the slowest rank's time."""
    t = max(ms_per_rank)
    return sum(queries_per_rank) / (t * 1e-3) if t > 0 else 0.0
