"""Host-side logic of the multi-GPU mode: replicas that each serve a shard of the query stream.

Queries are independent (paper Section 2.1: a stream of queries, each answered by one SubNet), so the
only multi-GPU structure is data parallelism over queries with one SuperNet replica per GPU.  There is
no data-path collective; torch.distributed is used for the barrier and for the max of the timings.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


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


def rotated_stream(items: Sequence, rank: int, n: int, stride: int = 131) -> List:
    """Weak-scaling stream of a replica: n queries of the same distribution, starting at a
    rank-dependent offset of the base stream."""
    m = len(items)
    return [items[(i + stride * rank) % m] for i in range(n)]


def aggregate_throughput(queries_per_rank: Sequence[int], ms_per_rank: Sequence[float]) -> float:
    """Whole-job queries/s: all queries served divided by the slowest rank's time."""
    t = max(ms_per_rank)
    return sum(queries_per_rank) / (t * 1e-3) if t > 0 else 0.0
