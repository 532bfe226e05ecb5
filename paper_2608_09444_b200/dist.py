"""Multi-GPU plumbing.  The path shards by sequence: every GPU holds a weight replica, its own page pool
and its own scheduler, and processes its own sequences; there is no data-path collective.  The only
communication is the barrier around a timed region and the max-over-ranks of its duration."""
from __future__ import annotations

import os


def env_rank():
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def shard(items, world: int, rank: int):
    """Round-robin share of `items` for `rank`: disjoint, complete, sizes differ by at most one."""
    return list(items)[rank::world]


def rank_seed(base: int, rank: int) -> int:
    """Seed of a rank's own synthetic workload (weak scaling: every rank gets fresh rows)."""
    return base + rank


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's value; a plain float when there is one rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def route_least_loaded(arrivals, kv_tokens, out_lens, world: int, est_s_per_token: float = 0.01):
    """Front-end assignment of requests to replicas: each request, in arrival order, goes to the replica
    that holds the fewest reserved KV tokens at its arrival time (ties: lowest rank).  A request reserves
    kv_tokens[i] (prompt + output) from its arrival until its estimated finish, arrival + out_lens[i] *
    est_s_per_token.  A pure function of the trace, so every rank computes the same assignment without
    talking to the others.  Returns the replica index of every request."""
    import heapq
    load = [0] * world
    releases = []                                   # (time, rank, tokens)
    out = []
    for i in range(len(arrivals)):
        t = float(arrivals[i])
        while releases and releases[0][0] <= t:
            _, r, k = heapq.heappop(releases)
            load[r] -= k
        r = min(range(world), key=lambda j: (load[j], j))
        load[r] += int(kv_tokens[i])
        heapq.heappush(releases, (t + int(out_lens[i]) * est_s_per_token, r, int(kv_tokens[i])))
        out.append(r)
    return out


def gather_objects(obj):
    """[obj of rank 0, obj of rank 1, ...] on every rank; [obj] when there is one rank."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [obj]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, obj)
    return out
