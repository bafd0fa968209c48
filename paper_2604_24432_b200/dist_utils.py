"""Multi-GPU plumbing of the benchmark and of batch sharding (host logic only, no data-path collective).

The KSA forward pass shards without any exchange: by whole sequences of a packed batch (each
rank takes a subset of the sequences) or by KV-head groups.  ``shard_sequences`` assigns the
sequences of a packed batch to ranks, longest processing time first, with the closed-form visible
pair count of Eq. 3 as the cost.  The timing helpers implement the "max over ranks" rule."""
from __future__ import annotations

import dataclasses
from typing import List, Sequence


def visible_pairs_of_sequence(n: int, k: int, m: int, C: int) -> int:
    """Closed-form number of visible (query, key) pairs of one sequence and one head (Eq. 3 text rows
    plus the summary rows with self visibility)."""
    total = 0
    for c in range((n + k - 1) // k):
        rows = min(n, c * k + k) - c * k
        far = max(0, c - C)
        first = c * k - far * k + 1 + far * m          # visible keys of the chunk's first row
        total += rows * first + rows * (rows - 1) // 2
    total += (n // k) * sum(k + r + 1 for r in range(m))
    return total


def shard_sequences(text_lens: Sequence[int], k: int, m: int, C: int, world: int) -> List[List[int]]:
    """Indices of the sequences each rank processes (every sequence exactly once): longest first onto
    the least loaded rank; ties go to the lower rank, so every rank computes the same table."""
    cost = [visible_pairs_of_sequence(n, k, m, C) for n in text_lens]
    order = sorted(range(len(text_lens)), key=lambda i: (-cost[i], i))
    load = [0] * world
    shards: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda j: (load[j], j))
        shards[r].append(i)
        load[r] += cost[i]
    return [sorted(s) for s in shards]


def shard_kv_heads(num_kv_heads: int, world: int) -> List[range]:
    """Contiguous KV-head ranges per rank (each rank also takes the query heads of its KV heads)."""
    base, rem = divmod(num_kv_heads, world)
    out, h = [], 0
    for r in range(world):
        n = base + (1 if r < rem else 0)
        out.append(range(h, h + n))
        h += n
    return out


def rank_workload(wl, rank: int):
    """Independent batch per rank (weak scaling): same shape, another seed."""
    return dataclasses.replace(wl, seed=wl.seed + 1000 * rank)


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a timing (identity without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    if t.is_cuda:
        t = t.float()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job rate: the units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)
