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


def visible_pairs_of_rows(n: int, k: int, m: int, C: int, aug_begin: int, aug_end: int) -> int:
    """Visible (query, key) pairs of the augmented rows [aug_begin, aug_end) of one sequence of n text tokens and
    one head: text rows by Eq. 3, summary rows their own chunk with self visibility."""
    total = 0
    s = k + m
    full = (n // k) * s
    for a in range(aug_begin, aug_end):
        if a < full and a % s >= k:                        # summary row r of its chunk
            total += k + (a % s - k) + 1
            continue
        i = (a // s) * k + a % s if a < full else (n // k) * k + (a - full)
        c = i // k
        far = max(0, c - C)
        total += i - far * k + 1 + far * m
    return total


def kv_rows_needed(aug_end: int) -> range:
    """Rows of k and v a sequence-parallel rank needs for query rows that end at aug_end (exclusive): a text row
    attends to rows at or before its own, a summary row to its own chunk, so everything before aug_end and
    nothing after it.  (Rows of the window's far side that only summaries cover could be skipped as well; the
    all-gather below does not bother.)"""
    return range(0, aug_end)


def all_gather_rows(local_rows, ranges, total_rows):
    """The exchange step of a sequence-parallel run: every rank contributes its rows [begin, end) of k (or v) and
    receives the whole tensor.  `local_rows`: this rank's [end - begin, H, D] tensor; `ranges`: the (begin, end)
    of every rank, in rank order.  Uses one all_gather over equally sized (padded) buffers."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size()
    longest = max(e - b for b, e in ranges)
    pad = torch.zeros((longest,) + tuple(local_rows.shape[1:]), dtype=local_rows.dtype, device=local_rows.device)
    pad[:local_rows.shape[0]] = local_rows
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    full = torch.zeros((total_rows,) + tuple(local_rows.shape[1:]), dtype=local_rows.dtype, device=local_rows.device)
    for (b, e), t in zip(ranges, parts):
        full[b:e] = t[:e - b]
    return full


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
