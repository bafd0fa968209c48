"""The N > 1 host logic under a real process group: two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import dist_utils, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, lens, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shards = dist_utils.shard_sequences(lens, 8, 1, 128, world)
        mine = shards[rank]
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        # every rank computed the same table, and the shards tile the batch
        assert gathered == shards
        assert sorted(i for s in gathered for i in s) == list(range(len(lens)))
        # timing rule: the slowest rank decides
        t = dist_utils.max_over_ranks(10.0 + rank)
        assert t == 10.0 + (world - 1)
        wl = dist_utils.rank_workload(synth.WORKLOADS["tiny"], rank)
        seeds = [None] * world
        dist.all_gather_object(seeds, wl.seed)
        assert len(set(seeds)) == world
        rate = dist_utils.aggregate_rate(100.0, world, t)
        assert abs(rate - world * 100.0 / (t * 1e-3)) < 1e-6
        ret[rank] = "ok"
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_time():
    lens = synth.varlen_text_lens()
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, port, lens, ret), nprocs=2, join=True)
    assert dict(ret) == {0: "ok", 1: "ok"}


def test_sequence_cost_is_the_oracle_pair_count():
    for n, k, m, C in [(100, 8, 1, 2), (37, 4, 2, 0), (513, 64, 8, 1), (64, 8, 0, 3)]:
        L = orc.aug_len(n, k, m)
        want = sum(orc.visible_count(n, k, m, C, p) for p in range(L))
        assert dist_utils.visible_pairs_of_sequence(n, k, m, C) == want


def test_shards_are_balanced_and_head_ranges_tile():
    lens = synth.varlen_text_lens()
    cost = [dist_utils.visible_pairs_of_sequence(n, 8, 1, 128) for n in lens]
    for world in (1, 2, 4, 8):
        shards = dist_utils.shard_sequences(lens, 8, 1, 128, world)
        loads = [sum(cost[i] for i in s) for s in shards]
        assert sum(loads) == sum(cost)
        assert max(loads) - min(loads) <= max(cost)          # longest-first never does worse than one item
        ranges = dist_utils.shard_kv_heads(8, world)
        assert [h for r in ranges for h in r] == list(range(8))
