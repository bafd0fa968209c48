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


def _split_rows_by_work(n, k, m, C, world):
    """Contiguous augmented row ranges of about equal visible pairs (what the library's ksa_part_rows does at tile
    granularity; here row by row, for the CPU test)."""
    L = orc.aug_len(n, k, m)
    cost = [dist_utils.visible_pairs_of_rows(n, k, m, C, a, a + 1) for a in range(L)]
    total, acc, cuts = sum(cost), 0, [0]
    for a, c in enumerate(cost):
        acc += c
        while len(cuts) < world and acc * world >= total * len(cuts):
            cuts.append(a + 1)
    cuts += [L] * (world + 1 - len(cuts))
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def _seq_parallel_worker(rank, world, port, ret):
    """Sequence-parallel forward over gloo: every rank owns a part of the rows of one sequence, contributes its rows
    of k and v to an all-gather, computes its own query rows (here with the oracle standing in for the kernel:
    it only reads k, v rows before the part's end) and the parts together equal the whole."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n, k, m, C, Hq, Hkv, D = 150, 8, 1, 3, 2, 1, 16
        wl = synth.Workload("sp", 5, [n], Hq, Hkv, D)
        L = orc.aug_len(n, k, m)
        q, kk, v = synth.make_qkv(wl, L)                     # every rank draws the same tensors ...
        ranges = _split_rows_by_work(n, k, m, C, world)
        b, e = ranges[rank]
        k_full = dist_utils.all_gather_rows(kk[b:e].clone(), ranges, L)     # ... but only contributes its own rows
        v_full = dist_utils.all_gather_rows(v[b:e].clone(), ranges, L)
        assert torch.equal(k_full, kk) and torch.equal(v_full, v)
        # what the rank may look at: its own q rows, k and v before the end of its part (Eq. 3)
        need = dist_utils.kv_rows_needed(e)
        k_loc, v_loc = torch.zeros_like(kk), torch.zeros_like(v)
        k_loc[need.start:need.stop] = k_full[need.start:need.stop]
        v_loc[need.start:need.stop] = v_full[need.start:need.stop]
        rows = list(range(b, e))
        out_part, lse_part, _ = orc.fwd(synth.bits(q), synth.bits(k_loc), synth.bits(v_loc), [n], k, m, C, wl.scale, rows=rows)
        out_ref, lse_ref, _ = orc.fwd(synth.bits(q), synth.bits(kk), synth.bits(v), [n], k, m, C, wl.scale, rows=rows)
        assert (out_part == out_ref).all() and (lse_part == lse_ref).all()
        # the parts tile the rows and carry about the same work
        work = [dist_utils.visible_pairs_of_rows(n, k, m, C, x, y) for x, y in ranges]
        assert sum(work) == dist_utils.visible_pairs_of_sequence(n, k, m, C)
        assert ranges[0][0] == 0 and ranges[-1][1] == L and all(r0[1] == r1[0] for r0, r1 in zip(ranges, ranges[1:]))
        assert max(work) <= 1.25 * sum(work) / world
        ret[rank] = "ok"
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_sequence_parallel_exchange():
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_seq_parallel_worker, args=(2, port, ret), nprocs=2, join=True)
    assert dict(ret) == {0: "ok", 1: "ok"}


def test_row_costs_add_up_to_the_oracle_pair_count():
    for n, k, m, C in [(100, 8, 1, 2), (37, 4, 2, 0), (130, 64, 8, 1)]:
        L = orc.aug_len(n, k, m)
        for a in (0, 1, L // 2, L - 1):
            assert dist_utils.visible_pairs_of_rows(n, k, m, C, a, a + 1) == orc.visible_count(n, k, m, C, a)
        assert dist_utils.visible_pairs_of_rows(n, k, m, C, 0, L) == dist_utils.visible_pairs_of_sequence(n, k, m, C)


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` outside torchrun starts two ranks of itself (here with the stand-in step over gloo: no
    GPU in this test), the slower rank sets the time and rank 0 alone prints one line with n_gpus = 2."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["KSA_BENCH_LAUNCH_TEST"] = "1"
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "5", "--warmup", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    assert lines[0]["n_gpus"] == 2 and lines[0]["built_by_launcher"]
    assert lines[0]["ms_per_step"] >= 2.0           # rank 1 sleeps 2 ms per step: the MAX over ranks


def test_bench_gpus_flag_fails_loudly_without_enough_gpus():
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "KSA_BENCH_LAUNCH_TEST")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "64", "--steps", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode != 0
    assert "GPU" in (r.stderr + r.stdout) or "CUDA" in (r.stderr + r.stdout)
