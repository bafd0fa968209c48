"""Pins for the oracle's visibility rule (Eq. 1, Eq. 3, summary scope).  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import ksa_oracle as orc
from tests.helpers import aug_positions, dense_mask, visible_sets

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq3_n6_k2.txt")


def _name_to_pos(name, tp, sp):
    return tp[int(name[1:])] if name[0] == "t" else sp[(int(name[1:]), 0)]


def test_hand_fixture_eq3():
    """The worked n=6, k=2 example enumerated by hand from Eq. 3."""
    tp, sp, L = aug_positions(6, 2, 1)
    assert L == 9 and orc.aug_len(6, 2, 1) == 9
    n_lines = 0
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, rest = line.split("|")
        _, C, variant = head.split()
        qname, keys = rest.split(":")
        flags = orc.SUMMARY_TEXT_ONLY if variant == "strict" else 0
        pq = _name_to_pos(qname.strip(), tp, sp)
        want = np.zeros(L, dtype=np.uint8)
        for kn in keys.split():
            want[_name_to_pos(kn, tp, sp)] = 1
        got = orc.mask_row(6, 2, 1, int(C), pq, flags)
        assert got.tolist() == want.tolist(), line
        n_lines += 1
    assert n_lines == 24


def test_augmented_order_eq1():
    """Eq. 1: chunk_j = [t_jk .. t_jk+k-1, s_j]; position decoding round-trips."""
    for n, k, m in [(6, 2, 1), (17, 4, 1), (17, 4, 3), (8, 8, 1), (5, 8, 2), (24, 3, 0)]:
        tp, sp, L = aug_positions(n, k, m)
        assert orc.aug_len(n, k, m) == L == n + (n // k) * m
        for i, p in tp.items():
            assert orc.decode_pos(n, k, m, p) == (False, i, 0)
        for (j, r), p in sp.items():
            assert orc.decode_pos(n, k, m, p) == (True, j, r)
        with pytest.raises(ValueError):
            orc.decode_pos(n, k, m, L)


@pytest.mark.parametrize("text_only", [False, True])
def test_mask_equals_enumerated_sets(text_only):
    """Brute force: the predicate's explicit mask equals the sets Eq. 3 lists, for
    every (k, m, C) with k <= 8, m <= 3, C <= 4 and all tail lengths."""
    flags = orc.SUMMARY_TEXT_ONLY if text_only else 0
    for k, m, C in itertools.product([1, 2, 3, 5, 8], [0, 1, 2, 3], [0, 1, 2, 4]):
        for n in sorted({1, k, 2 * k + 1, 5 * k - 1, 6 * k, min(64, 9 * k + k // 2)}):
            if n < 1:
                continue
            want = dense_mask(n, k, m, C, text_only)
            got = orc.mask(n, k, m, C, flags).astype(bool)
            assert got.shape == want.shape
            assert (got == want).all(), (n, k, m, C)


def _closed_form_text(i, k, m, C):
    c = i // k
    far = max(0, c - C)
    return (i - k * far + 1) + m * far


@pytest.mark.parametrize("n,k,m,C", [(1024, 8, 1, 128), (1024, 8, 1, 2), (1024, 64, 8, 16),
                                      (1024, 64, 8, 2), (1000, 8, 1, 3), (777, 64, 8, 1),
                                      (300, 7, 2, 0), (513, 16, 1, 4)])
def test_closed_form_counts(n, k, m, C):
    """Per-row popcount of the explicit mask equals the closed form implied by the
    chunk layout: text row i: (i - k*max(0,c-C) + 1) + m*max(0,c-C);
    summary row (j, r): k + r + 1 (k under the strict rule)."""
    tp, sp, L = aug_positions(n, k, m)
    for i, p in tp.items():
        assert orc.visible_count(n, k, m, C, p) == _closed_form_text(i, k, m, C)
    for (j, r), p in sp.items():
        assert orc.visible_count(n, k, m, C, p) == k + r + 1
        assert orc.visible_count(n, k, m, C, p, orc.SUMMARY_TEXT_ONLY) == k
    total = sum(_closed_form_text(i, k, m, C) for i in range(n)) + (n // k) * sum(k + r + 1 for r in range(m))
    assert orc.total_pairs([n], k, m, C) == total


def test_workload_pair_totals():
    """Visible pairs per head of the 8K workload (both layouts) by popcount of every
    mask row equal the closed-form sum; packed sequences add up."""
    for k, m, C in [(8, 1, 128), (64, 8, 16)]:
        n = 8192
        i = np.arange(n, dtype=np.int64)
        far = np.maximum(0, i // k - C)
        total = int(((i - k * far + 1) + m * far).sum()) + (n // k) * sum(k + r + 1 for r in range(m))
        assert orc.total_pairs([n], k, m, C) == total
    assert orc.total_pairs([8192], 8, 1, 128) == 11113984  # 1.1114e7 pairs per head
    a = orc.total_pairs([100, 37, 64], 8, 1, 2)
    assert a == sum(orc.total_pairs([x], 8, 1, 2) for x in (100, 37, 64))


def test_partition_property():
    """Every earlier full chunk is either fully visible as text (and none of its
    summaries), or visible only through all of its summaries (Sec. 2.2.2, last
    paragraph): no intermediate state."""
    for n, k, m, C in [(64, 4, 1, 2), (61, 4, 2, 3), (40, 8, 1, 0), (50, 5, 3, 1)]:
        tp, sp, L = aug_positions(n, k, m)
        for i in range(n):
            row = orc.mask_row(n, k, m, C, tp[i])
            for j in range(i // k):
                text_vis = [row[tp[x]] for x in range(j * k, j * k + k)]
                summ_vis = [row[sp[(j, r)]] for r in range(m)]
                all_text = all(text_vis) and not any(summ_vis)
                all_summ = (not any(text_vis)) and all(summ_vis)
                assert all_text != all_summ or m == 0, (n, k, m, C, i, j)
                if m == 0:
                    assert all(text_vis) or not any(text_vis)
            # own chunk: causal prefix, never its own summaries
            c = i // k
            for x in range(c * k, min(n, c * k + k)):
                assert row[tp[x]] == (x <= i)
            for r in range(m):
                if (c, r) in sp:
                    assert row[sp[(c, r)]] == 0


def test_summary_rows_see_only_their_chunk():
    n, k, m, C = 40, 4, 2, 1
    tp, sp, L = aug_positions(n, k, m)
    for (j, r), p in sp.items():
        row = orc.mask_row(n, k, m, C, p)
        want = {tp[x] for x in range(j * k, j * k + k)} | {sp[(j, rr)] for rr in range(r + 1)}
        assert set(np.nonzero(row)[0].tolist()) == want


def test_decode_cache_equivalence():
    """Sec. 2.3.1: at decode step i the cache holds [summary buffer | sliding chunk
    text ring | current chunk]; its contents equal row i's visible set."""
    n, k, m, C = 53, 4, 1, 3
    tp, sp, L = aug_positions(n, k, m)
    summaries, ring, current = [], [], []   # lists of augmented positions
    for i in range(n):
        current.append(tp[i])
        cache = set(summaries) | {x for ch in ring for x in ch} | set(current)
        row = orc.mask_row(n, k, m, C, tp[i])
        assert set(np.nonzero(row)[0].tolist()) == cache, i
        if len(current) == k:                       # chunk filled
            j = i // k
            srow = orc.mask_row(n, k, m, C, sp[(j, 0)])
            assert set(np.nonzero(srow)[0].tolist()) == set(current) | {sp[(j, 0)]}
            ring.append(current)                    # copy chunk into the ring
            current = []
            if len(ring) > C:                       # oldest chunk leaves the window:
                old = ring.pop(0)                   # from now on reached through its summary
                summaries.append(sp[(tp_inv(tp, old[0]) // k, 0)])


def tp_inv(tp, pos):
    for i, p in tp.items():
        if p == pos:
            return i
    raise KeyError(pos)


def test_bad_arguments():
    assert orc.aug_len(-1, 8, 1) == -1
    with pytest.raises(ValueError):
        orc.visible(8, 2, 1, -1, 0, 0)
    with pytest.raises(ValueError):
        orc.visible(8, 2, 1, 1, 0, 99)
