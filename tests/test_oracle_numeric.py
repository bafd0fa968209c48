"""Pins for the oracle's numeric path (masked softmax attention, LSE, GQA).  CPU only."""
import itertools

import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from tests.helpers import (aug_positions, bf16_bits_to_f64, dense_attention, dense_mask,
                           rand_bf16)


def _inputs(rng, L, Hq, Hkv, D, qs=1.0):
    qb, q = rand_bf16(rng, (L, Hq, D), qs)
    kb, k = rand_bf16(rng, (L, Hkv, D))
    vb, v = rand_bf16(rng, (L, Hkv, D))
    return (qb, kb, vb), (q, k, v)


def test_causal_reduction_vs_torch_sdpa():
    """With C >= number of chunks no summary is ever visible to text, and the text
    rows are ordinary causal attention over the text-only subsequence: compare with
    torch's scaled_dot_product_attention(is_causal=True) in fp64, GQA 4/2."""
    rng = np.random.default_rng(10)
    n, k, m, C, Hq, Hkv, D = 96, 8, 1, 12, 4, 2, 16
    tp, sp, L = aug_positions(n, k, m)
    (qb, kb, vb), (q, kk, v) = _inputs(rng, L, Hq, Hkv, D)
    scale = 1.0 / np.sqrt(D)
    out, lse, cnt = orc.fwd(qb, kb, vb, [n], k, m, C, scale)
    text = np.array([tp[i] for i in range(n)])
    qt = torch.from_numpy(q[text]).permute(1, 0, 2)[None]                  # [1,Hq,n,D]
    kt = torch.from_numpy(kk[text]).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    vt = torch.from_numpy(v[text]).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(out[text] - ref).max() < 1e-12
    s = scale * torch.einsum("hid,hjd->hij", qt[0], kt[0])
    s = s.masked_fill(~torch.tril(torch.ones(n, n, dtype=torch.bool)), float("-inf"))
    ref_lse = torch.logsumexp(s, dim=-1).T.numpy()
    assert np.abs(lse[text] - ref_lse).max() < 1e-12
    assert (cnt[text] == np.arange(1, n + 1)).all()


def test_sliding_window_reduction():
    """m = 0, k = 1 turns Eq. 2 into a token-level sliding window of width C + 1."""
    rng = np.random.default_rng(11)
    n, C, H, D = 50, 6, 2, 8
    (qb, kb, vb), (q, kk, v) = _inputs(rng, n, H, H, D)
    out, lse, cnt = orc.fwd(qb, kb, vb, [n], 1, 0, C, 0.3)
    i = np.arange(n)
    band = (i[None, :] <= i[:, None]) & (i[None, :] >= i[:, None] - C)
    ref, ref_lse = dense_attention(q, kk, v, band, 0.3)
    assert np.abs(out - ref).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-12
    assert (cnt == np.minimum(i, C) + 1).all()


@pytest.mark.parametrize("text_only", [False, True])
def test_brute_force_dense(text_only):
    """Tiny inputs, every (k, m, C) of a small grid and ragged tails: the oracle equals
    a dense-mask softmax written separately; the softmax weights of a row sum to 1
    (checked through V = all-ones => out = 1)."""
    rng = np.random.default_rng(12)
    flags = orc.SUMMARY_TEXT_ONLY if text_only else 0
    for k, m, C in itertools.product([1, 2, 3, 8], [0, 1, 3], [0, 1, 4]):
        for n in (k, 4 * k + (k // 2), 37):
            mask = dense_mask(n, k, m, C, text_only)
            L = mask.shape[0]
            (qb, kb, vb), (q, kk, v) = _inputs(rng, L, 4, 2, 8, qs=2.0)
            out, lse, cnt = orc.fwd(qb, kb, vb, [n], k, m, C, 0.5, flags)
            ref, ref_lse = dense_attention(q, kk, v, mask, 0.5, G=2)
            assert np.abs(out - ref).max() < 1e-12, (n, k, m, C)
            assert np.abs(lse - ref_lse).max() < 1e-12
            assert (cnt == mask.sum(1)).all()
            ones = np.full_like(vb, 0x3F80)           # bf16 1.0
            out1, _, _ = orc.fwd(qb, kb, ones, [n], k, m, C, 0.5, flags)
            assert np.abs(out1 - 1.0).max() < 1e-14


def test_zero_query_gives_log_count_and_mean():
    """Q = 0 => every visible score is 0: lse = ln(count), out = mean of visible V."""
    rng = np.random.default_rng(13)
    n, k, m, C, H, D = 70, 8, 2, 2, 2, 8
    mask = dense_mask(n, k, m, C)
    L = mask.shape[0]
    (qb, kb, vb), (q, kk, v) = _inputs(rng, L, H, H, D)
    qb[:] = 0
    out, lse, cnt = orc.fwd(qb, kb, vb, [n], k, m, C, 1.0)
    assert np.abs(lse - np.log(mask.sum(1))[:, None]).max() < 1e-13
    for h in range(H):
        mean = (mask.astype(np.float64) @ v[:, h, :]) / mask.sum(1, keepdims=True)
        assert np.abs(out[:, h, :] - mean).max() < 1e-13


def test_perturbation_invariance_and_packing():
    """Changing K/V at invisible positions, or in another packed sequence, leaves the
    result bit-identical; a packed batch equals its sequences run one by one."""
    rng = np.random.default_rng(14)
    lens, k, m, C, Hq, Hkv, D = [45, 23, 64], 8, 1, 1, 4, 2, 8
    Ls = [orc.aug_len(n, k, m) for n in lens]
    tot = sum(Ls)
    (qb, kb, vb), _ = _inputs(rng, tot, Hq, Hkv, D)
    out, lse, _ = orc.fwd(qb, kb, vb, lens, k, m, C, 0.4)
    off = np.concatenate([[0], np.cumsum(Ls)])
    for b, n in enumerate(lens):
        sl = slice(off[b], off[b + 1])
        o1, l1, _ = orc.fwd(qb[sl], kb[sl], vb[sl], [n], k, m, C, 0.4)
        assert (o1 == out[sl]).all() and (l1 == lse[sl]).all()
    # pick a row of sequence 0, scramble everything it cannot see
    row = off[0] + 40
    vis = orc.mask_row(lens[0], k, m, C, 40).astype(bool)
    kb2, vb2 = kb.copy(), vb.copy()
    hidden = np.ones(tot, dtype=bool)
    hidden[: Ls[0]][vis] = False
    kb2[hidden] = rand_bf16(rng, kb2[hidden].shape, 5.0)[0]
    vb2[hidden] = rand_bf16(rng, vb2[hidden].shape, 5.0)[0]
    o2, l2, _ = orc.fwd(qb, kb2, vb2, lens, k, m, C, 0.4, rows=[row])
    assert (o2[0] == out[row]).all() and (l2[0] == lse[row]).all()
    # and a visible key does matter
    kb3 = kb.copy()
    kb3[np.nonzero(vis)[0][0]] ^= 0x8000
    o3, _, _ = orc.fwd(qb, kb3, vb, lens, k, m, C, 0.4, rows=[row])
    assert not (o3[0] == out[row]).all()


def test_merge_identity():
    """Attention over the summary set and over the text band computed separately and
    merged through their LSEs equals the joint result (what a two-part kernel uses)."""
    rng = np.random.default_rng(15)
    n, k, m, C, H, D = 64, 4, 1, 2, 2, 8
    tp, sp, L = aug_positions(n, k, m)
    mask = dense_mask(n, k, m, C)
    (qb, kb, vb), (q, kk, v) = _inputs(rng, L, H, H, D)
    out, lse, _ = orc.fwd(qb, kb, vb, [n], k, m, C, 0.5)
    is_sum = np.zeros(L, dtype=bool)
    is_sum[list(sp.values())] = True
    for i in range(4 * k, n):                # rows that see at least one summary
        p = tp[i]
        ms = (mask[p] & is_sum)[None, :].repeat(L, 0)
        mt = (mask[p] & ~is_sum)[None, :].repeat(L, 0)
        o_s, l_s = dense_attention(q, kk, v, ms, 0.5)
        o_t, l_t = dense_attention(q, kk, v, mt, 0.5)
        l_joint = np.logaddexp(l_s[p], l_t[p])
        o_joint = (np.exp(l_s[p] - l_joint)[:, None] * o_s[p] + np.exp(l_t[p] - l_joint)[:, None] * o_t[p])
        assert np.abs(o_joint - out[p]).max() < 1e-12
        assert np.abs(l_joint - lse[p]).max() < 1e-12


def test_peaked_scores_stay_finite():
    """Large score magnitudes (|x| ~ 1e3) must not overflow: the max is subtracted."""
    rng = np.random.default_rng(16)
    n, k, m, C, H, D = 32, 4, 1, 1, 1, 8
    L = orc.aug_len(n, k, m)
    (qb, kb, vb), (q, kk, v) = _inputs(rng, L, H, H, D, qs=60.0)
    out, lse, _ = orc.fwd(qb, kb, vb, [n], k, m, C, 8.0)
    ref, ref_lse = dense_attention(q, kk, v, dense_mask(n, k, m, C), 8.0)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    assert np.abs(out - ref).max() < 1e-10
    assert np.abs(lse - ref_lse).max() < 1e-9


def test_rows_subset_matches_full():
    rng = np.random.default_rng(17)
    lens, k, m, C = [30, 50], 8, 1, 1
    tot = sum(orc.aug_len(n, k, m) for n in lens)
    (qb, kb, vb), _ = _inputs(rng, tot, 2, 1, 8)
    out, lse, cnt = orc.fwd(qb, kb, vb, lens, k, m, C, 0.3)
    rows = np.array([0, 5, 33, 34, tot - 1])
    o2, l2, c2 = orc.fwd(qb, kb, vb, lens, k, m, C, 0.3, rows=rows)
    assert (o2 == out[rows]).all() and (l2 == lse[rows]).all() and (c2 == cnt[rows]).all()
    with pytest.raises(ValueError):
        orc.fwd(qb, kb, vb, lens, k, m, C, 0.3, rows=[tot])
