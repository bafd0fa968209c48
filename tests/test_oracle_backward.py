"""Pins of the oracle's backward pass against things other than itself: torch autograd on the
cases that reduce to textbook attention, finite differences through the oracle's FORWARD pass,
a dense-mask numpy restatement, and identities of softmax-attention gradients."""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from tests import helpers


def _rand(seed, total, Hq, Hkv, D, scale=1.0):
    rng = np.random.default_rng(seed)
    qb, q = helpers.rand_bf16(rng, (total, Hq, D), scale)
    kb, k = helpers.rand_bf16(rng, (total, Hkv, D), scale)
    vb, v = helpers.rand_bf16(rng, (total, Hkv, D), scale)
    gb, g = helpers.rand_bf16(rng, (total, Hq, D), scale)
    return (qb, kb, vb, gb), (q, k, v, g)


def test_causal_reduction_against_torch_autograd():
    """No summaries, window wider than the sequence: plain causal attention, whose gradients torch
    computes by automatic differentiation of its own softmax (fp64, grouped heads)."""
    n, Hq, Hkv, D, scale = 45, 4, 2, 16, 0.3
    bits, (q, k, v, g) = _rand(1, n, Hq, Hkv, D)
    dq, dk, dv = orc.bwd(*bits, [n], 8, 0, 100, scale)
    tq = torch.tensor(q, requires_grad=True); tk = torch.tensor(k, requires_grad=True); tv = torch.tensor(v, requires_grad=True)
    kk = tk.repeat_interleave(Hq // Hkv, dim=1); vv = tv.repeat_interleave(Hq // Hkv, dim=1)
    s = torch.einsum("ihd,jhd->hij", tq, kk) * scale
    s = s.masked_fill(~torch.tril(torch.ones(n, n, dtype=torch.bool)), float("-inf"))
    o = torch.einsum("hij,jhd->ihd", torch.softmax(s, dim=-1), vv)
    (o * torch.tensor(g)).sum().backward()
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("n,k,m,C,flags", [(37, 4, 1, 2, 0), (50, 8, 2, 1, 0), (29, 3, 1, 0, orc.SUMMARY_TEXT_ONLY)])
def test_dense_mask_restatement_with_torch_autograd(n, k, m, C, flags):
    """The KSA mask enumerated independently (tests/helpers.py writes the visible sets of Eq. 3 out as
    lists), dense masked attention differentiated by torch autograd, packed batch of two sequences."""
    Hq, Hkv, D, scale = 2, 1, 8, 0.4
    lens = [n, n - 5]
    Ls = [orc.aug_len(x, k, m) for x in lens]
    bits, (q, kk, v, g) = _rand(2, sum(Ls), Hq, Hkv, D)
    dq, dk, dv = orc.bwd(*bits, lens, k, m, C, scale, flags)
    tq = torch.tensor(q, requires_grad=True); tk = torch.tensor(kk, requires_grad=True); tv = torch.tensor(v, requires_grad=True)
    loss = 0.0
    off = 0
    for x, L in zip(lens, Ls):
        M = torch.tensor(helpers.dense_mask(x, k, m, C, text_only=bool(flags)))
        s = torch.einsum("ihd,jhd->hij", tq[off:off + L], tk[off:off + L].repeat_interleave(Hq, dim=1)) * scale
        p = torch.softmax(s.masked_fill(~M, float("-inf")), dim=-1)
        o = torch.einsum("hij,jhd->ihd", p, tv[off:off + L].repeat_interleave(Hq, dim=1))
        loss = loss + (o * torch.tensor(g[off:off + L])).sum()
        off += L
    loss.backward()
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_finite_differences_through_the_oracle_forward():
    """d/dx sum(out * dO) by central differences of the oracle's own forward pass, on inputs moved by
    whole bf16 steps so that both evaluations are exact bf16 inputs."""
    n, k, m, C, Hq, Hkv, D, scale = 40, 4, 1, 2, 4, 2, 8, 0.35
    L = orc.aug_len(n, k, m)
    (qb, kb, vb, gb), (q, kk, v, g) = _rand(3, L, Hq, Hkv, D)
    dq, dk, dv = orc.bwd(qb, kb, vb, gb, [n], k, m, C, scale)

    def loss(qb_, kb_, vb_):
        out, _, _ = orc.fwd(qb_, kb_, vb_, [n], k, m, C, scale)
        return float((out * g).sum())

    rng = np.random.default_rng(4)
    for which, grad, arr in (("q", dq, qb), ("k", dk, kb), ("v", dv, vb)):
        for _ in range(6):
            idx = tuple(int(rng.integers(0, s)) for s in arr.shape)
            steps = 8                                   # 8 bf16 ulps each way: h is about 3 % of |x|
            hi, lo = arr.copy(), arr.copy()
            hi[idx] = arr[idx] + steps; lo[idx] = arr[idx] - steps      # same sign and exponent for these draws
            x_hi = helpers.bf16_bits_to_f64(np.array([hi[idx]], dtype=np.uint16))[0]
            x_lo = helpers.bf16_bits_to_f64(np.array([lo[idx]], dtype=np.uint16))[0]
            args_hi = {"q": (hi, kb, vb), "k": (qb, hi, vb), "v": (qb, kb, hi)}[which]
            args_lo = {"q": (lo, kb, vb), "k": (qb, lo, vb), "v": (qb, kb, lo)}[which]
            fd = (loss(*args_hi) - loss(*args_lo)) / (x_hi - x_lo)
            assert abs(fd - grad[idx]) <= 2e-3 * max(1.0, abs(grad[idx])) + 2e-3 * np.abs(grad).max(), (which, idx, fd, grad[idx])


def test_gradient_identities():
    """sum_i <q_i, dq_i> = sum_j <k_j, dk_j> (the scores depend on q and k through their products only);
    sum_j dv_j = sum over rows and the heads of the group of dO (softmax rows sum to one); keys no row
    can see keep zero gradients; sequences of a packed batch do not mix."""
    lens, k, m, C, Hq, Hkv, D, scale = [33, 20], 4, 1, 1, 4, 2, 8, 0.5
    Ls = [orc.aug_len(x, k, m) for x in lens]
    (qb, kb, vb, gb), (q, kk, v, g) = _rand(5, sum(Ls), Hq, Hkv, D)
    dq, dk, dv = orc.bwd(qb, kb, vb, gb, lens, k, m, C, scale)
    assert abs((q * dq).sum() - (kk * dk).sum()) < 1e-9 * max(1.0, np.abs(q * dq).sum())
    G = Hq // Hkv
    np.testing.assert_allclose(dv.sum(axis=0), g.reshape(sum(Ls), Hkv, G, D).sum(axis=(0, 2)), rtol=1e-10, atol=1e-12)
    # the trailing summary of a sequence (last full chunk's summary) is seen by itself only (self-visible rule):
    # its dk is the self term alone, and under the strict rule exactly zero
    dq2, dk2, dv2 = orc.bwd(qb, kb, vb, gb, lens, k, m, C, scale, orc.SUMMARY_TEXT_ONLY)
    last_summ = (lens[0] // k) * (k + m) - 1
    assert np.all(dk2[last_summ] == 0) and np.all(dv2[last_summ] == 0)
    # isolation: gradients of sequence 0 do not change when sequence 1's inputs change
    qb3, kb3, vb3 = qb.copy(), kb.copy(), vb.copy()
    qb3[Ls[0]:] ^= 0x0101; kb3[Ls[0]:] ^= 0x0101; vb3[Ls[0]:] ^= 0x0101
    dq3, dk3, dv3 = orc.bwd(qb3, kb3, vb3, gb, lens, k, m, C, scale)
    assert np.array_equal(dq3[:Ls[0]], dq[:Ls[0]]) and np.array_equal(dk3[:Ls[0]], dk[:Ls[0]]) and np.array_equal(dv3[:Ls[0]], dv[:Ls[0]])


def test_sampled_rows_equal_the_full_gradients():
    """ksa_oracle_bwd_rows (the gradients of a sample of rows, used where the full computation is too long) returns
    exactly the corresponding rows of ksa_oracle_bwd, whose arithmetic the tests above pin: packed sequences, GQA,
    ragged tail, keys that are text and keys that are summaries, rows in every sequence."""
    rng = np.random.default_rng(3)
    lens, k, m, C, Hq, Hkv, D = [70, 33, 9], 4, 2, 3, 4, 2, 8
    total = sum(orc.aug_len(n, k, m) for n in lens)
    rand_bf16 = helpers.rand_bf16
    qb, _ = rand_bf16(rng, (total, Hq, D))
    kb, _ = rand_bf16(rng, (total, Hkv, D))
    vb, _ = rand_bf16(rng, (total, Hkv, D))
    gb, _ = rand_bf16(rng, (total, Hq, D))
    dq, dk, dv = orc.bwd(qb, kb, vb, gb, lens, k, m, C, 0.35)
    q_rows = np.array([0, 3, 5, 17, 60, total - 1, orc.aug_len(70, k, m), orc.aug_len(70, k, m) + 20], dtype=np.int64)
    k_rows = np.array([0, 4, 5, 11, 40, 104, 105 + 7, total - 2], dtype=np.int64)     # rows 4, 5, 11: summaries of sequence 0
    sq, sk, sv = orc.bwd_rows(qb, kb, vb, gb, lens, k, m, C, 0.35, q_rows, k_rows)
    np.testing.assert_allclose(sq, dq[q_rows], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(sk, dk[k_rows], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(sv, dv[k_rows], rtol=1e-12, atol=1e-14)
    assert np.abs(sk).max() > 0 and np.abs(sq).max() > 0
    # the strict summary rule goes through the same predicate
    dq2, dk2, dv2 = orc.bwd(qb, kb, vb, gb, lens, k, m, C, 0.35, orc.SUMMARY_TEXT_ONLY)
    sq2, sk2, sv2 = orc.bwd_rows(qb, kb, vb, gb, lens, k, m, C, 0.35, q_rows, k_rows, orc.SUMMARY_TEXT_ONLY)
    np.testing.assert_allclose(sq2, dq2[q_rows], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(sk2, dk2[k_rows], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(sv2, dv2[k_rows], rtol=1e-12, atol=1e-14)
