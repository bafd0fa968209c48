"""GPU parity of the backward pass (dQ, dK, dV) against the oracle's fp64 gradients.

Tolerances: the gradients are bf16 and the kernel feeds bf16 probabilities / dS to the tensor
cores, so every product carries a relative error of about 2^-9; with magnitudes that vary by
orders between rows the bound is relative to the tensor's scale:
max |err| <= 2e-2 * max |ref| + 1e-5 and mean |err| <= 1e-2 * mean |ref| + 1e-5."""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    ksa_build.build()
    c = ksa.Context(0)
    yield c
    c.close()


def _check(name, got, ref):
    assert np.isfinite(got).all(), name
    err = np.abs(got - ref)
    # 1e-5: floor for gradients that are exactly zero (a row with a single visible key has dS = 0)
    assert err.max() <= 2e-2 * np.abs(ref).max() + 1e-5, (name, err.max(), np.abs(ref).max())
    assert err.mean() <= 1e-2 * np.abs(ref).mean() + 1e-5, (name, err.mean(), np.abs(ref).mean())


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D,flags", [
    ([300, 77], 8, 1, 2, 4, 2, 128, 0),
    ([1000], 8, 1, 16, 8, 2, 128, 0),                 # several summary tiles, G = 4
    ([520, 130], 3, 2, 5, 6, 2, 64, 0),               # k does not divide the tile, m = 2, G = 3, D = 64
    ([700], 16, 0, 7, 4, 4, 128, 0),                  # no summaries
    ([450], 8, 1, 3, 4, 1, 128, ksa.KSA_FLAG_SUMMARY_TEXT_ONLY),
    ([1], 8, 1, 2, 2, 2, 64, 0),
    ([2100, 640], 8, 1, 16, 8, 2, 128, 0),            # several query segments per summary key tile
    ([2500], 64, 8, 4, 4, 2, 128, 0),                 # long chunks with 8 summaries each
    ([600, 9], 8, 1, 0, 4, 2, 128, 0),                # no window beyond the own chunk
    ([900], 8, 1, 1000, 4, 2, 128, 0),                # window longer than the sequence: plain causal attention
    ([5, 130, 64, 1, 257], 8, 1, 4, 8, 1, 128, 0),    # many short sequences, one KV head for 8 query heads
    # whole chunks everywhere: the tensor-core kernels read q, k, v, dout in place (no packed copies)
    ([1024, 264, 8], 8, 1, 4, 4, 2, 128, 0),          # sequences that end inside a 128-row tile
    ([1280], 64, 8, 4, 4, 2, 128, 0),
    ([704, 48], 16, 0, 7, 4, 4, 128, 0),
    ([640], 8, 1, 3, 4, 1, 128, ksa.KSA_FLAG_SUMMARY_TEXT_ONLY),
    ([500], 8, 3, 2, 4, 2, 128, 0),                   # three summaries per chunk: packed streams, 128 % m != 0
    ([400, 136], 8, 1, 2, 4, 4, 128, 0),              # one query head per KV head, with summaries
    # head_dim 64 on the tcgen05 kernels
    ([1000, 300], 8, 1, 16, 8, 2, 64, 0),
    ([2500], 64, 8, 4, 4, 2, 64, 0),
    ([2100, 640], 8, 1, 16, 4, 4, 64, 0),
    ([700], 16, 0, 7, 4, 4, 64, 0),
    ([450], 8, 1, 3, 4, 1, 64, ksa.KSA_FLAG_SUMMARY_TEXT_ONLY),
    ([1024, 264, 8], 8, 1, 4, 4, 2, 64, 0),           # whole chunks: read in place
    ([1280], 64, 8, 4, 4, 2, 64, 0),
    # summary-row gradients on mma.sync tiles (8 <= m G <= 128 query rows per chunk and KV head, 12 < k + m <= 128)
    ([1000, 200], 24, 3, 2, 12, 2, 128, 0),           # 18 rows (a ragged second tile), 27 keys
    ([600], 56, 8, 1, 4, 4, 64, 0),                   # one query head per KV head, head_dim 64
    ([1000], 120, 8, 1, 16, 1, 128, 0),               # the largest block: 128 rows, 128 keys
    ([512, 40], 13, 8, 3, 8, 2, 128, ksa.KSA_FLAG_SUMMARY_TEXT_ONLY),
    ([4096], 64, 8, 16, 32, 4, 128, 0),               # the 64 + 8 layout with eight query heads per KV head
    # the mma.sync kernels (the on-device cross-check of the tcgen05 kernels)
    ([1000], 8, 1, 16, 8, 2, 128, ksa.KSA_FLAG_BWD_MMA_SYNC_KERNELS),
    ([520, 130], 3, 2, 5, 6, 2, 64, ksa.KSA_FLAG_BWD_MMA_SYNC_KERNELS),
    ([1024, 264, 8], 8, 1, 4, 4, 2, 128, ksa.KSA_FLAG_BWD_MMA_SYNC_KERNELS),
])
def test_backward_matches_oracle(ctx, lens, k, m, C, Hq, Hkv, D, flags):
    wl = synth.Workload("bwd", 31, lens, Hq, Hkv, D)
    total = sum(orc.aug_len(n, k, m) for n in lens)
    q, kk, v = synth.make_qkv(wl, total)
    g = torch.Generator("cpu").manual_seed(77)
    dout = torch.randn((total, Hq, D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, D, wl.scale, flags)
    qd, kd, vd, gd = q.to(dev), kk.to(dev), v.to(dev), dout.to(dev)
    out = torch.empty_like(qd); lse = torch.empty((Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out, lse, ws)
    dq = torch.full_like(qd, 7.0); dk = torch.full_like(kd, 7.0); dv = torch.full_like(vd, 7.0)
    wsb = torch.full((ksa.bwd_workspace_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)    # NaN patterns
    for _ in range(2):                          # twice: the accumulators must be cleared by the call itself
        ctx.attn_bwd(prob, qd, kd, vd, out, lse, gd, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    oflags = orc.SUMMARY_TEXT_ONLY if (flags & ksa.KSA_FLAG_SUMMARY_TEXT_ONLY) else 0
    rdq, rdk, rdv = orc.bwd(synth.bits(q), synth.bits(kk), synth.bits(v), synth.bits(dout), lens, k, m, C, wl.scale, oflags)
    _check("dq", dq.double().cpu().numpy(), rdq)
    _check("dk", dk.double().cpu().numpy(), rdk)
    _check("dv", dv.double().cpu().numpy(), rdv)


@pytest.mark.parametrize("workload", ["32k", "128k", "varlen"])
def test_backward_full_size_identities(ctx, workload):
    """Full-size workloads, in the launch configuration the bench times: two identities that hold for the exact
    gradients at any size and involve every element of dq, dk and dv.

    (a) The scores only see q k^T, so scaling q by t and k by 1/t changes nothing: d/dt at t = 1 gives
        sum <q, dq> = sum <k, dk> over the rows and the query heads of every KV head.
    (b) out is linear in v: sum <v, dv> = sum <out, dout> over the rows and the query heads of every KV head.
    Both sides are sums of terms of either sign; bf16 gradients (relative error about 2^-9 per element, random
    sign) keep the difference far below 2e-3 of the sum of the absolute terms."""
    wl = synth.WORKLOADS[workload]
    lay = synth.LAYOUT_P
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(wl.text_lens, lay.k, lay.m, lay.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    total = ksa.total_aug_len(prob)
    q, kk, v = synth.make_qkv(wl, total)
    qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
    g = torch.Generator("cpu").manual_seed(5)
    gd = torch.randn((total, wl.Hq, wl.D), generator=g, dtype=torch.float32).to(torch.bfloat16).to(dev)
    out = torch.empty_like(qd); lse = torch.empty((wl.Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out, lse, ws)
    dq = torch.full_like(qd, 7.0); dk = torch.full_like(kd, 7.0); dv = torch.full_like(vd, 7.0)
    wsb = torch.full((ksa.bwd_workspace_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)
    ctx.attn_bwd(prob, qd, kd, vd, out, lse, gd, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for t in (dq, dk, dv):
        assert torch.isfinite(t.float()).all()
    G = wl.Hq // wl.Hkv

    def per_kv_head(a, b, heads_per_kv):       # sum over rows and elements of a * b, and of |a * b|, per KV head
        prod = (a.double() * b.double()).sum(dim=2)                        # [rows, heads]
        absum = (a.double() * b.double()).abs().sum(dim=2)
        prod = prod.sum(dim=0).reshape(wl.Hkv, heads_per_kv).sum(dim=1)
        absum = absum.sum(dim=0).reshape(wl.Hkv, heads_per_kv).sum(dim=1)
        return prod.cpu().numpy(), absum.cpu().numpy()

    qdq, qabs = per_kv_head(qd, dq, G)
    kdk, kabs = per_kv_head(kd, dk, 1)
    vdv, vabs = per_kv_head(vd, dv, 1)
    odo, oabs = per_kv_head(out, gd, G)
    assert (np.abs(qdq - kdk) <= 2e-3 * (qabs + kabs)).all(), (qdq, kdk, qabs)
    assert (np.abs(vdv - odo) <= 2e-3 * (vabs + oabs)).all(), (vdv, odo, vabs)
    # the identities are not met by zeros only: the gradients have their expected size
    assert (qabs > 0).all() and (vabs > 0).all()


def _aug_of_text(n, k, m, i):
    J = n // k
    return (i // k) * (k + m) + i % k if i < J * k else J * (k + m) + (i - J * k)


def _check_rows(name, got, ref):
    """Sampled rows: the same bounds as _check, with each tensor's scale taken from the sample."""
    assert np.isfinite(got).all(), name
    err = np.abs(got - ref)
    assert err.max() <= 2e-2 * np.abs(ref).max() + 1e-5, (name, err.max(), np.abs(ref).max())
    assert err.mean() <= 1e-2 * np.abs(ref).mean() + 1e-5, (name, err.mean(), np.abs(ref).mean())
    # row by row as well: a row that is wrong as a whole must not hide behind the sample's largest row
    rerr = err.reshape(err.shape[0], -1).max(axis=1)
    rref = np.abs(ref).reshape(ref.shape[0], -1).max(axis=1)
    assert (rerr <= 4e-2 * rref + 2e-2 * np.abs(ref).max() * 0.05 + 1e-5).all(), (name, rerr, rref)


@pytest.mark.parametrize("workload", ["32k", "128k", "varlen"])
def test_backward_full_size_sampled_rows(ctx, workload):
    """Full-size workloads in the launch configuration the bench times, element by element on sampled rows against
    the oracle's fp64 gradients (ksa_oracle_bwd_rows: dq of a row needs that row only; dk, dv of a key need every
    query row that sees it under Eq. 3, each with its complete softmax).

    Query rows: first and last rows, rows either side of tile and window boundaries, summary rows, random rows.
    Key rows: text keys (first, last, tile edges, random) -- each is seen by the window's ~1,032 query rows, i.e. by
    nine query tiles -- and summary keys.  At 32k a summary key of the first chunks is sampled, which every later
    row sees: 256 query tiles, sixteen accumulation segments of the dK/dV kernel, four query heads per KV head.
    At 128k and in the long sequences of varlen the sampled summary keys are late ones (seen by the last few
    thousand rows: two segments), because the oracle needs the complete softmax of every row that sees a sampled
    key; there the early keys stay covered by the sum identities of the test above."""
    wl = synth.WORKLOADS[workload]
    lay = synth.LAYOUT_P
    k, m, C = lay.k, lay.m, lay.C
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(wl.text_lens, k, m, C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    total = ksa.total_aug_len(prob)
    q, kk, v = synth.make_qkv(wl, total)
    qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
    g = torch.Generator("cpu").manual_seed(5)
    dout = torch.randn((total, wl.Hq, wl.D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    gd = dout.to(dev)
    out = torch.empty_like(qd); lse = torch.empty((wl.Hq, total), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out, lse, ws)
    dq = torch.full_like(qd, 7.0); dk = torch.full_like(kd, 7.0); dv = torch.full_like(vd, 7.0)
    wsb = torch.full((ksa.bwd_workspace_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)
    ctx.attn_bwd(prob, qd, kd, vd, out, lse, gd, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0

    rng = np.random.default_rng(17)
    q_rows, k_rows = [], []
    base = 0
    lens = list(wl.text_lens)
    # which sequences get key samples: all at 32k, the one sequence at 128k, the shortest and the longest of varlen
    key_seqs = set(range(len(lens))) if len(lens) <= 2 else {int(np.argmin(lens)), int(np.argmax(lens))}
    for b, n in enumerate(lens):
        L = orc.aug_len(n, k, m)
        J = n // k
        text = [0, 1, 127, 128, C * k - 1, C * k + k, n // 2, n - 129, n - 2, n - 1] + [int(t) for t in rng.integers(0, n, size=4)]
        text = sorted(set(min(max(t, 0), n - 1) for t in text))
        q_rows += [base + _aug_of_text(n, k, m, t) for t in text]
        q_rows += [base + j * (k + m) + k for j in (0, J // 2, J - 1)]              # summary rows
        if b in key_seqs:
            tk = [0, 127, 128, n - 1, n - 130] + [int(t) for t in rng.integers(0, n, size=3)]
            k_rows += [base + _aug_of_text(n, k, m, min(max(t, 0), n - 1)) for t in sorted(set(tk))]
            late = [J - 1, J - C - 2, J - C - 2 - 200]                                # seen by nobody / few / ~1,600 text rows
            early = [1] if n <= 40000 else []                                        # seen by nearly every row
            k_rows += [base + j * (k + m) + k for j in late + early if 0 <= j < J]
        base += L
    q_rows = np.unique(np.asarray(q_rows, dtype=np.int64))
    k_rows = np.unique(np.asarray(k_rows, dtype=np.int64))
    rdq, rdk, rdv = orc.bwd_rows(synth.bits(q), synth.bits(kk), synth.bits(v), synth.bits(dout), lens, k, m, C, wl.scale,
                                 q_rows, k_rows)
    tq = torch.from_numpy(q_rows).to(dev); tk_ = torch.from_numpy(k_rows).to(dev)
    _check_rows("dq", dq[tq].double().cpu().numpy(), rdq)
    _check_rows("dk", dk[tk_].double().cpu().numpy(), rdk)
    _check_rows("dv", dv[tk_].double().cpu().numpy(), rdv)


def test_full_causal_mode_against_torch_attention(ctx):
    """m = 0 and a window that covers every chunk reduce the operator to plain causal attention: forward and
    backward against torch's scaled_dot_product_attention and autograd in fp32 on the same bf16 inputs (a library
    routine, at a size the CPU oracle would need minutes for)."""
    n, k, Hq, Hkv, D = 4096, 8, 8, 2, 128
    G = Hq // Hkv
    dev = torch.device("cuda", 0)
    wl = synth.Workload("causal", 51, [n], Hq, Hkv, D)
    prob = ksa.Problem([n], k, 0, 1 << 20, Hq, Hkv, D, wl.scale, 0)
    q, kk, v = synth.make_qkv(wl, n)
    g = torch.Generator("cpu").manual_seed(52)
    dout = torch.randn((n, Hq, D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    qd, kd, vd, gd = q.to(dev), kk.to(dev), v.to(dev), dout.to(dev)
    out = torch.empty_like(qd); lse = torch.empty((Hq, n), dtype=torch.float32, device=dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out, lse, ws)
    dq = torch.empty_like(qd); dk = torch.empty_like(kd); dv = torch.empty_like(vd)
    wsb = torch.empty(ksa.bwd_workspace_bytes(prob), dtype=torch.uint8, device=dev)
    ctx.attn_bwd(prob, qd, kd, vd, out, lse, gd, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    # reference: [heads, n, D] in fp32, K / V heads repeated over their group
    qr = qd.float().transpose(0, 1).contiguous().requires_grad_(True)
    kr = kd.float().transpose(0, 1).contiguous().requires_grad_(True)
    vr = vd.float().transpose(0, 1).contiguous().requires_grad_(True)
    from torch.nn.attention import SDPBackend, sdpa_kernel
    with sdpa_kernel(SDPBackend.MATH):
        ref = torch.nn.functional.scaled_dot_product_attention(
            qr[None], kr.repeat_interleave(G, dim=0)[None], vr.repeat_interleave(G, dim=0)[None],
            is_causal=True, scale=wl.scale)[0]
    ref.backward(gd.float().transpose(0, 1))
    got = out.float().transpose(0, 1)
    assert (got - ref.detach()).abs().max().item() <= 2e-2
    assert (got - ref.detach()).abs().mean().item() <= 2e-3
    # natural-log LSE of the scaled scores over the visible keys, by torch
    scores = torch.einsum("hid,hjd->hij", qr.detach(), kr.detach().repeat_interleave(G, dim=0)) * wl.scale
    scores = scores.masked_fill(torch.ones(n, n, dtype=torch.bool, device=dev).triu(1), float("-inf"))
    lse_ref = torch.logsumexp(scores, dim=2)
    assert ((lse - lse_ref).abs() <= 1e-3 * lse_ref.abs().clamp(min=1.0)).all()
    for name, mine, theirs in (("dq", dq, qr.grad), ("dk", dk, kr.grad), ("dv", dv, vr.grad)):
        err = (mine.float().transpose(0, 1) - theirs).abs()
        assert err.max().item() <= 2e-2 * theirs.abs().max().item() + 1e-5, name
        assert err.mean().item() <= 1e-2 * theirs.abs().mean().item() + 1e-5, name
