"""Decode path (Summary KV cache, Sec. 2.3.1): host-side slice arithmetic on CPU, and on the GPU
token-by-token decoding against the oracle's prefill rows (a decode step of token i must equal
row i of the forward pass over the whole sequence)."""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity


@pytest.mark.parametrize("k,C", [(8, 128), (8, 3), (4, 0), (1, 5), (64, 16)])
def test_cache_slice_has_the_visible_count_of_eq3(k, C):
    """The contiguous slice the cache layout gives a step has exactly as many rows as the oracle's
    mask has visible keys for that position (text rows and summary rows, self-visible and strict)."""
    n = 40 * k + 3
    for flags, oflags in ((0, 0), (ksa.KSA_FLAG_SUMMARY_TEXT_ONLY, orc.SUMMARY_TEXT_ONLY)):
        spec = ksa.CacheSpec(1, k, C, n // k + 1, 8, 2, 128, 0.1, flags)
        assert ksa.cache_rows(spec) == 1 + k + C * k + n // k + 1
        for i in range(n):
            lo, hi = ksa.cache_slice(spec, i, False)
            p = (i // k) * (k + 1) + i % k
            assert hi - lo == orc.visible_count(n, k, 1, C, p, oflags), (i, lo, hi)
            assert lo >= 1 and hi <= ksa.cache_rows(spec)
        for j in range(1, n // k + 1):
            lo, hi = ksa.cache_slice(spec, j * k, True)
            p = (j - 1) * (k + 1) + k
            assert hi - lo == orc.visible_count(n, k, 1, C, p, oflags)


def test_cache_parameter_errors():
    good = ksa.CacheSpec(2, 8, 4, 16, 8, 2, 128, 0.1)
    assert ksa.cache_rows(good) > 0
    import dataclasses
    for bad in (dataclasses.replace(good, k=0), dataclasses.replace(good, Hq=7), dataclasses.replace(good, D=96),
                dataclasses.replace(good, Hq=34, Hkv=2), dataclasses.replace(good, max_summaries=0)):
        assert ksa.cache_rows(bad) < 0
        with pytest.raises(ksa.KsaError):
            ksa.cache_bytes(bad)
    with pytest.raises(ksa.KsaError):
        ksa.cache_slice(good, 5, True)          # a summary step needs a full chunk


@pytest.fixture(scope="module")
def ctx():
    ksa_build.build()
    c = ksa.Context(0)
    yield c
    c.close()


def _decode_all(ctx, lens, k, C, Hq, Hkv, D, flags, start_from_prefill_at=0, seed=21):
    """Decodes every sequence of a batch token by token (all sequences have the same length) and
    returns (out, lse) in the augmented layout next to the oracle's forward pass."""
    n = lens[0]
    assert all(x == n for x in lens)
    B = len(lens)
    wl = synth.Workload("dec", seed, lens, Hq, Hkv, D)
    L = orc.aug_len(n, k, 1)
    q, kk, v = synth.make_qkv(wl, B * L)
    oflags = orc.SUMMARY_TEXT_ONLY if flags else 0
    ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(kk), synth.bits(v), lens, k, 1, C, wl.scale, oflags)
    dev = torch.device("cuda", 0)
    qd, kd, vd = (t.to(dev).view(B, L, -1, D) for t in (q, kk, v))
    spec = ksa.CacheSpec(B, k, C, n // k + 1, Hq, Hkv, D, wl.scale, flags)
    cache = ksa.DecodeCache(ctx, spec)
    cache.kcache.fill_(float("nan")); cache.vcache.fill_(float("nan"))     # nothing unwritten may be read
    got_out = torch.full((B, L, Hq, D), 7.0, dtype=torch.bfloat16, device=dev)
    got_lse = torch.full((B, L, Hq), -1.0, dtype=torch.float32, device=dev)
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=dev)
    first = 0
    if start_from_prefill_at:
        n0 = start_from_prefill_at
        L0 = orc.aug_len(n0, k, 1)
        prob0 = ksa.Problem([n0] * B, k, 1, C, Hq, Hkv, D, wl.scale, flags)
        k0 = kd[:, :L0].contiguous().view(B * L0, Hkv, D); v0 = vd[:, :L0].contiguous().view(B * L0, Hkv, D)
        cache.fill_from_prefill(prob0, k0, v0)
        first = n0
        got_out[:, :L0] = torch.from_numpy(ref_out.reshape(B, L, Hq, D)[:, :L0]).to(dev).to(torch.bfloat16)
        got_lse[:, :L0] = torch.from_numpy(ref_lse.reshape(B, L, Hq)[:, :L0]).to(dev).float()
    else:
        cache.reset()
    ctx.clear_device_status()
    for i in range(first, n):
        p = (i // k) * (k + 1) + i % k
        cache.decode_text(qd[:, p].contiguous(), kd[:, p].contiguous(), vd[:, p].contiguous(), out, lse)
        got_out[:, p] = out; got_lse[:, p] = lse
        if (i + 1) % k == 0:
            ps = p + 1
            cache.decode_summary(qd[:, ps].contiguous(), kd[:, ps].contiguous(), vd[:, ps].contiguous(), out, lse)
            got_out[:, ps] = out; got_lse[:, ps] = lse
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    st = cache.state.cpu().numpy()
    assert (st[:, 0] == n).all() and (st[:, 1] == n // k).all()
    return (got_out.double().cpu().numpy().reshape(B * L, Hq, D), got_lse.double().cpu().numpy().reshape(B * L, Hq),
            ref_out, ref_lse)


@pytest.mark.gpu
@pytest.mark.parametrize("n,k,C,Hq,Hkv,D,flags", [
    (100, 8, 3, 8, 2, 128, 0),       # ring wraps several times, G = 4
    (70, 8, 128, 16, 2, 128, 0),     # window wider than the sequence: plain causal over the text, G = 8
    (45, 4, 0, 4, 4, 64, 0),         # no sliding chunks at all (summaries only), MHA, D = 64
    (50, 8, 2, 6, 2, 128, ksa.KSA_FLAG_SUMMARY_TEXT_ONLY),   # strict summary rule, G = 3
    (330, 8, 5, 8, 1, 128, 0),       # longer than one 64-row tile per split
])
def test_decode_token_by_token_equals_prefill(ctx, n, k, C, Hq, Hkv, D, flags):
    got_out, got_lse, ref_out, ref_lse = _decode_all(ctx, [n, n], k, C, Hq, Hkv, D, flags)
    parity.compare(got_out, got_lse, ref_out, ref_lse, "decode")


@pytest.mark.gpu
def test_decode_continues_a_prefill(ctx):
    """Cache built from a prefill's K/V (mid-chunk and on a chunk boundary), then decoded on."""
    for n0 in (61, 64):
        got_out, got_lse, ref_out, ref_lse = _decode_all(ctx, [120, 120, 120], 8, 4, 8, 2, 128, 0, start_from_prefill_at=n0)
        parity.compare(got_out, got_lse, ref_out, ref_lse, f"decode after prefill of {n0}")


@pytest.mark.gpu
def test_decode_text_step_refuses_a_pending_summary(ctx):
    spec = ksa.CacheSpec(1, 4, 2, 8, 4, 2, 128, 0.1)
    cache = ksa.DecodeCache(ctx, spec)
    dev = cache.kcache.device
    q = torch.zeros((1, 4, 128), dtype=torch.bfloat16, device=dev); kv = torch.zeros((1, 2, 128), dtype=torch.bfloat16, device=dev)
    out = torch.empty_like(q); lse = torch.empty((1, 4), dtype=torch.float32, device=dev)
    ctx.clear_device_status()
    for _ in range(4):
        cache.decode_text(q, kv, kv, out, lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    cache.decode_text(q, kv, kv, out, lse)          # chunk is full, its summary has not been inserted
    torch.cuda.synchronize()
    assert ctx.device_status() == 101
    assert cache.state.cpu().numpy().tolist() == [[4, 0]]
    ctx.clear_device_status()
    cache.decode_summary(q, kv, kv, out, lse)
    cache.decode_text(q, kv, kv, out, lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0 and cache.state.cpu().numpy().tolist() == [[5, 1]]
