"""The allocation-free entry point ``ksa_attn_fwd_noalloc`` against ``ksa_attn_fwd``.

Some callers cannot obtain device memory when they need attention (the GPU belongs to a
server's own memory pool, or an allocation's device-wide synchronisation is not
acceptable), so the library offers a variant whose scratch is a fixed array inside the
library.  This file is collected last on purpose: a failure here cannot hide another.
"""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity


def _run_both(ctx, wl, k, m, C):
    dev = torch.device("cuda", 0)
    total = sum(orc.aug_len(n, k, m) for n in wl.text_lens)
    q, kk, v = (t.to(dev) for t in synth.make_qkv(wl, total))
    prob = ksa.Problem(wl.text_lens, k, m, C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    ref_out, ref_lse = ksa.attn_fwd(ctx, prob, q, kk, v)
    out = torch.full_like(ref_out, 3.0)
    lse = torch.full_like(ref_lse, -7.0)
    ksa.attn_fwd_noalloc(prob, q, kk, v, out, lse)
    torch.cuda.synchronize()
    return out, lse, ref_out, ref_lse


@pytest.mark.gpu
def test_noalloc_matches_regular_entry_point_twice():
    """Two calls in a row (the second smaller, so stale scratch from the first would show)
    give what the regular entry point gives, within the parity tolerances."""
    ksa_build.build()
    torch.cuda.set_device(0)
    ctx = ksa.Context(0)
    cases = [
        (synth.Workload("na1", 21, [1500, 700], 8, 2, 128), 8, 1, 4),
        (synth.Workload("na2", 22, [333], 4, 4, 64), 8, 1, 2),
    ]
    for wl, k, m, C in cases:
        out, lse, ref_out, ref_lse = _run_both(ctx, wl, k, m, C)
        parity.compare(out.double().cpu().numpy(), lse.double().cpu().numpy().T,
                       ref_out.double().cpu().numpy(), ref_lse.double().cpu().numpy().T, wl.name)
    ctx.close()


@pytest.mark.gpu
def test_noalloc_rejects_oversized_problem():
    """A problem whose scratch exceeds the fixed array is refused before any GPU work."""
    ksa_build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    prob = ksa.Problem([8189], 8, 1, 128, 32, 8, 128, 0.0884)      # not whole chunks: the packed streams are needed
    assert ksa.workspace_bytes(prob) > ksa.NOALLOC_MAX_SCRATCH_BYTES
    total = ksa.total_aug_len(prob)
    q = torch.zeros((total, 32, 128), dtype=torch.bfloat16, device=dev)
    kv = torch.zeros((total, 8, 128), dtype=torch.bfloat16, device=dev)
    out = torch.full_like(q, 5.0)
    lse = torch.zeros((32, total), dtype=torch.float32, device=dev)
    with pytest.raises(ksa.KsaError) as e:
        ksa.attn_fwd_noalloc(prob, q, kv, kv, out, lse)
    assert e.value.status == ksa.KSA_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (out == 5.0).all()
