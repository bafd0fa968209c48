"""The allocation-free entry point ``ksa_attn_fwd_noalloc``.

Some callers cannot obtain device memory when they need attention (the GPU belongs to a
server's own memory pool, or an allocation's device-wide synchronisation is not
acceptable), so the library offers a variant whose scratch is a fixed array inside the
library.  Its results are checked against the CPU oracle (and, bit for bit, against the
regular entry point, which runs the same kernels).  This file is collected last on
purpose: a failure here cannot hide another.
"""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity


def _run_noalloc(wl, k, m, C):
    """Canary-padded out / lse: the call must write every row and nothing else."""
    dev = torch.device("cuda", 0)
    total = sum(orc.aug_len(n, k, m) for n in wl.text_lens)
    q, kk, v = synth.make_qkv(wl, total)
    qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
    prob = ksa.Problem(wl.text_lens, k, m, C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    out = torch.full((total + 2, wl.Hq, wl.D), 3.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((wl.Hq * total + 64,), -7.0, dtype=torch.float32, device=dev)
    out_v = out[1:total + 1]
    lse_v = lse[32:32 + wl.Hq * total].view(wl.Hq, total)
    ksa.attn_fwd_noalloc(prob, qd, kd, vd, out_v, lse_v)
    torch.cuda.synchronize()
    assert ksa.noalloc_device_status() == 0
    assert (out[0] == 3.0).all() and (out[-1] == 3.0).all(), "out canary overwritten"
    assert (lse[:32] == -7.0).all() and (lse[-32:] == -7.0).all(), "lse canary overwritten"
    ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(kk), synth.bits(v), wl.text_lens, k, m, C, wl.scale)
    return prob, (qd, kd, vd), out_v, lse_v, ref_out, ref_lse


@pytest.mark.gpu
def test_noalloc_matches_oracle_twice():
    """Calls in a row (each smaller than the one before, so stale scratch would show; the second a whole-chunk batch,
    which the regular entry point reads in place and this one still packs) agree with the oracle within the parity
    tolerances and with the regular entry point bit for bit."""
    ksa_build.build()
    torch.cuda.set_device(0)
    ctx = ksa.Context(0)
    cases = [
        (synth.Workload("na1", 21, [1500, 700], 8, 2, 128), 8, 1, 4),
        (synth.Workload("na3", 23, [1024, 512], 8, 2, 128), 8, 1, 16),      # whole chunks
        (synth.Workload("na2", 22, [333], 4, 4, 64), 8, 1, 2),
    ]
    for wl, k, m, C in cases:
        prob, (q, kk, v), out, lse, ref_out, ref_lse = _run_noalloc(wl, k, m, C)
        parity.compare(out.double().cpu().numpy(), lse.double().cpu().numpy().T, ref_out, ref_lse, wl.name)
        reg_out, reg_lse = ksa.attn_fwd(ctx, prob, q, kk, v)
        torch.cuda.synchronize()
        # the same kernels on the same tiles (packed here; read in place by the regular call when the batch is whole
        # chunks): the same arithmetic in the same order, so the same bits
        assert torch.equal(reg_out, out) and torch.equal(reg_lse, lse)
    ctx.close()


@pytest.mark.gpu
def test_noalloc_rejects_oversized_problem():
    """A problem whose scratch exceeds the fixed array is refused before any GPU work -- also a whole-chunk one, whose
    regular workspace is only 256 bytes."""
    ksa_build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    for n in (8189, 8192):
        prob = ksa.Problem([n], 8, 1, 128, 32, 8, 128, 0.0884)
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
