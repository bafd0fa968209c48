"""Sequence-parallel parts (ksa_attn_fwd_part) on one GPU: the parts, run one after the other, give bit for bit
what the whole call gives; a part writes its own rows only and does not need k, v of later rows."""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D,num_parts", [
    ([4096], 8, 1, 16, 4, 2, 128, 4),                 # whole chunks: tiles read in place
    ([3000, 1100, 77], 8, 1, 8, 4, 2, 128, 3),        # ragged: packed streams; parts cross sequence boundaries
    ([2048], 64, 8, 4, 2, 2, 64, 2),
    ([700], 16, 0, 7, 4, 4, 128, 8),                  # more parts than there is work for some of them
])
def test_parts_equal_the_whole(ctx, lens, k, m, C, Hq, Hkv, D, num_parts):
    dev = torch.device("cuda", 0)
    wl = synth.Workload("parts", 41, lens, Hq, Hkv, D)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, D, wl.scale, 0)
    total = ksa.total_aug_len(prob)
    q, kk, v = synth.make_qkv(wl, total)
    qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    out_ref = torch.empty_like(qd); lse_ref = torch.empty((Hq, total), dtype=torch.float32, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out_ref, lse_ref, ws)
    torch.cuda.synchronize()
    # the parts tile the rows
    ranges = [ctx.part_rows(prob, r, num_parts) for r in range(num_parts)]
    assert ranges[0][0] == 0 and ranges[-1][1] == total
    for (b0, e0), (b1, e1) in zip(ranges, ranges[1:]):
        assert b0 <= e0 == b1 <= e1
    out = torch.full_like(qd, float("nan")); lse = torch.full_like(lse_ref, float("nan"))
    for r, (b, e) in enumerate(ranges):
        # what a rank of a sequence-parallel run holds: its own q rows, k and v up to its last row (zeros after)
        kr, vr = kd.clone(), vd.clone()
        kr[e:] = 0; vr[e:] = 0
        qr = torch.zeros_like(qd); qr[b:e] = qd[b:e]
        before = out.clone()
        ctx.attn_fwd_part(prob, qr, kr, vr, out, lse, ws, r, num_parts)
        torch.cuda.synchronize()
        # rows outside the part are untouched (NaN patterns included: compare bits)
        same = (out.view(torch.int16) == before.view(torch.int16))
        assert same[:b].all() and same[e:].all()
    assert ctx.device_status() == 0
    assert torch.equal(out.view(torch.int16), out_ref.view(torch.int16))
    assert torch.equal(lse.view(torch.int32), lse_ref.view(torch.int32))


def test_parts_are_balanced(ctx):
    """Under Eq. 3 later rows see more keys: equal row counts would be unbalanced, the parts are cut by work."""
    wl = synth.WORKLOADS["32k"]
    lay = synth.LAYOUT_P
    prob = ksa.Problem([32768], lay.k, lay.m, lay.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    ranges = [ctx.part_rows(prob, r, 4) for r in range(4)]
    sizes = [e - b for b, e in ranges]
    assert sizes[0] > sizes[-1]                       # the first part has the cheapest rows, hence the most
    from paper_2604_24432_b200 import dist_utils
    work = [dist_utils.visible_pairs_of_rows(32768, lay.k, lay.m, lay.C, b, e) for b, e in ranges]
    assert max(work) <= 1.15 * (sum(work) / 4)
