"""Seeded random configurations (shapes the hand-picked cases may miss): forward, backward, the sequence-parallel
parts and the host-buffer entry point against the oracle, element by element, at sizes the oracle finishes in a
moment."""
import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    ksa_build.build()
    c = ksa.Context(0)
    yield c
    c.close()


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    k = int(rng.choice([1, 2, 3, 4, 8, 16, 32, 64]))
    m = int(rng.choice([0, 1, 1, 2, 4, 8]))
    C = int(rng.choice([0, 1, 2, 5, 17, 200]))
    Hq, Hkv = [(2, 2), (4, 2), (4, 1), (6, 2), (8, 2)][int(rng.integers(0, 5))]
    D = int(rng.choice([64, 128, 128]))
    nseq = int(rng.integers(1, 4))
    hi = 520 if seed < 24 else 1100                          # the later seeds span more tiles
    if rng.random() < 0.4:                                   # whole chunks everywhere (tiles read in place when k, m divide 128)
        lens = [int(rng.integers(1, max(2, hi // k))) * k for _ in range(nseq)]
    else:
        lens = [int(rng.integers(1, hi)) for _ in range(nseq)]
    flags = ksa.KSA_FLAG_SUMMARY_TEXT_ONLY if rng.random() < 0.25 else 0
    return lens, k, m, C, Hq, Hkv, D, flags


@pytest.mark.parametrize("seed", range(48))
def test_random_configuration(ctx, seed):
    lens, k, m, C, Hq, Hkv, D, flags = _draw(seed)
    what = f"lens={lens} k={k} m={m} C={C} heads={Hq}/{Hkv} D={D} flags={flags}"
    wl = synth.Workload("fuzz", 2000 + seed, lens, Hq, Hkv, D)
    total = sum(orc.aug_len(n, k, m) for n in lens)
    q, kk, v = synth.make_qkv(wl, total)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, D, wl.scale, flags)
    oflags = orc.SUMMARY_TEXT_ONLY if flags else 0
    # ---- forward ----
    got_out, got_lse = parity.run_gpu(ctx, prob, q, kk, v)
    ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(kk), synth.bits(v), lens, k, m, C, wl.scale, oflags)
    parity.compare(got_out, got_lse, ref_out, ref_lse, what)
    # ---- sequence-parallel parts: bit for bit the whole call ----
    dev = torch.device("cuda", 0)
    qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    out_w = torch.empty_like(qd); lse_w = torch.empty((Hq, total), dtype=torch.float32, device=dev)
    ctx.attn_fwd(prob, qd, kd, vd, out_w, lse_w, ws)
    out_p = torch.full_like(qd, float("nan")); lse_p = torch.full_like(lse_w, float("nan"))
    parts = 1 + seed % 3
    for r in range(parts):
        ctx.attn_fwd_part(prob, qd, kd, vd, out_p, lse_p, ws, r, parts)
    torch.cuda.synchronize()
    assert torch.equal(out_p.view(torch.int16), out_w.view(torch.int16)), what
    assert torch.equal(lse_p.view(torch.int32), lse_w.view(torch.int32)), what
    # ---- host buffers in, host buffers out: the same bits again ----
    out_h = torch.full((total, Hq, D), 7.0, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.full((Hq, total), -1.0, dtype=torch.float32).pin_memory()
    staging = torch.full((ksa.host_staging_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)
    ctx.attn_fwd_host(prob, q, kk, v, out_h, lse_h, staging)
    assert ctx.device_status() == 0, what
    assert torch.equal(out_h.view(torch.int16), out_w.cpu().view(torch.int16)), what
    assert torch.equal(lse_h.view(torch.int32), lse_w.cpu().view(torch.int32)), what
    # ---- backward ----
    g = torch.Generator("cpu").manual_seed(3000 + seed)
    dout = torch.randn((total, Hq, D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    dq = torch.full_like(qd, 7.0); dk = torch.full_like(kd, 7.0); dv = torch.full_like(vd, 7.0)
    wsb = torch.full((ksa.bwd_workspace_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)
    ctx.attn_bwd(prob, qd, kd, vd, out_w, lse_w, dout.to(dev), dq, dk, dv, wsb)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0, what
    rdq, rdk, rdv = orc.bwd(synth.bits(q), synth.bits(kk), synth.bits(v), synth.bits(dout), lens, k, m, C, wl.scale, oflags)
    for name, got, ref in (("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        got = got.double().cpu().numpy()
        assert np.isfinite(got).all(), (what, name)
        err = np.abs(got - ref)
        assert err.max() <= 2e-2 * np.abs(ref).max() + 1e-5, (what, name, err.max(), np.abs(ref).max())
        assert err.mean() <= 1e-2 * np.abs(ref).mean() + 1e-5, (what, name, err.mean(), np.abs(ref).mean())
