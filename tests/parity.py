"""Shared code of the GPU parity tests: run the CUDA library and the oracle on the same
seeded inputs and compare element by element.

Tolerances (bf16 output against the fp64 oracle): max |out - ref| <= 2e-2 and
mean |out - ref| <= 2e-3; LSE: |lse - ref| <= 1e-3 * max(1, |ref|)."""
import numpy as np
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import synth

OUT_MAX_ABS = 2e-2
OUT_MEAN_ABS = 2e-3
LSE_REL = 1e-3


def run_gpu(ctx, prob, q, k, v):
    """q, k, v: CPU bf16 tensors.  Returns (out float64 [L,Hq,D], lse float64 [L,Hq])."""
    dev = torch.device("cuda", 0)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    total = q.shape[0]
    # canary-padded outputs: the kernels must write every row and nothing else
    out = torch.full((total + 2, prob.Hq, prob.D), 7.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((prob.Hq * total + 64,), -12345.0, dtype=torch.float32, device=dev)
    ws = torch.empty(ksa.workspace_bytes(prob) + 256, dtype=torch.uint8, device=dev)
    ws_al = ws[(256 - ws.data_ptr() % 256) % 256:]
    out_v = out[1:total + 1]
    lse_v = lse[32:32 + prob.Hq * total].view(prob.Hq, total)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qd, kd, vd, out_v, lse_v, ws_al[:ksa.workspace_bytes(prob)])
    torch.cuda.synchronize()
    assert ctx.device_status() == 0, "a device-side wait gave up: code %d" % ctx.device_status()
    assert (out[0] == 7.0).all() and (out[-1] == 7.0).all(), "out canary overwritten"
    assert (lse[:32] == -12345.0).all() and (lse[-32:] == -12345.0).all(), "lse canary overwritten"
    return out_v.double().cpu().numpy(), lse_v.double().cpu().numpy().T.copy()


def compare(got_out, got_lse, ref_out, ref_lse, what=""):
    assert np.isfinite(got_out).all(), what + ": non-finite output"
    assert np.isfinite(got_lse).all(), what + ": non-finite lse"
    err = np.abs(got_out - ref_out)
    lerr = np.abs(got_lse - ref_lse) / np.maximum(1.0, np.abs(ref_lse))
    stats = dict(out_max=float(err.max()), out_mean=float(err.mean()), lse_rel=float(lerr.max()))
    assert stats["out_max"] <= OUT_MAX_ABS, (what, stats)
    assert stats["out_mean"] <= OUT_MEAN_ABS, (what, stats)
    assert stats["lse_rel"] <= LSE_REL, (what, stats)
    return stats


def sample_rows(text_lens, k, m, n_random, seed, tile=128):
    """Global augmented rows: every row of the first, the last and a few boundary query
    tiles of each sequence (in augmented coordinates), plus random rows."""
    rng = np.random.default_rng(seed)
    rows = []
    off = 0
    for n in text_lens:
        L = orc.aug_len(n, k, m)
        s = k + m
        tiles = {0, max(0, (n - 1) // tile), max(0, (n - 1) // tile - 1), min((n - 1) // tile, 9), (n // tile) // 2}
        for t in sorted(tiles):
            i0, i1 = t * tile, min(n, t * tile + tile)
            p0 = (i0 // k) * s + i0 % k
            p1 = min(L, ((i1 - 1) // k) * s + (i1 - 1) % k + 1 + m)
            rows.extend(range(off + p0, off + p1))
        rows.extend((off + rng.integers(0, L, size=n_random // len(text_lens))).tolist())
        off += L
    return np.unique(np.asarray(rows, dtype=np.int64))


def check_workload(ctx, wl, layout, flags=0, rows=None, C=None, n_random=0, seed=0):
    C = layout.C if C is None else C
    total = sum(orc.aug_len(n, layout.k, layout.m) for n in wl.text_lens)
    q, k, v = synth.make_qkv(wl, total)
    prob = ksa.Problem(wl.text_lens, layout.k, layout.m, C, wl.Hq, wl.Hkv, wl.D, wl.scale, flags)
    assert ksa.total_aug_len(prob) == total
    got_out, got_lse = run_gpu(ctx, prob, q, k, v)
    if rows is None and n_random:
        rows = sample_rows(wl.text_lens, layout.k, layout.m, n_random, seed)
    oflags = orc.SUMMARY_TEXT_ONLY if (flags & ksa.KSA_FLAG_SUMMARY_TEXT_ONLY) else 0
    ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(k), synth.bits(v), wl.text_lens,
                                  layout.k, layout.m, C, wl.scale, oflags, rows=rows)
    if rows is not None:
        got_out, got_lse = got_out[rows], got_lse[rows]
    return compare(got_out, got_lse, ref_out, ref_lse, f"{wl.name}/{layout.name}/C={C}/flags={flags}")
