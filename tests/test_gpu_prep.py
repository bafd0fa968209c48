"""GPU parity of the Q/K/V preparation pass (position ids, interpolation at summary positions, rotary embedding)
against the fp64 oracle, element by element, through the C ABI.

Tolerance: the kernel takes the angles in double precision and does the interpolation and the rotation in fp32
on bf16 inputs (errors of about 1e-7 relative), then rounds once to bf16: |err| <= 2^-8 |ref| + 1e-6 per element
(half an ulp of bf16 is 2^-9 relative; the factor 2 covers values next to a binade boundary)."""
import numpy as np
import pytest
import torch

from oracle import ksa_prep_oracle as prep
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    ksa_build.build()
    c = ksa.Context(0)
    yield c
    c.close()


def _rand(shape, seed):
    g = torch.Generator("cpu").manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)


@pytest.mark.parametrize("lens,k,m,Hq,Hkv,D,lam,theta,flags", [
    ([300, 77], 8, 1, 4, 2, 128, 0.3, 1.0e4, 0),
    ([1000], 8, 1, 8, 2, 128, 1.0, 1.0e6, 0),
    ([130, 5, 64], 64, 8, 2, 2, 64, 0.75, 1.0e6, 0),              # several summaries per chunk, head_dim 64
    ([40], 3, 2, 3, 1, 64, 0.0, 1.0e4, 0),                         # lambda = 0: no summary projections needed
    ([257], 16, 0, 2, 2, 128, 0.5, 1.0e4, 0),                      # no summary tokens at all
    ([96, 31], 8, 1, 4, 4, 128, 0.6, 0.0, ksa.KSA_PREP_NO_ROPE),   # interpolation only
    ([131072 - 8, 8], 8, 1, 1, 1, 128, 0.5, 1.0e6, 0),             # positions up to 131,071: angles need more than fp32
])
def test_prepare_matches_oracle(ctx, lens, k, m, Hq, Hkv, D, lam, theta, flags):
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(lens, k, m, 4, Hq, Hkv, D, 1.0 / np.sqrt(D), 0)
    L = ksa.total_aug_len(prob)
    S = ksa.total_summary_rows(prob)
    assert S == sum((n // k) * m for n in lens)
    qm, km, vm = _rand((L, Hq, D), 1), _rand((L, Hkv, D), 2), _rand((L, Hkv, D), 3)
    need_summ = lam != 0.0 and S > 0
    qs, ks, vs = (_rand((S, Hq, D), 4), _rand((S, Hkv, D), 5), _rand((S, Hkv, D), 6)) if need_summ else (None, None, None)
    qd, kd, vd = qm.to(dev), km.to(dev), vm.to(dev)
    to = lambda t: None if t is None else t.to(dev)
    qo, ko, vo = torch.full_like(qd, 7.0), torch.full_like(kd, 7.0), torch.full_like(vd, 7.0)
    ctx.qkv_prepare(prob, qd, kd, vd, to(qs), to(ks), to(vs), qo, ko, vo, lam, theta, flags)
    torch.cuda.synchronize()
    # the position ids the library reports are the oracle's
    assert ksa.position_ids(prob).tolist() == prep.position_ids(lens, k, m).tolist()
    # oracle on a bounded number of rows for the long case: the first and the last rows and a seeded sample
    rows = np.arange(L)
    if L > 4096:
        rng = np.random.default_rng(0)
        rows = np.unique(np.concatenate([np.arange(64), np.arange(L - 64, L), rng.integers(0, L, 512)]))
    pos, is_summ = prep.position_ids(lens, k, m), prep.summary_rows(lens, k, m)
    summ_index = np.cumsum(is_summ) - 1
    f64 = lambda t: t.double().numpy()
    for name, main, summ, out, rotate in (("q", qm, qs, qo, True), ("k", km, ks, ko, True), ("v", vm, vs, vo, False)):
        got = out.cpu().double().numpy()
        for r in rows:
            x = f64(main[r])
            if is_summ[r] and need_summ:
                x = lam * f64(summ[summ_index[r]]) + (1.0 - lam) * x
            ref = prep.rope_row(x, pos[r], theta) if (rotate and not flags) else x
            err = np.abs(got[r] - ref)
            assert (err <= 2.0 ** -8 * np.abs(ref) + 1e-6).all(), (name, int(r), float(err.max()))


def test_prepare_in_place_and_whole_oracle(ctx):
    """Outputs may alias the inputs; the whole-tensor oracle routine (not only its row function) agrees."""
    lens, k, m, Hq, Hkv, D, lam, theta = [45, 16], 8, 1, 2, 1, 64, 0.25, 1.0e4
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(lens, k, m, 4, Hq, Hkv, D, 0.125, 0)
    L, S = ksa.total_aug_len(prob), ksa.total_summary_rows(prob)
    qm, km, vm = _rand((L, Hq, D), 11), _rand((L, Hkv, D), 12), _rand((L, Hkv, D), 13)
    qs, ks, vs = _rand((S, Hq, D), 14), _rand((S, Hkv, D), 15), _rand((S, Hkv, D), 16)
    rq, rk, rv = prep.prepare(qm.double().numpy(), km.double().numpy(), vm.double().numpy(),
                              qs.double().numpy(), ks.double().numpy(), vs.double().numpy(), lens, k, m, lam, theta)
    qd, kd, vd = qm.to(dev), km.to(dev), vm.to(dev)
    ctx.qkv_prepare(prob, qd, kd, vd, qs.to(dev), ks.to(dev), vs.to(dev), qd, kd, vd, lam, theta)
    torch.cuda.synchronize()
    for got, ref in ((qd, rq), (kd, rk), (vd, rv)):
        err = np.abs(got.cpu().double().numpy() - ref)
        assert (err <= 2.0 ** -8 * np.abs(ref) + 1e-6).all()


def test_anneal_lambda_matches_oracle():
    for step in (0, 99, 100, 101, 150, 299, 300, 10 ** 9):
        assert ksa.anneal_lambda(step, 100, 300) == pytest.approx(prep.anneal_lambda(step, 100, 300), abs=1e-7)


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D,lam,theta,flags", [
    ([300, 77], 8, 1, 4, 4, 2, 128, 0.3, 1.0e4, 0),                  # ragged lengths
    ([1024, 512], 8, 1, 16, 8, 2, 128, 0.6, 1.0e6, 0),               # whole chunks (the plain forward call would read these in place)
    ([1500], 8, 1, 16, 8, 2, 128, 1.0, 1.0e6, 0),                    # several summary tiles
    ([400, 130], 64, 8, 2, 4, 2, 128, 0.75, 1.0e4, 0),               # eight summaries per chunk
    ([333], 3, 2, 5, 6, 2, 64, 0.5, 1.0e4, 0),                       # head_dim 64, odd group size
    ([257], 16, 0, 3, 2, 2, 128, 0.5, 1.0e4, 0),                     # no summary tokens
    ([200], 8, 1, 2, 4, 2, 128, 0.4, 0.0, ksa.KSA_PREP_NO_ROPE),     # interpolation only
])
def test_prepared_forward_equals_prepare_then_forward_and_the_oracles(ctx, lens, k, m, C, Hq, Hkv, D, lam, theta, flags):
    """ksa_attn_fwd_prepared (preparation folded into the pack pass) against (a) ksa_qkv_prepare followed by ksa_attn_fwd:
    the same arithmetic on the same rows, so the same bits, and (b) the two oracles chained: the fp64 preparation oracle,
    rounded once to bf16 as the operator's inputs are, then the fp64 attention oracle."""
    from oracle import ksa_oracle as orc
    from tests import parity
    dev = torch.device("cuda", 0)
    scale = 1.0 / np.sqrt(D)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, D, scale, 0)
    L, S = ksa.total_aug_len(prob), ksa.total_summary_rows(prob)
    qm, km, vm = _rand((L, Hq, D), 11), _rand((L, Hkv, D), 12), _rand((L, Hkv, D), 13)
    need_summ = lam != 0.0 and S > 0
    qs, ks, vs = (_rand((S, Hq, D), 14), _rand((S, Hkv, D), 15), _rand((S, Hkv, D), 16)) if need_summ else (None, None, None)
    to = lambda t: None if t is None else t.to(dev)
    qd, kd, vd = qm.to(dev), km.to(dev), vm.to(dev)
    # (a) two calls
    qo, ko, vo = torch.empty_like(qd), torch.empty_like(kd), torch.empty_like(vd)
    ctx.qkv_prepare(prob, qd, kd, vd, to(qs), to(ks), to(vs), qo, ko, vo, lam, theta, flags)
    out2 = torch.empty_like(qd); lse2 = torch.empty((Hq, L), dtype=torch.float32, device=dev)
    ws2 = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    ctx.clear_device_status()
    ctx.attn_fwd(prob, qo, ko, vo, out2, lse2, ws2)
    # one call; canary-padded outputs, NaN-filled workspace
    out = torch.full((L + 2, Hq, D), 7.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((Hq * L + 64,), -5.0, dtype=torch.float32, device=dev)
    out_v, lse_v = out[1:L + 1], lse[32:32 + Hq * L].view(Hq, L)
    ws = torch.full((ksa.prepared_workspace_bytes(prob),), 0xFF, dtype=torch.uint8, device=dev)
    ctx.attn_fwd_prepared(prob, qd, kd, vd, to(qs), to(ks), to(vs), lam, theta, out_v, lse_v, ws, flags)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert (out[0] == 7.0).all() and (out[-1] == 7.0).all() and (lse[:32] == -5.0).all() and (lse[-32:] == -5.0).all()
    # text rows: the same tensor-core kernel on the same tiles -> the same bits; summary rows come from another kernel
    is_summ = torch.from_numpy(prep.summary_rows(lens, k, m).astype(bool)).to(dev)
    assert torch.equal(out_v[~is_summ], out2[~is_summ]) and torch.equal(lse_v[:, ~is_summ], lse2[:, ~is_summ])
    # (b) the oracles
    f64 = lambda t: None if t is None else t.double().numpy()
    if flags & ksa.KSA_PREP_NO_ROPE:
        pos, summ = prep.position_ids(lens, k, m), prep.summary_rows(lens, k, m)
        idx = np.cumsum(summ) - 1
        def blend(main, s_):
            x = f64(main).copy()
            if need_summ:
                x[summ.astype(bool)] = lam * f64(s_)[idx[summ.astype(bool)]] + (1.0 - lam) * x[summ.astype(bool)]
            return x
        rq, rk, rv = blend(qm, qs), blend(km, ks), blend(vm, vs)
    else:
        rq, rk, rv = prep.prepare(f64(qm), f64(km), f64(vm), f64(qs), f64(ks), f64(vs), lens, k, m, lam if need_summ else 0.0, theta)
    bits = lambda x: (torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    ref_out, ref_lse, _ = orc.fwd(bits(rq), bits(rk), bits(rv), lens, k, m, C, scale)
    parity.compare(out_v.double().cpu().numpy(), lse_v.double().cpu().numpy().T, ref_out, ref_lse, "prepared")
