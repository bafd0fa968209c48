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
