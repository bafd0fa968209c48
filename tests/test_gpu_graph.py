"""A training step's attention (forward, then backward) captured once in a CUDA graph and replayed on new inputs:
after the first call with a set of lengths the library does no host synchronisation, allocation or blocking copy, so
the two calls record into a graph like any kernel launch.  The replay has to give the bits of the plain calls."""
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


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D", [
    ([1024, 640], 8, 1, 16, 8, 2, 128),        # whole chunks: tiles read in place, tensor-core backward
    ([1000, 333], 8, 1, 16, 4, 2, 128),        # ragged: packed streams
    ([700], 64, 8, 2, 4, 4, 64),               # head_dim 64
])
def test_forward_backward_replayed_from_a_graph(ctx, lens, k, m, C, Hq, Hkv, D):
    dev = torch.device("cuda", 0)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, D, float(D) ** -0.5)
    total = ksa.total_aug_len(prob)
    wl_a = synth.Workload("graph-a", 11, lens, Hq, Hkv, D)
    wl_b = synth.Workload("graph-b", 12, lens, Hq, Hkv, D)
    g = torch.Generator("cpu").manual_seed(13)
    douts = [torch.randn((total, Hq, D), generator=g).to(torch.bfloat16).to(dev) for _ in range(2)]
    inputs = [tuple(t.to(dev) for t in synth.make_qkv(w, total)) for w in (wl_a, wl_b)]

    def buffers():
        return dict(out=torch.empty((total, Hq, D), dtype=torch.bfloat16, device=dev),
                    lse=torch.empty((Hq, total), dtype=torch.float32, device=dev),
                    dq=torch.empty((total, Hq, D), dtype=torch.bfloat16, device=dev),
                    dk=torch.empty((total, Hkv, D), dtype=torch.bfloat16, device=dev),
                    dv=torch.empty((total, Hkv, D), dtype=torch.bfloat16, device=dev))

    ws = torch.empty(max(256, ksa.workspace_bytes(prob)), dtype=torch.uint8, device=dev)
    wsb = torch.empty(ksa.bwd_workspace_bytes(prob), dtype=torch.uint8, device=dev)

    def step(q, kk, v, dout, b):
        ctx.attn_fwd(prob, q, kk, v, b["out"], b["lse"], ws)
        ctx.attn_bwd(prob, q, kk, v, b["out"], b["lse"], dout, b["dq"], b["dk"], b["dv"], wsb)

    # plain calls: the expected bits for both input sets (the first one also caches the schedule)
    want = []
    for (q, kk, v), dout in zip(inputs, douts):
        b = buffers()
        step(q, kk, v, dout, b)
        torch.cuda.synchronize()
        want.append({name: t.clone() for name, t in b.items()})
    assert ctx.device_status() == 0

    # capture once on static buffers, replay twice with the inputs swapped in
    sq, sk, sv = (torch.empty_like(t) for t in inputs[0])
    sdout = torch.empty_like(douts[0])
    sb = buffers()
    launches0 = ctx.launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(sq, sk, sv, sdout, sb)
    assert ctx.launch_count() > launches0            # the calls did record kernels
    for i in (1, 0, 1):
        q, kk, v = inputs[i]
        sq.copy_(q); sk.copy_(kk); sv.copy_(v); sdout.copy_(douts[i])
        for t in sb.values():
            t.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for name, t in sb.items():
            a = t.view(torch.int16) if t.dtype == torch.bfloat16 else t.view(torch.int32)
            w = want[i][name]
            w = w.view(torch.int16) if w.dtype == torch.bfloat16 else w.view(torch.int32)
            if name in ("out", "lse", "dq"):
                assert torch.equal(a, w), (name, i)
            else:
                # dk, dv are sums of fp32 atomic adds whose order is not fixed: equal up to rounding order
                d = (t.float() - want[i][name].float()).abs().max().item()
                assert d <= 2e-2 * want[i][name].float().abs().max().item(), (name, i, d)
