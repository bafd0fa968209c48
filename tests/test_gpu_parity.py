"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from paper_2604_24432_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

REF = ksa.KSA_FLAG_REFERENCE_KERNEL
STRICT = ksa.KSA_FLAG_SUMMARY_TEXT_ONLY


@pytest.fixture(scope="module")
def ctx():
    ksa_build.build()
    c = ksa.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("kernel_flag", [REF, 0], ids=["ref", "tc"])
@pytest.mark.parametrize("layout", [synth.LAYOUT_P, synth.LAYOUT_G], ids=["P", "G"])
@pytest.mark.parametrize("C", [None, 0, 1, 2, 4])
def test_tiny_full(ctx, kernel_flag, layout, C):
    """1,024 text tokens, 4/4 heads, D = 64: every row against the oracle, at the paper's
    window (pure causal over text) and at small windows that make summaries visible."""
    parity.check_workload(ctx, synth.WORKLOADS["tiny"], layout, kernel_flag, C=C)


@pytest.mark.parametrize("kernel_flag", [REF, 0], ids=["ref", "tc"])
def test_tiny_strict_summary_rule(ctx, kernel_flag):
    parity.check_workload(ctx, synth.WORKLOADS["tiny"], synth.LAYOUT_G, kernel_flag | STRICT, C=2)
    parity.check_workload(ctx, synth.WORKLOADS["tiny"], synth.LAYOUT_P, kernel_flag | STRICT, C=2)


@pytest.mark.parametrize("kernel_flag", [REF, 0], ids=["ref", "tc"])
def test_8k_full(ctx, kernel_flag):
    """8,192 text tokens, GQA 32/8, D = 128, K scaled by 0.5 (flat softmax): every row."""
    parity.check_workload(ctx, synth.WORKLOADS["8k"], synth.LAYOUT_P, kernel_flag)


def test_8k_layout_g_sampled(ctx):
    parity.check_workload(ctx, synth.WORKLOADS["8k"], synth.LAYOUT_G, 0, n_random=512, seed=1)


@pytest.mark.parametrize("name,n_random", [("32k", 768), ("128k", 512), ("varlen", 1024)])
def test_full_size_sampled(ctx, name, n_random):
    """The three large workloads at full size, in the launch configuration the benchmark times:
    every row of the first, last and a few boundary query tiles of each sequence plus random
    rows, all heads, against the oracle (which computes the sampled rows one by one)."""
    parity.check_workload(ctx, synth.WORKLOADS[name], synth.LAYOUT_P, 0, n_random=n_random, seed=11)


@pytest.mark.parametrize("name,n_random", [("32k", 384), ("128k", 256), ("varlen", 512)])
def test_full_size_layout_g_sampled(ctx, name, n_random):
    """The large workloads at the 64 + 8 chunk layout (m = 8 summaries per chunk), sampled rows (boundary tiles of every
    sequence plus random rows)."""
    parity.check_workload(ctx, synth.WORKLOADS[name], synth.LAYOUT_G, 0, n_random=n_random, seed=12)


@pytest.mark.parametrize("name,layout,n_random", [("8k", "P", 0), ("32k", "P", 384), ("128k", "P", 256), ("varlen", "P", 384),
                                                  ("32k", "G", 256), ("128k", "G", 192)])
def test_cta_pair_kernel(ctx, name, layout, n_random):
    """The CTA-pair text kernel (opt-in flag) on the workloads it applies to, against the oracle; the ragged varlen
    batch goes through the packed streams, the others are read in place."""
    lay = {"P": synth.LAYOUT_P, "G": synth.LAYOUT_G}[layout]
    parity.check_workload(ctx, synth.WORKLOADS[name], lay, ksa.KSA_FLAG_CTA_PAIR_KERNEL, n_random=n_random, seed=13)


@pytest.mark.parametrize("kernel_flag", [REF, 0], ids=["ref", "tc"])
@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D", [
    ([1], 8, 1, 2, 2, 2, 64),              # a single token
    ([7], 8, 1, 2, 2, 1, 128),             # shorter than a chunk: no summary at all
    ([127, 129, 128], 8, 1, 3, 4, 2, 64),  # ragged tiles, packed
    ([333, 1000], 3, 2, 5, 6, 2, 128),     # k does not divide the tile, m = 2, G = 3 (one head per item)
    ([777], 16, 0, 7, 4, 4, 64),           # m = 0: sliding chunk attention alone (Eq. 2)
    ([640], 1, 1, 100, 2, 1, 128),         # k = 1
    ([1290], 200, 3, 1, 4, 1, 128),        # chunk longer than a tile
    ([2100], 8, 1, 16, 8, 2, 128),         # several summary tiles
    ([2048, 640, 1336], 8, 1, 16, 8, 2, 128),   # whole chunks everywhere: direct views, sequences not on tile boundaries
    ([1024, 320], 4, 2, 9, 4, 2, 64),      # direct views with m = 2, D = 64
    ([768], 128, 1, 2, 2, 1, 128),         # a chunk is a whole tile
    ([1300], 200, 8, 1, 8, 1, 128),        # long chunks, 64 summary tasks per chunk (several task blocks, rows read from global memory)
    ([900], 96, 4, 2, 4, 2, 64),           # head_dim 64, summary rows from staged chunk rows
])
def test_edge_shapes(ctx, kernel_flag, lens, k, m, C, Hq, Hkv, D):
    wl = synth.Workload("edge", 99, lens, Hq, Hkv, D)
    parity.check_workload(ctx, wl, synth.Layout("edge", k, m, C), kernel_flag)


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D", [
    ([2048, 1500, 333], 8, 1, 16, 16, 16, 128),   # multi-head attention (the paper's 16/16 model): every pair has two KV heads
    ([2048, 640], 8, 1, 16, 8, 8, 64),            # the same at head_dim 64, whole chunks (tiles read in place)
    ([1900], 64, 8, 4, 6, 2, 128),                # three query heads per KV head: pairs (0,1), (2,3) across KV heads, (4,5)
    ([1500, 700], 8, 1, 5, 10, 2, 128),           # five per KV head
    ([900], 16, 2, 3, 3, 3, 64),                  # an odd number of query heads: single-head work items
])
def test_head_pairs_across_kv_heads(ctx, lens, k, m, C, Hq, Hkv, D):
    """Work items pair consecutive query heads; where the two belong to different KV heads the kernel streams K and V per
    head (four ring stages per key tile).  Several tiles, several work items per CTA, packed and in-place inputs."""
    wl = synth.Workload("mha", 96, lens, Hq, Hkv, D)
    parity.check_workload(ctx, wl, synth.Layout("edge", k, m, C), 0)


def test_thousands_of_short_sequences(ctx):
    """3,000 packed sequences of 1 .. 89 tokens (most shorter than a tile, many shorter than a chunk): sampled rows against
    the oracle."""
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(1, 90, size=3000)]
    wl = synth.Workload("many", 9, lens, 4, 2, 128)
    parity.check_workload(ctx, wl, synth.Layout("p", 8, 1, 2), 0, n_random=600, seed=4)
    assert ctx.device_status() == 0


def test_one_million_tokens(ctx):
    """One sequence of 2^20 text tokens (1,179,648 augmented rows, 8,192 query tiles, up to 1,033 key tiles per work item;
    8/2 heads keep it at a few GB): sampled rows against the oracle, no bounded wait gave up."""
    wl = synth.Workload("1m", 7, [1 << 20], 8, 2, 128)
    parity.check_workload(ctx, wl, synth.LAYOUT_P, 0, n_random=400, seed=3)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("strict", [0, STRICT])
@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv,D", [
    ([700, 200], 24, 3, 2, 12, 2, 128),    # 18 query rows per chunk and KV head (two 16-row tiles, one ragged), 27 keys
    ([1000], 120, 8, 1, 16, 1, 128),       # the largest block: 128 query rows (eight tiles for four warps), 128 keys
    ([600], 56, 8, 1, 4, 4, 64),           # one query head per KV head, head_dim 64
    ([512, 40], 13, 8, 3, 8, 2, 128),      # odd chunk length, a sequence of three chunks and a tail
    ([300], 16, 2, 2, 8, 2, 128),          # the smallest block: 8 query rows, 18 keys
])
def test_summary_rows_on_mma_tiles(ctx, lens, k, m, C, Hq, Hkv, D, strict):
    """Chunks longer than the short-chunk kernel takes, with at least 8 (summary row, query head) pairs per chunk and KV
    head and at most 128 of them and 128 keys: the summary rows run on the mma.sync kernel.  Every row against the oracle,
    with and without the chunk's own summaries visible (Sec. 2.2.1)."""
    wl = synth.Workload("summ-mma", 97, lens, Hq, Hkv, D)
    parity.check_workload(ctx, wl, synth.Layout("edge", k, m, C), strict)


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv", [
    ([1], 8, 1, 2, 2, 1), ([7], 8, 1, 2, 2, 1), ([127, 129, 128], 8, 1, 3, 4, 2), ([333, 1000], 3, 2, 5, 4, 2),
    ([777], 16, 0, 7, 4, 2), ([640], 1, 1, 100, 2, 1), ([1290], 200, 3, 1, 4, 1), ([2048, 640, 1336], 8, 1, 16, 8, 2),
    ([768], 128, 1, 2, 2, 1), ([2100], 8, 1, 16, 8, 2), ([4096], 64, 8, 4, 4, 2), ([130], 8, 1, 0, 16, 2),
])
@pytest.mark.parametrize("strict", [0, STRICT])
def test_cta_pair_kernel_edge_shapes(ctx, lens, k, m, C, Hq, Hkv, strict):
    """Edge shapes through the CTA-pair kernel (head_dim 128, even group sizes): single tokens, ragged tiles, chunks that do
    not divide a tile (falls back to packed streams), no summaries, items of one and two tiles (the tile stream runs
    across work items), more work items than pairs and fewer."""
    wl = synth.Workload("pair-edge", 98, lens, Hq, Hkv, 128)
    parity.check_workload(ctx, wl, synth.Layout("edge", k, m, C), ksa.KSA_FLAG_CTA_PAIR_KERNEL | strict)


@pytest.mark.parametrize("n", [900, 896])     # 896: whole chunks, tiles are read straight from the strided views
def test_strided_inputs_and_stream(ctx, n):
    """Non-contiguous q/k/v/out views (packed QKV buffer) on a side stream."""
    wl = synth.Workload("strided", 5, [n], 8, 2, 128)
    lay = synth.Layout("s", 8, 1, 4)
    total = orc.aug_len(n, 8, 1)
    q, k, v = synth.make_qkv(wl, total)
    dev = torch.device("cuda", 0)
    packed = torch.zeros((total, 8 + 2 + 2 + 1, 128), dtype=torch.bfloat16, device=dev)
    packed[:, :8] = q.to(dev); packed[:, 8:10] = k.to(dev); packed[:, 10:12] = v.to(dev)
    qd, kd, vd = packed[:, :8], packed[:, 8:10], packed[:, 10:12]
    outbuf = torch.zeros((total, 9, 128), dtype=torch.bfloat16, device=dev)
    out = outbuf[:, 1:]
    lse = torch.empty((8, total), dtype=torch.float32, device=dev)
    prob = ksa.Problem([n], 8, 1, 4, 8, 2, 128, wl.scale)
    ws = torch.empty(ksa.workspace_bytes(prob), dtype=torch.uint8, device=dev)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        ctx.attn_fwd(prob, qd, kd, vd, out, lse, ws, stream=st.cuda_stream)
    st.synchronize()
    ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(k), synth.bits(v), [n], 8, 1, 4, wl.scale)
    parity.compare(out.double().cpu().numpy(), lse.double().cpu().numpy().T, ref_out, ref_lse, "strided")
    assert (outbuf[:, 0] == 0).all()


@pytest.mark.parametrize("lens,k,m,C,Hq,Hkv", [
    ([500, 300], 8, 1, 2, 4, 2),          # shorter than a row chunk each
    ([6000], 8, 1, 16, 8, 2),             # one sequence cut into several upload/compute/download stages
    ([5000, 1300, 77], 3, 2, 5, 6, 2),    # k does not divide the tile, m = 2, ragged lengths, G = 3
    ([3000, 2100], 16, 0, 7, 4, 4),       # no summaries
])
def test_host_entry_point(ctx, lens, k, m, C, Hq, Hkv):
    """Host tensors in, host tensors out (the pipelined entry point).  The staging buffer starts
    out filled with NaN bit patterns: nothing that a stage has not written yet may leak into a result."""
    wl = synth.Workload("host", 6, lens, Hq, Hkv, 128)
    total = sum(orc.aug_len(n, k, m) for n in lens)
    q, kk, v = synth.make_qkv(wl, total, pin=True)
    prob = ksa.Problem(lens, k, m, C, Hq, Hkv, 128, wl.scale)
    out = torch.empty((total, Hq, 128), dtype=torch.bfloat16).pin_memory()
    lse = torch.empty((Hq, total), dtype=torch.float32).pin_memory()
    staging = torch.full((ksa.host_staging_bytes(prob),), 0xFF, dtype=torch.uint8, device="cuda:0")
    for _ in range(2):                    # the second call reuses the cached chunked schedule
        out.fill_(7.0); lse.fill_(-1.0)
        ctx.clear_device_status()
        ctx.attn_fwd_host(prob, q, kk, v, out, lse, staging)
        assert ctx.device_status() == 0
        ref_out, ref_lse, _ = orc.fwd(synth.bits(q), synth.bits(kk), synth.bits(v), lens, k, m, C, wl.scale)
        parity.compare(out.double().numpy(), lse.double().numpy().T, ref_out, ref_lse, "host")


def test_runtime_argument_errors(ctx):
    dev = torch.device("cuda", 0)
    prob = ksa.Problem([300], 8, 1, 2, 4, 2, 64, 0.125)
    total = ksa.total_aug_len(prob)
    q = torch.zeros((total, 4, 64), dtype=torch.bfloat16, device=dev)
    k = torch.zeros((total, 2, 64), dtype=torch.bfloat16, device=dev)
    out = torch.zeros_like(q)
    lse = torch.zeros((4, total), dtype=torch.float32, device=dev)
    ws = torch.empty(ksa.workspace_bytes(prob), dtype=torch.uint8, device=dev)
    before = ctx.launch_count()
    with pytest.raises(ksa.KsaError) as e:
        ctx.attn_fwd(prob, q, k, k, out, lse, ws[:1024])
    assert e.value.status == ksa.KSA_ERR_WORKSPACE
    with pytest.raises(ksa.KsaError) as e:
        ctx.attn_fwd(prob, q.view(-1)[1:].view(-1)[: (total - 1) * 256].view(total - 1, 4, 64), k, k, out, lse, ws)
    assert e.value.status == ksa.KSA_ERR_INVALID_ARG     # misaligned q
    bad = dataclasses.replace(prob, k=0)
    with pytest.raises(ksa.KsaError):
        ctx.attn_fwd(bad, q, k, k, out, lse, ws)
    assert ctx.launch_count() == before                  # nothing was launched
    ctx.attn_fwd(prob, q, k, k, out, lse, ws)
    torch.cuda.synchronize()
    assert ctx.launch_count() == before + 3


def test_q_zero_gives_log_count(ctx):
    """Q = 0: lse = ln(visible count) and out = mean of the visible V rows, for every row."""
    wl = synth.Workload("q0", 7, [1500], 4, 2, 128)
    lay = synth.Layout("q0", 8, 1, 16)
    total = orc.aug_len(1500, 8, 1)
    q, k, v = synth.make_qkv(wl, total)
    q.zero_()
    prob = ksa.Problem([1500], 8, 1, 16, 4, 2, 128, wl.scale)
    out, lse = parity.run_gpu(ctx, prob, q, k, v)
    cnt = np.array([orc.visible_count(1500, 8, 1, 16, p) for p in range(total)])
    assert np.abs(lse - np.log(cnt)[:, None]).max() < 1e-4
