"""Host-side logic of the CUDA library, checked on CPU: exports, layout helpers, argument
validation and the block-sparse schedule against the oracle's explicit mask."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from oracle import ksa_oracle as orc
from paper_2604_24432_b200 import binding as ksa
from paper_2604_24432_b200 import build as ksa_build
from tests.helpers import aug_positions

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    ksa_build.build()


def test_exports_match_header():
    declared = set()
    inc = os.path.join(ROOT, "include")
    for name in sorted(os.listdir(inc)):            # every header of the C ABI
        hdr = open(os.path.join(inc, name)).read()
        hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
        declared |= set(re.findall(r"\b(ksa_[a-z_]+)\s*\(", hdr))
    assert declared == set(ksa.EXPORTS)
    L = ksa.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert ctypes.sizeof(ksa.ksa_params) == 120
    assert ctypes.sizeof(ksa.ksa_tile_rec) == 32
    assert ctypes.sizeof(ksa.ksa_cache_params) == 40


def test_aug_len_and_pairs_match_oracle():
    for n, k, m in [(0, 8, 1), (7, 8, 1), (8, 8, 1), (1000, 8, 1), (1000, 64, 8), (5, 1, 0)]:
        assert ksa.aug_len(n, k, m) == orc.aug_len(n, k, m)
    assert ksa.aug_len(-1, 8, 1) == -1 and ksa.aug_len(8, 0, 1) == -1
    for lens, k, m, C in [([300], 8, 1, 2), ([100, 37, 64], 8, 1, 2), ([257], 64, 8, 1), ([513, 9], 4, 0, 3)]:
        prob = ksa.Problem(lens, k, m, C, 4, 2, 64, 0.125)
        assert ksa.total_aug_len(prob) == sum(orc.aug_len(n, k, m) for n in lens)
        assert ksa.visible_pairs(prob) == orc.total_pairs(lens, k, m, C)
        prob.flags = ksa.KSA_FLAG_SUMMARY_TEXT_ONLY
        assert ksa.visible_pairs(prob) == orc.total_pairs(lens, k, m, C, orc.SUMMARY_TEXT_ONLY)


def test_workload_visible_flops():
    """Visible pairs of the 128K workload (closed form) -> 19.52 TFLOP at 32 heads, D = 128."""
    prob = ksa.Problem([131072], 8, 1, 128, 32, 4, 128, 0.0883)
    pairs = ksa.visible_pairs(prob)
    i = np.arange(131072, dtype=np.int64)
    far = np.maximum(0, i // 8 - 128)
    assert pairs == int(((i - 8 * far + 1) + far).sum()) + 16384 * 9
    assert abs(4 * 128 * 32 * pairs / 1e12 - 19.52) < 0.01


@pytest.mark.parametrize("lens,k,m,C", [
    ([700], 8, 1, 2), ([700], 8, 1, 20), ([700], 8, 1, 128), ([515], 64, 8, 1), ([1030], 64, 8, 0),
    ([300, 129, 128, 5], 8, 1, 3), ([640], 1, 1, 100), ([900], 3, 2, 50), ([777], 16, 0, 7),
    ([2100], 8, 1, 16), ([1500], 2, 1, 0), ([1280], 128, 128, 1), ([1290], 200, 3, 1),
])
def test_schedule_bit_exact_against_oracle_mask(lens, k, m, C):
    """The visited tiles are exactly the tiles holding >= 1 visible pair of the oracle's
    explicit mask; they cover every visible pair of every text row once; is_full is set
    iff every pair of the rectangle is visible."""
    prob = ksa.Problem(lens, k, m, C, 4, 2, 64, 0.125)
    recs = ksa.schedule_dump(prob)
    TM = 128
    for b, n in enumerate(lens):
        tp, sp, L = aug_positions(n, k, m)
        tpos = np.array([tp[i] for i in range(n)])
        spos = np.array([sp[(u // m, u % m)] for u in range((n // k) * m)], dtype=np.int64) if m else np.zeros(0, np.int64)
        mask = orc.mask(n, k, m, C).astype(bool)
        vis_text = mask[tpos][:, tpos]                    # [text query, text key]
        vis_summ = mask[tpos][:, spos] if len(spos) else np.zeros((n, 0), bool)
        cover_t = np.zeros_like(vis_text, dtype=np.int32)
        cover_s = np.zeros_like(vis_summ, dtype=np.int32)
        rb = recs[recs["seq"] == b]
        seen = set()
        for r in rb:
            assert r["q_stream"] == ksa.KSA_STREAM_TEXT
            assert r["q_row0"] % TM == 0 and r["kv_row0"] % TM == 0
            assert 1 <= r["q_rows"] <= TM and 1 <= r["kv_rows"] <= TM
            qs = slice(r["q_row0"], r["q_row0"] + r["q_rows"])
            ks_ = slice(r["kv_row0"], r["kv_row0"] + r["kv_rows"])
            assert qs.stop <= n
            if r["kv_stream"] == ksa.KSA_STREAM_TEXT:
                assert ks_.stop <= n
                sub = vis_text[qs, ks_]
                cover_t[qs, ks_] += 1
            else:
                assert ks_.stop <= len(spos)
                sub = vis_summ[qs, ks_]
                cover_s[qs, ks_] += 1
            assert sub.any(), tuple(r)
            assert bool(r["is_full"]) == bool(sub.all()), tuple(r)
            key = (int(r["q_row0"]), int(r["kv_stream"]), int(r["kv_row0"]))
            assert key not in seen
            seen.add(key)
        # every visible pair is inside exactly one visited tile
        assert (cover_t[vis_text] == 1).all() and (cover_s[vis_summ] == 1).all()
        # exhaustive tile grid: any tile with a visible pair must be listed
        for q0 in range(0, n, TM):
            for a0 in range(0, n, TM):
                if vis_text[q0:q0 + TM, a0:a0 + TM].any():
                    assert (q0, ksa.KSA_STREAM_TEXT, a0) in seen
            for u0 in range(0, len(spos), TM):
                if vis_summ[q0:q0 + TM, u0:u0 + TM].any():
                    assert (q0, ksa.KSA_STREAM_SUMMARY, u0) in seen


def _check_query_tile(recs_tile, n, k, m, C, q0, TM=128):
    """One query tile of one sequence against the oracle's explicit mask rows (every key position of the
    sequence is put through the oracle's predicate): visited tiles <=> a visible pair, is_full <=> all visible,
    nothing visited twice."""
    tp, sp, L = None, None, orc.aug_len(n, k, m)
    s_len = k + m
    J = n // k
    i = np.arange(n, dtype=np.int64)
    tpos = np.where(i < J * k, (i // k) * s_len + i % k, J * s_len + (i - J * k))          # Eq. 1
    u = np.arange(J * m, dtype=np.int64)
    spos = (u // max(m, 1)) * s_len + k + u % max(m, 1) if m else np.zeros(0, np.int64)
    q1 = min(n, q0 + TM)
    rows = np.stack([orc.mask_row(n, k, m, C, int(tpos[r])) for r in range(q0, q1)]).astype(bool)
    vis_t, vis_s = rows[:, tpos], rows[:, spos]
    assert rows.sum() == vis_t.sum() + vis_s.sum()
    want = {}
    for a0 in range(0, n, TM):
        sub = vis_t[:, a0:a0 + TM]
        if sub.any():
            want[(ksa.KSA_STREAM_TEXT, a0)] = (min(TM, n - a0), bool(sub.all()))
    for u0 in range(0, len(spos), TM):
        sub = vis_s[:, u0:u0 + TM]
        if sub.any():
            want[(ksa.KSA_STREAM_SUMMARY, u0)] = (min(TM, len(spos) - u0), bool(sub.all()))
    got = {}
    for r in recs_tile:
        key = (int(r["kv_stream"]), int(r["kv_row0"]))
        assert key not in got, key
        assert int(r["q_rows"]) == q1 - q0
        got[key] = (int(r["kv_rows"]), bool(r["is_full"]))
    assert got == want


@pytest.mark.parametrize("layout", ["P", "G"])
def test_schedule_bit_exact_8k_workload(layout):
    """The 8K workload, every query tile, both layouts."""
    from paper_2604_24432_b200 import synth
    wl, lay = synth.WORKLOADS["8k"], {"P": synth.LAYOUT_P, "G": synth.LAYOUT_G}[layout]
    prob = ksa.Problem(wl.text_lens, lay.k, lay.m, lay.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    recs = ksa.schedule_dump(prob)
    n = wl.text_lens[0]
    for q0 in range(0, n, 128):
        _check_query_tile(recs[(recs["seq"] == 0) & (recs["q_row0"] == q0)], n, lay.k, lay.m, lay.C, q0)
    assert len(recs) == sum(len(recs[(recs["seq"] == 0) & (recs["q_row0"] == q0)]) for q0 in range(0, n, 128))


@pytest.mark.parametrize("name,layout", [("tiny", "P"), ("tiny", "G"), ("32k", "P"), ("32k", "G"), ("128k", "P"), ("128k", "G"),
                                         ("varlen", "P"), ("varlen", "G")])
def test_schedule_bit_exact_workloads_sampled(name, layout):
    """The other workloads at full size: in every sequence the first and last query tiles, the tiles on either side of
    the point where the window stops reaching token 0, the tile in the middle and seeded random tiles, each checked
    tile by tile against the oracle's mask rows."""
    from paper_2604_24432_b200 import synth
    wl, lay = synth.WORKLOADS[name], {"P": synth.LAYOUT_P, "G": synth.LAYOUT_G}[layout]
    prob = ksa.Problem(wl.text_lens, lay.k, lay.m, lay.C, wl.Hq, wl.Hkv, wl.D, wl.scale)
    recs = ksa.schedule_dump(prob)
    rng = np.random.default_rng(7)
    for b, n in enumerate(wl.text_lens):
        n_t = (n + 127) // 128
        edge = (lay.C * lay.k) // 128                      # first tile whose rows start to lose token 0
        tiles = {0, n_t - 1, max(0, n_t - 2), min(n_t - 1, edge), min(n_t - 1, edge + 1), max(0, min(n_t - 1, edge - 1)), n_t // 2}
        tiles |= set(int(t) for t in rng.integers(0, n_t, size=2 if len(wl.text_lens) > 2 else 4))
        rb = recs[recs["seq"] == b]
        for t in sorted(tiles):
            _check_query_tile(rb[rb["q_row0"] == t * 128], n, lay.k, lay.m, lay.C, t * 128)


def test_schedule_tile_counts_128k():
    """Per-head visited tiles of the 128K workload: 65,024 summary + 9,180 text tiles."""
    prob = ksa.Problem([131072], 8, 1, 128, 32, 4, 128, 0.0883)
    recs = ksa.schedule_dump(prob)
    assert int((recs["kv_stream"] == ksa.KSA_STREAM_SUMMARY).sum()) == 65024
    assert int((recs["kv_stream"] == ksa.KSA_STREAM_TEXT).sum()) == 9180


def _status_of(fn):
    try:
        fn()
    except ksa.KsaError as e:
        return e.status
    return ksa.KSA_OK


def test_invalid_arguments_are_rejected():
    good = dict(text_lens=[100], k=8, m=1, C=2, Hq=4, Hkv=2, D=64, scale=0.125)
    assert _status_of(lambda: ksa.workspace_bytes(ksa.Problem(**good))) == ksa.KSA_OK
    bad = [
        (dict(k=0), ksa.KSA_ERR_INVALID_ARG), (dict(m=-1), ksa.KSA_ERR_INVALID_ARG),
        (dict(C=-1), ksa.KSA_ERR_INVALID_ARG), (dict(Hq=3), ksa.KSA_ERR_INVALID_ARG),
        (dict(D=96), ksa.KSA_ERR_UNSUPPORTED), (dict(scale=0.0), ksa.KSA_ERR_INVALID_ARG),
        (dict(text_lens=[10, 0, 5]), ksa.KSA_ERR_INVALID_ARG), (dict(flags=0x80), ksa.KSA_ERR_INVALID_ARG),
        (dict(scale=float("nan")), ksa.KSA_ERR_INVALID_ARG),
    ]
    for change, want in bad:
        prob = ksa.Problem(**{**good, **change})
        assert _status_of(lambda: ksa.workspace_bytes(prob)) == want, change
        assert _status_of(lambda: ksa.schedule_dump(prob)) == want, change
    # wrong struct_size
    p = ksa.Problem(**good).params()
    p.struct_size = 8
    n = ctypes.c_size_t()
    assert ksa.lib().ksa_workspace_bytes(None, ctypes.byref(p), ctypes.byref(n)) == ksa.KSA_ERR_INVALID_ARG
    assert ksa.lib().ksa_workspace_bytes(None, None, ctypes.byref(n)) == ksa.KSA_ERR_INVALID_ARG
    assert ksa.strerror(ksa.KSA_ERR_WORKSPACE).startswith("workspace")


def test_create_fails_loudly_without_device():
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(ksa.KsaError) as ei:
        ksa.Context(0)
    assert ei.value.status in (ksa.KSA_ERR_CUDA, ksa.KSA_ERR_INVALID_ARG)
    assert ksa.lib().ksa_destroy(None) == ksa.KSA_OK
    assert ksa.lib().ksa_attn_fwd(None, None, None, None, None, None, None, 0, None, None) == ksa.KSA_ERR_INVALID_ARG


def test_workspace_size_formula():
    prob = ksa.Problem([1000, 300], 8, 1, 4, 8, 2, 128, 0.088)
    text_rows = 1024 + 384
    summ_rows = 128 + 128
    want = (8 + 2 + 2) * text_rows * 256 + 4 * summ_rows * 256
    got = ksa.workspace_bytes(prob)
    assert want <= got <= want + 5 * 1024


def test_no_pack_mode_needs_no_workspace():
    """Whole chunks everywhere and a tile that is a whole number of chunks: nothing is packed."""
    assert ksa.workspace_bytes(ksa.Problem([1024, 640], 8, 1, 4, 8, 2, 128, 0.088)) == 256
    assert ksa.workspace_bytes(ksa.Problem([1024, 640], 8, 0, 4, 8, 2, 128, 0.088)) == 256
    assert ksa.workspace_bytes(ksa.Problem([1024, 641], 8, 1, 4, 8, 2, 128, 0.088)) > 256      # ragged tail
    assert ksa.workspace_bytes(ksa.Problem([1020], 3, 1, 4, 8, 2, 128, 0.088)) > 256           # 128 % k != 0
    assert ksa.workspace_bytes(ksa.Problem([1024], 8, 3, 4, 8, 2, 128, 0.088)) > 256           # 128 % m != 0
    ref = ksa.Problem([1024, 640], 8, 1, 4, 8, 2, 128, 0.088, ksa.KSA_FLAG_REFERENCE_KERNEL)
    assert ksa.workspace_bytes(ref) > 256                                                      # cross-check kernel reads the packed streams


def test_backward_workspace_and_limits():
    prob = ksa.Problem([1000, 300], 8, 1, 4, 8, 2, 128, 0.088)
    text_rows, summ_rows = 1024 + 384, 128 + 128
    fwd = (8 + 2 + 2) * text_rows * 256 + 4 * summ_rows * 256
    extra = 8 * text_rows * 256 + 2 * 8 * text_rows * 4 + 2 * 2 * (text_rows + summ_rows) * 128 * 4
    got = ksa.bwd_workspace_bytes(prob)
    assert fwd + extra <= got <= fwd + extra + 16 * 1024
    # whole chunks and head_dim 128: q, k, v, dout are read in place -- only the row scalars and the fp32 accumulators
    direct = ksa.Problem([1024, 640], 8, 1, 4, 8, 2, 128, 0.088)
    text_rows, summ_rows = 1024 + 640, 128 + 128
    small = 2 * 8 * text_rows * 4 + 2 * 2 * (text_rows + summ_rows) * 128 * 4
    assert small <= ksa.bwd_workspace_bytes(direct) <= small + 16 * 1024
    many = ksa.Problem([8] * 70000, 8, 1, 2, 4, 2, 64, 0.125)
    assert _status_of(lambda: ksa.workspace_bytes(many)) == ksa.KSA_ERR_UNSUPPORTED
