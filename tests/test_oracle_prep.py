"""Pins of the Q/K/V preparation oracle (position ids, interpolation at summary positions, rotary embedding)
against what the paper and the mathematics fix; no GPU."""
import os

import numpy as np
import pytest

from oracle import ksa_prep_oracle as prep

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "position_ids_n10_k4.txt")


def test_position_ids_hand_written_example():
    want = [int(x) for line in open(GOLDEN) if not line.startswith("#") for x in line.split()]
    got = prep.position_ids([10], 4, 1)
    assert got.tolist() == want
    assert prep.summary_rows([10], 4, 1).tolist() == [False] * 4 + [True] + [False] * 4 + [True] + [False] * 2


@pytest.mark.parametrize("lens,k,m", [([37, 8, 1], 8, 1), ([130], 64, 8), ([25, 25], 5, 2), ([9], 3, 0)])
def test_position_ids_closed_form(lens, k, m):
    ids = prep.position_ids(lens, k, m)
    flags = prep.summary_rows(lens, k, m)
    assert len(ids) == sum(n + (n // k) * m for n in lens)              # Eq. 1: L = n + floor(n / k) m
    off = 0
    for n in lens:
        for j in range(n // k):
            base = off + j * (k + m)
            assert ids[base:base + k].tolist() == list(range(j * k, (j + 1) * k))
            assert ids[base + k:base + k + m].tolist() == [(j + 1) * k - 1] * m     # the chunk's last text token
            assert not flags[base:base + k].any() and flags[base + k:base + k + m].all()
        tail = off + (n // k) * (k + m)
        assert ids[tail:off + n + (n // k) * m].tolist() == list(range((n // k) * k, n))
        off += n + (n // k) * m


def test_anneal_lambda_schedule():
    assert prep.anneal_lambda(0, 100, 300) == 1.0 and prep.anneal_lambda(100, 100, 300) == 1.0
    assert prep.anneal_lambda(300, 100, 300) == 0.0 and prep.anneal_lambda(10 ** 6, 100, 300) == 0.0
    assert prep.anneal_lambda(200, 100, 300) == pytest.approx(0.5)
    assert prep.anneal_lambda(150, 100, 300) == pytest.approx(0.75)
    vals = [prep.anneal_lambda(s, 100, 300) for s in range(0, 400, 7)]
    assert all(a >= b for a, b in zip(vals, vals[1:]))                  # never increases


def test_rope_is_a_rotation_of_complex_pairs():
    """(x[d] + i x[d + D/2]) * exp(i pos theta^(-2d/D)): the same numbers by complex arithmetic."""
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 16))
    theta, pos = 1.0e4, 37
    got = prep.rope_row(x, pos, theta)
    z = x[:, :8] + 1j * x[:, 8:]
    w = z * np.exp(1j * pos * theta ** (-2.0 * np.arange(8) / 16))
    np.testing.assert_allclose(got[:, :8], w.real, rtol=0, atol=1e-12)
    np.testing.assert_allclose(got[:, 8:], w.imag, rtol=0, atol=1e-12)
    np.testing.assert_allclose(prep.rope_row(x, 0, theta), x, rtol=0, atol=0)             # position 0: identity
    np.testing.assert_allclose((got ** 2).sum(axis=1), (x ** 2).sum(axis=1), rtol=1e-12)  # norms are kept
    # d = 0 turns by exactly pos radians, the last pair by pos * theta^(-(D-2)/D)
    a, b = x[0, 0], x[0, 8]
    assert got[0, 0] == pytest.approx(a * np.cos(37.0) - b * np.sin(37.0))
    a, b = x[0, 7], x[0, 15]
    ang = 37.0 * theta ** (-14.0 / 16.0)
    assert got[0, 15] == pytest.approx(b * np.cos(ang) + a * np.sin(ang))


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, 32)), rng.standard_normal((1, 32))
    ref = (prep.rope_row(q, 100, 1e6) * prep.rope_row(k, 93, 1e6)).sum()
    for shift in (1, 17, 4096):
        got = (prep.rope_row(q, 100 + shift, 1e6) * prep.rope_row(k, 93 + shift, 1e6)).sum()
        assert got == pytest.approx(ref, abs=1e-9)
    other = (prep.rope_row(q, 100, 1e6) * prep.rope_row(k, 92, 1e6)).sum()
    assert abs(other - ref) > 1e-6                                      # ... and do depend on it


def test_prepare_special_cases():
    rng = np.random.default_rng(3)
    lens, k, m, Hq, Hkv, D, theta = [11, 4], 4, 1, 2, 1, 8, 1.0e4
    L = sum(n + (n // k) * m for n in lens)
    S = sum((n // k) * m for n in lens)
    qm, km, vm = rng.standard_normal((L, Hq, D)), rng.standard_normal((L, Hkv, D)), rng.standard_normal((L, Hkv, D))
    qs, ks, vs = rng.standard_normal((S, Hq, D)), rng.standard_normal((S, Hkv, D)), rng.standard_normal((S, Hkv, D))
    pos, flags = prep.position_ids(lens, k, m), prep.summary_rows(lens, k, m)
    q1, k1, v1 = prep.prepare(qm, km, vm, qs, ks, vs, lens, k, m, 1.0, theta)
    q0, k0, v0 = prep.prepare(qm, km, vm, qs, ks, vs, lens, k, m, 0.0, theta)
    qh, kh, vh = prep.prepare(qm, km, vm, qs, ks, vs, lens, k, m, 0.25, theta)
    srows = np.flatnonzero(flags)
    assert len(srows) == S
    for s, row in enumerate(srows):
        # lambda = 1: the summary weights alone; lambda = 0: the shared weights alone
        np.testing.assert_allclose(q1[row], prep.rope_row(qs[s], pos[row], theta), atol=1e-12)
        np.testing.assert_allclose(k0[row], prep.rope_row(km[row], pos[row], theta), atol=1e-12)
        np.testing.assert_allclose(v1[row], vs[s], atol=0)
        np.testing.assert_allclose(v0[row], vm[row], atol=0)
    for row in np.flatnonzero(~flags):
        # text rows: the shared projection, whatever lambda is; v is never rotated
        np.testing.assert_allclose(q1[row], q0[row], atol=0)
        np.testing.assert_allclose(kh[row], prep.rope_row(km[row], pos[row], theta), atol=1e-12)
        np.testing.assert_allclose(vh[row], vm[row], atol=0)
    # linear in lambda (interpolation and rotation are both linear)
    np.testing.assert_allclose(qh, 0.25 * q1 + 0.75 * q0, atol=1e-12)
    np.testing.assert_allclose(kh, 0.25 * k1 + 0.75 * k0, atol=1e-12)
    np.testing.assert_allclose(vh, 0.25 * v1 + 0.75 * v0, atol=1e-12)
    # the second sequence starts again at position 0
    first_of_second = lens[0] + (lens[0] // k) * m
    np.testing.assert_allclose(q0[first_of_second], qm[first_of_second], atol=0)
