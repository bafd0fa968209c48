"""Plain numpy (fp64) statement of what happens to Q, K, V between the projections and the KSA attention
operator: the position ids of the augmented sequence, the interpolation of the two projections at summary
positions and the rotary position embedding.

TEST INFRASTRUCTURE ONLY: imported by the tests and by the benchmark's CPU-baseline leg.  The CUDA package never
imports this module and this module never imports the CUDA package.  Everything is written row by row, in the
order the paper states it; nothing is vectorised across rows.

What the paper fixes
  * the augmented sequence: m summary tokens after every full chunk of k text tokens (Eq. 1);
  * the position id of a summary token is that of its own chunk's last text token (second bullet of
    Sec. 2.2.1); text tokens keep their own index in the original sequence;
  * at a summary position the Q, K, V fed into the attention are lambda x_s + (1 - lambda) x_s^main, the two
    projections of the same hidden state, with lambda following a linear ramp between two training steps
    ("Parameter annealing for CPT", Sec. 4.1);
  * RoPE is applied to every key before it is cached (Sec. 2.3.1), with base theta (Table 3).
What it leaves open (readings)
  * the rotary embedding itself: taken as in the model family the paper continues training from -- element d
    of the first half of a head is paired with element d + D/2, the pair is rotated by the angle
    pos * theta^(-2 d / D);
  * with several summary tokens per chunk, all of them take the chunk's last text token's position id;
  * the interpolation comes before the rotation (both are linear and the two projections share the position,
    so the order does not change the result).
"""
from __future__ import annotations

import numpy as np


def position_ids(text_lens, k, m):
    """Position id of every row of the augmented batch, sequence after sequence (Eq. 1 and Sec. 2.2.1)."""
    ids = []
    for n in text_lens:
        in_chunk = 0
        for i in range(n):
            ids.append(i)                       # a text token keeps its index in the original sequence
            in_chunk += 1
            if in_chunk == k:                   # chunk complete: its summary tokens follow
                for _ in range(m):
                    ids.append(i)               # ... with the position id of the chunk's last text token
                in_chunk = 0
    return np.asarray(ids, dtype=np.int64)


def summary_rows(text_lens, k, m):
    """Boolean per augmented row: is it a summary token (Eq. 1)."""
    flags = []
    for n in text_lens:
        in_chunk = 0
        for _ in range(n):
            flags.append(False)
            in_chunk += 1
            if in_chunk == k:
                flags.extend([True] * m)
                in_chunk = 0
    return np.asarray(flags, dtype=bool)


def anneal_lambda(step, s_start, s_end):
    """Interpolation coefficient of the annealing schedule (Sec. 4.1, "Parameter annealing for CPT")."""
    if step <= s_start:
        return 1.0
    if step >= s_end:
        return 0.0
    return 1.0 - (step - s_start) / float(s_end - s_start)


def rope_row(x, pos, theta):
    """Rotary embedding of one row x[H, D] at position pos: the pair (d, d + D/2) turns by pos * theta^(-2d/D)."""
    H, D = x.shape
    half = D // 2
    out = np.empty_like(x, dtype=np.float64)
    for h in range(H):
        for d in range(half):
            angle = float(pos) * float(theta) ** (-2.0 * d / D)
            c, s = np.cos(angle), np.sin(angle)
            a, b = float(x[h, d]), float(x[h, d + half])
            out[h, d] = a * c - b * s
            out[h, d + half] = b * c + a * s
    return out


def prepare(q_main, k_main, v_main, q_summ, k_summ, v_summ, text_lens, k, m, lam, theta):
    """Attention inputs from the projections.

    q_main [L, Hq, D], k_main / v_main [L, Hkv, D]: projections with the shared weights at every augmented row;
    q_summ / k_summ / v_summ [S, H, D]: projections with the summary weights at the S summary rows, in order.
    Returns (q, k, v) in fp64: interpolated at summary rows, q and k rotated, v not."""
    pos = position_ids(text_lens, k, m)
    is_summ = summary_rows(text_lens, k, m)
    L = len(pos)
    assert q_main.shape[0] == L and k_main.shape[0] == L and v_main.shape[0] == L
    q = np.empty(q_main.shape, dtype=np.float64)
    kk = np.empty(k_main.shape, dtype=np.float64)
    v = np.empty(v_main.shape, dtype=np.float64)
    s = 0                                        # running index into the summary projections
    for row in range(L):
        xq = np.asarray(q_main[row], dtype=np.float64)
        xk = np.asarray(k_main[row], dtype=np.float64)
        xv = np.asarray(v_main[row], dtype=np.float64)
        if is_summ[row]:
            xq = lam * np.asarray(q_summ[s], dtype=np.float64) + (1.0 - lam) * xq
            xk = lam * np.asarray(k_summ[s], dtype=np.float64) + (1.0 - lam) * xk
            xv = lam * np.asarray(v_summ[s], dtype=np.float64) + (1.0 - lam) * xv
            s += 1
        q[row] = rope_row(xq, pos[row], theta)
        kk[row] = rope_row(xk, pos[row], theta)
        v[row] = xv
    return q, kk, v
