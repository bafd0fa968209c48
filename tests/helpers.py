"""Independent restatements used to pin the oracle (pure Python / numpy, tiny sizes).

Nothing here calls the oracle's predicate: the visible sets are enumerated as the
lists Eq. 3 writes out, and mapped to augmented positions through Eq. 1.
"""
import numpy as np


def aug_positions(n, k, m):
    """Eq. 1 (m summaries per full chunk, none for a trailing partial chunk).

    Returns (text_pos[i], summ_pos[(j, r)], L)."""
    text_pos, summ_pos, p = {}, {}, 0
    J = n // k
    for j in range(J):
        for o in range(k):
            text_pos[j * k + o] = p
            p += 1
        for r in range(m):
            summ_pos[(j, r)] = p
            p += 1
    for i in range(J * k, n):
        text_pos[i] = p
        p += 1
    return text_pos, summ_pos, p


def visible_sets(n, k, m, C, text_only=False):
    """dict: augmented query position -> set of visible augmented key positions,
    enumerated as the lists of Eq. 3 / the summary rule."""
    tp, sp, L = aug_positions(n, k, m)
    J = n // k
    vis = {}
    for i in range(n):
        c = i // k
        keys = set()
        for j in range(0, c - C):             # s_0 .. s_{c-C-1}
            if j < J:
                for r in range(m):
                    keys.add(sp[(j, r)])
        start = max(0, c - C) * k             # t_{(c-C)k} .. t_i
        for ip in range(start, i + 1):
            keys.add(tp[ip])
        vis[tp[i]] = keys
    for j in range(J):
        for r in range(m):
            keys = {tp[i] for i in range(j * k, j * k + k)}
            if not text_only:
                keys |= {sp[(j, rr)] for rr in range(r + 1)}
            vis[sp[(j, r)]] = keys
    return vis, L


def dense_mask(n, k, m, C, text_only=False):
    vis, L = visible_sets(n, k, m, C, text_only)
    M = np.zeros((L, L), dtype=bool)
    for p, keys in vis.items():
        M[p, list(keys)] = True
    return M


def bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dense_attention(q, k, v, mask, scale, G=1):
    """Textbook masked softmax attention in fp64.  q [L,Hq,D], k/v [L,Hkv,D] float64,
    mask [L,L] bool.  Returns out [L,Hq,D], lse [L,Hq]."""
    L, Hq, D = q.shape
    out = np.zeros((L, Hq, D))
    lse = np.zeros((L, Hq))
    for h in range(Hq):
        s = scale * (q[:, h, :] @ k[:, h // G, :].T)
        s = np.where(mask, s, -np.inf)
        mx = s.max(axis=1, keepdims=True)
        p = np.exp(s - mx)
        l = p.sum(axis=1, keepdims=True)
        out[:, h, :] = (p / l) @ v[:, h // G, :]
        lse[:, h] = (mx + np.log(l))[:, 0]
    return out, lse


def rand_bf16(rng, shape, scale=1.0):
    """Random values exactly representable in bf16, returned as (uint16 bits, float64)."""
    x = (rng.standard_normal(shape) * scale).astype(np.float32)
    b = (x.view(np.uint32) >> 16).astype(np.uint16)      # truncation is fine for test data
    return b, bf16_bits_to_f64(b)
