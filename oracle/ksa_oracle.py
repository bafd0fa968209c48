"""ctypes wrapper around the plain C KSA oracle (``ksa_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and this
module never imports the CUDA package.

The wrapper only marshals numpy arrays; all arithmetic lives in the C file, which
states the KSA operator exactly as the paper defines it (Eq. 1, Eq. 3, the summary
visibility bullet of Sec. 2.2.1 and the masked-softmax equation of Sec. 4.1.4).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ksa_oracle.c")
_HDR = os.path.join(_HERE, "ksa_oracle.h")
_LIB = os.path.join(_HERE, "libksa_oracle.so")

SUMMARY_TEXT_ONLY = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3, OpenMP).  Returns the path of the library."""
    stale = (
        force
        or not os.path.exists(_LIB)
        or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    )
    if stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    i32, i64, u32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32
    vp = ctypes.c_void_p
    lib.ksa_oracle_aug_len.restype = i64
    lib.ksa_oracle_aug_len.argtypes = [i64, i32, i32]
    lib.ksa_oracle_decode_pos.restype = ctypes.c_int
    lib.ksa_oracle_decode_pos.argtypes = [i64, i32, i32, i64, vp, vp, vp]
    lib.ksa_oracle_visible.restype = ctypes.c_int
    lib.ksa_oracle_visible.argtypes = [i64, i32, i32, i32, u32, i64, i64]
    lib.ksa_oracle_mask_row.restype = i64
    lib.ksa_oracle_mask_row.argtypes = [i64, i32, i32, i32, u32, i64, vp]
    lib.ksa_oracle_visible_count.restype = i64
    lib.ksa_oracle_visible_count.argtypes = [i64, i32, i32, i32, u32, i64]
    lib.ksa_oracle_total_pairs.restype = i64
    lib.ksa_oracle_total_pairs.argtypes = [i32, vp, i32, i32, i32, u32]
    lib.ksa_oracle_fwd.restype = ctypes.c_int
    lib.ksa_oracle_fwd.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, i32,
                                   ctypes.c_double, u32, vp, i64, vp, vp, vp]
    lib.ksa_oracle_bwd.argtypes = [vp, vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, i32, ctypes.c_double, u32, vp, vp, vp]
    lib.ksa_oracle_bwd_rows.argtypes = [vp, vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, i32, ctypes.c_double, u32,
                                        vp, i64, vp, vp, i64, vp, vp]
    lib.ksa_oracle_num_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def aug_len(n_text: int, k: int, m: int) -> int:
    return int(_load().ksa_oracle_aug_len(n_text, k, m))


def decode_pos(n_text: int, k: int, m: int, p: int):
    """-> (is_summary, index, r): text token index, or (chunk j, summary slot r)."""
    a, b, c = ctypes.c_int32(), ctypes.c_int64(), ctypes.c_int32()
    rc = _load().ksa_oracle_decode_pos(n_text, k, m, p, ctypes.addressof(a),
                                       ctypes.addressof(b), ctypes.addressof(c))
    if rc != 0:
        raise ValueError("position out of range")
    return bool(a.value), int(b.value), int(c.value)


def visible(n_text, k, m, C, pq, pk, flags=0) -> bool:
    rc = _load().ksa_oracle_visible(n_text, k, m, C, flags, pq, pk)
    if rc < 0:
        raise ValueError("bad argument")
    return bool(rc)


def mask_row(n_text, k, m, C, pq, flags=0) -> np.ndarray:
    L = aug_len(n_text, k, m)
    row = np.zeros(L, dtype=np.uint8)
    rc = _load().ksa_oracle_mask_row(n_text, k, m, C, flags, pq, row.ctypes.data)
    if rc < 0:
        raise ValueError("bad argument")
    return row


def mask(n_text, k, m, C, flags=0) -> np.ndarray:
    """Full explicit mask [L, L] of one sequence (small sequences only)."""
    L = aug_len(n_text, k, m)
    out = np.zeros((L, L), dtype=np.uint8)
    for p in range(L):
        out[p] = mask_row(n_text, k, m, C, p, flags)
    return out


def visible_count(n_text, k, m, C, pq, flags=0) -> int:
    return int(_load().ksa_oracle_visible_count(n_text, k, m, C, flags, pq))


def total_pairs(text_lens, k, m, C, flags=0) -> int:
    cu = np.concatenate([[0], np.cumsum(np.asarray(text_lens, dtype=np.int64))]).astype(np.int32)
    return int(_load().ksa_oracle_total_pairs(len(text_lens), cu.ctypes.data, k, m, C, flags))


def num_threads() -> int:
    return int(_load().ksa_oracle_num_threads())


def fwd(q_bits, k_bits, v_bits, text_lens, k, m, C, scale, flags=0, rows=None):
    """KSA forward in fp64.

    q_bits [total_aug, Hq, D], k_bits/v_bits [total_aug, Hkv, D]: uint16 arrays holding
    bf16 bit patterns.  ``rows``: optional global augmented row indices to evaluate.
    Returns (out [R, Hq, D] float64, lse [R, Hq] float64, count [R] int64).
    """
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    total, Hq, D = q_bits.shape
    Hkv = k_bits.shape[1]
    assert k_bits.shape == (total, Hkv, D) and v_bits.shape == (total, Hkv, D)
    cu = np.concatenate([[0], np.cumsum(np.asarray(text_lens, dtype=np.int64))]).astype(np.int32)
    assert sum(aug_len(int(n), k, m) for n in text_lens) == total, "layout/shape mismatch"
    if rows is None:
        R, rows_ptr = total, None
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        R, rows_ptr = rows.shape[0], rows.ctypes.data
    out = np.empty((R, Hq, D), dtype=np.float64)
    lse = np.empty((R, Hq), dtype=np.float64)
    cnt = np.empty((R,), dtype=np.int64)
    rc = _load().ksa_oracle_fwd(q_bits.ctypes.data, k_bits.ctypes.data, v_bits.ctypes.data,
                                len(text_lens), cu.ctypes.data, k, m, C, Hq, Hkv, D,
                                float(scale), flags, rows_ptr, R,
                                out.ctypes.data, lse.ctypes.data, cnt.ctypes.data)
    if rc != 0:
        raise ValueError("ksa_oracle_fwd: bad argument")
    return out, lse, cnt


def bwd(q_bits, k_bits, v_bits, dout_bits, text_lens, k, m, C, scale, flags=0):
    """Gradients (dq, dk, dv) in fp64 for the upstream gradient dout (bf16 bit patterns), all rows."""
    lib = _load()
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    dout_bits = np.ascontiguousarray(dout_bits, dtype=np.uint16)
    total, Hq, D = q_bits.shape
    Hkv = k_bits.shape[1]
    cu = np.concatenate([[0], np.cumsum(np.asarray(text_lens, dtype=np.int64))]).astype(np.int32)
    dq = np.empty((total, Hq, D), dtype=np.float64)
    dk = np.empty((total, Hkv, D), dtype=np.float64)
    dv = np.empty((total, Hkv, D), dtype=np.float64)
    rc = lib.ksa_oracle_bwd(q_bits.ctypes.data, k_bits.ctypes.data, v_bits.ctypes.data, dout_bits.ctypes.data,
                            len(text_lens), cu.ctypes.data, k, m, C, Hq, Hkv, D, float(scale), flags,
                            dq.ctypes.data, dk.ctypes.data, dv.ctypes.data)
    if rc != 0:
        raise ValueError("ksa_oracle_bwd: bad arguments")
    return dq, dk, dv


def bwd_rows(q_bits, k_bits, v_bits, dout_bits, text_lens, k, m, C, scale, q_rows, k_rows, flags=0):
    """Gradients on a sample: dq [len(q_rows), Hq, D] of the query rows and dk, dv [len(k_rows), Hkv, D] of the key rows
    (global augmented row indices), all float64."""
    lib = _load()
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    dout_bits = np.ascontiguousarray(dout_bits, dtype=np.uint16)
    total, Hq, D = q_bits.shape
    Hkv = k_bits.shape[1]
    cu = np.concatenate([[0], np.cumsum(np.asarray(text_lens, dtype=np.int64))]).astype(np.int32)
    q_rows = np.ascontiguousarray(q_rows, dtype=np.int64)
    k_rows = np.ascontiguousarray(k_rows, dtype=np.int64)
    dq = np.empty((len(q_rows), Hq, D), dtype=np.float64)
    dk = np.empty((len(k_rows), Hkv, D), dtype=np.float64)
    dv = np.empty((len(k_rows), Hkv, D), dtype=np.float64)
    rc = lib.ksa_oracle_bwd_rows(q_bits.ctypes.data, k_bits.ctypes.data, v_bits.ctypes.data, dout_bits.ctypes.data,
                                 len(text_lens), cu.ctypes.data, k, m, C, Hq, Hkv, D, float(scale), flags,
                                 q_rows.ctypes.data, len(q_rows), dq.ctypes.data,
                                 k_rows.ctypes.data, len(k_rows), dk.ctypes.data, dv.ctypes.data)
    if rc != 0:
        raise ValueError("ksa_oracle_bwd_rows: bad arguments (%d)" % rc)
    return dq, dk, dv
