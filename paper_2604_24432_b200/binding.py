"""Thin ctypes binding of ``include/ksa.h`` (same names, argument marshalling only).

Every step of the forward pass runs inside the shared library's CUDA kernels; this
module allocates nothing on the device except through torch tensors the caller (or the
convenience wrapper ``attn_fwd``) owns.  If the shared library is missing the import of
this module still succeeds, but every entry point raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# KSA_B200_LIB_VARIANT=debug / asan selects a test variant of the library (see build.py); unset: the product library
LIB_PATH = os.path.join(_HERE, "libksa_b200%s.so" % ("_" + os.environ["KSA_B200_LIB_VARIANT"] if os.environ.get("KSA_B200_LIB_VARIANT") else ""))

KSA_OK = 0
KSA_ERR_INVALID_ARG, KSA_ERR_UNSUPPORTED, KSA_ERR_WORKSPACE = -1, -2, -3
KSA_ERR_CUDA, KSA_ERR_TIMEOUT, KSA_ERR_NOMEM, KSA_ERR_INTERNAL = -4, -5, -6, -7
KSA_PREP_NO_ROPE = 1
KSA_FLAG_SUMMARY_TEXT_ONLY = 0x1
KSA_FLAG_REFERENCE_KERNEL = 0x2
KSA_FLAG_SINGLE_CTA_KERNEL = 0x4
KSA_FLAG_CTA_PAIR_KERNEL = 0x8
KSA_FLAG_BWD_MMA_SYNC_KERNELS = 0x10
KSA_STREAM_TEXT, KSA_STREAM_SUMMARY = 0, 1

EXPORTS = [
    "ksa_create", "ksa_destroy", "ksa_aug_len", "ksa_total_aug_len", "ksa_workspace_bytes",
    "ksa_visible_pairs", "ksa_attn_fwd", "ksa_host_staging_bytes", "ksa_attn_fwd_host",
    "ksa_attn_fwd_noalloc", "ksa_noalloc_last_device_status", "ksa_bwd_workspace_bytes", "ksa_attn_bwd",
    "ksa_schedule_dump", "ksa_selftest_bounded_wait", "ksa_last_device_status", "ksa_clear_device_status",
    "ksa_last_cuda_error", "ksa_launch_count", "ksa_device_info", "ksa_enable_kernel_timing", "ksa_text_kernel_ms",
    "ksa_strerror",
    "ksa_cache_rows", "ksa_cache_bytes", "ksa_cache_slice", "ksa_cache_reset", "ksa_cache_fill_from_prefill",
    "ksa_decode_text", "ksa_decode_summary",
    "ksa_anneal_lambda", "ksa_position_ids", "ksa_total_summary_rows", "ksa_qkv_prepare",
    "ksa_prepared_workspace_bytes", "ksa_attn_fwd_prepared",
    "ksa_part_rows", "ksa_attn_fwd_part",
]


class ksa_params(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("num_seqs", ctypes.c_int32),
        ("cu_text_lens", ctypes.c_void_p),
        ("chunk_len", ctypes.c_int32), ("summaries_per_chunk", ctypes.c_int32),
        ("window_chunks", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("q_stride_tok", ctypes.c_int64), ("q_stride_head", ctypes.c_int64),
        ("k_stride_tok", ctypes.c_int64), ("k_stride_head", ctypes.c_int64),
        ("v_stride_tok", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
        ("o_stride_tok", ctypes.c_int64), ("o_stride_head", ctypes.c_int64),
        ("flags", ctypes.c_uint32), ("reserved", ctypes.c_uint32),
    ]


class ksa_cache_params(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("batch", ctypes.c_int32), ("chunk_len", ctypes.c_int32),
        ("window_chunks", ctypes.c_int32), ("max_summaries", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_uint32),
    ]


class ksa_tile_rec(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("seq", "q_stream", "q_row0", "q_rows", "kv_stream", "kv_row0", "kv_rows", "is_full")]


class KsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


_lib = None


def lib():
    """Loads the shared library (built by ``paper_2604_24432_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2604_24432_b200.build` "
            "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    pp = ctypes.POINTER(ksa_params)
    L.ksa_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
    L.ksa_destroy.argtypes = [vp]
    L.ksa_aug_len.restype = i64
    L.ksa_aug_len.argtypes = [i64, i32, i32]
    L.ksa_total_aug_len.restype = i64
    L.ksa_total_aug_len.argtypes = [pp]
    L.ksa_workspace_bytes.argtypes = [vp, pp, ctypes.POINTER(ctypes.c_size_t)]
    L.ksa_visible_pairs.argtypes = [pp, ctypes.POINTER(i64)]
    L.ksa_attn_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, pp, vp]
    L.ksa_host_staging_bytes.argtypes = [vp, pp, ctypes.POINTER(ctypes.c_size_t)]
    L.ksa_attn_fwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, pp, vp]
    L.ksa_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, vp, pp, vp]
    L.ksa_noalloc_last_device_status.argtypes = [ctypes.POINTER(i32)]
    L.ksa_bwd_workspace_bytes.argtypes = [vp, pp, ctypes.POINTER(ctypes.c_size_t)]
    L.ksa_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, pp, vp]
    L.ksa_part_rows.argtypes = [vp, pp, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.ksa_attn_fwd_part.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, pp, i32, i32, vp]
    L.ksa_anneal_lambda.argtypes = [i64, i64, i64, ctypes.POINTER(ctypes.c_float)]
    L.ksa_position_ids.argtypes = [pp, vp]
    L.ksa_total_summary_rows.restype = i64
    L.ksa_total_summary_rows.argtypes = [pp]
    L.ksa_qkv_prepare.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, pp, vp]
    L.ksa_prepared_workspace_bytes.argtypes = [vp, pp, ctypes.POINTER(ctypes.c_size_t)]
    L.ksa_attn_fwd_prepared.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, vp, vp, vp, ctypes.c_size_t, pp, vp]
    L.ksa_schedule_dump.argtypes = [vp, pp, ctypes.POINTER(ksa_tile_rec), i64, ctypes.POINTER(i64)]
    L.ksa_last_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    L.ksa_selftest_bounded_wait.argtypes = [vp, i64, vp, vp]
    L.ksa_clear_device_status.argtypes = [vp]
    L.ksa_last_cuda_error.argtypes = [vp]
    L.ksa_launch_count.restype = i64
    L.ksa_launch_count.argtypes = [vp]
    L.ksa_device_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.ksa_enable_kernel_timing.argtypes = [vp, ctypes.c_int]
    L.ksa_text_kernel_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    cp = ctypes.POINTER(ksa_cache_params)
    szp = ctypes.POINTER(ctypes.c_size_t)
    L.ksa_cache_rows.restype = i64
    L.ksa_cache_rows.argtypes = [cp]
    L.ksa_cache_bytes.argtypes = [cp, szp, szp, szp]
    L.ksa_cache_slice.argtypes = [cp, i64, ctypes.c_int, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.ksa_cache_reset.argtypes = [vp, vp, cp, vp]
    L.ksa_cache_fill_from_prefill.argtypes = [vp, vp, vp, vp, vp, vp, pp, cp, vp]
    L.ksa_decode_text.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, cp, vp]
    L.ksa_decode_summary.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, cp, vp]
    L.ksa_strerror.restype = ctypes.c_char_p
    L.ksa_strerror.argtypes = [ctypes.c_int]
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().ksa_strerror(status).decode()


def _check(status: int, where: str):
    if status != KSA_OK:
        raise KsaError(status, where)


@dataclass
class Problem:
    """Python-side holder of a ``ksa_params`` plus the host array it points to."""
    text_lens: Sequence[int]
    k: int
    m: int
    C: int
    Hq: int
    Hkv: int
    D: int
    scale: float
    flags: int = 0

    def params(self, q=None, k=None, v=None, o=None) -> ksa_params:
        cu = np.concatenate([[0], np.cumsum(np.asarray(self.text_lens, dtype=np.int64))]).astype(np.int32)
        self._cu = cu  # keep alive
        p = ksa_params()
        p.struct_size = ctypes.sizeof(ksa_params)
        p.num_seqs = len(self.text_lens)
        p.cu_text_lens = cu.ctypes.data
        p.chunk_len, p.summaries_per_chunk, p.window_chunks = self.k, self.m, self.C
        p.num_q_heads, p.num_kv_heads, p.head_dim = self.Hq, self.Hkv, self.D
        p.softmax_scale = self.scale
        p.flags = self.flags
        p.reserved = 0

        def strides(t, H):
            if t is None:
                return H * self.D, self.D
            assert t.stride(2) == 1, "head_dim must be contiguous"
            return t.stride(0), t.stride(1)

        p.q_stride_tok, p.q_stride_head = strides(q, self.Hq)
        p.k_stride_tok, p.k_stride_head = strides(k, self.Hkv)
        p.v_stride_tok, p.v_stride_head = strides(v, self.Hkv)
        p.o_stride_tok, p.o_stride_head = strides(o, self.Hq)
        return p


def aug_len(n_text: int, k: int, m: int) -> int:
    return int(lib().ksa_aug_len(n_text, k, m))


def total_aug_len(prob: Problem) -> int:
    p = prob.params()
    r = int(lib().ksa_total_aug_len(ctypes.byref(p)))
    if r < 0:
        raise KsaError(r, "ksa_total_aug_len")
    return r


def workspace_bytes(prob: Problem) -> int:
    p = prob.params()
    n = ctypes.c_size_t()
    _check(lib().ksa_workspace_bytes(None, ctypes.byref(p), ctypes.byref(n)), "ksa_workspace_bytes")
    return int(n.value)


def bwd_workspace_bytes(prob: Problem) -> int:
    p = prob.params()
    n = ctypes.c_size_t()
    _check(lib().ksa_bwd_workspace_bytes(None, ctypes.byref(p), ctypes.byref(n)), "ksa_bwd_workspace_bytes")
    return int(n.value)


def anneal_lambda(step: int, s_start: int, s_end: int) -> float:
    lam = ctypes.c_float()
    _check(lib().ksa_anneal_lambda(step, s_start, s_end, ctypes.byref(lam)), "ksa_anneal_lambda")
    return float(lam.value)


def prepared_workspace_bytes(prob: Problem) -> int:
    b = ctypes.c_size_t()
    p = prob.params()
    _check(lib().ksa_prepared_workspace_bytes(None, ctypes.byref(p), ctypes.byref(b)), "ksa_prepared_workspace_bytes")
    return int(b.value)


def position_ids(prob: Problem):
    """Position id of every augmented row (numpy int32), computed by the library on the host."""
    import numpy as np
    p = prob.params()
    out = np.zeros(total_aug_len(prob), dtype=np.int32)
    _check(lib().ksa_position_ids(ctypes.byref(p), out.ctypes.data), "ksa_position_ids")
    return out


def total_summary_rows(prob: Problem) -> int:
    p = prob.params()
    return int(lib().ksa_total_summary_rows(ctypes.byref(p)))


def host_staging_bytes(prob: Problem) -> int:
    p = prob.params()
    n = ctypes.c_size_t()
    _check(lib().ksa_host_staging_bytes(None, ctypes.byref(p), ctypes.byref(n)), "ksa_host_staging_bytes")
    return int(n.value)


def visible_pairs(prob: Problem) -> int:
    p = prob.params()
    n = ctypes.c_int64()
    _check(lib().ksa_visible_pairs(ctypes.byref(p), ctypes.byref(n)), "ksa_visible_pairs")
    return int(n.value)


def schedule_dump(prob: Problem, ctx: Optional["Context"] = None) -> np.ndarray:
    """Structured numpy array of the visited (query tile, kv tile) records."""
    p = prob.params()
    cnt = ctypes.c_int64()
    h = ctx.handle if ctx is not None else None
    _check(lib().ksa_schedule_dump(h, ctypes.byref(p), None, 0, ctypes.byref(cnt)), "ksa_schedule_dump")
    arr = (ksa_tile_rec * max(1, cnt.value))()
    _check(lib().ksa_schedule_dump(h, ctypes.byref(p), arr, cnt.value, ctypes.byref(cnt)), "ksa_schedule_dump")
    dt = np.dtype([(n, np.int32) for n, _ in ksa_tile_rec._fields_])
    return np.frombuffer(arr, dtype=dt, count=cnt.value).copy()


class Context:
    """Owns a ``ksa_ctx``."""

    def __init__(self, device: int = 0):
        h = ctypes.c_void_p()
        _check(lib().ksa_create(ctypes.byref(h), device), "ksa_create")
        self.handle = h
        self.device = device

    def close(self):
        if self.handle:
            lib().ksa_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def attn_fwd(self, prob: Problem, q, k, v, out, lse, workspace, stream: Optional[int] = None):
        """ksa_attn_fwd on torch CUDA tensors (q, k, v, out bf16; lse fp32; workspace uint8)."""
        import torch
        p = prob.params(q, k, v, out)
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        _check(lib().ksa_attn_fwd(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                  lse.data_ptr(), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                  ctypes.byref(p), stream), "ksa_attn_fwd")

    def attn_bwd(self, prob: Problem, q, k, v, out, lse, dout, dq, dk, dv, workspace, stream: Optional[int] = None):
        """ksa_attn_bwd on torch CUDA tensors (dout like out, dq like q, dk / dv like k / v)."""
        import torch
        p = prob.params(q, k, v, out)
        assert dout.stride() == out.stride() and dq.stride() == q.stride() and dk.stride() == k.stride() and dv.stride() == v.stride()
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        _check(lib().ksa_attn_bwd(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                  dout.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), workspace.data_ptr(),
                                  workspace.numel() * workspace.element_size(), ctypes.byref(p), stream), "ksa_attn_bwd")

    def part_rows(self, prob: Problem, part: int, num_parts: int):
        """Augmented row range [begin, end) of part `part` of `num_parts` (ksa_part_rows)."""
        p = prob.params()
        b, e = ctypes.c_int64(), ctypes.c_int64()
        _check(lib().ksa_part_rows(self.handle, ctypes.byref(p), part, num_parts, ctypes.byref(b), ctypes.byref(e)), "ksa_part_rows")
        return int(b.value), int(e.value)

    def attn_fwd_part(self, prob: Problem, q, k, v, out, lse, workspace, part: int, num_parts: int, stream: Optional[int] = None):
        """ksa_attn_fwd_part on torch CUDA tensors: only the query rows of the part are computed."""
        import torch
        p = prob.params(q, k, v, out)
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        _check(lib().ksa_attn_fwd_part(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                       workspace.data_ptr(), workspace.numel() * workspace.element_size(), ctypes.byref(p),
                                       part, num_parts, stream), "ksa_attn_fwd_part")

    def qkv_prepare(self, prob: Problem, q_main, k_main, v_main, q_summ, k_summ, v_summ, q_out, k_out, v_out,
                    lam: float, rope_theta: float, flags: int = 0, stream: Optional[int] = None):
        """ksa_qkv_prepare on torch CUDA tensors (outputs laid out like their _main inputs; summ tensors may be None)."""
        import torch
        p = prob.params(q_main, k_main, v_main, q_main)
        assert q_out.stride() == q_main.stride() and k_out.stride() == k_main.stride() and v_out.stride() == v_main.stride()
        for t in (q_summ, k_summ, v_summ):
            assert t is None or t.is_contiguous()
        if stream is None:
            stream = torch.cuda.current_stream(q_main.device).cuda_stream
        ptr = lambda t: None if t is None else t.data_ptr()
        _check(lib().ksa_qkv_prepare(self.handle, q_main.data_ptr(), k_main.data_ptr(), v_main.data_ptr(),
                                     ptr(q_summ), ptr(k_summ), ptr(v_summ), q_out.data_ptr(), k_out.data_ptr(), v_out.data_ptr(),
                                     ctypes.c_float(lam), ctypes.c_float(rope_theta), ctypes.c_uint32(flags),
                                     ctypes.byref(p), stream), "ksa_qkv_prepare")

    def attn_fwd_prepared(self, prob: Problem, q_main, k_main, v_main, q_summ, k_summ, v_summ, lam: float, rope_theta: float,
                          out, lse, workspace, flags: int = 0, stream: Optional[int] = None):
        """ksa_attn_fwd_prepared: preparation (position ids, interpolation, rotation) folded into the pack pass, then attention."""
        import torch
        p = prob.params(q_main, k_main, v_main, out)
        if stream is None:
            stream = torch.cuda.current_stream(q_main.device).cuda_stream
        ptr = lambda t: None if t is None else t.data_ptr()
        _check(lib().ksa_attn_fwd_prepared(self.handle, q_main.data_ptr(), k_main.data_ptr(), v_main.data_ptr(),
                                           ptr(q_summ), ptr(k_summ), ptr(v_summ), ctypes.c_float(lam), ctypes.c_float(rope_theta),
                                           ctypes.c_uint32(flags), out.data_ptr(), lse.data_ptr(), workspace.data_ptr(),
                                           workspace.numel() * workspace.element_size(), ctypes.byref(p), stream),
               "ksa_attn_fwd_prepared")

    def attn_fwd_host(self, prob: Problem, q, k, v, out, lse, staging, stream: Optional[int] = None):
        """ksa_attn_fwd_host: q, k, v, out, lse are contiguous HOST tensors (pinned recommended)."""
        import torch
        p = prob.params()
        if stream is None:
            stream = torch.cuda.current_stream(staging.device).cuda_stream
        _check(lib().ksa_attn_fwd_host(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                       lse.data_ptr(), staging.data_ptr(), staging.numel() * staging.element_size(),
                                       ctypes.byref(p), stream), "ksa_attn_fwd_host")

    def device_status(self) -> int:
        s = ctypes.c_int32()
        rc = lib().ksa_last_device_status(self.handle, ctypes.byref(s))
        if rc not in (KSA_OK, KSA_ERR_TIMEOUT):          # KSA_ERR_TIMEOUT: the status word is non-zero, returned below
            _check(rc, "ksa_last_device_status")
        return int(s.value)

    def device_status_rc(self) -> int:
        """The return code of ksa_last_device_status itself (KSA_OK or KSA_ERR_TIMEOUT)."""
        s = ctypes.c_int32()
        return int(lib().ksa_last_device_status(self.handle, ctypes.byref(s)))

    def selftest_bounded_wait(self, limit_cycles: int, report, stream: Optional[int] = None):
        _check(lib().ksa_selftest_bounded_wait(self.handle, int(limit_cycles), report.data_ptr(), stream),
               "ksa_selftest_bounded_wait")

    def clear_device_status(self):
        _check(lib().ksa_clear_device_status(self.handle), "ksa_clear_device_status")

    def last_cuda_error(self) -> int:
        return int(lib().ksa_last_cuda_error(self.handle))

    def launch_count(self) -> int:
        return int(lib().ksa_launch_count(self.handle))

    def device_info(self):
        """(SM count, two-CTA clusters the device runs at once)."""
        n, c = ctypes.c_int32(), ctypes.c_int32()
        _check(lib().ksa_device_info(self.handle, ctypes.byref(n), ctypes.byref(c)), "ksa_device_info")
        return int(n.value), int(c.value)

    def enable_kernel_timing(self, on: bool = True):
        _check(lib().ksa_enable_kernel_timing(self.handle, int(on)), "ksa_enable_kernel_timing")

    def text_kernel_ms(self) -> float:
        ms = ctypes.c_float()
        _check(lib().ksa_text_kernel_ms(self.handle, ctypes.byref(ms)), "ksa_text_kernel_ms")
        return float(ms.value)


NOALLOC_MAX_SCRATCH_BYTES = 32 * 1024 * 1024


def noalloc_device_status() -> int:
    """Status word of the allocation-free entry point on the current device (0 = no wait gave up)."""
    st = ctypes.c_int32()
    rc = lib().ksa_noalloc_last_device_status(ctypes.byref(st))
    if rc not in (KSA_OK, KSA_ERR_TIMEOUT):
        _check(rc, "ksa_noalloc_last_device_status")
    return int(st.value)


def attn_fwd_noalloc(prob: Problem, q, k, v, out, lse, stream: Optional[int] = None):
    """ksa_attn_fwd_noalloc: the forward pass for callers that may not allocate device
    memory (no context, no workspace; the library's fixed internal scratch is used).
    q, k, v, out, lse are torch CUDA tensors on the current device, owned by the caller."""
    import torch
    p = prob.params(q, k, v, out)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    _check(lib().ksa_attn_fwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                      lse.data_ptr(), ctypes.byref(p), stream), "ksa_attn_fwd_noalloc")


def attn_fwd(ctx: Context, prob: Problem, q, k, v):
    """Convenience wrapper: allocates out, lse and the workspace with torch and calls
    ``ksa_attn_fwd`` on the current stream.  Returns (out, lse)."""
    import torch
    total = q.shape[0]
    out = torch.empty((total, prob.Hq, prob.D), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((prob.Hq, total), dtype=torch.float32, device=q.device)
    ws = torch.empty(workspace_bytes(prob), dtype=torch.uint8, device=q.device)
    ctx.attn_fwd(prob, q, k, v, out, lse, ws)
    return out, lse


@dataclass
class CacheSpec:
    """Python-side holder of a ``ksa_cache_params`` (decode path, Sec. 2.3.1)."""
    batch: int
    k: int
    C: int
    max_summaries: int
    Hq: int
    Hkv: int
    D: int
    scale: float
    flags: int = 0

    def params(self) -> ksa_cache_params:
        p = ksa_cache_params()
        p.struct_size = ctypes.sizeof(ksa_cache_params)
        p.batch, p.chunk_len, p.window_chunks, p.max_summaries = self.batch, self.k, self.C, self.max_summaries
        p.num_q_heads, p.num_kv_heads, p.head_dim = self.Hq, self.Hkv, self.D
        p.softmax_scale, p.flags = self.scale, self.flags
        return p


def cache_rows(spec: CacheSpec) -> int:
    p = spec.params()
    return int(lib().ksa_cache_rows(ctypes.byref(p)))


def cache_bytes(spec: CacheSpec):
    """(bytes of kcache = vcache, bytes of the state array, bytes of the decode workspace)"""
    p = spec.params()
    a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().ksa_cache_bytes(ctypes.byref(p), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "ksa_cache_bytes")
    return int(a.value), int(b.value), int(c.value)


def cache_slice(spec: CacheSpec, text_tokens_before: int, is_summary: bool):
    p = spec.params()
    lo, hi = ctypes.c_int64(), ctypes.c_int64()
    _check(lib().ksa_cache_slice(ctypes.byref(p), text_tokens_before, int(is_summary), ctypes.byref(lo), ctypes.byref(hi)),
           "ksa_cache_slice")
    return int(lo.value), int(hi.value)


class DecodeCache:
    """Torch tensors of one Summary KV cache plus the calls that step it (argument marshalling only)."""

    def __init__(self, ctx: "Context", spec: CacheSpec):
        import torch
        self.ctx, self.spec = ctx, spec
        dev = torch.device("cuda", ctx.device)
        rows = cache_rows(spec)
        _, _, wsb = cache_bytes(spec)
        self.kcache = torch.zeros((spec.batch, spec.Hkv, rows, spec.D), dtype=torch.bfloat16, device=dev)
        self.vcache = torch.zeros_like(self.kcache)
        self.state = torch.zeros((spec.batch, 2), dtype=torch.int32, device=dev)
        self.workspace = torch.empty(max(wsb, 256), dtype=torch.uint8, device=dev)

    def _stream(self, stream):
        import torch
        return torch.cuda.current_stream(self.kcache.device).cuda_stream if stream is None else stream

    def reset(self, stream=None):
        p = self.spec.params()
        _check(lib().ksa_cache_reset(self.ctx.handle, self.state.data_ptr(), ctypes.byref(p), self._stream(stream)), "ksa_cache_reset")

    def fill_from_prefill(self, prob: Problem, k, v, stream=None):
        p = self.spec.params()
        pp_ = prob.params(None, k, v, None)
        _check(lib().ksa_cache_fill_from_prefill(self.ctx.handle, self.kcache.data_ptr(), self.vcache.data_ptr(), self.state.data_ptr(),
                                                 k.data_ptr(), v.data_ptr(), ctypes.byref(pp_), ctypes.byref(p), self._stream(stream)),
               "ksa_cache_fill_from_prefill")

    def _step(self, fn, name, q, k_new, v_new, out, lse, stream):
        p = self.spec.params()
        _check(fn(self.ctx.handle, self.kcache.data_ptr(), self.vcache.data_ptr(), self.state.data_ptr(), q.data_ptr(),
                  k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(), lse.data_ptr(), self.workspace.data_ptr(),
                  self.workspace.numel(), ctypes.byref(p), self._stream(stream)), name)

    def decode_text(self, q, k_new, v_new, out, lse, stream=None):
        self._step(lib().ksa_decode_text, "ksa_decode_text", q, k_new, v_new, out, lse, stream)

    def decode_summary(self, q, k_new, v_new, out, lse, stream=None):
        self._step(lib().ksa_decode_summary, "ksa_decode_summary", q, k_new, v_new, out, lse, stream)
