"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module only draws random tensors and names workloads.  It holds none of the
method's arithmetic: callers compute the augmented length with their own side's
layout routine and pass it in as ``total_aug``.

Recipe (one CPU generator per workload, so the CPU oracle and the CUDA library are
handed the very same bits): ``g = torch.Generator('cpu').manual_seed(seed)``; Q, K, V
are drawn in that order with ``torch.randn(total_aug, H, D, generator=g)`` in fp32,
then the workload's scaling is applied, then everything is rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np
import torch


@dataclass(frozen=True)
class Layout:
    """Chunk layout: k text tokens then m summary tokens per chunk, window of C chunks."""
    name: str
    k: int
    m: int
    C: int


# Table 2 of the paper: chunk size 8, one summary token per chunk, 128 sliding chunks.
LAYOUT_P = Layout("P", 8, 1, 128)
# Same 8x compression and 1,024-token window with 64-token chunks and 8 summaries each.
LAYOUT_G = Layout("G", 64, 8, 16)
# The full-attention layers of the hybrid stack (one in four, Table 2): no summary tokens, a window that covers
# every chunk, i.e. plain causal attention through the same entry points.
LAYOUT_F = Layout("F", 8, 0, 1 << 20)


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    text_lens: List[int]
    Hq: int
    Hkv: int
    D: int
    k_scale: float = 1.0          # K <- k_scale * K
    peaked_frac: float = 0.0      # fraction of token positions whose K rows are multiplied by 4
    note: str = ""

    @property
    def scale(self) -> float:
        return float(np.float32(1.0 / np.sqrt(self.D)))


def varlen_text_lens() -> List[int]:
    """Eight text lengths drawn uniformly from [4096, 65536] with numpy seed 4."""
    return [int(x) for x in np.random.default_rng(4).integers(4096, 65537, size=8)]


WORKLOADS = {
    "tiny": Workload("tiny", 0, [1024], 4, 4, 64, note="1,024 text tokens, MHA 4 heads, D=64"),
    "8k": Workload("8k", 1, [8192], 32, 8, 128, k_scale=0.5, note="8,192 text tokens, K scaled by 0.5"),
    "32k": Workload("32k", 2, [32768, 32768], 32, 8, 128, note="two sequences of 32,768 text tokens"),
    "128k": Workload("128k", 3, [131072], 32, 4, 128, peaked_frac=0.01,
                     note="131,072 text tokens, 1% of K rows scaled by 4"),
    "varlen": Workload("varlen", 4, varlen_text_lens(), 32, 8, 128,
                       note="8 packed sequences, lengths uniform in [4096, 65536]"),
}


def make_qkv(wl: Workload, total_aug: int, device: str = "cpu", pin: bool = False):
    """Draw (q, k, v) as bf16 tensors [total_aug, H, D] for workload ``wl``.

    Q and V are drawn in slabs (the fp32 staging stays below ~1 GB); K is drawn in
    one piece and kept in fp32 until its scaling has been applied, so that it is
    rounded to bf16 once.  The draw order is Q, K, V, then the peaked positions.
    """
    g = torch.Generator("cpu").manual_seed(wl.seed)

    def draw_bf16(H):
        out = torch.empty((total_aug, H, wl.D), dtype=torch.bfloat16, pin_memory=pin)
        slab = max(1, (1 << 28) // (H * wl.D))
        for r0 in range(0, total_aug, slab):
            r1 = min(total_aug, r0 + slab)
            x = torch.randn((r1 - r0, H, wl.D), generator=g, dtype=torch.float32)
            out[r0:r1] = x.to(torch.bfloat16)
        return out

    q = draw_bf16(wl.Hq)
    kf = torch.randn((total_aug, wl.Hkv, wl.D), generator=g, dtype=torch.float32)
    v = draw_bf16(wl.Hkv)
    if wl.k_scale != 1.0:
        kf *= wl.k_scale
    if wl.peaked_frac > 0.0:
        cnt = int(round(wl.peaked_frac * total_aug))
        pos = torch.randperm(total_aug, generator=g)[:cnt]
        kf[pos] *= 4.0
    k = torch.empty((total_aug, wl.Hkv, wl.D), dtype=torch.bfloat16, pin_memory=pin)
    k.copy_(kf.to(torch.bfloat16))
    del kf
    if device != "cpu":
        q, k, v = q.to(device), k.to(device), v.to(device)
    return q, k, v


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array of its bit patterns (CPU)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
