"""Reporting helpers over the library's outputs (not part of the compression pass).

cross_segment_rate: the statistic behind the paper's motivation (Sec. 2.3, Fig. 2a): the share of
fixed-size blocks, laid out from position 0 as block-level eviction methods do, that contain
tokens of more than one semantic segment.  block_size_histogram: how often each block size was
chosen by the adaptive search, over the segments that retain something (Sec. 4.5, Fig. 9).
Both take the tensors the library wrote (segment ids from sablock_segment, g*_k and b_k from
sablock_select) and reduce them with torch on the device they live on.
"""
from __future__ import annotations

from typing import Dict, Sequence

import torch


def cross_segment_rate(seg_id: torch.Tensor, block: int) -> float:
    """Share of the blocks [j * block, (j + 1) * block) of the compressible region whose first and
    last token lie in different segments (segment ids are non-decreasing, so that is the case
    exactly when the block holds tokens of more than one segment)."""
    T = seg_id.numel()
    if T == 0 or block < 1:
        return 0.0
    first = torch.arange(0, T, block, device=seg_id.device)
    last = torch.clamp(first + block - 1, max=T - 1)
    return float((seg_id[first] != seg_id[last]).double().mean().item())


def block_size_histogram(seg_block: torch.Tensor, seg_budget: torch.Tensor, n_seg: int,
                         candidates: Sequence[int]) -> Dict[int, int]:
    """Number of segments with b_k > 0 that chose each candidate block size."""
    g = seg_block[:n_seg][seg_budget[:n_seg] > 0]
    return {int(c): int((g == int(c)).sum().item()) for c in candidates}
