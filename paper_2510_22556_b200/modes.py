"""Named parameter settings of the compression pass: the method itself and the variants its
ablation study compares it with (Sec. 4.5, Tables 3 and 4).

Every variant is the same kernels run with other parameters; nothing here computes anything.
A preset is (overrides of the parameter block, block-size candidates).

  sablock             the method: segment-guided scores (alpha = 0.9, eta = 1.0), adaptive block
                      size from the caller's candidate set with fidelity threshold tau = 0.85
  token_level         token-level eviction: the only candidate is g = 1, so every segment keeps
                      exactly its share of the global Top-B (T_k(1) = T_topB within S_k)
  fixed_block(g)      a fixed granularity: candidates {1, g} and tau = 0, so every segment whose
                      implicit budget and length allow a block of g tokens uses it, whatever the
                      fidelity (g = 1 remains for the segments that cannot hold one block)
  no_segment_scoring  alpha = 0: the refined score equals the window score (Eq. 8), segments still
                      bound the blocks
"""
from __future__ import annotations

from typing import Dict, Sequence, Tuple

Preset = Tuple[Dict[str, float], Tuple[int, ...]]


def sablock(candidates: Sequence[int]) -> Preset:
    return {}, tuple(candidates)


def token_level() -> Preset:
    return {}, (1,)


def fixed_block(g: int) -> Preset:
    if g < 1:
        raise ValueError("block size must be positive")
    return {"tau": 0.0}, ((1,) if g == 1 else (1, int(g)))


def no_segment_scoring(candidates: Sequence[int]) -> Preset:
    return {"alpha": 0.0}, tuple(candidates)


def ablation_presets(candidates: Sequence[int]) -> Dict[str, Preset]:
    """The rows of the paper's ablation tables as presets (Tables 3 and 4)."""
    return {
        "sablock": sablock(candidates),
        "token_level": token_level(),
        "fixed_block_5": fixed_block(5),
        "fixed_block_10": fixed_block(10),
        "no_segment_scoring": no_segment_scoring(candidates),
    }
