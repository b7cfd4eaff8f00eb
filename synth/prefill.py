"""Stand-in for what the PREFILL hands to the compression pass in its single-sweep mode.

The pass runs right after a FlashAttention prefill (Sec. 4.1), whose attention kernel keeps the log
of the softmax normaliser of every query row.  No prefill runs in this repository, so this module
produces that by-product for the last W query rows from the same stored q_win and K, in fp32 with
torch.  It is an INPUT of the CUDA path only: the CPU checker never reads it (it computes its own
normalisers), and a CPU test pins it against the checker's attention weights.
"""
from __future__ import annotations

import math
from typing import Sequence

import torch


def prefill_row_lse(q_win: torch.Tensor, k: torch.Tensor, cu_seqlens: Sequence[int]) -> torch.Tensor:
    """What a prefill attention kernel would hand over for the last W query rows of every
    (layer, sequence): the natural log of the softmax normaliser over the causal keys,
    row_lse[l, i, h, w] = ln sum_{j <= T+w} exp(q[l,i,h,w] . k[l,j,kv(h)] / sqrt(D)), in fp32
    (products of the stored values, fp32 accumulation), as FlashAttention keeps it per query row.
    An input of the single-sweep mode, produced here because no prefill runs in this repository.

    q_win [n_layers, n_seqs, H, W, D]; k [n_layers, total_tokens, Hkv, D]; returns fp32
    [n_layers, n_seqs, H, W] on k's device."""
    nl, ns, H, W, D = q_win.shape
    Hkv = k.shape[2]
    G = H // Hkv
    out = torch.empty(nl, ns, H, W, dtype=torch.float32, device=k.device)
    for l in range(nl):
        for i in range(ns):
            a, z = cu_seqlens[i], cu_seqlens[i + 1]
            L = z - a
            T = L - W
            if T <= 0:
                out[l, i] = 0.0
                continue
            visible = torch.arange(L, device=k.device)[None, :] <= (T + torch.arange(W, device=k.device))[:, None]
            for j in range(Hkv):
                qj = q_win[l, i, j * G:(j + 1) * G].float().reshape(G * W, D)
                kj = k[l, a:z, j].float()
                logits = (qj @ kj.t()) / math.sqrt(D)                       # [G*W, L]
                logits = logits.view(G, W, L).masked_fill(~visible[None], float("-inf"))
                out[l, i, j * G:(j + 1) * G] = torch.logsumexp(logits, dim=-1)
    return out
