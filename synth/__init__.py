"""Seeded synthetic inputs for the SABlock compression pass.

This module only draws inputs (keys, values, window queries, token ids, the
delimiter set).  It holds none of the method's arithmetic and is shared by the
CPU checker's tests and by the CUDA path's tests and benchmark, so that both
sides read exactly the same stored values.

The paper evaluates on LongBench / needle-in-a-haystack prompts run through
Llama-3 / Mistral models (Sec. 4.1); neither the datasets nor the weights are
available offline, so these generators stand in for them with the same tensor
shapes (Llama-3-8B: 32 query heads, 8 KV heads, head_dim 128), heavy-tailed
attention logits (a shared low-rank component in K), planted "needle" spans
whose keys align with the mean window query, and token streams whose
delimiters arrive at geometric gaps (sentences ~25 tokens, one in six
delimiters a paragraph break).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class Config:
    """One workload shape.  Names follow the paper's notation where it has one."""
    name: str
    n_layers: int
    n_q_heads: int          # H
    n_kv_heads: int         # Hkv
    head_dim: int           # D
    window: int             # W = n_rcnt
    seq_lens: Tuple[int, ...]   # L per sequence (batch = len)
    budgets: Tuple[int, ...]
    candidates: Tuple[int, ...]
    dtype: str              # "f32" | "bf16"
    vocab: int
    rank: int               # r of the shared low-rank key component
    kappa: float            # its scale
    mean_gap: int           # mean tokens between delimiters
    needle_depths: Tuple[float, ...] = ()
    base_seed: int = 0

    @property
    def total_tokens(self) -> int:
        return sum(self.seq_lens)


def _ragged_lengths(seed: int, n: int, lo: int, hi: int) -> Tuple[int, ...]:
    g = torch.Generator().manual_seed(seed)
    return tuple(int(x) for x in torch.randint(lo, hi + 1, (n,), generator=g))


CONFIGS = {
    # 0: tiny fp32 reference case
    "tiny": Config("tiny", 1, 4, 1, 64, 16, (512,), (64,), (1, 2, 4, 8), "f32",
                   32000, 8, 2.0, 20, (), 0),
    # 1: Llama-3-8B-shaped single layer
    "layer8k": Config("layer8k", 1, 32, 8, 128, 32, (8192,), (96, 128, 256), (1, 2, 4, 8, 16),
                      "bf16", 128256, 16, 2.0, 25, (0.37,), 1),
    # 2: 32-layer stack at 32K, budget sweep
    "stack32k": Config("stack32k", 32, 32, 8, 128, 32, (32768,), (128, 256, 512, 1024, 2048),
                       (1, 2, 4, 8, 16, 32), "bf16", 128256, 16, 2.0, 25, (0.10, 0.50, 0.90), 2),
    # 3: headline, 128K context, budget 1024
    "headline128k": Config("headline128k", 32, 32, 8, 128, 32, (131072,), (1024,),
                           (1, 2, 4, 8, 16, 32), "bf16", 128256, 16, 2.0, 25, (0.62,), 3),
    # 4: ragged batch of 16
    "ragged16": Config("ragged16", 32, 32, 8, 128, 32, _ragged_lengths(4, 16, 4096, 16384), (512,),
                       (1, 2, 4, 8, 16), "bf16", 128256, 16, 2.0, 25, (), 4),
    # the paper's own settings (Sec. 4.1 and 4.5): observation window n_rcnt = 8, search set
    # {1, 2, 3, 5, 7, 9, 11, 13} (g_max = 13), its budget range, on the same 32-layer stack at 32K
    "paper8": Config("paper8", 32, 32, 8, 128, 8, (32768,), (128, 256, 512, 1024, 2048),
                     (1, 2, 3, 5, 7, 9, 11, 13), "bf16", 128256, 16, 2.0, 25, (0.10, 0.50, 0.90), 5),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def delimiter_ids(vocab: int) -> Tuple[int, int]:
    """Two reserved ids: (sentence delimiter, paragraph delimiter)."""
    return vocab - 2, vocab - 1


def delimiter_bitmap(vocab: int, ids: Optional[Sequence[int]] = None) -> torch.Tensor:
    """Bitmap over the vocabulary (int32 words, bit i of word i//32 set iff id i delimits)."""
    if ids is None:
        ids = delimiter_ids(vocab)
    words = torch.zeros((vocab + 31) // 32, dtype=torch.int64)
    for i in ids:
        words[i // 32] |= (1 << (i % 32))
    # store as int32 with the same bit pattern
    words = torch.where(words >= 2 ** 31, words - 2 ** 32, words)
    return words.to(torch.int32)


def make_token_ids(L: int, vocab: int, mean_gap: int, seed: int,
                   with_delimiters: bool = True) -> torch.Tensor:
    """Token ids uniform over the non-delimiter vocabulary; a delimiter follows each
    geometric(mean_gap) run of ordinary tokens; one delimiter in six is a paragraph break."""
    g = torch.Generator().manual_seed(seed)
    sent, para = delimiter_ids(vocab)
    ids = torch.randint(0, vocab - 2, (L,), generator=g, dtype=torch.int64)
    if with_delimiters and L > 0:
        p = 1.0 / mean_gap
        # geometric gaps >= 1 by inversion
        n_draw = max(16, int(3 * L / mean_gap) + 16)
        u = torch.rand(n_draw, generator=g, dtype=torch.float64).clamp_(1e-12, 1 - 1e-12)
        gaps = torch.floor(torch.log(u) / math.log(1.0 - p)).to(torch.int64) + 1
        pos = torch.cumsum(gaps, 0) - 1
        pos = pos[pos < L]
        kind = torch.rand(pos.numel(), generator=g) < (1.0 / 6.0)
        ids[pos] = torch.where(kind, torch.tensor(para), torch.tensor(sent))
    return ids.to(torch.int32)


def _unit(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-30)


def make_layer(cfg: Config, L: int, seed: int, device: str = "cpu",
               needle_depths: Optional[Sequence[float]] = None):
    """One (layer, sequence) worth of tensors.

    Returns q_win [H, W, D], k [L, Hkv, D], v [L, Hkv, D] in cfg.dtype, and the list of
    needle (start, length) spans.  Values are drawn in fp32 and then cast, so the stored
    values are what every consumer sees.
    """
    H, Hkv, D, W, r = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.rank
    G = H // Hkv
    g = torch.Generator(device=device).manual_seed(seed)
    kw = dict(generator=g, device=device, dtype=torch.float32)
    z = torch.randn(L, Hkv, D, **kw)
    c = torch.randn(L, r, **kw)
    Gm = torch.randn(Hkv, r, D, **kw)
    k = z + (cfg.kappa / math.sqrt(r)) * torch.einsum("tr,jrd->tjd", c, Gm)
    del z, c
    v = torch.randn(L, Hkv, D, **kw)
    u = _unit(torch.randn(Hkv, D, **kw))
    q = torch.randn(H, W, D, **kw) + 3.0 * u.repeat_interleave(G, dim=0)[:, None, :]
    spans: List[Tuple[int, int]] = []
    depths = cfg.needle_depths if needle_depths is None else needle_depths
    T = L - W
    n_len = 24
    rho = math.sqrt(D * (1.0 + cfg.kappa ** 2))
    for depth in depths:
        start = max(0, min(T - n_len, int(depth * T)))
        if T < n_len:
            break
        mhat = _unit(q.view(Hkv, G * W, D).mean(dim=1))                 # [Hkv, D]
        nz = torch.randn(n_len, Hkv, D, **kw)
        nz = nz - (nz * mhat[None]).sum(-1, keepdim=True) * mhat[None]
        nhat = _unit(nz)
        k[start:start + n_len] = rho * (0.9 * mhat[None] + math.sqrt(1 - 0.81) * nhat)
        spans.append((start, n_len))
    dt = torch_dtype(cfg.dtype)
    return q.to(dt), k.to(dt), v.to(dt), spans


def layer_seed(cfg: Config, layer: int, seq: int) -> int:
    return cfg.base_seed * 1_000_003 + 1000 * layer + seq


def token_seed(cfg: Config, seq: int) -> int:
    return 7_000_000 + cfg.base_seed * 1009 + seq


@dataclass
class Batch:
    """A packed (layers x sequences) workload in the layout the library consumes.

    q_win: [n_layers, n_seqs, H, W, D]; k, v: [n_layers, total_tokens, Hkv, D];
    token_ids: [total_tokens] int32 (shared by all layers); cu_seqlens: python list.
    """
    cfg: Config
    q_win: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    token_ids: torch.Tensor
    cu_seqlens: List[int]
    bitmap: torch.Tensor
    spans: List[List[Tuple[int, int]]] = field(default_factory=list)


def make_batch(cfg: Config, device: str = "cpu", n_layers: Optional[int] = None,
               seq_lens: Optional[Sequence[int]] = None, with_delimiters: bool = True) -> Batch:
    nl = cfg.n_layers if n_layers is None else n_layers
    lens = list(cfg.seq_lens if seq_lens is None else seq_lens)
    cu = [0]
    for L in lens:
        cu.append(cu[-1] + L)
    dt = torch_dtype(cfg.dtype)
    H, Hkv, D, W = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
    q = torch.empty(nl, len(lens), H, W, D, dtype=dt, device=device)
    k = torch.empty(nl, cu[-1], Hkv, D, dtype=dt, device=device)
    v = torch.empty(nl, cu[-1], Hkv, D, dtype=dt, device=device)
    spans_all: List[List[Tuple[int, int]]] = []
    for l in range(nl):
        for s, L in enumerate(lens):
            qi, ki, vi, sp = make_layer(cfg, L, layer_seed(cfg, l, s), device)
            q[l, s] = qi
            k[l, cu[s]:cu[s + 1]] = ki
            v[l, cu[s]:cu[s + 1]] = vi
            if l == 0:
                spans_all.append(sp)
    ids = torch.cat([make_token_ids(L, cfg.vocab, cfg.mean_gap, token_seed(cfg, s), with_delimiters)
                     for s, L in enumerate(lens)]).to(device)
    return Batch(cfg, q, k, v, ids, cu, delimiter_bitmap(cfg.vocab).to(device), spans_all)


from .prefill import prefill_row_lse  # noqa: E402,F401  (stand-in for the prefill attention kernel's output)
