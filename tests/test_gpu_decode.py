"""Decoding over the compacted cache (Sec. 4.4): sablock_decode_attention against the float64 oracle,
on caches the compression pass wrote and on full caches, element by element (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as build_lib

pytestmark = pytest.mark.gpu

# fp32 accumulation over up to 131072 rows of bf16 products; weights are exp2 of fp32 logits
REL, ABS = 2e-3, 1e-5


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_lib()
    B.lib()


def _check(out, lse, q, k, v, n_valid=None):
    for i in range(q.shape[0]):
        n = k.shape[1] if n_valid is None else int(n_valid[i])
        ref, ref_lse = oracle.decode_attention(q[i], k[i, :n], v[i, :n])
        got = out[i].cpu().double().numpy()
        assert np.isfinite(got).all()
        assert (np.abs(got - ref) <= ABS + REL * np.abs(ref)).all(), float(np.abs(got - ref).max())
        if lse is not None:
            np.testing.assert_allclose(lse[i].cpu().double().numpy(), ref_lse, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("H,Hkv,D,dtype,n_rows,n_prob", [
    (32, 8, 128, torch.bfloat16, 1024, 3),        # the headline's compacted cache
    (32, 8, 128, torch.bfloat16, 1, 1),           # a single row
    (32, 8, 128, torch.bfloat16, 257, 2),         # one row more than a chunk
    (32, 8, 128, torch.bfloat16, 70001, 1),       # ragged splits over a long cache
    (4, 1, 64, torch.float32, 512, 2),            # the tiny configuration's shape
    (8, 8, 64, torch.bfloat16, 300, 2),           # no grouping, 128-byte rows
    (16, 8, 128, torch.float32, 999, 1),          # two query heads per KV head, 512-byte rows
])
def test_decode_attention_matches_oracle(H, Hkv, D, dtype, n_rows, n_prob):
    g = torch.Generator().manual_seed(n_rows + H)
    q = (torch.randn(n_prob, H, D, generator=g) * 1.5).to(dtype)
    k = torch.randn(n_prob, n_rows, Hkv, D, generator=g).to(dtype)
    v = torch.randn(n_prob, n_rows, Hkv, D, generator=g).to(dtype)
    p = B.make_params(H, Hkv, D, 8, dtype)
    out, lse = B.decode_attention(p, q.cuda(), k.cuda(), v.cuda(), want_lse=True)
    torch.cuda.synchronize()
    _check(out, lse, q, k, v)
    out2 = B.decode_attention(p, q.cuda(), k.cuda(), v.cuda())
    torch.cuda.synchronize()
    assert torch.equal(out, out2)                  # fixed summation order: runs are bit-identical


def test_decode_over_the_cache_the_pass_wrote():
    """Compress two layers of ragged sequences, then decode over out_k / out_v with out_n_keep as the row
    counts (a short sequence is returned whole and fills fewer rows), against the oracle on the same rows;
    and over the full cache of one sequence."""
    cfg = synth.CONFIGS["ragged16"]
    lens = [3000, 100, 700]
    b = synth.make_batch(cfg, device="cuda", n_layers=2, seq_lens=lens)
    p = B.make_params(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, torch.bfloat16, b.bitmap, cfg.vocab)
    ws = B.alloc_workspace(p, b.cu_seqlens[-1], max(lens), 3, 2)
    out = B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 256, cfg.candidates, ws)
    out.out_k[0, 1, 100:] = 0                      # rows beyond n_keep are never read
    out.out_v[0, 1, 100:] = 0
    torch.cuda.synchronize()
    g = torch.Generator().manual_seed(7)
    q_new = torch.randn(6, cfg.n_q_heads, cfg.head_dim, generator=g).to(torch.bfloat16).cuda()
    kc = out.out_k.view(6, 256, cfg.n_kv_heads, cfg.head_dim)
    vc = out.out_v.view(6, 256, cfg.n_kv_heads, cfg.head_dim)
    n_valid = out.n_keep.view(6)
    res = B.decode_attention(p, q_new, kc, vc, n_valid=n_valid)
    torch.cuda.synchronize()
    assert n_valid.cpu().tolist() == [256, 100, 256] * 2
    _check(res, None, q_new.cpu(), kc.cpu(), vc.cpu(), n_valid.cpu().tolist())
    # the full cache of sequence 0, layer 1
    full = B.decode_attention(p, q_new[3:4], b.k[1:2, :3000], b.v[1:2, :3000])
    torch.cuda.synchronize()
    _check(full, None, q_new[3:4].cpu(), b.k[1:2, :3000].cpu(), b.v[1:2, :3000].cpu())


def test_decode_rejects_what_it_does_not_take():
    import ctypes as C
    p = B.make_params(32, 4, 128, 8, torch.bfloat16)          # eight query heads per KV head
    assert B.lib().sablock_decode_workspace_bytes(C.addressof(p), 1, 100) == 0
    p = B.make_params(32, 8, 96, 8, torch.bfloat16)           # 192-byte rows
    assert B.lib().sablock_decode_workspace_bytes(C.addressof(p), 1, 100) == 0
    p = B.make_params(32, 8, 128, 8, torch.bfloat16)
    fake = C.c_void_p(256)
    assert B.lib().sablock_decode_attention(C.addressof(p), 1, fake, fake, fake, 0, None, fake, None, fake, 1 << 30, None) == 1
    assert B.lib().sablock_decode_attention(C.addressof(p), 1, fake, fake, fake, 100, None, fake, None, fake, 16, None) == 3
