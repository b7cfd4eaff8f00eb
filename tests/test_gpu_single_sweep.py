"""Single-sweep mode: the caller passes the log of Eq. 2's normaliser for every window row (what a
FlashAttention prefill keeps per query row, Sec. 4.1), and the scores are computed in one sweep
over K.  The oracle stays as it is (it computes its own normaliser); the row log-sum-exps are
computed in fp32 from the same stored inputs; tolerances and the index protocol are those of the
two-sweep mode (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as build_lib
from parity import assert_scores_close
from test_gpu_compress import check_invariants_every_layer, run_batch, _params

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_lib()
    B.lib()


def _with_lse(cfg, batch, budget, layers_to_check=None, **kw):
    lse = synth.prefill_row_lse(batch.q_win, batch.k, batch.cu_seqlens)
    return run_batch(cfg, batch, budget, layers_to_check=layers_to_check, row_lse=lse, **kw)


@pytest.mark.parametrize("impl", [B.SCORE_SIMT, B.SCORE_TENSOR, B.SCORE_FUSED])
def test_score_stage_with_row_lse(impl):
    cfg = synth.CONFIGS["layer8k"]
    b = synth.make_batch(cfg, device="cuda", seq_lens=[2048 + 77])
    L = b.cu_seqlens[-1]
    lse = synth.prefill_row_lse(b.q_win, b.k, b.cu_seqlens)
    p = _params(cfg, b.bitmap, score_impl=impl, row_lse=lse)
    ws = B.alloc_workspace(p, L, L)
    _, seg_start, n_seg = B.segment(p, b.token_ids, ws)
    s, e, sr, _ = B.score(p, b.q_win[0, 0], b.k[0], seg_start, n_seg, ws)
    torch.cuda.synchronize()
    assert B.read_status(ws) == 0
    _, s_ref, e_ref = oracle.scores(b.q_win[0, 0], b.k[0], eps=float(np.float32(1e-6)))
    assert_scores_close(s, s_ref, "s")
    assert_scores_close(e, e_ref, "e", abs_=1e-4)


def test_tiny_config_fp32_with_row_lse():
    cfg = synth.CONFIGS["tiny"]
    b = synth.make_batch(cfg, device="cuda")
    out, infos = _with_lse(cfg, b, 64)
    assert out.n_keep.item() == 64


@pytest.mark.parametrize("budget", [96, 128, 256])
def test_layer8k_config_single_sweep(budget):
    cfg = synth.CONFIGS["layer8k"]
    b = synth.make_batch(cfg, device="cuda")
    out, infos = _with_lse(cfg, b, budget, score_impl=B.SCORE_FUSED)
    two, _ = run_batch(cfg, b, budget)
    assert torch.equal(out.out_idx, two.out_idx)          # both modes retain the same positions here


def test_single_sweep_runs_are_bit_identical():
    cfg = synth.CONFIGS["ragged16"]
    b = synth.make_batch(cfg, device="cuda", n_layers=3, seq_lens=[5000, 129, 2222, 100, 777])
    lse = synth.prefill_row_lse(b.q_win, b.k, b.cu_seqlens)
    p = _params(cfg, b.bitmap, row_lse=lse)
    total, max_L = b.cu_seqlens[-1], 5000
    ws = B.alloc_workspace(p, total, max_L, 5, 3)
    runs = []
    out = B.LayersOut(p, 3, 5, 128, b.k.dtype)          # rows beyond n_keep of a short sequence are never written
    out.out_idx.fill_(-1)
    for _ in range(2):
        out = B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 128, cfg.candidates, ws, out)
        torch.cuda.synchronize()
        assert B.read_status(ws) == 0
        runs.append((B.workspace_view(p, ws, "s", total, max_L, 5, 3).clone(), out.out_idx.clone()))
    assert torch.equal(runs[0][0], runs[1][0]) and torch.equal(runs[0][1], runs[1][1])


def test_many_short_phases_single_sweep():
    """Short sequences give every CTA one tile step per (problem, KV head) phase, the case in which the
    producer runs furthest ahead of the epilogue relative to the per-phase buffers (query blocks,
    log-sum-exps).  64 layers of eight such sequences, twice: identical runs, two problems against the oracle."""
    cfg = synth.CONFIGS["ragged16"]
    lens = [2000, 1900, 2100, 1500, 2048, 1800, 2200, 1700]
    b = synth.make_batch(cfg, device="cuda", n_layers=64, seq_lens=lens)
    lse = synth.prefill_row_lse(b.q_win, b.k, b.cu_seqlens)
    p = _params(cfg, b.bitmap, row_lse=lse)
    total, max_L = b.cu_seqlens[-1], max(lens)
    ws = B.alloc_workspace(p, total, max_L, len(lens), 64)
    out = B.LayersOut(p, 64, len(lens), 128, b.k.dtype)
    runs = []
    for _ in range(3):
        B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 128, cfg.candidates, ws, out)
        torch.cuda.synchronize()
        assert B.read_status(ws) == 0
        runs.append((B.workspace_view(p, ws, "s", total, max_L, len(lens), 64).clone(), out.out_idx.clone()))
    for r in runs[1:]:
        assert torch.equal(runs[0][0], r[0]) and torch.equal(runs[0][1], r[1])
    s = runs[0][0]
    for (l, i) in ((0, 0), (63, 7), (31, 3)):
        a, z = b.cu_seqlens[i], b.cu_seqlens[i + 1]
        _, s_ref, _ = oracle.scores(b.q_win[l, i], b.k[l, a:z], eps=float(np.float32(1e-6)))
        assert_scores_close(s[l, a:z - cfg.window], s_ref, "s")


def test_ragged_and_edge_lengths_single_sweep():
    cfg = synth.CONFIGS["ragged16"]
    lens = [128 * 3 - 1, 128 * 3, 128 * 3 + 33, 100, 1024 + 32, 4096 + 17, 33]
    b = synth.make_batch(cfg, device="cuda", n_layers=2, seq_lens=lens)
    out, infos = _with_lse(cfg, b, 128)
    assert out.n_keep[0].cpu().tolist() == [128, 128, 128, 100, 128, 128, 33]


def test_ragged16_config_full_size_single_sweep():
    cfg = synth.CONFIGS["ragged16"]
    b = synth.make_batch(cfg, device="cuda")
    out, infos = _with_lse(cfg, b, 512, layers_to_check=[7])
    check_invariants_every_layer(cfg, b, out, 512)


def test_headline_config_full_size_single_sweep():
    """The benchmark's launch configuration in single-sweep mode: layers 0 and 31 against the oracle in
    full, every layer for the invariants and the gathered rows."""
    cfg = synth.CONFIGS["headline128k"]
    b = synth.make_batch(cfg, device="cuda")
    out, infos = _with_lse(cfg, b, 1024, layers_to_check=[0, 31])
    idx = out.out_idx[:, 0].cpu().numpy()
    L, W = cfg.seq_lens[0], cfg.window
    assert (out.n_keep.cpu().numpy() == 1024).all()
    assert (np.diff(idx, axis=1) > 0).all()
    assert (idx[:, -W:] == np.arange(L - W, L)[None]).all()
    for l in range(cfg.n_layers):
        sel = torch.from_numpy(idx[l]).cuda().long()
        assert torch.equal(out.out_k[l, 0], b.k[l, sel]) and torch.equal(out.out_v[l, 0], b.v[l, sel])
