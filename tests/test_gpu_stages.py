"""Per-stage parity of the CUDA library against the float64 oracle (needs a B200)."""
import math

import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as build_lib
from parity import ABS, REL, assert_scores_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_lib()
    B.lib()


def _sync_ok(ws):
    torch.cuda.synchronize()
    assert B.read_status(ws) == 0


# ------------------------------------------------------------------ stage 1
@pytest.mark.parametrize("L,W,gap,delims", [
    (512, 16, 20, True), (8192, 32, 25, True), (5000, 32, 3, True), (70001, 8, 25, True),
    (4096, 32, 25, False), (2049 + 32, 32, -1, True), (33, 32, 2, True), (131072, 32, 25, True),
])
def test_segment_bit_exact(L, W, gap, delims):
    vocab = 128256
    ids = synth.make_token_ids(L, vocab, abs(gap) + 1, seed=L + W, with_delimiters=delims)
    if gap < 0:                                         # every token a delimiter
        ids[:] = synth.delimiter_ids(vocab)[0]
    bm = synth.delimiter_bitmap(vocab)
    ref_id, ref_start = oracle.segment(ids, W, bm, vocab)
    p = B.make_params(32, 8, 128, W, torch.bfloat16, bm.cuda(), vocab)
    ws = B.alloc_workspace(p, L, L)
    seg_id, seg_start, n_seg = B.segment(p, ids.cuda(), ws)
    _sync_ok(ws)
    n = int(n_seg.item())
    assert n == len(ref_start) - 1
    assert torch.equal(seg_id[: L - W].cpu(), torch.from_numpy(ref_id))
    assert torch.equal(seg_start[: n + 1].cpu(), torch.from_numpy(ref_start))


# ------------------------------------------------------------------ stages 2 + 3
def _score_case(H, Hkv, D, W, L, dtype, impl, seed, gap=25, pool=(1, 0), kappa=2.0):
    cfg = synth.Config("t", 1, H, Hkv, D, W, (L,), (64,), (1, 2), "bf16" if dtype == torch.bfloat16 else "f32",
                       128256, 8, kappa, gap, (0.4,), seed)
    q, k, v, _ = synth.make_layer(cfg, L, seed)
    ids = synth.make_token_ids(L, cfg.vocab, gap, seed + 1)
    bm = synth.delimiter_bitmap(cfg.vocab)
    bm_d = bm.cuda()
    p = B.make_params(H, Hkv, D, W, dtype, bm_d, cfg.vocab, score_impl=impl, pool_kernel=pool[0], pool_mode=pool[1])
    ws = B.alloc_workspace(p, L, L)
    seg_id, seg_start, n_seg = B.segment(p, ids.cuda(), ws)
    s, e, sr, stats = B.score(p, q.cuda(), k.cuda(), seg_start, n_seg, ws, want_stats=True)
    _sync_ok(ws)
    abar, s_ref, e_ref = oracle.scores(q, k, eps=1e-6)
    if pool[0] > 1:
        s_ref = oracle.pool(s_ref, pool[0], pool[1])
    _, st_ref = oracle.segment(ids, W, bm, cfg.vocab)
    I, Dk, om, sr_ref = oracle.refine(s_ref, e_ref, st_ref)
    errs = dict(
        s=assert_scores_close(s, s_ref, "s"),
        e=assert_scores_close(e, e_ref, "e", abs_=1e-4),
        sr=assert_scores_close(sr, sr_ref, "s_refined"),
    )
    ns = len(st_ref) - 1
    assert_scores_close(stats[0, :ns], I, "I_k")
    assert_scores_close(stats[1, :ns], Dk, "D_k", abs_=1e-4)
    assert_scores_close(stats[2, :ns], om, "omega_k")
    # tighter than the stated tolerance: relative error of s well below 2e-3 everywhere it matters
    g = s.cpu().double().numpy()
    big = s_ref > 1e-7
    assert (np.abs(g[big] - s_ref[big]) / s_ref[big]).max() < 2e-3
    return errs


def test_score_simt_tiny_fp32():
    _score_case(4, 1, 64, 16, 512, torch.float32, B.SCORE_SIMT, 0, gap=20)


@pytest.mark.parametrize("H,Hkv,D,W,L", [(8, 2, 32, 5, 300), (6, 3, 48, 16, 1000), (4, 4, 128, 32, 777), (2, 1, 256, 64, 400)])
def test_score_simt_odd_shapes_fp32(H, Hkv, D, W, L):
    _score_case(H, Hkv, D, W, L, torch.float32, B.SCORE_SIMT, L)


def test_score_simt_bf16_llama_shape():
    _score_case(32, 8, 128, 32, 2048 + 77, torch.bfloat16, B.SCORE_SIMT, 3)


@pytest.mark.parametrize("H,Hkv,D,W,L", [
    (32, 8, 128, 32, 8192),        # Llama-3-8B shape, several tiles
    (32, 8, 128, 32, 4096 + 55),   # ragged tail, window straddles a tile boundary
    (8, 2, 128, 32, 160),          # two tiles only
    (8, 2, 128, 32, 129),          # T < one tile
    (16, 4, 128, 16, 3000),        # W = 16: 64 query rows per KV head
    (16, 4, 128, 8, 2500),         # W = 8: 32 rows
    (16, 16, 128, 8, 1500),        # no grouping: 8 rows per KV head
    (12, 4, 128, 32, 1111),        # G = 3: 96 rows (partial last column group)
    (32, 8, 64, 32, 5000),         # head_dim 64
])
def test_score_tensor_core_bf16(H, Hkv, D, W, L):
    _score_case(H, Hkv, D, W, L, torch.bfloat16, B.SCORE_TENSOR, L + W)


def test_score_tensor_core_heavy_tails():
    # large logits: kappa 6 gives |logit| of several tens; the running-max path must hold
    _score_case(32, 8, 128, 32, 3000, torch.bfloat16, B.SCORE_TENSOR, 9, kappa=6.0)


@pytest.mark.parametrize("H,Hkv,L", [
    (32, 8, 8192),         # Llama-3-8B shape, 64 tiles: fewer tiles than CTAs
    (32, 8, 4096 + 55),    # ragged tail, window straddles a tile boundary
    (32, 8, 20000),        # more tiles than CTAs: some CTAs hold two
    (8, 2, 160),           # two tiles only
    (8, 2, 129),           # T < one tile; the second tile holds window keys only
    (8, 2, 128),           # one tile in all: 96 compressible tokens and the window
    (4, 1, 128 * 3 + 32),  # T a whole number of tiles: the window has a tile of its own
])
def test_score_fused_bf16(H, Hkv, L):
    _score_case(H, Hkv, 128, 32, L, torch.bfloat16, B.SCORE_FUSED, L + 3)


def test_score_fused_heavy_tails():
    # large logits: the row sums' reference exponents must move without losing the sum
    _score_case(32, 8, 128, 32, 3000, torch.bfloat16, B.SCORE_FUSED, 9, kappa=6.0)


def test_score_fused_agrees_with_two_launch_path():
    # two implementations of the same arithmetic up to the order of the fp32 sums
    cfg = synth.Config("t", 1, 32, 8, 128, 32, (6000,), (64,), (1, 2), "bf16", 128256, 8, 2.0, 25, (0.4,), 21)
    q, k, v, _ = synth.make_layer(cfg, 6000, 21)
    ids = synth.make_token_ids(6000, cfg.vocab, 25, 22)
    bm = synth.delimiter_bitmap(cfg.vocab).cuda()
    outs = []
    for impl in (B.SCORE_FUSED, B.SCORE_TENSOR):
        p = B.make_params(32, 8, 128, 32, torch.bfloat16, bm, cfg.vocab, score_impl=impl)
        ws = B.alloc_workspace(p, 6000, 6000)
        _, seg_start, n_seg = B.segment(p, ids.cuda(), ws)
        s, e, sr, _ = B.score(p, q.cuda(), k.cuda(), seg_start, n_seg, ws)
        _sync_ok(ws)
        outs.append((s.double().cpu().numpy(), e.double().cpu().numpy()))
    (s0, e0), (s1, e1) = outs
    assert np.abs(s0 - s1).max() <= 1e-7 + 2e-5 * np.abs(s1).max()
    assert np.abs(e0 - e1).max() <= 1e-4


def test_score_fused_refuses_what_it_cannot_run():
    bm = synth.delimiter_bitmap(128256).cuda()
    p = B.make_params(16, 4, 64, 32, torch.bfloat16, bm, 128256, score_impl=B.SCORE_FUSED)     # head_dim 64
    with pytest.raises(B.SablockError):
        B.alloc_workspace(p, 4096, 4096)
    # fewer key rows than one 128-row TMA box: forced FUSED says so, AUTO takes the SIMT kernels
    with pytest.raises(B.SablockError):
        _score_case(8, 2, 128, 32, 33, torch.bfloat16, B.SCORE_FUSED, 5)
    _score_case(8, 2, 128, 32, 33, torch.bfloat16, B.SCORE_AUTO, 5)


@pytest.mark.parametrize("pool", [(7, 0), (7, 1), (3, 1)])
def test_score_with_pooling(pool):
    _score_case(32, 8, 128, 32, 2000, torch.bfloat16, B.SCORE_AUTO, 4, pool=pool)


def test_score_runs_are_bit_identical():
    cfg = synth.CONFIGS["layer8k"]
    b = synth.make_batch(cfg, device="cuda")
    p = B.make_params(32, 8, 128, 32, torch.bfloat16, b.bitmap, cfg.vocab)
    ws = B.alloc_workspace(p, 8192, 8192)
    _, seg_start, n_seg = B.segment(p, b.token_ids, ws)
    outs = []
    for _ in range(2):
        s, e, sr, _ = B.score(p, b.q_win[0, 0], b.k[0], seg_start, n_seg, ws)
        torch.cuda.synchronize()
        outs.append((s.clone(), e.clone(), sr.clone()))
    for a, c in zip(*outs):
        assert torch.equal(a, c)


# ------------------------------------------------------------------ stage 4
def _select_case(T, W, seg_lens, B_tok, cands, tau, quantised, seed):
    rng = np.random.default_rng(seed)
    st = np.concatenate([[0], np.cumsum(seg_lens)]).astype(np.int32)
    assert st[-1] == T
    base = np.repeat(rng.random(len(seg_lens)) ** 3, seg_lens)
    sr = (base * (0.5 + 0.5 * rng.random(T))).astype(np.float32)
    if quantised:
        sr = (np.round(sr * 40) / 40).astype(np.float32)
    L = T + W
    p = B.make_params(32, 8, 128, W, torch.bfloat16, tau=tau)
    ws = B.alloc_workspace(p, L, L)
    seg_start = torch.zeros(T + 1, dtype=torch.int32, device="cuda")
    seg_start[: len(st)] = torch.from_numpy(st).cuda()
    n_seg = torch.tensor([len(seg_lens)], dtype=torch.int32, device="cuda")
    budget = B_tok + W
    out_idx, seg_g, seg_b = B.select(p, torch.from_numpy(sr).cuda(), L, seg_start, n_seg, budget, cands, ws,
                                     want_segments=True)
    _sync_ok(ws)
    r = oracle.select(sr.astype(np.float64), st, B_tok, cands, tau=float(np.float32(tau)))
    idx = out_idx.cpu().numpy()
    assert idx[:B_tok].tolist() == r["keep"].tolist()
    assert idx[B_tok:].tolist() == list(range(T, L))
    ns = len(seg_lens)
    assert seg_b[:ns].cpu().numpy().tolist() == r["b_k"].tolist()
    assert seg_g[:ns].cpu().numpy().tolist() == r["g_star"].tolist()
    return r


@pytest.mark.parametrize("quantised", [False, True])
@pytest.mark.parametrize("tau", [0.0, 0.85, 1.0])
def test_select_matches_oracle(quantised, tau):
    rng = np.random.default_rng(17)
    for trial in range(6):
        n_seg = int(rng.integers(1, 400))
        seg_lens = rng.geometric(1 / 20.0, n_seg).astype(np.int64)
        T = int(seg_lens.sum())
        B_tok = int(rng.integers(1, max(2, T // 2)))
        _select_case(T, 32, seg_lens, B_tok, [1, 2, 4, 8, 16, 32], tau, quantised, trial)


def test_select_paper_candidate_set():
    rng = np.random.default_rng(3)
    seg_lens = rng.geometric(1 / 25.0, 300).astype(np.int64)
    r = _select_case(int(seg_lens.sum()), 8, seg_lens, 1500, [1, 2, 3, 5, 7, 9, 11, 13], 0.85, False, 5)
    assert (r["g_star"] > 1).any()


def test_select_long_segments_and_degenerates():
    # one segment longer than the shared-memory path takes, next to short ones
    _select_case(3000 + 40, 32, np.array([10, 3000, 30]), 700, [1, 2, 4, 8, 16, 32], 0.85, False, 1)
    # no delimiters at all: a single segment
    _select_case(4064, 32, np.array([4064]), 480, [1, 2, 4, 8, 16], 0.85, False, 2)
    _select_case(4064, 32, np.array([4064]), 480, [1, 2, 4, 8, 16], 0.5, True, 3)
    # every token its own segment
    _select_case(1000, 32, np.ones(1000, np.int64), 100, [1, 2, 4], 0.85, False, 4)
    # all scores equal: ties everywhere, lower index wins
    T, W = 640, 32
    p = B.make_params(32, 8, 128, W, torch.bfloat16)
    ws = B.alloc_workspace(p, T + W, T + W)
    st = np.arange(0, T + 1, 64).astype(np.int32)
    seg_start = torch.zeros(T + 1, dtype=torch.int32, device="cuda")
    seg_start[: len(st)] = torch.from_numpy(st).cuda()
    n_seg = torch.tensor([len(st) - 1], dtype=torch.int32, device="cuda")
    sr = torch.full((T,), 0.25, device="cuda")
    out_idx, _, _ = B.select(p, sr, T + W, seg_start, n_seg, 100 + W, [1, 2, 4, 8], ws)
    _sync_ok(ws)
    r = oracle.select(np.full(T, 0.25), st, 100, [1, 2, 4, 8], tau=float(np.float32(0.85)))
    assert out_idx.cpu().numpy()[:100].tolist() == r["keep"].tolist() == list(range(100))


@pytest.mark.parametrize("quantised", [False, True])
def test_select_very_long_segments(quantised):
    """A prompt with few or no delimiters is one segment of the whole compressible region (Sec. 3.1):
    the search must stay linear in the segment length.  Exact against the oracle, ties included."""
    # the whole 128K region as one segment, at several budgets (the block scores repeat when quantised)
    for B_tok, tau in ((992, 0.85), (20000, 0.85), (5001, 0.0), (992, 1.0)):
        _select_case(131040, 32, np.array([131040]), B_tok, [1, 2, 4, 8, 16, 32], tau, quantised, 11 + B_tok)
    # a 20000-token segment between short ones, odd candidate sizes (short last blocks)
    rng = np.random.default_rng(9)
    lens = np.concatenate([rng.geometric(1 / 20.0, 40), [20000], rng.geometric(1 / 20.0, 40), [777, 600]]).astype(np.int64)
    _select_case(int(lens.sum()), 8, lens, 3000, [1, 2, 3, 5, 7, 9, 11, 13], 0.85, quantised, 12)
    _select_case(int(lens.sum()), 8, lens, 9000, [1, 3, 7, 13], 0.6, quantised, 13)


# ------------------------------------------------------------------ stage 5
@pytest.mark.parametrize("dtype,Hkv,D", [(torch.bfloat16, 8, 128), (torch.float32, 1, 64), (torch.bfloat16, 2, 64)])
def test_compact_bytes(dtype, Hkv, D):
    L = 3001
    g = torch.Generator().manual_seed(1)
    k = torch.randn(L, Hkv, D, generator=g).to(dtype)
    v = torch.randn(L, Hkv, D, generator=g).to(dtype)
    idx = torch.sort(torch.randperm(L, generator=g)[:517]).values.to(torch.int32)
    p = B.make_params(Hkv, Hkv, D, 32, dtype)
    ok, ov = B.compact(p, k.cuda(), v.cuda(), idx.cuda())
    torch.cuda.synchronize()
    assert (oracle.gather(k, idx.numpy()) == ok.cpu().view(torch.uint8).numpy().reshape(517, -1)).all()
    assert (oracle.gather(v, idx.numpy()) == ov.cpu().view(torch.uint8).numpy().reshape(517, -1)).all()
