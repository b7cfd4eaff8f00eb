"""Pins for the float64 CPU checker: each test ties one part of it to something other
than itself (hand-worked traces, library routines, closed forms, brute force, invariants
the paper states).  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alg2_examples.txt")


def _golden(kind):
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, *fields = [x.strip() for x in line.split("|")]
            k, name = head.split()
            if k == kind:
                out.append((name, fields))
    return out


def _nums(s, t=float):
    return [t(x) for x in s.split()]


# ------------------------------------------------------------------ Sec. 3.1 segmentation
def _brute_segments(ids, W, delims):
    T = len(ids) - W
    seg_id = [sum(1 for u in range(t) if ids[u] in delims) for t in range(T)]
    starts = [0] + [t for t in range(1, T) if ids[t - 1] in delims] + [T]
    return seg_id, starts


@pytest.mark.parametrize("L,W,gap,seed", [(64, 8, 5, 0), (200, 16, 20, 1), (33, 32, 3, 2), (300, 4, 2, 3)])
def test_segment_matches_brute_force(L, W, gap, seed):
    vocab = 1000
    ids = synth.make_token_ids(L, vocab, gap, seed)
    bm = synth.delimiter_bitmap(vocab)
    seg_id, seg_start = oracle.segment(ids, W, bm, vocab)
    b_id, b_start = _brute_segments(ids.tolist(), W, set(synth.delimiter_ids(vocab)))
    assert seg_id.tolist() == b_id
    assert seg_start.tolist() == b_start


def test_segment_edge_cases():
    vocab = 64
    bm = synth.delimiter_bitmap(vocab)
    sent, para = synth.delimiter_ids(vocab)
    # no delimiters: one segment
    ids = torch.arange(0, 20, dtype=torch.int32)
    seg_id, st = oracle.segment(ids, 4, bm, vocab)
    assert seg_id.tolist() == [0] * 16 and st.tolist() == [0, 16]
    # consecutive delimiters give one-token segments; a delimiter closes its own segment
    ids = torch.tensor([1, sent, para, sent, 2, 3, para, 9, 9, 9], dtype=torch.int32)
    seg_id, st = oracle.segment(ids, 3, bm, vocab)        # T = 7; delimiter at T-1 opens nothing
    assert seg_id.tolist() == [0, 0, 1, 2, 3, 3, 3]
    assert st.tolist() == [0, 2, 3, 4, 7]
    # delimiters inside the window do not matter
    ids = torch.tensor([1, 2, 3, sent, sent], dtype=torch.int32)
    seg_id, st = oracle.segment(ids, 2, bm, vocab)
    assert st.tolist() == [0, 3]
    # out-of-vocabulary ids never delimit
    ids = torch.tensor([-5, 1000, 1, 1, 1, 1], dtype=torch.int32)
    assert oracle.segment(ids, 1, bm, vocab)[1].tolist() == [0, 5]


# ------------------------------------------------------------------ Eq. 2 / Sec. 3.2 attention
def _torch_attention(q, k, W):
    """Library route: causal-masked logits -> torch.softmax in float64, GQA by repeat_interleave."""
    q = q.double(); k = k.double()
    H, _, D = q.shape
    L, Hkv, _ = k.shape
    T = L - W
    kk = k.permute(1, 0, 2).repeat_interleave(H // Hkv, dim=0)            # [H, L, D]
    logits = torch.einsum("hwd,hld->hwl", q, kk) / math.sqrt(D)
    pos_q = T + torch.arange(W)[:, None]
    mask = torch.arange(L)[None, :] > pos_q
    logits = logits.masked_fill(mask[None], float("-inf"))
    return torch.softmax(logits, dim=-1)[:, :, :T]


@pytest.mark.parametrize("H,Hkv,D,W,L", [(4, 1, 64, 16, 100), (8, 4, 32, 5, 37), (6, 2, 16, 1, 20), (3, 3, 8, 7, 9)])
def test_attention_equals_library_softmax(H, Hkv, D, W, L):
    g = torch.Generator().manual_seed(L)
    q = torch.randn(H, W, D, generator=g) * 1.5
    k = torch.randn(L, Hkv, D, generator=g) * 1.5
    A = oracle.attention(q, k, W)
    ref = _torch_attention(q, k, W).numpy()
    np.testing.assert_allclose(A, ref, rtol=1e-11, atol=1e-15)
    abar, s, e = oracle.scores(q, k, eps=1e-6)
    np.testing.assert_allclose(abar, ref.mean(axis=0), rtol=1e-11, atol=1e-15)   # Eq. 3
    np.testing.assert_allclose(s, ref.mean(axis=0).sum(axis=0), rtol=1e-11)      # Eq. 4


def test_scores_closed_form_identical_keys():
    """All keys equal => every causal softmax row is uniform over its T+w+1 keys, so
    s_t = sum_w 1/(T+w+1) for every t (Eqs. 2-4), whatever the queries."""
    H, Hkv, D, W, L = 4, 2, 16, 6, 50
    T = L - W
    g = torch.Generator().manual_seed(1)
    q = torch.randn(H, W, D, generator=g)
    k = torch.randn(1, 1, D, generator=g).expand(L, Hkv, D).contiguous()
    abar, s, e = oracle.scores(q, k, eps=0.0)
    expect = sum(1.0 / (T + w + 1) for w in range(W))
    np.testing.assert_allclose(s, np.full(T, expect), rtol=1e-12)
    from scipy.stats import entropy
    prof = np.array([1.0 / (T + w + 1) for w in range(W)])
    np.testing.assert_allclose(e, np.full(T, entropy(prof)), rtol=1e-12)       # library entropy, eps = 0


def test_entropy_bounds_and_library():
    """0 <= e_t <= ln W (Eq. 6 inner sum); with eps = 0 it is the Shannon entropy (scipy)."""
    from scipy.stats import entropy
    g = torch.Generator().manual_seed(5)
    q = torch.randn(8, 8, 32, generator=g) * 2
    k = torch.randn(120, 2, 32, generator=g) * 2
    abar, s, e0 = oracle.scores(q, k, eps=0.0)
    np.testing.assert_allclose(e0, entropy(abar, axis=0), rtol=1e-10)
    _, _, e = oracle.scores(q, k, eps=1e-6)
    assert (e <= math.log(8) + 1e-12).all() and (e >= -1e-5).all()
    # eps only lowers each term slightly: |e - e0| <= W * eps
    assert np.abs(e - e0).max() <= 8e-6
    # W = 1: Ahat = 1, e = -log(1 + eps)
    _, _, e1 = oracle.scores(q[:, :1].contiguous(), k, eps=1e-6)
    np.testing.assert_allclose(e1, -math.log1p(1e-6), rtol=1e-9)


def test_scores_single_head_single_query_is_softmax():
    g = torch.Generator().manual_seed(9)
    q = torch.randn(1, 1, 16, generator=g)
    k = torch.randn(30, 1, 16, generator=g)
    _, s, _ = oracle.scores(q, k)
    ref = torch.softmax((k[:, 0].double() @ q[0, 0].double()) / 4.0, dim=0)[:29]
    np.testing.assert_allclose(s, ref.numpy(), rtol=1e-12)


def test_gqa_group_mapping():
    """Query head h reads KV head h // (H/Hkv): make KV head 1 all zeros, so the heads of
    group 1 attend uniformly while group 0 does not."""
    H, Hkv, D, W, L = 4, 2, 8, 2, 12
    g = torch.Generator().manual_seed(3)
    q = torch.randn(H, W, D, generator=g)
    k = torch.randn(L, Hkv, D, generator=g)
    k[:, 1] = 0
    A = oracle.attention(q, k, W)
    T = L - W
    for h in (2, 3):
        for w in range(W):
            np.testing.assert_allclose(A[h, w], 1.0 / (T + w + 1), rtol=1e-12)
    assert np.abs(A[0, 0] - 1.0 / (T + 1)).max() > 1e-3


def test_prefill_row_lse_generator_is_the_normaliser_of_eq2():
    """The input generator of the single-sweep mode against the checker: exp(logit - row_lse) must be
    the attention weight A[h, w, t] of Eq. 2 (logits retyped here from the stored values)."""
    cfg = synth.Config("lse", 1, 8, 2, 32, 8, (90,), (32,), (1, 2), "bf16", 5000, 4, 2.0, 9, (), 33)
    b = synth.make_batch(cfg)
    lse = synth.prefill_row_lse(b.q_win, b.k, b.cu_seqlens)[0, 0].double().numpy()      # [H, W]
    q, k = b.q_win[0, 0].double(), b.k[0].double()
    A = oracle.attention(b.q_win[0, 0], b.k[0], cfg.window)
    T = 90 - cfg.window
    for h in range(cfg.n_q_heads):
        logits = (q[h] @ k[:T, h // 4].t()).numpy() / math.sqrt(cfg.head_dim)            # [W, T]
        np.testing.assert_allclose(np.exp(logits - lse[h][:, None]), A[h], rtol=2e-5)


def test_pooling_against_library():
    g = torch.Generator().manual_seed(2)
    s = torch.rand(57, generator=g, dtype=torch.float64)
    for kern in (3, 7):
        mx = torch.nn.functional.max_pool1d(s[None, None], kern, 1, kern // 2)[0, 0]
        np.testing.assert_allclose(oracle.pool(s.numpy(), kern, 0), mx.numpy(), rtol=0)
        av = torch.nn.functional.avg_pool1d(s[None, None], kern, 1, kern // 2, count_include_pad=False)[0, 0]
        np.testing.assert_allclose(oracle.pool(s.numpy(), kern, 1), av.numpy(), rtol=1e-12)
    np.testing.assert_array_equal(oracle.pool(s.numpy(), 1, 0), s.numpy())


# ------------------------------------------------------------------ Eqs. 5-8 refinement
def test_refine_hand_example():
    for name, f in _golden("refine"):
        s, e, st = _nums(f[0]), _nums(f[1]), _nums(f[2], int)
        I, Dk, om, sr = oracle.refine(s, e, st, alpha=float(f[3]), eta=float(f[4]))
        np.testing.assert_allclose(I, _nums(f[5]), rtol=1e-12)
        np.testing.assert_allclose(Dk, _nums(f[6]), rtol=1e-12)
        np.testing.assert_allclose(om, _nums(f[7]), rtol=1e-12)
        np.testing.assert_allclose(sr, _nums(f[8]), rtol=1e-12)


def test_refine_invariants():
    rng = np.random.default_rng(0)
    s = rng.random(200); e = rng.random(200) * 2
    st = np.array([0, 1, 5, 80, 81, 200], np.int32)
    I, Dk, om, sr = oracle.refine(s, e, st)
    # within a segment the order of tokens is unchanged (Sec. 3.2, last paragraph)
    for a, b in zip(st[:-1], st[1:]):
        assert (np.argsort(-s[a:b], kind="stable") == np.argsort(-sr[a:b], kind="stable")).all()
        ratio = sr[a:b] / s[a:b]
        np.testing.assert_allclose(ratio, ratio[0], rtol=1e-12)
    # alpha = 0 leaves the scores alone; eta = 0 makes omega = I
    np.testing.assert_array_equal(oracle.refine(s, e, st, alpha=0.0)[3], s)
    np.testing.assert_allclose(oracle.refine(s, e, st, eta=0.0)[2], I, rtol=1e-15)
    np.testing.assert_allclose(I, [s[a:b].mean() for a, b in zip(st[:-1], st[1:])], rtol=1e-12)
    np.testing.assert_allclose(Dk, [e[a:b].mean() for a, b in zip(st[:-1], st[1:])], rtol=1e-12)


# ------------------------------------------------------------------ Algorithm 2
def test_fill_hand_traces():
    for name, f in _golden("fill"):
        sv, b, g = _nums(f[0]), int(f[1]), int(f[2])
        taken, score, blocks = oracle.segment_fill(sv, b, g)
        assert np.flatnonzero(taken).tolist() == _nums(f[3], int), name
        assert score == float(f[4]), name


def test_select_hand_traces():
    for name, f in _golden("select"):
        r = oracle.select(_nums(f[0]), _nums(f[1], int), int(f[2]), _nums(f[3], int), tau=float(f[4]))
        assert r["keep"].tolist() == _nums(f[5], int), name
        assert r["g_star"].tolist() == _nums(f[6], int), name
        assert r["b_k"].tolist() == _nums(f[7], int), name


def _margin(tok):
    if tok == "inf":
        return math.inf
    num, _, den = tok.partition("/")
    return float(num) / float(den or 1)


def test_decision_margins_hand_traces():
    """The four decision margins the comparison protocol gates on, against hand-worked values."""
    fills = dict(_golden("fill"))
    for name, f in _golden("fillmargins"):
        src = fills[name]
        *_, m = oracle.segment_fill(_nums(src[0]), int(src[1]), int(src[2]), want_margins=True)
        np.testing.assert_allclose(m, [_margin(x) for x in f], rtol=1e-12, atol=1e-15, err_msg=name)
    selects = dict(_golden("select"))
    for name, f in _golden("selectmargins"):
        src = selects[name]
        r = oracle.select(_nums(src[0]), _nums(src[1], int), int(src[2]), _nums(src[3], int), tau=float(src[4]))
        np.testing.assert_allclose(r["margins"], [_margin(x) for x in f], rtol=1e-12, atol=1e-15, err_msg=name)


def _random_problem(rng, quantised):
    n_seg = int(rng.integers(1, 6))
    lens = rng.integers(1, 9, n_seg)
    st = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(st[-1])
    sr = rng.random(T) ** 3
    if quantised:
        sr = np.round(sr * 6) / 6 + 0.0          # many exact ties
    B = int(rng.integers(0, T + 1))
    return sr, st, T, B


@pytest.mark.parametrize("quantised", [False, True])
def test_topB_equals_full_sort_and_budgets(quantised):
    rng = np.random.default_rng(11 + quantised)
    for _ in range(200):
        sr, st, T, B = _random_problem(rng, quantised)
        r = oracle.select(sr, st, B, [1], tau=0.85)            # g = 1 only: T* = T_topB (Alg. 2)
        order = np.argsort(-sr, kind="stable")                 # library sort, ties to the lower index
        top = np.sort(order[:B])
        assert r["keep"].tolist() == top.tolist()
        assert r["b_k"].sum() == B                             # sum_k b_k = B (Eq. 10)
        assert [int(np.isin(top, np.arange(a, z)).sum()) for a, z in zip(st[:-1], st[1:])] == r["b_k"].tolist()
        rest = np.setdiff1d(np.arange(T), top)
        if len(top) and len(rest):
            assert sr[rest].max() <= sr[top].min()             # nth-element property


@pytest.mark.parametrize("quantised", [False, True])
def test_search_against_brute_force(quantised):
    rng = np.random.default_rng(5 + quantised)
    cands = [1, 2, 3, 4, 5, 8]
    for trial in range(300):
        sr, st, T, B = _random_problem(rng, quantised)
        tau = float(rng.choice([0.0, 0.5, 0.85, 0.95, 1.0]))
        r = oracle.select(sr, st, B, cands, tau=tau)
        keep = r["keep"]
        assert len(keep) == B and (np.diff(keep) > 0).all() and (keep < T).all()       # Eq. 13
        top = np.sort(np.argsort(-sr, kind="stable")[:B])
        for k, (a, z) in enumerate(zip(st[:-1], st[1:])):
            n, b = z - a, int(r["b_k"][k])
            mine = keep[(keep >= a) & (keep < z)] - a
            assert len(mine) == b                                                      # |T_k*| = b_k
            if b == 0:
                assert r["g_star"][k] == 0
                continue
            sv = sr[a:z]
            # (i) the token-level baseline is the best b-subset, so R_k(g) <= 1
            base = max(sum(c) for c in itertools.combinations(sv.tolist(), b))
            t1, sc1, _ = oracle.segment_fill(sv, b, 1)
            assert abs(sc1 - base) <= 1e-12 * max(1.0, base)
            # (iii) T_k(1) = T_topB within the segment
            assert np.flatnonzero(t1).tolist() == (top[(top >= a) & (top < z)] - a).tolist()
            # (ii) g* = max{g in G_k : Score(g) >= tau * base} by evaluating every g (Eq. 12)
            feas = [g for g in cands if g <= min(n, b)]
            ok = []
            for g in feas:
                tg, sc, blocks = oracle.segment_fill(sv, b, g)
                assert tg.sum() == b                                                   # (iv)
                assert sc <= sc1 + 1e-12
                assert abs(sc - sv[tg].sum()) < 1e-12
                # blocks are aligned to the segment start and stay inside the segment
                for (ba, bz) in blocks:
                    assert ba % g == 0 and 0 <= ba < bz <= n and bz - ba <= g
                covered = np.zeros(n, bool)
                for (ba, bz) in blocks:
                    covered[ba:bz] = True
                assert covered[tg].all()
                if g == 1 or sc >= tau * sc1:
                    ok.append(g)
            assert r["g_star"][k] == max(ok)
            tg, _, _ = oracle.segment_fill(sv, b, int(r["g_star"][k]))
            assert np.flatnonzero(tg).tolist() == mine.tolist()
            if tau == 0.0:
                assert r["g_star"][k] == max(feas)                                     # (v)
        # no selected block crosses a segment boundary
        for (ba, bz) in r["blocks"]:
            k = np.searchsorted(st, ba, side="right") - 1
            assert st[k] <= ba and bz <= st[k + 1]


def test_block_size_grows_with_budget():
    """Larger budgets favour larger blocks (Sec. 3.3, last paragraph): mean g* over active
    segments is non-decreasing along a budget sweep on a smooth synthetic score profile."""
    rng = np.random.default_rng(0)
    T = 4000
    st = np.arange(0, T + 1, 40).astype(np.int32)
    base = np.repeat(rng.random(len(st) - 1) ** 4, 40)
    sr = base * (0.6 + 0.4 * rng.random(T))
    means = []
    for B in (50, 200, 800, 2400):
        r = oracle.select(sr, st, B, [1, 2, 4, 8, 16, 32])
        act = r["g_star"][r["b_k"] > 0]
        means.append(act.mean())
    assert all(b >= a for a, b in zip(means, means[1:])), means


# ------------------------------------------------------------------ whole pass
def test_compress_invariants_tiny_config():
    cfg = synth.CONFIGS["tiny"]
    b = synth.make_batch(cfg)
    L, W = cfg.seq_lens[0], cfg.window
    r = oracle.compress(b.q_win[0, 0], b.k[0], b.token_ids, b.bitmap, cfg.vocab, 64, cfg.candidates)
    idx = r["out_idx"]
    assert r["n_keep"] == 64 and len(idx) == 64
    assert (np.diff(idx) > 0).all()
    assert idx[-W:].tolist() == list(range(L - W, L))              # window always kept (Sec. 3.1)
    assert r["b_k"].sum() == 64 - W
    assert 0 < r["s"].sum() < W                                    # window keys take some mass
    # every g* is a candidate no larger than min(|S_k|, b_k)
    lens = np.diff(r["seg_start"])
    for g, n, bk in zip(r["g_star"], lens, r["b_k"]):
        assert (bk == 0 and g == 0) or (g in cfg.candidates and g <= min(n, bk))
    # cache untouched when the budget covers the prompt
    r2 = oracle.compress(b.q_win[0, 0], b.k[0], b.token_ids, b.bitmap, cfg.vocab, L, cfg.candidates)
    assert r2["out_idx"].tolist() == list(range(L))
    kb = oracle.gather(b.k[0], r2["out_idx"])
    assert (kb == b.k[0].contiguous().view(torch.uint8).numpy().reshape(L, -1)).all()


def _compose(q, k, ids, bitmap, vocab, W, n_out, cands, pool_kernel, pool_mode, alpha=0.9, eta=1.0, tau=0.85):
    """The pass put together from the stage functions, each of which is pinned on its own above."""
    seg_id, seg_start = oracle.segment(ids, W, bitmap, vocab)
    _, s, e = oracle.scores(q, k, eps=1e-6)                     # entropy from the unpooled attention
    sp = oracle.pool(s, pool_kernel, pool_mode) if pool_kernel > 1 else s
    I, Dk, om, sr = oracle.refine(sp, e, seg_start, alpha=alpha, eta=eta)
    sel = oracle.select(sr, seg_start, n_out - W, cands, tau=tau)
    T = k.shape[0] - W
    return dict(seg_id=seg_id, seg_start=seg_start, s=sp, e=e, s_ref=sr, g_star=sel["g_star"], b_k=sel["b_k"],
                out_idx=np.concatenate([sel["keep"], np.arange(T, T + W, dtype=np.int32)]))


@pytest.mark.parametrize("shape", ["tiny", "gqa8"])
@pytest.mark.parametrize("pool_kernel,pool_mode", [(1, 0), (7, 0), (7, 1)])
def test_compress_is_the_composition_of_its_stages(shape, pool_kernel, pool_mode):
    """The glue of the whole-pass function: segmentation, scores, pooling of s only (the entropy keeps
    the unpooled attention), refinement of the pooled s, Algorithm 2 with B = budget - W, window last.
    A swapped argument or a wrong order there changes one of the compared arrays."""
    if shape == "tiny":
        cfg = synth.CONFIGS["tiny"]
        budget = 64
    else:
        cfg = synth.Config("gqa8", 1, 8, 2, 32, 8, (300,), (48,), (1, 2, 3, 5), "bf16", 5000, 4, 2.0, 9, (0.4,), 21)
        budget = 48
    b = synth.make_batch(cfg)
    q, k, ids, W = b.q_win[0, 0], b.k[0], b.token_ids, cfg.window
    r = oracle.compress(q, k, ids, b.bitmap, cfg.vocab, budget, cfg.candidates, pool_kernel=pool_kernel,
                        pool_mode=pool_mode, alpha=0.7, eta=0.5, tau=0.9)
    c = _compose(q, k, ids, b.bitmap, cfg.vocab, W, budget, cfg.candidates, pool_kernel, pool_mode, 0.7, 0.5, 0.9)
    for name in ("seg_id", "seg_start", "g_star", "b_k", "out_idx"):
        assert r[name].tolist() == c[name].tolist(), name
    for name in ("s", "e", "s_ref"):
        np.testing.assert_array_equal(r[name], c[name], err_msg=name)
    if pool_kernel > 1:                                         # pooling did change the scores it was given
        assert not np.array_equal(c["s"], oracle.scores(q, k, eps=1e-6)[1])
    # the other reading of "budget" (Eq. 13 and the sentence after it): B = budget, W more entries come out
    r0 = oracle.compress(q, k, ids, b.bitmap, cfg.vocab, budget - W, cfg.candidates, pool_kernel=pool_kernel,
                         pool_mode=pool_mode, alpha=0.7, eta=0.5, tau=0.9, budget_includes_window=0)
    assert r0["n_keep"] == budget and r0["out_idx"].tolist() == r["out_idx"].tolist()
    L = k.shape[0]
    full = oracle.compress(q, k, ids, b.bitmap, cfg.vocab, L - W, cfg.candidates, budget_includes_window=0)
    assert full["out_idx"].tolist() == list(range(L))           # budget + W >= L: nothing is evicted


def test_ablation_settings_reduce_to_their_definitions():
    """What the ablation presets mean in the checker (Sec. 4.5): token-level retention is the global
    Top-B of the refined scores; alpha = 0 switches the segment-guided refinement off (Eq. 8); a fixed
    block size g with tau = 0 is used by every segment that can hold one block of g tokens."""
    cfg = synth.Config("abl", 1, 8, 2, 32, 8, (400,), (72,), (1, 2, 4, 8), "bf16", 5000, 4, 2.0, 9, (0.4,), 41)
    b = synth.make_batch(cfg)
    q, k, ids, W = b.q_win[0, 0], b.k[0], b.token_ids, cfg.window
    args = (q, k, ids, b.bitmap, cfg.vocab, 72)
    tok = oracle.compress(*args, (1,))
    top = np.sort(np.argsort(-tok["s_ref"], kind="stable")[: 72 - W])
    assert tok["out_idx"][: 72 - W].tolist() == top.tolist()
    assert set(tok["g_star"][tok["b_k"] > 0].tolist()) == {1}
    plain = oracle.compress(*args, cfg.candidates, alpha=0.0)
    np.testing.assert_array_equal(plain["s_ref"], plain["s"])
    fixed = oracle.compress(*args, (1, 5), tau=0.0)
    lens = np.diff(fixed["seg_start"])
    for g, n, bk in zip(fixed["g_star"], lens, fixed["b_k"]):
        assert g == (0 if bk == 0 else (5 if min(n, bk) >= 5 else 1))


def test_cross_segment_rate_helper_against_brute_force():
    """The motivation statistic of Sec. 2.3 (share of fixed-size blocks that hold tokens of more than one
    segment): the reporting helper against a per-block recount of the checker's segment ids."""
    from paper_2510_22556_b200 import diagnostics
    vocab, W = 1000, 8
    ids = synth.make_token_ids(3000, vocab, 12, 4)
    seg_id, _ = oracle.segment(ids, W, synth.delimiter_bitmap(vocab), vocab)
    T = len(seg_id)
    for g in (1, 2, 5, 7, 64):
        crossing = sum(1 for a in range(0, T, g) if len(set(seg_id[a:a + g].tolist())) > 1)
        n_blocks = (T + g - 1) // g
        assert abs(diagnostics.cross_segment_rate(torch.from_numpy(seg_id), g) - crossing / n_blocks) < 1e-12
    assert diagnostics.cross_segment_rate(torch.from_numpy(seg_id), 1) == 0.0


@pytest.mark.parametrize("H,Hkv,D,n", [(8, 2, 32, 50), (4, 4, 16, 1), (32, 8, 128, 300), (6, 1, 8, 17)])
def test_decode_attention_equals_library_softmax(H, Hkv, D, n):
    """Decoding over a cache (Sec. 4.4): the checker against torch's float64 softmax and matmul, with the
    grouped-query mapping written out by repeat_interleave."""
    g = torch.Generator().manual_seed(n)
    q = torch.randn(H, D, generator=g) * 1.5
    k = torch.randn(n, Hkv, D, generator=g)
    v = torch.randn(n, Hkv, D, generator=g)
    out, lse = oracle.decode_attention(q, k, v)
    kk = k.double().permute(1, 0, 2).repeat_interleave(H // Hkv, dim=0)        # [H, n, D]
    vv = v.double().permute(1, 0, 2).repeat_interleave(H // Hkv, dim=0)
    logits = torch.einsum("hd,hnd->hn", q.double(), kk) / math.sqrt(D)
    ref = torch.einsum("hn,hnd->hd", torch.softmax(logits, dim=-1), vv)
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-12)


def test_decode_attention_closed_forms():
    """Identical keys: uniform weights, the output is the mean of the values.  One dominant key: its value."""
    g = torch.Generator().manual_seed(0)
    q = torch.randn(4, 16, generator=g)
    k = torch.randn(1, 2, 16, generator=g).expand(9, 2, 16).contiguous()
    v = torch.randn(9, 2, 16, generator=g)
    out, lse = oracle.decode_attention(q, k, v)
    mean_v = v.double().mean(dim=0)                                            # [Hkv, D]
    np.testing.assert_allclose(out, mean_v.repeat_interleave(2, dim=0).numpy(), rtol=1e-12)
    k2 = torch.zeros(5, 1, 16)
    k2[3, 0] = q[0] * 100.0
    v2 = torch.randn(5, 1, 16, generator=g)
    out2, _ = oracle.decode_attention(q[:1], k2, v2)
    np.testing.assert_allclose(out2[0], v2[3, 0].double().numpy(), rtol=1e-9, atol=1e-12)


def test_gather_is_byte_exact():
    x = torch.randn(50, 2, 8).to(torch.bfloat16)
    idx = np.array([3, 4, 10, 49], np.int32)
    out = oracle.gather(x, idx)
    ref = x[idx.tolist()].contiguous().view(torch.uint8).numpy().reshape(4, -1)
    assert (out == ref).all()
