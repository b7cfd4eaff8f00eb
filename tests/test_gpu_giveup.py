"""The give-up paths of the bounded device-side waits, exercised without hanging anything: a second
build of the library has the waits shortened to about a millisecond and hooks that make ONE producer
withhold its post (a tile of the segmentation scan never publishes its state; one CTA of the Top-B
select never reports its histogram; one CTA of the persistent score kernel never reports its row
sums).  The waiting side must run into its limit, the kernel must return, the status word must say
TIMEOUT and the word after it must name the wait.  Nothing traps or faults; the product library is
not involved (needs a B200)."""
import numpy as np
import pytest
import torch

import synth
from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as pkg_build
from paper_2510_22556_b200.build import build_test_hooks

pytestmark = pytest.mark.gpu

TIMEOUT = 5          # SABLOCK_ERR_TIMEOUT
HOOK_SEGMENT, HOOK_TOPB, HOOK_SCORE = 1, 2, 4


@pytest.fixture(scope="module")
def hooked():
    pkg_build()
    path = build_test_hooks()
    with B.use_library(path) as l:
        assert l.sablock_test_set_hooks(0) == 0
        yield l
        l.sablock_test_set_hooks(0)


def _code(word):
    return word & 0xff


def test_segmentation_lookback_gives_up(hooked):
    vocab, W, L = 128256, 32, 5 * 2048 + 32
    bitmap = synth.delimiter_bitmap(vocab).cuda()
    ids = synth.make_token_ids(L, vocab, 25, 3).cuda()
    p = B.make_params(32, 8, 128, W, torch.bfloat16, bitmap, vocab)
    ws = B.alloc_workspace(p, L, L)
    # with the hook off the shortened waits are long enough for a normal run
    B.segment(p, ids, ws)
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0)
    assert hooked.sablock_test_set_hooks(HOOK_SEGMENT) == 0
    B.segment(p, ids, ws)
    torch.cuda.synchronize()                                  # the kernel came back
    code, raw, where = B.read_status_detail(ws)
    assert code == TIMEOUT and raw & 1
    assert _code(where) == 30                                 # the look-back of the segmentation scan
    hooked.sablock_test_set_hooks(0)
    B.segment(p, ids, ws)                                     # and the context is as usable as before
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0)


def test_topb_select_gives_up(hooked):
    T, W = 16384, 32
    L = T + W
    p = B.make_params(32, 8, 128, W, torch.bfloat16)
    ws = B.alloc_workspace(p, L, L)
    rng = np.random.default_rng(0)
    sr = torch.from_numpy(rng.random(T).astype(np.float32)).cuda()
    st = np.arange(0, T + 1, 32).astype(np.int32)
    seg_start = torch.zeros(T + 1, dtype=torch.int32, device="cuda")
    seg_start[: len(st)] = torch.from_numpy(st).cuda()
    n_seg = torch.tensor([len(st) - 1], dtype=torch.int32, device="cuda")
    out_idx, _, _ = B.select(p, sr, L, seg_start, n_seg, 256 + W, [1, 2, 4], ws)
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0)
    good = out_idx.clone()
    assert hooked.sablock_test_set_hooks(HOOK_TOPB) == 0
    out_idx, _, _ = B.select(p, sr, L, seg_start, n_seg, 256 + W, [1, 2, 4], ws)
    torch.cuda.synchronize()
    code, raw, where = B.read_status_detail(ws)
    assert code == TIMEOUT and raw & 1 and _code(where) == 31
    idx = out_idx.cpu().numpy()
    assert ((idx >= 0) & (idx < L)).all()                     # whatever was produced stays inside the sequence
    hooked.sablock_test_set_hooks(0)
    out_idx, _, _ = B.select(p, sr, L, seg_start, n_seg, 256 + W, [1, 2, 4], ws)
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0) and torch.equal(out_idx, good)


def test_score_kernel_handover_gives_up(hooked):
    cfg = synth.CONFIGS["layer8k"]
    b = synth.make_batch(cfg, device="cuda")
    L = b.cu_seqlens[-1]
    p = B.make_params(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, torch.bfloat16, b.bitmap, cfg.vocab,
                      score_impl=B.SCORE_FUSED)
    ws = B.alloc_workspace(p, L, L)
    out = B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 256, cfg.candidates, ws)
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0)
    good = out.out_idx.clone()
    assert hooked.sablock_test_set_hooks(HOOK_SCORE) == 0
    out = B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 256, cfg.candidates, ws)
    torch.cuda.synchronize()                                  # every role of every CTA left its loop
    code, raw, where = B.read_status_detail(ws)
    assert code == TIMEOUT and raw & 1
    assert 1 <= _code(where) <= 21                            # one of the score kernel's waits
    idx = out.out_idx.cpu().numpy()
    assert ((idx >= 0) & (idx < L)).all()
    hooked.sablock_test_set_hooks(0)
    out = B.compress_layers(p, b.q_win, b.k, b.v, b.token_ids, b.cu_seqlens, 256, cfg.candidates, ws)
    torch.cuda.synchronize()
    assert B.read_status_detail(ws) == (0, 0, 0) and torch.equal(out.out_idx, good)
