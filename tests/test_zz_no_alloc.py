"""sablock_segment_static: segmentation for callers that cannot allocate device memory.

A server with a frozen memory pool, or a plug-in that only ever sees its input and output
buffers, has no workspace to hand to sablock_segment.  The static variant keeps the scan's
scratch in a fixed array inside the library instead.  This test calls it through the C ABI twice
in a row (the array keeps the previous call's contents, so the second call checks that the entry
point clears what it must) and compares with sablock_segment and with the CPU checker bit for bit:
segment ids are integers, so the tolerance of the other segmentation tests applies, which is exact
equality.  It also checks that torch's allocator handed out no device memory during the calls.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import ctypes as C

import pytest
import torch

import oracle
import synth
from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as build_lib

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_lib()
    B.lib()


def _reference(p, ids):
    ws = B.alloc_workspace(p, ids.numel(), ids.numel())
    seg_id, seg_start, n_seg = B.segment(p, ids, ws)
    torch.cuda.synchronize()
    assert B.read_status(ws) == 0
    return seg_id, seg_start, n_seg


def test_static_segmentation_matches_workspace_version_twice_in_a_row():
    vocab, W = 128256, 32
    bitmap = synth.delimiter_bitmap(vocab).cuda()
    p = B.make_params(32, 8, 128, W, torch.bfloat16, bitmap, vocab)
    # two different prompts, the second shorter than the first (stale tile states beyond its end)
    cases = [synth.make_token_ids(100_000 + 77, vocab, 25, 5).cuda(), synth.make_token_ids(9_000 + 3, vocab, 7, 6).cuda()]
    # every buffer of the static call is made before it; the call itself allocates nothing
    bufs = []
    for ids in cases:
        T = ids.numel() - W
        bufs.append((torch.full((T,), -1, dtype=torch.int32, device="cuda"),
                     torch.full((T + 1,), -1, dtype=torch.int32, device="cuda"),
                     torch.zeros(1, dtype=torch.int32, device="cuda"),
                     torch.zeros(1, dtype=torch.int32, device="cuda")))
    torch.cuda.synchronize()
    reserved, allocated = torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
    for ids, (seg_id, seg_start, n_seg, status) in zip(cases, bufs):       # back to back on one stream
        B.segment_static(p, ids, seg_id, seg_start, n_seg, status)
    torch.cuda.synchronize()
    assert (torch.cuda.memory_reserved(), torch.cuda.memory_allocated()) == (reserved, allocated)
    for ids, (seg_id, seg_start, n_seg, status) in zip(cases, bufs):
        ref_id, ref_start, ref_n = _reference(p, ids)
        n = int(ref_n.item())
        assert status.item() == 0
        assert n_seg.item() == n
        assert torch.equal(seg_id, ref_id)
        assert torch.equal(seg_start[: n + 1], ref_start[: n + 1])
        cpu_id, cpu_start = oracle.segment(ids, W, bitmap, vocab)          # the CPU checker, not only CUDA against CUDA
        assert seg_id.cpu().tolist() == cpu_id.tolist()
        assert seg_start[: n + 1].cpu().tolist() == cpu_start.tolist()
    # private status word (status = NULL) and a third call after the others
    seg_id, seg_start, n_seg, _ = bufs[1]
    seg_id.fill_(-1)
    B.segment_static(p, cases[1], seg_id, seg_start, n_seg, None)
    torch.cuda.synchronize()
    assert torch.equal(seg_id, _reference(p, cases[1])[0])


def test_static_segmentation_rejects_what_it_cannot_hold():
    vocab, W = 128256, 32
    bitmap = synth.delimiter_bitmap(vocab).cuda()
    p = B.make_params(32, 8, 128, W, torch.bfloat16, bitmap, vocab)
    fake = C.c_void_p(256)                       # never dereferenced: the call must fail on the host
    too_long = B.SEGMENT_STATIC_MAX_T + W + 1
    rc = B.lib().sablock_segment_static(C.addressof(p), fake, too_long, fake, fake, fake, None, None)
    assert rc == 2                               # SABLOCK_ERR_UNSUPPORTED
    assert B.lib().sablock_segment_static(C.addressof(p), fake, W, fake, fake, fake, None, None) == 1
    assert B.lib().sablock_segment_static(C.addressof(p), None, 4096, fake, fake, fake, None, None) == 1
