"""Host-side checks that need no GPU: the library loads, exports every declared symbol,
validates arguments before touching the device, and sizes its workspace sensibly."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2510_22556_b200 import binding as B
from paper_2510_22556_b200 import build as build_lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_lib()
    return B.lib()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "sablock.h")).read()
    declared = set(re.findall(r"\b(sablock_[a-z_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in sablock.h but not exported"
    assert declared == set(B.EXPORTS)
    assert lib.sablock_params_sizeof() == C.sizeof(B.Params)
    assert lib.sablock_version() >= 100


def test_defaults_follow_the_paper(lib):
    p = B.Params()
    lib.sablock_params_default(C.addressof(p))
    assert (round(p.alpha, 6), round(p.eta, 6), round(p.tau, 6)) == (0.9, 1.0, 0.85)
    assert abs(p.eps - 1e-6) < 1e-12
    assert p.pool_kernel == 1 and p.budget_includes_window == 1


def _params(**kw):
    base = dict(n_q_heads=32, n_kv_heads=8, head_dim=128, window=32, dtype=torch.bfloat16)
    base.update(kw)
    return B.make_params(**base)


def test_workspace_bytes(lib):
    p = _params()
    small = B.workspace_bytes(p, 8192, 8192)
    big = B.workspace_bytes(p, 131072, 131072, 1, 32)
    assert 0 < small < big < 2 * 1024 ** 3
    bad = _params(n_q_heads=30)
    assert lib.sablock_workspace_bytes(C.addressof(bad), 100, 100, 1, 1) == 0
    assert lib.sablock_workspace_bytes(C.addressof(p), 100, 100, 65, 1) == 0


@pytest.mark.parametrize("kw,code", [
    (dict(n_q_heads=30), 1), (dict(window=0), 1), (dict(pool_kernel=4), 1), (dict(score_impl=7), 1),
    (dict(window=128), 2), (dict(head_dim=512), 2), (dict(head_dim=100, score_impl=B.SCORE_TENSOR), 2),
    (dict(dtype=torch.float32, score_impl=B.SCORE_TENSOR), 2),
])
def test_invalid_params_rejected_before_any_device_work(lib, kw, code):
    p = _params(**kw)
    one = C.c_int(0)
    cand = (C.c_int * 2)(1, 2)
    # Non-null but never dereferenced pointers: validation must fail first.
    fake = C.c_void_p(256)
    st = lib.sablock_compress(C.addressof(p), fake, fake, fake, fake, 4096, 256, cand, 2, fake, fake, fake, fake,
                              fake, 1 << 40, None)
    assert st == code


def test_argument_checks(lib):
    p = _params()
    fake = C.c_void_p(256)
    ok_c = (C.c_int * 3)(1, 2, 4)
    big = 1 << 40

    def compress(L=4096, budget=256, cand=ok_c, n=3, ws=fake, ws_bytes=big, q=fake):
        return lib.sablock_compress(C.addressof(p), q, fake, fake, fake, L, budget, cand, n, fake, fake, fake, fake,
                                    ws, ws_bytes, None)

    assert compress(budget=32) == 1                       # budget must exceed the window
    assert compress(budget=0) == 1
    assert compress(L=0) == 1
    assert compress(cand=(C.c_int * 3)(2, 4, 8)) == 1     # 1 must be a candidate
    assert compress(cand=(C.c_int * 3)(1, 4, 4)) == 1     # strictly ascending
    assert compress(n=0) == 1 and compress(n=17) == 1
    assert compress(q=None) == 1
    assert compress(ws_bytes=1024) == 3                   # workspace too small
    assert compress(ws=None) == 3
    cu_bad = (C.c_int * 3)(1, 10, 20)
    assert lib.sablock_compress_layers(C.addressof(p), 1, 2, fake, fake, fake, fake, cu_bad, 256, ok_c, 3, fake, fake,
                                       fake, fake, fake, big, None) == 1
    cu_empty = (C.c_int * 3)(0, 10, 10)
    assert lib.sablock_compress_layers(C.addressof(p), 1, 2, fake, fake, fake, fake, cu_empty, 256, ok_c, 3, fake,
                                       fake, fake, fake, fake, big, None) == 1
    assert lib.sablock_segment(C.addressof(p), fake, 32, fake, fake, fake, fake, big, None) == 1   # L <= W
    assert lib.sablock_status_string(3).decode().startswith("workspace")


def test_host_buffer_entry_point_checks_before_copying(lib):
    """sablock_compress_layers_host sizes its copies from cu_seqlens, the budget and the shapes: all of
    them, the candidates and every pointer are checked before the first copy is enqueued."""
    p = _params()
    fake = C.c_void_p(256)                                # never dereferenced: each call must fail on the host
    ok_c = (C.c_int * 3)(1, 2, 4)
    big = 1 << 40

    def call(cu=(0, 4096), budget=256, cand=ok_c, n=3, ws=fake, ws_bytes=big, dev_out=fake, h_in=fake):
        cu_arr = (C.c_int * len(cu))(*cu)
        return lib.sablock_compress_layers_host(C.addressof(p), 1, len(cu) - 1, h_in, fake, fake, fake, cu_arr, budget,
                                                cand, n, fake, fake, fake, fake, fake, fake, fake, fake, dev_out, fake,
                                                fake, fake, ws, ws_bytes, None)

    assert call(cu=(5, 4096)) == 1                        # cu_seqlens[0] must be 0
    assert call(cu=(0, 4096, 4096)) == 1                  # an empty sequence
    assert call(cu=(0, 4096, 100)) == 1                   # a negative length
    assert call(budget=32) == 1 and call(budget=-7) == 1
    assert call(cand=(C.c_int * 3)(2, 4, 8)) == 1
    assert call(n=0) == 1
    assert call(dev_out=None) == 1                        # device outputs may not be NULL
    assert call(h_in=None) == 1
    assert call(ws=None) == 3 and call(ws_bytes=4096) == 3
    bad = _params(n_q_heads=30)
    cu_arr = (C.c_int * 2)(0, 4096)
    assert lib.sablock_compress_layers_host(C.addressof(bad), 1, 1, fake, fake, fake, fake, cu_arr, 256, ok_c, 3, fake,
                                            fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, big,
                                            None) == 1


def test_read_status_detail_rejects_null(lib):
    raw = (C.c_int * 2)()
    assert lib.sablock_read_status_detail(None, None, C.addressof(raw)) == 1
    assert lib.sablock_read_status_detail(C.c_void_p(256), None, None) == 1


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libsablock.so")
    with pytest.raises(ImportError):
        B.lib()


def test_workspace_regions(lib):
    p = _params()
    total = B.workspace_bytes(p, 20000, 8192, 3, 2)
    seen = []
    for name in ("s", "e", "s_refined", "seg_id", "seg_start", "n_seg"):
        off, nb = C.c_size_t(0), C.c_size_t(0)
        st = lib.sablock_workspace_region(C.addressof(p), 20000, 8192, 3, 2, name.encode(), C.addressof(off),
                                          C.addressof(nb))
        assert st == 0 and off.value % 256 == 0 and off.value + nb.value <= total
        seen.append((off.value, off.value + nb.value))
    seen.sort()
    assert all(a[1] <= b[0] for a, b in zip(seen, seen[1:]))          # regions do not overlap
    off, nb = C.c_size_t(0), C.c_size_t(0)
    assert lib.sablock_workspace_region(C.addressof(p), 20000, 8192, 3, 2, b"nope", C.addressof(off),
                                        C.addressof(nb)) == 1
    ws = torch.zeros(total, dtype=torch.uint8)
    v = B.workspace_view(p, ws, "s_refined", 20000, 8192, 3, 2)
    assert v.shape == (2, 20000) and v.dtype == torch.float32
