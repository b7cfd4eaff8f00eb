"""Thin ctypes binding of libsablock.so (include/sablock.h): argument marshalling only.

Every function takes torch CUDA tensors (or raw pointers), passes their device pointers
through the C ABI and enqueues on torch's current stream.  No step of the pass runs in
Python or torch; if the library is missing the import of `lib()` fails loudly.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsablock.so")

OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE_TOO_SMALL", 4: "CUDA", 5: "TIMEOUT",
                6: "INTERNAL"}
F32, BF16 = 0, 1
SCORE_AUTO, SCORE_SIMT, SCORE_TENSOR, SCORE_FUSED = 0, 1, 2, 3

EXPORTS = [
    "sablock_params_default", "sablock_status_string", "sablock_version", "sablock_workspace_bytes",
    "sablock_read_status", "sablock_segment", "sablock_score", "sablock_select", "sablock_compact",
    "sablock_compress", "sablock_compress_layers", "sablock_compress_layers_host", "sablock_last_launch_count",
    "sablock_params_sizeof", "sablock_workspace_region", "sablock_profile_enable", "sablock_profile_read",
    "sablock_profile_stage_name", "sablock_segment_static", "sablock_last_cuda_error", "sablock_read_status_detail",
    "sablock_decode_workspace_bytes", "sablock_decode_attention",
]


class Params(C.Structure):
    _fields_ = [
        ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int), ("window", C.c_int),
        ("dtype", C.c_int),
        ("k_stride_token", C.c_longlong), ("k_stride_head", C.c_longlong), ("k_stride_layer", C.c_longlong),
        ("v_stride_token", C.c_longlong), ("v_stride_head", C.c_longlong), ("v_stride_layer", C.c_longlong),
        ("alpha", C.c_float), ("eta", C.c_float), ("eps", C.c_float), ("tau", C.c_float),
        ("pool_kernel", C.c_int), ("pool_mode", C.c_int), ("budget_includes_window", C.c_int),
        ("delim_bitmap", C.c_void_p), ("vocab_size", C.c_int),
        ("score_impl", C.c_int), ("debug_sync", C.c_int), ("row_lse", C.c_void_p), ("reproducible", C.c_int), ("reserved", C.c_int * 5),
    ]


class SablockError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = lib().sablock_last_cuda_error().decode() if code == 4 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({lib().sablock_status_string(code).decode()})"
                         + (f" [{detail}]" if detail else ""))


_lib = None


def _load(path: str):
    """dlopens one build of the library and declares the argument types of its entry points."""
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2510_22556_b200.build` "
                          "or __graft_entry__.build()")
    l = C.CDLL(path)
    l.sablock_status_string.restype = C.c_char_p
    l.sablock_last_cuda_error.restype = C.c_char_p
    l.sablock_params_sizeof.restype = C.c_size_t
    if l.sablock_params_sizeof() != C.sizeof(Params):
        raise ImportError("sablock_params_t layout mismatch between the library and the binding")
    l.sablock_workspace_bytes.restype = C.c_size_t
    l.sablock_workspace_bytes.argtypes = [C.c_void_p, C.c_longlong, C.c_int, C.c_int, C.c_int]
    vp, ci, sz = C.c_void_p, C.c_int, C.c_size_t
    l.sablock_read_status.argtypes = [vp, vp, vp]
    l.sablock_read_status_detail.argtypes = [vp, vp, vp]
    l.sablock_workspace_region.argtypes = [vp, C.c_longlong, ci, ci, ci, C.c_char_p, vp, vp]
    l.sablock_params_default.argtypes = [vp]
    l.sablock_profile_read.argtypes = [ci, vp, ci]
    l.sablock_profile_stage_name.restype = C.c_char_p
    l.sablock_segment.argtypes = [vp, vp, ci, vp, vp, vp, vp, sz, vp]
    l.sablock_segment_static.argtypes = [vp, vp, ci, vp, vp, vp, vp, vp]
    l.sablock_score.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    l.sablock_select.argtypes = [vp, vp, ci, vp, vp, ci, vp, ci, vp, vp, vp, vp, sz, vp]
    l.sablock_compact.argtypes = [vp, vp, vp, ci, vp, ci, vp, vp, vp]
    l.sablock_compress.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, ci, vp, vp, vp, vp, vp, sz, vp]
    l.sablock_compress_layers.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, ci, vp, vp, vp, vp, vp, sz, vp]
    l.sablock_compress_layers_host.argtypes = [vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, ci, vp, vp, vp, vp,
                                               vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    l.sablock_decode_workspace_bytes.restype = C.c_size_t
    l.sablock_decode_workspace_bytes.argtypes = [vp, ci, ci]
    l.sablock_decode_attention.argtypes = [vp, ci, vp, vp, vp, ci, vp, vp, vp, vp, sz, vp]
    return l


def lib():
    """The CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        _lib = _load(LIB_PATH)
    return _lib


@contextlib.contextmanager
def use_library(path: str):
    """Routes every call of this module through another build of the library (the tests of the
    give-up paths use one with shortened waits) for the duration of the block."""
    global _lib
    saved = _lib
    _lib = _load(path)
    try:
        yield _lib
    finally:
        _lib = saved


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != OK:
        raise SablockError(code, where)


def _iarr(xs: Sequence[int]):
    return (C.c_int * len(xs))(*[int(x) for x in xs])


def make_params(n_q_heads: int, n_kv_heads: int, head_dim: int, window: int, dtype: torch.dtype,
                delim_bitmap: Optional[torch.Tensor] = None, vocab_size: int = 0, **kw) -> Params:
    p = Params()
    lib().sablock_params_default(C.addressof(p))
    p.n_q_heads, p.n_kv_heads, p.head_dim, p.window = n_q_heads, n_kv_heads, head_dim, window
    p.dtype = {torch.float32: F32, torch.bfloat16: BF16}[dtype]
    if delim_bitmap is not None:
        p.delim_bitmap = delim_bitmap.data_ptr()
        p.vocab_size = vocab_size
        p._bitmap_ref = delim_bitmap          # keep the device buffer alive as long as the block
    for k, v in kw.items():
        if not hasattr(p, k):
            raise AttributeError(k)
        if k == "row_lse" and isinstance(v, torch.Tensor):
            if v.dtype != torch.float32 or not v.is_contiguous():
                raise TypeError("row_lse must be a contiguous float32 tensor")
            p._row_lse_ref = v                # keep the device buffer alive as long as the block
            v = v.data_ptr()
        setattr(p, k, v)
    return p


def workspace_bytes(p: Params, total_tokens: int, max_L: int, n_seqs: int = 1, n_layers: int = 1) -> int:
    n = lib().sablock_workspace_bytes(C.addressof(p), total_tokens, max_L, n_seqs, n_layers)
    if n == 0:
        raise SablockError(1, "sablock_workspace_bytes")
    return int(n)


def workspace_view(p: Params, ws: torch.Tensor, name: str, total_tokens: int, max_L: int, n_seqs: int = 1,
                   n_layers: int = 1) -> torch.Tensor:
    """A typed view of one of the fused call's intermediate arrays inside the workspace."""
    off, nb = C.c_size_t(0), C.c_size_t(0)
    _check(lib().sablock_workspace_region(C.addressof(p), total_tokens, max_L, n_seqs, n_layers, name.encode(),
                                          C.addressof(off), C.addressof(nb)), "sablock_workspace_region")
    raw = ws[off.value: off.value + nb.value]
    dt = torch.float32 if name in ("s", "e", "s_refined") else torch.int32
    v = raw.view(dt)
    return v.view(n_layers, total_tokens) if dt == torch.float32 else v


def alloc_workspace(p: Params, total_tokens: int, max_L: int, n_seqs: int = 1, n_layers: int = 1,
                    device="cuda") -> torch.Tensor:
    return torch.empty(workspace_bytes(p, total_tokens, max_L, n_seqs, n_layers), dtype=torch.uint8, device=device)


def read_status(ws: torch.Tensor) -> int:
    raw = C.c_int(0)
    code = lib().sablock_read_status(_ptr(ws), _stream(), C.addressof(raw))
    return code


def read_status_detail(ws: torch.Tensor):
    """(status code, raw status word, code | CTA << 8 | warp << 20 of the first wait that gave up)."""
    raw = (C.c_int * 2)()
    code = lib().sablock_read_status_detail(_ptr(ws), _stream(), C.addressof(raw))
    return code, int(raw[0]), int(raw[1])


def profile_enable(slots: int) -> None:
    _check(lib().sablock_profile_enable(int(slots)), "sablock_profile_enable")


def profile_read(slot: int):
    """Stage name -> milliseconds for the fused call that used event slot `slot`."""
    buf = (C.c_float * 16)()
    n = lib().sablock_profile_read(slot, C.addressof(buf), 16)
    return {lib().sablock_profile_stage_name(i).decode(): float(buf[i]) for i in range(n)}


def last_launch_count() -> int:
    return int(lib().sablock_last_launch_count())


def segment(p: Params, token_ids: torch.Tensor, ws: torch.Tensor):
    L = token_ids.numel()
    T = L - p.window
    seg_id = torch.empty(max(T, 1), dtype=torch.int32, device=token_ids.device)
    seg_start = torch.empty(max(T, 1) + 1, dtype=torch.int32, device=token_ids.device)
    n_seg = torch.zeros(1, dtype=torch.int32, device=token_ids.device)
    _check(lib().sablock_segment(C.addressof(p), _ptr(token_ids), L, _ptr(seg_id), _ptr(seg_start), _ptr(n_seg),
                                 _ptr(ws), ws.numel(), _stream()), "sablock_segment")
    return seg_id, seg_start, n_seg


SEGMENT_STATIC_MAX_T = 1024 * 2048


def segment_static(p: Params, token_ids: torch.Tensor, seg_id: torch.Tensor, seg_start: torch.Tensor,
                   n_seg: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    """sablock_segment without a workspace: the caller supplies every buffer (outputs included),
    the scan's scratch is a fixed array inside the library.  Nothing is allocated here."""
    _check(lib().sablock_segment_static(C.addressof(p), _ptr(token_ids), token_ids.numel(), _ptr(seg_id),
                                        _ptr(seg_start), _ptr(n_seg), _ptr(status), _stream()),
           "sablock_segment_static")


def score(p: Params, q_win: torch.Tensor, k: torch.Tensor, seg_start: torch.Tensor, n_seg: torch.Tensor,
          ws: torch.Tensor, want_stats: bool = False):
    L = k.shape[0]
    T = L - p.window
    dev = k.device
    s = torch.empty(T, dtype=torch.float32, device=dev)
    e = torch.empty(T, dtype=torch.float32, device=dev)
    sr = torch.empty(T, dtype=torch.float32, device=dev)
    stats = torch.zeros(3 * T, dtype=torch.float32, device=dev) if want_stats else None
    _check(lib().sablock_score(C.addressof(p), _ptr(q_win), _ptr(k), L, _ptr(seg_start), _ptr(n_seg), _ptr(s), _ptr(e),
                               _ptr(sr), _ptr(stats), _ptr(ws), ws.numel(), _stream()), "sablock_score")
    return s, e, sr, (stats.view(3, T) if want_stats else None)


def rows_out(p: Params, budget: int, L: int) -> int:
    n = budget if p.budget_includes_window else budget + p.window
    return L if n >= L else n


def select(p: Params, s_refined: torch.Tensor, L: int, seg_start: torch.Tensor, n_seg: torch.Tensor, budget: int,
           candidates: Sequence[int], ws: torch.Tensor, want_segments: bool = False):
    dev = s_refined.device
    T = L - p.window
    out_idx = torch.empty(rows_out(p, budget, L), dtype=torch.int32, device=dev)
    seg_g = torch.zeros(max(T, 1), dtype=torch.int32, device=dev) if want_segments else None
    seg_b = torch.zeros(max(T, 1), dtype=torch.int32, device=dev) if want_segments else None
    cand = _iarr(candidates)
    _check(lib().sablock_select(C.addressof(p), _ptr(s_refined), L, _ptr(seg_start), _ptr(n_seg), budget, cand,
                                len(candidates), _ptr(out_idx), _ptr(seg_g), _ptr(seg_b), _ptr(ws), ws.numel(),
                                _stream()), "sablock_select")
    return out_idx, seg_g, seg_b


def compact(p: Params, k: torch.Tensor, v: torch.Tensor, out_idx: torch.Tensor):
    n = out_idx.numel()
    out_k = torch.empty((n,) + tuple(k.shape[1:]), dtype=k.dtype, device=k.device)
    out_v = torch.empty_like(out_k)
    _check(lib().sablock_compact(C.addressof(p), _ptr(k), _ptr(v), k.shape[0], _ptr(out_idx), n, _ptr(out_k),
                                 _ptr(out_v), _stream()), "sablock_compact")
    return out_k, out_v


def compress(p: Params, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, token_ids: torch.Tensor, budget: int,
             candidates: Sequence[int], ws: torch.Tensor):
    """One layer of one sequence.  Returns (out_k, out_v, out_idx, n_keep tensor)."""
    L = k.shape[0]
    n = rows_out(p, budget, L)
    out_k = torch.empty((n,) + tuple(k.shape[1:]), dtype=k.dtype, device=k.device)
    out_v = torch.empty_like(out_k)
    out_idx = torch.empty(n, dtype=torch.int32, device=k.device)
    n_keep = torch.zeros(1, dtype=torch.int32, device=k.device)
    cand = _iarr(candidates)
    _check(lib().sablock_compress(C.addressof(p), _ptr(q_win), _ptr(k), _ptr(v), _ptr(token_ids), L, budget, cand,
                                  len(candidates), _ptr(out_k), _ptr(out_v), _ptr(out_idx), _ptr(n_keep), _ptr(ws),
                                  ws.numel(), _stream()), "sablock_compress")
    return out_k, out_v, out_idx, n_keep


class LayersOut:
    """Pre-allocated outputs of compress_layers: out_k/out_v [layers, seqs, n_out, Hkv, D], out_idx, n_keep."""

    def __init__(self, p: Params, n_layers: int, n_seqs: int, budget: int, dtype, device="cuda", pinned_host=False):
        n_out = budget if p.budget_includes_window else budget + p.window
        kw = dict(device="cpu", pin_memory=True) if pinned_host else dict(device=device)
        self.n_out = n_out
        self.out_k = torch.empty(n_layers, n_seqs, n_out, p.n_kv_heads, p.head_dim, dtype=dtype, **kw)
        self.out_v = torch.empty(n_layers, n_seqs, n_out, p.n_kv_heads, p.head_dim, dtype=dtype, **kw)
        self.out_idx = torch.empty(n_layers, n_seqs, n_out, dtype=torch.int32, **kw)
        self.n_keep = torch.zeros(n_layers, n_seqs, dtype=torch.int32, **kw)


def compress_layers(p: Params, q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, token_ids: torch.Tensor,
                    cu_seqlens: Sequence[int], budget: int, candidates: Sequence[int], ws: torch.Tensor,
                    out: Optional[LayersOut] = None) -> LayersOut:
    n_layers, n_seqs = q_win.shape[0], q_win.shape[1]
    if out is None:
        out = LayersOut(p, n_layers, n_seqs, budget, k.dtype, k.device)
    cu = _iarr(cu_seqlens)
    cand = _iarr(candidates)
    _check(lib().sablock_compress_layers(C.addressof(p), n_layers, n_seqs, _ptr(q_win), _ptr(k), _ptr(v),
                                         _ptr(token_ids), cu, budget, cand, len(candidates), _ptr(out.out_k),
                                         _ptr(out.out_v), _ptr(out.out_idx), _ptr(out.n_keep), _ptr(ws), ws.numel(),
                                         _stream()), "sablock_compress_layers")
    return out


def compress_layers_host(p: Params, h_q, h_k, h_v, h_ids, cu_seqlens, budget, candidates, h_out: LayersOut,
                         d_q, d_k, d_v, d_ids, d_out: LayersOut, ws: torch.Tensor) -> LayersOut:
    """End-to-end variant: host (ideally pinned) inputs and outputs, device staging supplied by the caller."""
    n_layers, n_seqs = h_q.shape[0], h_q.shape[1]
    cu = _iarr(cu_seqlens)
    cand = _iarr(candidates)
    _check(lib().sablock_compress_layers_host(
        C.addressof(p), n_layers, n_seqs, _ptr(h_q), _ptr(h_k), _ptr(h_v), _ptr(h_ids), cu, budget, cand,
        len(candidates), _ptr(h_out.out_k), _ptr(h_out.out_v), _ptr(h_out.out_idx), _ptr(h_out.n_keep),
        _ptr(d_q), _ptr(d_k), _ptr(d_v), _ptr(d_ids), _ptr(d_out.out_k), _ptr(d_out.out_v), _ptr(d_out.out_idx),
        _ptr(d_out.n_keep), _ptr(ws), ws.numel(), _stream()), "sablock_compress_layers_host")
    return h_out


def decode_attention(p: Params, q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                     n_valid: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                     want_lse: bool = False):
    """One decode step's attention over a cache.  q [n_prob, H, D]; k_cache, v_cache
    [n_prob, n_rows, Hkv, D] (contiguous).  Returns out f32 [n_prob, H, D] (and lse [n_prob, H])."""
    n_prob, H, D = q.shape
    n_rows = k_cache.shape[1]
    if ws is None:
        nb = int(lib().sablock_decode_workspace_bytes(C.addressof(p), n_prob, n_rows))
        if nb == 0:
            raise SablockError(2, "sablock_decode_workspace_bytes")
        ws = torch.empty(nb, dtype=torch.uint8, device=q.device)
    out = torch.empty(n_prob, H, D, dtype=torch.float32, device=q.device)
    lse = torch.empty(n_prob, H, dtype=torch.float32, device=q.device) if want_lse else None
    _check(lib().sablock_decode_attention(C.addressof(p), n_prob, _ptr(q), _ptr(k_cache), _ptr(v_cache), n_rows,
                                          _ptr(n_valid), _ptr(out), _ptr(lse), _ptr(ws), ws.numel(), _stream()),
           "sablock_decode_attention")
    return (out, lse) if want_lse else out
