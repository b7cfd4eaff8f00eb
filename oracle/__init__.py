"""ctypes front end of the float64 CPU checker (oracle/sablock_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sablock_oracle.c")
_LIB = os.path.join(_HERE, "libsablock_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc (OpenMP on the outer window loop)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.sabo_segment_fill.restype = C.c_double
    return _lib


def _p(a: Optional[np.ndarray], t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _f32(x) -> np.ndarray:
    """Stored values widened exactly to fp32 (torch tensors, bf16 included, or arrays)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _u32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x).view(np.uint32)


def num_threads() -> int:
    return int(lib().sabo_num_threads())


def set_num_threads(n: int) -> None:
    lib().sabo_set_num_threads(int(n))


def segment(token_ids, W: int, bitmap, vocab: int):
    ids = _i32(token_ids)
    L = ids.shape[0]
    T = max(L - W, 0)
    seg_id = np.zeros(T, np.int32)
    seg_start = np.zeros(T + 1, np.int32)
    n = lib().sabo_segment(_p(ids, C.c_int32), L, W, _p(_u32(bitmap), C.c_uint32), vocab,
                           _p(seg_id, C.c_int32), _p(seg_start, C.c_int32))
    return seg_id, seg_start[: n + 1].copy()


def attention(q, k, W: int):
    """A[h, w, t] of Sec. 3.2 (small inputs)."""
    qf, kf = _f32(q), _f32(k)
    H, Wq, D = qf.shape
    L, Hkv, _ = kf.shape
    assert Wq == W
    A = np.zeros((H, W, L - W), np.float64)
    lib().sabo_attention(_p(qf, C.c_float), _p(kf, C.c_float), L, H, Hkv, D, W,
                         C.c_longlong(Hkv * D), C.c_longlong(D), _p(A, C.c_double))
    return A


def scores(q, k, eps: float = 1e-6):
    """Returns (abar[W, T], s[T], e[T]) per Eqs. 3, 4 and the per-token sum of Eq. 6."""
    qf, kf = _f32(q), _f32(k)
    H, W, D = qf.shape
    L, Hkv, _ = kf.shape
    T = L - W
    abar = np.zeros((W, T), np.float64)
    s = np.zeros(T, np.float64)
    e = np.zeros(T, np.float64)
    lib().sabo_scores(_p(qf, C.c_float), _p(kf, C.c_float), L, H, Hkv, D, W,
                      C.c_longlong(Hkv * D), C.c_longlong(D), C.c_double(eps),
                      _p(abar, C.c_double), _p(s, C.c_double), _p(e, C.c_double))
    return abar, s, e


def pool(s, kernel: int, mode: int):
    s = np.ascontiguousarray(s, np.float64)
    out = np.zeros_like(s)
    lib().sabo_pool(_p(s, C.c_double), s.shape[0], kernel, mode, _p(out, C.c_double))
    return out


def refine(s, e, seg_start, alpha: float = 0.9, eta: float = 1.0):
    s = np.ascontiguousarray(s, np.float64)
    e = np.ascontiguousarray(e, np.float64)
    ss = _i32(seg_start)
    n_seg = ss.shape[0] - 1
    I = np.zeros(n_seg); Dk = np.zeros(n_seg); om = np.zeros(n_seg)
    sr = np.zeros_like(s)
    lib().sabo_refine(_p(s, C.c_double), _p(e, C.c_double), _p(ss, C.c_int32), n_seg,
                      C.c_double(alpha), C.c_double(eta), _p(I, C.c_double), _p(Dk, C.c_double),
                      _p(om, C.c_double), _p(sr, C.c_double))
    return I, Dk, om, sr


def segment_fill(sv, b: int, g: int, want_margins: bool = False):
    """Alg. 2 inner loop for one segment and one block size: (taken mask, Score_k(g), blocks),
    plus the four decision margins (inf where no such decision was taken) if asked for."""
    sv = np.ascontiguousarray(sv, np.float64)
    n = sv.shape[0]
    taken = np.zeros(n, np.uint8)
    blocks = np.zeros(2 * (n + 1), np.int32)
    nb = C.c_int(0)
    margins = np.full(4, np.inf)
    sc = lib().sabo_segment_fill(_p(sv, C.c_double), n, b, g, _p(taken, C.c_uint8),
                                 _p(blocks, C.c_int32), C.byref(nb), _p(margins, C.c_double))
    res = (taken.astype(bool), float(sc), blocks[: 2 * nb.value].reshape(-1, 2).copy())
    return res + (margins,) if want_margins else res


def select(s_ref, seg_start, B: int, candidates: Sequence[int], tau: float = 0.85):
    """Algorithm 2.  Returns dict(keep, g_star, b_k, margins, blocks)."""
    sr = np.ascontiguousarray(s_ref, np.float64)
    T = sr.shape[0]
    ss = _i32(seg_start)
    n_seg = ss.shape[0] - 1
    cand = np.ascontiguousarray(sorted(candidates), np.int32)
    keep = np.zeros(max(B, 1), np.int32)
    g_star = np.zeros(n_seg, np.int32)
    b_k = np.zeros(n_seg, np.int32)
    margins = np.full(4, np.inf)
    blocks = np.zeros(2 * max(B, 1), np.int32)
    nblk = C.c_int32(0)
    n = lib().sabo_select(_p(sr, C.c_double), T, _p(ss, C.c_int32), n_seg, B, _p(cand, C.c_int32),
                          cand.shape[0], C.c_double(tau), _p(keep, C.c_int32), _p(g_star, C.c_int32),
                          _p(b_k, C.c_int32), _p(margins, C.c_double), _p(blocks, C.c_int32),
                          C.byref(nblk))
    return dict(keep=keep[:n].copy(), g_star=g_star, b_k=b_k, margins=margins,
                blocks=blocks[: 2 * nblk.value].reshape(-1, 2).copy())


def gather(x, idx):
    """Rows of x[L, ...] at idx, as raw bytes (bit-exact copy)."""
    if hasattr(x, "detach"):
        import torch
        xb = x.detach().cpu().contiguous().view(torch.uint8).numpy() if x.dtype != torch.uint8 \
            else x.detach().cpu().numpy()
        xb = xb.reshape(x.shape[0], -1)
    else:
        xb = np.ascontiguousarray(x).view(np.uint8).reshape(x.shape[0], -1)
    xb = np.ascontiguousarray(xb)
    ii = _i32(idx)
    out = np.zeros((ii.shape[0], xb.shape[1]), np.uint8)
    lib().sabo_gather(_p(xb, C.c_uint8), C.c_longlong(xb.shape[1]), C.c_longlong(xb.shape[1]),
                      _p(ii, C.c_int32), ii.shape[0], _p(out, C.c_uint8))
    return out


def decode_attention(q, k, v):
    """Attention of one new query token over a cache: q [H, D]; k, v [n, Hkv, D] -> (out [H, D], lse [H])."""
    qf, kf, vf = _f32(q), _f32(k), _f32(v)
    H, D = qf.shape
    n, Hkv, _ = kf.shape
    out = np.zeros((H, D), np.float64)
    lse = np.zeros(H, np.float64)
    lib().sabo_decode_attention(_p(qf, C.c_float), _p(kf, C.c_float), _p(vf, C.c_float), n, H, Hkv, D,
                                _p(out, C.c_double), _p(lse, C.c_double))
    return out, lse


def compress(q, k, token_ids, bitmap, vocab: int, budget: int, candidates: Sequence[int],
             alpha: float = 0.9, eta: float = 1.0, eps: float = 1e-6, tau: float = 0.85,
             pool_kernel: int = 1, pool_mode: int = 0, budget_includes_window: int = 1):
    """The whole pass for one (layer, sequence).  Returns a dict of every stage's result."""
    qf, kf = _f32(q), _f32(k)
    H, W, D = qf.shape
    L, Hkv, _ = kf.shape
    T = L - W
    ids = _i32(token_ids)
    cand = np.ascontiguousarray(sorted(candidates), np.int32)
    n_out = budget if budget_includes_window else budget + W
    n_out = L if n_out >= L else n_out
    out_idx = np.zeros(max(n_out, 1), np.int32)
    seg_id = np.zeros(max(T, 1), np.int32)
    seg_start = np.zeros(max(T, 1) + 1, np.int32)
    n_seg = C.c_int32(0)
    s = np.zeros(max(T, 1)); e = np.zeros(max(T, 1)); sr = np.zeros(max(T, 1))
    g_star = np.zeros(max(T, 1), np.int32)
    b_k = np.zeros(max(T, 1), np.int32)
    margins = np.full(4, np.inf)
    n = lib().sabo_compress(_p(qf, C.c_float), _p(kf, C.c_float), _p(ids, C.c_int32), L, H, Hkv, D, W,
                            C.c_longlong(Hkv * D), C.c_longlong(D), _p(_u32(bitmap), C.c_uint32), vocab,
                            C.c_double(alpha), C.c_double(eta), C.c_double(eps), C.c_double(tau),
                            pool_kernel, pool_mode, budget, int(budget_includes_window), _p(cand, C.c_int32),
                            cand.shape[0],
                            _p(out_idx, C.c_int32), _p(seg_id, C.c_int32), _p(seg_start, C.c_int32),
                            C.byref(n_seg), _p(s, C.c_double), _p(e, C.c_double), _p(sr, C.c_double),
                            _p(g_star, C.c_int32), _p(b_k, C.c_int32), _p(margins, C.c_double))
    ns = n_seg.value
    return dict(out_idx=out_idx[:n].copy(), n_keep=n, seg_id=seg_id[:T], seg_start=seg_start[: ns + 1].copy(),
                n_seg=ns, s=s[:T], e=e[:T], s_ref=sr[:T], g_star=g_star[:ns].copy(), b_k=b_k[:ns].copy(),
                margins=margins)
