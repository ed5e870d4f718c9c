"""ctypes wrapper of the fp64 CPU oracle (purekv_oracle.cpp).

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product package.  `build()` compiles
the C++ file with g++ (OpenMP) next to this file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "purekv_oracle.cpp")
_LIB = os.path.join(_HERE, "libpurekv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


class MaskParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("grid_h", "grid_w", "anchor_frames", "spatial_radius",
                                         "temporal_depth", "temporal_stride", "temporal_radius",
                                         "dense_causal", "local_window", "atrous_dilation", "coarse_block")]


def mask_params(m) -> MaskParams:
    """From an inputs.STMask-like object (attribute access only)."""
    return MaskParams(m.grid_h, m.grid_w, m.anchor_frames, m.spatial_radius, m.temporal_depth,
                      m.temporal_stride, m.temporal_radius, 1 if m.dense_causal else 0,
                      getattr(m, "local_window", 0), getattr(m, "atrous_dilation", 0),
                      m.tile if getattr(m, "coarse", False) else 0)


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.pko_mask.restype = C.c_int32
        _lib.pko_select.restype = C.c_int32
        _lib.pko_select_sink_recent.restype = C.c_int32
        _lib.pko_spearman.restype = C.c_double
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def mask(mp: MaskParams, length: int, n_prefix: int, n_frames: int, i: int, j: int) -> bool:
    return bool(lib().pko_mask(C.byref(mp), int(length), int(n_prefix), int(n_frames), int(i), int(j)))


def mask_matrix(mp: MaskParams, length: int, n_prefix: int, n_frames: int) -> np.ndarray:
    length = int(length)
    out = np.zeros((length, length), dtype=np.uint8)
    lib().pko_mask_matrix(C.byref(mp), int(length), int(n_prefix), int(n_frames), _p(out, C.c_uint8))
    return out.astype(bool)


def prefill(q, k, v, cu_seqlens, n_prefix, n_frames, mp: MaskParams, scale: float = 0.0,
            rows: Optional[Sequence[int]] = None, heads: Optional[Sequence[int]] = None):
    """q [T,H,d], k,v [T,H_kv,d] float32.  Returns (out [n_rows,n_heads,d] f64, lse [n_heads,n_rows] f64)."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    t_tot, h, d = q.shape
    hkv = k.shape[1]
    cu, npre, nfr = _i32(cu_seqlens), _i32(n_prefix), _i32(n_frames)
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    heads_a = None if heads is None else _i32(heads)
    n_rows = t_tot if rows_a is None else len(rows_a)
    n_heads = h if heads_a is None else len(heads_a)
    out = np.zeros((n_rows, n_heads, d), dtype=np.float64)
    lse = np.zeros((n_heads, n_rows), dtype=np.float64)
    lib().pko_prefill(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float), C.c_int32(len(cu) - 1),
                      _p(cu, C.c_int32), _p(npre, C.c_int32), _p(nfr, C.c_int32), C.byref(mp),
                      C.c_int32(h), C.c_int32(hkv), C.c_int32(d), C.c_double(scale),
                      _p(rows_a, C.c_int64), C.c_int64(n_rows), _p(heads_a, C.c_int32), C.c_int32(n_heads),
                      _p(out, C.c_double), _p(lse, C.c_double))
    return out, lse


def lowlayer_score(q, k, cu_seqlens, window: int, scale: float = 0.0) -> np.ndarray:
    """Returns C [H_kv, T] float64 (Eq. 1-2)."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    t_tot, h, d = q.shape
    hkv = k.shape[1]
    cu = _i32(cu_seqlens)
    c = np.zeros((hkv, t_tot), dtype=np.float64)
    lib().pko_lowlayer_score(_p(q, C.c_float), _p(k, C.c_float), C.c_int32(len(cu) - 1), _p(cu, C.c_int32),
                             C.c_int32(window), C.c_int32(h), C.c_int32(hkv), C.c_int32(d),
                             C.c_double(scale), _p(c, C.c_double))
    return c


def lowlayer_score_ex(q, k, cu_seqlens, window: int, obs_rows: int = -1, pool: int = 1, scale: float = 0.0) -> np.ndarray:
    """C [H_kv, T] float64 under another reduction (App. A.1 / Table 6): the last obs_rows rows of each request are
    accumulated (all rows if negative), then averaged over `pool` neighbouring keys."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    t_tot, h, d = q.shape
    hkv = k.shape[1]
    cu = _i32(cu_seqlens)
    c = np.zeros((hkv, t_tot), dtype=np.float64)
    lib().pko_lowlayer_score_ex(_p(q, C.c_float), _p(k, C.c_float), C.c_int32(len(cu) - 1), _p(cu, C.c_int32),
                                C.c_int32(window), C.c_int32(obs_rows), C.c_int32(pool), C.c_int32(h), C.c_int32(hkv),
                                C.c_int32(d), C.c_double(scale), _p(c, C.c_double))
    return c


def select_sink_recent(cu_seqlens, window: int, h_keep, cu_kept, n_kv_heads: int) -> np.ndarray:
    """idx [H_kv, K_tot] of the score-free policy: the first h positions of each request, then its window."""
    cu, hk, ck = _i32(cu_seqlens), _i32(h_keep), _i32(cu_kept)
    idx = np.zeros((n_kv_heads, int(ck[-1])), dtype=np.int32)
    if lib().pko_select_sink_recent(C.c_int32(len(cu) - 1), _p(cu, C.c_int32), C.c_int32(window), _p(hk, C.c_int32),
                                    _p(ck, C.c_int32), C.c_int32(n_kv_heads), _p(idx, C.c_int32)) != 0:
        raise ValueError("select_sink_recent: a request's h is outside [0, l - w] or its kept count is not h + w")
    return idx


def spearman(a, b) -> float:
    """Eq. 7 on two equally long score vectors."""
    a = np.ascontiguousarray(a, dtype=np.float64).ravel()
    b = np.ascontiguousarray(b, dtype=np.float64).ravel()
    assert a.shape == b.shape
    return float(lib().pko_spearman(_p(a, C.c_double), _p(b, C.c_double), C.c_int64(a.size)))


def clie_rank_agreement(q_low, k_low, q_high, k_high, v_high, cu_seqlens, window: int) -> np.ndarray:
    """The validation study of Sec. 3.3 for one (low layer, high layer) pair: Spearman's rho between the estimate
    S_hat = C_low * ||V_high|| (Eq. 4) and S_high = C_high * ||V_high|| (Eq. 6) over each request's non-recent keys.
    Returns rho [H_kv, n_req].  CPU only; on synthetic inputs it checks the plumbing, not the paper's hypothesis."""
    cu = _i32(cu_seqlens)
    s_hat = vnorm_scores(lowlayer_score(q_low, k_low, cu, window), v_high)
    s_high = vnorm_scores(lowlayer_score(q_high, k_high, cu, window), v_high)
    out = np.full((s_hat.shape[0], len(cu) - 1), np.nan)
    for r in range(len(cu) - 1):
        nr = int(cu[r + 1] - cu[r]) - min(window, int(cu[r + 1] - cu[r]))
        for g in range(s_hat.shape[0]):
            if nr >= 2:
                out[g, r] = spearman(s_hat[g, cu[r]:cu[r] + nr], s_high[g, cu[r]:cu[r] + nr])
    return out


def vnorm_scores(c: np.ndarray, v: np.ndarray) -> np.ndarray:
    """S = C * ||V|| (Eq. 3/4) for one layer.  c [H_kv,T] f64, v [T,H_kv,d] f32 -> [H_kv,T] f64."""
    c = np.ascontiguousarray(c, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float32)
    t_tot, hkv, d = v.shape
    s = np.zeros((hkv, t_tot), dtype=np.float64)
    lib().pko_vnorm_scores(_p(c, C.c_double), _p(v, C.c_float), C.c_int64(t_tot), C.c_int32(hkv), C.c_int32(d),
                           _p(s, C.c_double))
    return s


def select(s: np.ndarray, cu_seqlens, window: int, h_keep, cu_kept):
    """Top-h + window for one layer.  Returns (idx [H_kv,K_tot] int32, kth [H_kv,n_req] f64)."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    cu, hk, ck = _i32(cu_seqlens), _i32(h_keep), _i32(cu_kept)
    hkv = s.shape[0]
    n_req = len(cu) - 1
    idx = np.zeros((hkv, int(ck[-1])), dtype=np.int32)
    kth = np.zeros((hkv, n_req), dtype=np.float64)
    rc = lib().pko_select(_p(s, C.c_double), C.c_int32(n_req), _p(cu, C.c_int32), C.c_int32(window),
                          _p(hk, C.c_int32), _p(ck, C.c_int32), C.c_int32(hkv), _p(idx, C.c_int32), _p(kth, C.c_double))
    if rc != 0:
        raise ValueError("select: a request's h is outside [0, l - w] or its kept count is not h + w")
    return idx, kth


def compact(src: np.ndarray, idx: np.ndarray, cu_seqlens, cu_kept) -> np.ndarray:
    """src [T,H_kv,d] any dtype -> [K_tot,H_kv,d], byte copy."""
    src = np.ascontiguousarray(src)
    idx = _i32(idx)
    cu, ck = _i32(cu_seqlens), _i32(cu_kept)
    t_tot, hkv, d = src.shape
    out = np.zeros((int(ck[-1]), hkv, d), dtype=src.dtype)
    lib().pko_compact(src.ctypes.data_as(C.POINTER(C.c_uint8)), _p(idx, C.c_int32), C.c_int32(len(cu) - 1),
                      _p(cu, C.c_int32), _p(ck, C.c_int32), C.c_int32(hkv), C.c_int64(d * src.itemsize),
                      out.ctypes.data_as(C.POINTER(C.c_uint8)))
    return out


def decode(q, kc, vc, cu_kept, scale: float = 0.0):
    """q [B,H,d], kc, vc [K_tot,H_kv,d] float32, cu_kept [B+1].  Returns (out [B,H,d] f64, lse [B,H] f64)."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    kc = np.ascontiguousarray(kc, dtype=np.float32)
    vc = np.ascontiguousarray(vc, dtype=np.float32)
    ck = _i32(cu_kept)
    b, h, d = q.shape
    hkv = kc.shape[1]
    assert len(ck) == b + 1 and kc.shape == vc.shape and kc.shape[0] >= int(ck[-1]) and kc.shape[2] == d
    out = np.zeros((b, h, d), dtype=np.float64)
    lse = np.zeros((b, h), dtype=np.float64)
    lib().pko_decode(_p(q, C.c_float), _p(kc, C.c_float), _p(vc, C.c_float), C.c_int32(b), _p(ck, C.c_int32),
                     C.c_int32(h), C.c_int32(hkv), C.c_int32(d), C.c_double(scale), _p(out, C.c_double),
                     _p(lse, C.c_double))
    return out, lse


def budget(length: int, window: int, keep_ratio: float):
    h, k = C.c_int32(), C.c_int32()
    lib().pko_budget(C.c_int32(length), C.c_int32(window), C.c_double(keep_ratio), C.byref(h), C.byref(k))
    return h.value, k.value


def budgets(seq_lens, window: int, keep_ratio: float):
    """Per-request (h_keep [n_req], cu_kept [n_req+1]) int32 arrays."""
    hk = [budget(int(l), window, keep_ratio) for l in seq_lens]
    h = np.array([x[0] for x in hk], dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum([x[1] for x in hk])]).astype(np.int32)
    return h, cu
