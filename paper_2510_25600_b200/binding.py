"""ctypes binding of libpurekv.so: argument marshalling only.

Every function here has the name of the C entry point it calls and passes torch
tensors' device pointers straight through; no step of the method runs in Python or
in torch.  torch supplies device memory and the current CUDA stream.  Importing
this module raises if the compiled library is missing: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpurekv.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_25600_b200.build`")
_lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_PLAN = range(7)
BF16, FP32 = 0, 1
FLAG_DENSE_CAUSAL = 1
FLAG_COARSE_BLOCKS = 2

EXPORTS = ("purekv_version", "purekv_last_error", "purekv_budget", "purekv_plan_bytes", "purekv_plan_build",
           "purekv_plan_build_host",
           "purekv_st_sparse_prefill", "purekv_score_ws_bytes", "purekv_lowlayer_score", "purekv_lowlayer_score_lse", "purekv_lowlayer_score_noalloc",
           "purekv_select_ws_bytes",
           "purekv_select_topk", "purekv_compact_kv", "purekv_decode_ws_bytes", "purekv_decode_attention",
           "purekv_poll_status", "purekv_set_wait_limit_ns", "purekv_score_ex_ws_bytes", "purekv_lowlayer_score_ex",
           "purekv_select_sink_recent", "purekv_select_compact")

_i32p = C.POINTER(C.c_int32)


class StParams(C.Structure):
    _fields_ = [("grid_h", C.c_int32), ("grid_w", C.c_int32), ("anchor_frames", C.c_int32),
                ("spatial_radius", C.c_int32), ("temporal_depth", C.c_int32), ("temporal_stride", C.c_int32),
                ("temporal_radius", C.c_int32), ("tile", C.c_int32), ("flags", C.c_uint32),
                ("local_window", C.c_int32), ("atrous_dilation", C.c_int32)]


class CBatch(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("total_tokens", C.c_int64), ("cu_seqlens", C.c_void_p),
                ("h_cu_seqlens", _i32p), ("h_n_prefix", _i32p), ("h_n_frames", _i32p)]


class PlanInfo(C.Structure):
    _fields_ = [("tile_q", C.c_int32), ("tile_k", C.c_int32), ("n_qtiles", C.c_int32), ("max_list", C.c_int32),
                ("tiles_kept", C.c_int64), ("tiles_causal", C.c_int64), ("pairs_kept", C.c_int64),
                ("tiles_full", C.c_int64), ("tiles_diag", C.c_int64), ("tiles_general", C.c_int64),
                ("bytes_used", C.c_int64), ("dtype", C.c_int32), ("head_dim", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("n_ctas", C.c_int32), ("n_units", C.c_int32),
                ("max_chunks", C.c_int32), ("ws_bytes", C.c_int64)]


class PlanHeaderView(C.Structure):
    """The first bytes of a plan buffer, field by field (tooling and tests that inspect or edit a host copy)."""
    _fields_ = [("magic", C.c_uint32), ("tile_q", C.c_int32), ("tile_k", C.c_int32), ("n_qtiles", C.c_int32),
                ("total_tokens", C.c_int64), ("n_entries", C.c_int64), ("n_mask_words", C.c_int64),
                ("off_qtiles", C.c_int64), ("off_order", C.c_int64), ("off_entries", C.c_int64), ("off_masks", C.c_int64),
                ("words_per_row", C.c_int32), ("n_ctas", C.c_int32), ("n_units", C.c_int32), ("n_counters", C.c_int32),
                ("off_units", C.c_int64), ("off_counters", C.c_int64), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("part_slots", C.c_int64), ("test_flags", C.c_uint32), ("pad_flags", C.c_uint32)]


UNIT_INT32S = 16        # a work unit of the tensor-core plan: q_start, q_rows, req_start, ent_begin, ent_count, pair,
                        # chunk, n_chunks, part_base, counter_base, q_start1, q_rows1 (a twin unit's second tile), 4 x padding

_lib.purekv_version.restype = C.c_char_p
_lib.purekv_set_wait_limit_ns.restype = None
_lib.purekv_set_wait_limit_ns.argtypes = [C.c_uint64]
_lib.purekv_plan_bytes.restype = C.c_size_t
_lib.purekv_score_ws_bytes.restype = C.c_size_t
_lib.purekv_select_ws_bytes.restype = C.c_size_t
_lib.purekv_plan_bytes.argtypes = [C.POINTER(CBatch), C.POINTER(StParams), C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_int32]
_lib.purekv_plan_build.argtypes = [C.POINTER(CBatch), C.POINTER(StParams), C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_void_p, C.c_size_t, C.POINTER(PlanInfo), C.c_void_p]
_lib.purekv_plan_build_host.argtypes = [C.POINTER(CBatch), C.POINTER(StParams), C.c_int, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.POINTER(PlanInfo)]
_lib.purekv_st_sparse_prefill.argtypes = [C.c_void_p] * 5 + [C.POINTER(CBatch), C.c_void_p, C.POINTER(PlanInfo),
                                                             C.c_int32, C.c_int32, C.c_int32, C.c_int, C.c_float,
                                                             C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
_lib.purekv_score_ws_bytes.argtypes = [C.POINTER(CBatch), C.c_int32, C.c_int32]
_lib.purekv_lowlayer_score.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(CBatch), C.c_int32, C.c_int32,
                                       C.c_int32, C.c_int32, C.c_int, C.c_float, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.purekv_score_ex_ws_bytes.restype = C.c_size_t
_lib.purekv_score_ex_ws_bytes.argtypes = [C.POINTER(CBatch), C.c_int32, C.c_int32, C.c_int32, C.c_int32]
_lib.purekv_lowlayer_score_ex.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(CBatch), C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int, C.c_float, C.c_void_p,
                                          C.c_size_t, C.c_void_p]
_lib.purekv_select_sink_recent.argtypes = [C.POINTER(CBatch), C.c_int32, C.c_void_p, _i32p, C.c_void_p, _i32p, C.c_int32,
                                           C.c_int32, C.c_void_p, C.c_void_p]
_lib.purekv_lowlayer_score_lse.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(CBatch), C.c_int32,
                                           C.c_int32, C.c_int32, C.c_int32, C.c_int, C.c_float, C.c_void_p, C.c_void_p]
_lib.purekv_lowlayer_score_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(CBatch), C.c_int32,
                                               C.c_int32, C.c_int32, C.c_int32, C.c_int, C.c_float, C.c_void_p]
_lib.purekv_decode_ws_bytes.restype = C.c_size_t
_lib.purekv_decode_ws_bytes.argtypes = [C.c_int32] * 5
_lib.purekv_decode_attention.argtypes = [C.c_void_p] * 7 + [C.c_int32] * 4 + [C.c_int, C.c_float, C.c_void_p, C.c_size_t,
                                                                             C.c_void_p]
_lib.purekv_select_ws_bytes.argtypes = [C.POINTER(CBatch), C.c_int32, C.c_int32]
_lib.purekv_select_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.POINTER(CBatch), C.c_int32,
                                    C.c_void_p, _i32p, C.c_void_p, _i32p, C.c_int32, C.c_int32, C.c_int, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.purekv_select_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.POINTER(CBatch), C.c_int32,
                                       C.c_void_p, _i32p, C.c_void_p, _i32p, C.c_int32, C.c_int32, C.c_int, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.purekv_compact_kv.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.POINTER(CBatch),
                                   C.c_void_p, _i32p, C.c_int32, C.c_int32, C.c_int, C.c_void_p, C.c_void_p,
                                   C.c_int64, C.c_void_p]
_lib.purekv_budget.argtypes = [C.c_int32, C.c_int32, C.c_double, _i32p, _i32p]
_lib.purekv_poll_status.argtypes = [C.c_void_p, _i32p, C.c_void_p]
_lib.purekv_last_error.argtypes = [C.c_char_p, C.c_size_t]


class PureKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        buf = C.create_string_buffer(512)
        _lib.purekv_last_error(buf, 512)
        self.status = status
        super().__init__(f"{where}: status {status}: {buf.value.decode(errors='replace')}")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise PureKVError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def purekv_version() -> str:
    return _lib.purekv_version().decode()


def purekv_budget(length: int, window: int, keep_ratio: float):
    h, k = C.c_int32(), C.c_int32()
    _check(_lib.purekv_budget(length, window, keep_ratio, C.byref(h), C.byref(k)), "purekv_budget")
    return h.value, k.value


class Batch:
    """Host arrays + the device copy of cu_seqlens the kernels read."""

    def __init__(self, seq_lens: Sequence[int], n_prefix: Sequence[int], n_frames: Sequence[int], device="cuda"):
        self.h_cu = _i32(np.concatenate([[0], np.cumsum(seq_lens)]))
        self.h_prefix = _i32(n_prefix)
        self.h_frames = _i32(n_frames)
        self.n_req = len(seq_lens)
        self.total_tokens = int(self.h_cu[-1])
        self.cu_seqlens = torch.from_numpy(self.h_cu.copy()).to(device) if device is not None else None
        self.c = CBatch(self.n_req, self.total_tokens, _ptr(self.cu_seqlens),
                        self.h_cu.ctypes.data_as(_i32p), self.h_prefix.ctypes.data_as(_i32p),
                        self.h_frames.ctypes.data_as(_i32p))

    @property
    def seq_lens(self) -> np.ndarray:
        return np.diff(self.h_cu)


class Budget:
    """Per-request h (top-h count) and the prefix sums of kept rows, on host and device."""

    def __init__(self, batch: Batch, window: int, keep_ratio: float, device="cuda"):
        hk = [purekv_budget(int(l), window, keep_ratio) for l in batch.seq_lens]
        self.window = window
        self.h_keep = _i32([x[0] for x in hk])
        self.h_cu_kept = _i32(np.concatenate([[0], np.cumsum([x[1] for x in hk])]))
        self.total_kept = int(self.h_cu_kept[-1])
        self.keep = torch.from_numpy(self.h_keep.copy()).to(device)
        self.cu_kept = torch.from_numpy(self.h_cu_kept.copy()).to(device)


def st_params(mask, tile: Optional[int] = None) -> StParams:
    """From an object with the STMask attributes."""
    return StParams(mask.grid_h, mask.grid_w, mask.anchor_frames, mask.spatial_radius, mask.temporal_depth,
                    mask.temporal_stride, mask.temporal_radius, tile if tile is not None else mask.tile,
                    (FLAG_DENSE_CAUSAL if mask.dense_causal else 0) | (FLAG_COARSE_BLOCKS if getattr(mask, "coarse", False) else 0),
                    getattr(mask, "local_window", 0), getattr(mask, "atrous_dilation", 0))


class Plan:
    def __init__(self, buf: torch.Tensor, info: PlanInfo):
        self.buf, self.info = buf, info


def purekv_plan_bytes(batch: Batch, params: StParams, dtype: int, head_dim: int, n_q_heads: int, n_kv_heads: int,
                      n_ctas: int = 0) -> int:
    return int(_lib.purekv_plan_bytes(C.byref(batch.c), C.byref(params), dtype, head_dim, n_q_heads, n_kv_heads, n_ctas))


def purekv_plan_build(batch: Batch, params: StParams, dtype: int, head_dim: int, n_q_heads: int, n_kv_heads: int,
                      buf: Optional[torch.Tensor] = None, n_ctas: int = 0) -> Plan:
    if buf is None:                 # size the buffer first (plans the batch once more); callers that plan often pass one
        n = purekv_plan_bytes(batch, params, dtype, head_dim, n_q_heads, n_kv_heads, n_ctas)
        if n == 0:
            _check(_lib.purekv_plan_build(C.byref(batch.c), C.byref(params), dtype, head_dim, n_q_heads, n_kv_heads,
                                          n_ctas, None, 0, C.byref(PlanInfo()), None), "purekv_plan_build")
        buf = torch.empty(n, dtype=torch.uint8, device="cuda")
    info = PlanInfo()
    _check(_lib.purekv_plan_build(C.byref(batch.c), C.byref(params), dtype, head_dim, n_q_heads, n_kv_heads, n_ctas,
                                  buf.data_ptr(), buf.numel(), C.byref(info), _stream()), "purekv_plan_build")
    return Plan(buf, info)


def purekv_plan_build_host(batch: Batch, params: StParams, dtype: int, head_dim: int, n_q_heads: int, n_kv_heads: int,
                           n_ctas: int = 0, out: Optional[torch.Tensor] = None):
    """Plan bytes in host memory + PlanInfo; makes no CUDA call.  Without `out` the bytes come back as a numpy
    uint8 array sized by a first planning pass; with `out` (a host uint8 tensor, e.g. pinned, large enough) they
    are written there in one pass and the used prefix of `out` is returned, ready for an asynchronous copy."""
    info = PlanInfo()
    if out is not None:
        _check(_lib.purekv_plan_build_host(C.byref(batch.c), C.byref(params), dtype, head_dim, n_q_heads, n_kv_heads,
                                           n_ctas, out.data_ptr(), out.numel(), C.byref(info)), "purekv_plan_build_host")
        return out[:info.bytes_used], info
    n = purekv_plan_bytes(batch, params, dtype, head_dim, n_q_heads, n_kv_heads, n_ctas)
    buf = np.zeros(max(n, 1), dtype=np.uint8)
    _check(_lib.purekv_plan_build_host(C.byref(batch.c), C.byref(params), dtype, head_dim, n_q_heads, n_kv_heads,
                                       n_ctas, buf.ctypes.data, n, C.byref(info)), "purekv_plan_build_host")
    return buf[:info.bytes_used], info


def purekv_st_sparse_prefill(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, batch: Batch, plan: Plan,
                             out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                             softmax_scale: float = 0.0, status: Optional[torch.Tensor] = None,
                             ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q [T,H,d], k,v [T,H_kv,d] contiguous on the GPU; returns O [T,H,d].  `ws`: workspace of
    plan.info.ws_bytes bytes (allocated here when not given)."""
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
    t, h, d = q.shape
    if out is None:
        out = torch.empty_like(q)
    if ws is None and plan.info.ws_bytes > 0:
        ws = torch.empty(plan.info.ws_bytes, dtype=torch.uint8, device=q.device)
    _check(_lib.purekv_st_sparse_prefill(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), _ptr(lse),
                                         C.byref(batch.c), plan.buf.data_ptr(), C.byref(plan.info), h, k.shape[1], d,
                                         _dtype_code(q), softmax_scale, _ptr(ws), 0 if ws is None else ws.numel(),
                                         _ptr(status), _stream()),
           "purekv_st_sparse_prefill")
    return out


def purekv_score_ws_bytes(batch: Batch, window: int, n_q_heads: int) -> int:
    return int(_lib.purekv_score_ws_bytes(C.byref(batch.c), window, n_q_heads))


def purekv_lowlayer_score(q: torch.Tensor, k: torch.Tensor, batch: Batch, window: int,
                          c_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                          softmax_scale: float = 0.0) -> torch.Tensor:
    """Returns C [H_kv, T] fp32 (Eq. 1-2)."""
    assert q.is_contiguous() and k.is_contiguous()
    t, h, d = q.shape
    hkv = k.shape[1]
    if c_out is None:
        c_out = torch.empty((hkv, t), dtype=torch.float32, device=q.device)
    if ws is None:
        ws = torch.empty(purekv_score_ws_bytes(batch, window, h), dtype=torch.uint8, device=q.device)
    _check(_lib.purekv_lowlayer_score(q.data_ptr(), k.data_ptr(), c_out.data_ptr(), C.byref(batch.c), window, h, hkv,
                                      d, _dtype_code(q), softmax_scale, ws.data_ptr(), ws.numel(), _stream()),
           "purekv_lowlayer_score")
    return c_out


def purekv_lowlayer_score_lse(q: torch.Tensor, k: torch.Tensor, lse: torch.Tensor, batch: Batch, window: int,
                              c_out: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                              status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """C [H_kv, T] fp32 from the rows' log-sum-exp `lse` [H, T] of the same layer's dense causal prefill."""
    assert q.is_contiguous() and k.is_contiguous() and lse.is_contiguous() and lse.dtype == torch.float32
    t, h, d = q.shape
    hkv = k.shape[1]
    if c_out is None:
        c_out = torch.empty((hkv, t), dtype=torch.float32, device=q.device)
    _check(_lib.purekv_lowlayer_score_lse(q.data_ptr(), k.data_ptr(), lse.data_ptr(), c_out.data_ptr(), C.byref(batch.c),
                                          window, h, hkv, d, _dtype_code(q), softmax_scale, _ptr(status), _stream()),
           "purekv_lowlayer_score_lse")
    return c_out


def purekv_score_ex_ws_bytes(batch: Batch, obs_rows: int, pool: int, n_q_heads: int, n_kv_heads: int) -> int:
    return int(_lib.purekv_score_ex_ws_bytes(C.byref(batch.c), obs_rows, pool, n_q_heads, n_kv_heads))


def purekv_lowlayer_score_ex(q: torch.Tensor, k: torch.Tensor, batch: Batch, window: int, obs_rows: int = -1,
                             pool: int = 1, c_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                             softmax_scale: float = 0.0) -> torch.Tensor:
    """C [H_kv, T] fp32 with the last `obs_rows` rows accumulated (all rows if negative) and averaged over `pool`
    neighbouring keys: the score reductions of the other eviction policies of App. A.1 / Table 6."""
    assert q.is_contiguous() and k.is_contiguous()
    t, h, d = q.shape
    hkv = k.shape[1]
    if c_out is None:
        c_out = torch.empty((hkv, t), dtype=torch.float32, device=q.device)
    if ws is None:
        ws = torch.empty(purekv_score_ex_ws_bytes(batch, obs_rows, pool, h, hkv), dtype=torch.uint8, device=q.device)
    _check(_lib.purekv_lowlayer_score_ex(q.data_ptr(), k.data_ptr(), c_out.data_ptr(), C.byref(batch.c), window, obs_rows,
                                         pool, h, hkv, d, _dtype_code(q), softmax_scale, ws.data_ptr(), ws.numel(),
                                         _stream()), "purekv_lowlayer_score_ex")
    return c_out


def purekv_select_sink_recent(batch: Batch, budget: "Budget", n_layers: int, n_kv_heads: int,
                              idx_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """idx [L, H_kv, K_tot] of the score-free policy: the first h positions of each request, then its window."""
    if idx_out is None:
        idx_out = torch.empty((n_layers, n_kv_heads, budget.total_kept), dtype=torch.int32, device="cuda")
    _check(_lib.purekv_select_sink_recent(C.byref(batch.c), budget.window, budget.keep.data_ptr(),
                                          budget.h_keep.ctypes.data_as(_i32p), budget.cu_kept.data_ptr(),
                                          budget.h_cu_kept.ctypes.data_as(_i32p), n_layers, n_kv_heads,
                                          idx_out.data_ptr(), _stream()), "purekv_select_sink_recent")
    return idx_out


NOALLOC_SCORE_MAX_ROWS = 262144


def purekv_lowlayer_score_noalloc(q: torch.Tensor, k: torch.Tensor, batch: Batch, window: int, c_out: torch.Tensor,
                                  softmax_scale: float = 0.0) -> torch.Tensor:
    """purekv_lowlayer_score for callers that cannot allocate: the scratch is an array inside the library, so
    this wrapper allocates nothing either -- `c_out` [H_kv, T] fp32 must be passed in.  Problems whose
    workspace need exceeds NOALLOC_SCORE_MAX_ROWS values raise PureKVError(ERR_WORKSPACE).  Calls share the scratch:
    keep them on one stream."""
    assert q.is_contiguous() and k.is_contiguous() and c_out.is_contiguous() and c_out.dtype == torch.float32
    t, h, d = q.shape
    _check(_lib.purekv_lowlayer_score_noalloc(q.data_ptr(), k.data_ptr(), c_out.data_ptr(), C.byref(batch.c), window,
                                              h, k.shape[1], d, _dtype_code(q), softmax_scale, _stream()),
           "purekv_lowlayer_score_noalloc")
    return c_out


def purekv_select_ws_bytes(batch: Batch, n_layers: int, n_kv_heads: int) -> int:
    return int(_lib.purekv_select_ws_bytes(C.byref(batch.c), n_layers, n_kv_heads))


def purekv_select_topk(c: torch.Tensor, v: torch.Tensor, batch: Batch, budget: Budget,
                       idx_out: Optional[torch.Tensor] = None, s_out: Optional[torch.Tensor] = None,
                       ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """c [H_kv,T] fp32, v [L,T,H_kv,d]; returns idx [L,H_kv,K_tot] int32 (request-relative positions)."""
    assert v.dim() == 4 and v.stride(3) == 1 and v[0].is_contiguous() and c.is_contiguous()
    n_layers, t, hkv, d = v.shape
    if idx_out is None:
        idx_out = torch.empty((n_layers, hkv, budget.total_kept), dtype=torch.int32, device=v.device)
    if s_out is None and ws is None:
        ws = torch.empty(purekv_select_ws_bytes(batch, n_layers, hkv), dtype=torch.uint8, device=v.device)
    _check(_lib.purekv_select_topk(c.data_ptr(), v.data_ptr(), v.stride(0), n_layers, C.byref(batch.c), budget.window,
                                   budget.keep.data_ptr(), budget.h_keep.ctypes.data_as(_i32p),
                                   budget.cu_kept.data_ptr(), budget.h_cu_kept.ctypes.data_as(_i32p), hkv, d,
                                   _dtype_code(v), idx_out.data_ptr(), _ptr(s_out), _ptr(ws),
                                   0 if ws is None else ws.numel(), _stream()), "purekv_select_topk")
    return idx_out


def purekv_select_compact(c: torch.Tensor, k: torch.Tensor, v: torch.Tensor, batch: Batch, budget: Budget,
                          idx_out: Optional[torch.Tensor] = None, s_out: Optional[torch.Tensor] = None,
                          k_out: Optional[torch.Tensor] = None, v_out: Optional[torch.Tensor] = None,
                          ws: Optional[torch.Tensor] = None):
    """Selection and compaction in one call.  c [H_kv,T]; k, v [L,T,H_kv,d]; returns (idx, k_c, v_c)."""
    assert k.dim() == 4 and k[0].is_contiguous() and v[0].is_contiguous() and k.stride(0) == v.stride(0) and c.is_contiguous()
    n_layers, t, hkv, d = v.shape
    if idx_out is None:
        idx_out = torch.empty((n_layers, hkv, budget.total_kept), dtype=torch.int32, device=v.device)
    if k_out is None:
        k_out = torch.empty((n_layers, budget.total_kept, hkv, d), dtype=k.dtype, device=k.device)
    if v_out is None:
        v_out = torch.empty_like(k_out)
    if s_out is None and ws is None:
        ws = torch.empty(purekv_select_ws_bytes(batch, n_layers, hkv), dtype=torch.uint8, device=v.device)
    _check(_lib.purekv_select_compact(c.data_ptr(), k.data_ptr(), v.data_ptr(), v.stride(0), n_layers, C.byref(batch.c),
                                      budget.window, budget.keep.data_ptr(), budget.h_keep.ctypes.data_as(_i32p),
                                      budget.cu_kept.data_ptr(), budget.h_cu_kept.ctypes.data_as(_i32p), hkv, d,
                                      _dtype_code(v), idx_out.data_ptr(), _ptr(s_out), k_out.data_ptr(), v_out.data_ptr(),
                                      k_out.stride(0), _ptr(ws), 0 if ws is None else ws.numel(), _stream()),
           "purekv_select_compact")
    return idx_out, k_out, v_out


def purekv_compact_kv(k: torch.Tensor, v: torch.Tensor, idx: torch.Tensor, batch: Batch, budget: Budget,
                      k_out: Optional[torch.Tensor] = None, v_out: Optional[torch.Tensor] = None):
    """k, v [L,T,H_kv,d]; idx [L,H_kv,K_tot]; returns (k_c, v_c) [L,K_tot,H_kv,d]."""
    assert k.dim() == 4 and k[0].is_contiguous() and v[0].is_contiguous() and k.stride(0) == v.stride(0)
    n_layers, t, hkv, d = k.shape
    if k_out is None:
        k_out = torch.empty((n_layers, budget.total_kept, hkv, d), dtype=k.dtype, device=k.device)
    if v_out is None:
        v_out = torch.empty_like(k_out)
    _check(_lib.purekv_compact_kv(k.data_ptr(), v.data_ptr(), k.stride(0), n_layers, idx.data_ptr(), C.byref(batch.c),
                                  budget.cu_kept.data_ptr(), budget.h_cu_kept.ctypes.data_as(_i32p), hkv, d,
                                  _dtype_code(k), k_out.data_ptr(), v_out.data_ptr(), k_out.stride(0), _stream()),
           "purekv_compact_kv")
    return k_out, v_out


def purekv_decode_ws_bytes(n_req: int, max_kept: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> int:
    return int(_lib.purekv_decode_ws_bytes(n_req, max_kept, n_q_heads, n_kv_heads, head_dim))


def purekv_decode_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, budget: Budget,
                            out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                            softmax_scale: float = 0.0, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q [B,H,d]; k_cache, v_cache [K_tot,H_kv,d] (one layer of the compact cache); returns o [B,H,d]."""
    assert q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous()
    b, h, d = q.shape
    hkv = k_cache.shape[1]
    if out is None:
        out = torch.empty_like(q)
    kept = np.diff(budget.h_cu_kept)
    need = purekv_decode_ws_bytes(b, int(kept.max()) if len(kept) else 0, h, hkv, d)
    if need and (ws is None or ws.numel() * ws.element_size() < need):
        ws = torch.empty(need, dtype=torch.uint8, device=q.device)
    _check(_lib.purekv_decode_attention(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr(), _ptr(lse),
                                        budget.cu_kept.data_ptr(), budget.h_cu_kept.ctypes.data_as(_i32p), b, h, hkv, d,
                                        _dtype_code(q), softmax_scale, _ptr(ws),
                                        ws.numel() * ws.element_size() if ws is not None else 0, _stream()),
           "purekv_decode_attention")
    return out


def purekv_set_wait_limit_ns(ns: int) -> None:
    """Limit of every device-side wait of the tensor-core kernels, process-wide; 0 restores the default (1 s)."""
    _lib.purekv_set_wait_limit_ns(int(ns))


def purekv_poll_status(status: Optional[torch.Tensor]) -> int:
    out = C.c_int32()
    _check(_lib.purekv_poll_status(_ptr(status), C.byref(out), _stream()), "purekv_poll_status")
    return out.value
