"""Helpers shared by the GPU parity tests: upload seeded inputs, run the CUDA path through
the C-ABI binding, compute the oracle on the same bits, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs

ATTN_TOL = {"bf16": 2e-2, "fp32": 1e-4}      # max abs error of the attention output
SCORE_RTOL = 1e-3                            # relative error of C and S ...
SCORE_FLOOR = 1e-6                           # ... measured against max(|o|, floor * max|o|)
INDEX_RTOL = 1e-5                            # an index may differ only if its oracle score is this close to the h-th


def pk():
    from paper_2510_25600_b200 import binding
    return binding


def upload(x: dict, name: str, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return torch.from_numpy(x[name + "_bits"].view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(x[name]).cuda()


def to_numpy_f32(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()


def device_batch(wl: inputs.Workload):
    b = wl.batch
    return pk().Batch(b.seq_lens, b.n_prefix, b.n_frames)


def gpu_prefill(wl: inputs.Workload, x: dict, want_lse: bool = True, mask=None, n_ctas: int = 0):
    P = pk()
    db = device_batch(wl)
    q, k, v = (upload(x, n, wl.dtype) for n in "qkv")
    code = P.BF16 if wl.dtype == "bf16" else P.FP32
    plan = P.purekv_plan_build(db, P.st_params(mask or wl.mask), code, wl.head_dim, wl.n_q_heads, wl.n_kv_heads,
                               n_ctas=n_ctas)
    lse = torch.full((wl.n_q_heads, db.total_tokens), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full_like(q, float("nan"))
    P.purekv_st_sparse_prefill(q, k, v, db, plan, out=out, lse=lse, status=status)
    assert P.purekv_poll_status(status) == 0
    return out, lse, plan


def check_prefill(wl: inputs.Workload, x: dict, rows=None, heads=None, mask=None, n_ctas: int = 0):
    out, lse, plan = gpu_prefill(wl, x, mask=mask, n_ctas=n_ctas)
    b = wl.batch
    ref, ref_lse = po.prefill(x["q"], x["k"], x["v"], b.cu_seqlens, b.n_prefix, b.n_frames,
                              po.mask_params(mask or wl.mask), rows=rows, heads=heads)
    got = to_numpy_f32(out)
    got_lse = lse.cpu().numpy()
    if rows is not None:
        got, got_lse = got[rows], got_lse[:, rows]
    if heads is not None:
        got, got_lse = got[:, heads], got_lse[heads]
    assert np.isfinite(got).all(), "prefill left unwritten or non-finite outputs"
    err = float(np.abs(got - ref).max())
    lerr = float(np.abs(got_lse - ref_lse).max())
    assert err <= ATTN_TOL[wl.dtype], f"attention max abs err {err}"
    assert lerr <= (1e-4 if wl.dtype == "fp32" else 2e-3), f"lse max abs err {lerr}"
    return err, plan


def score_error(got: np.ndarray, ref: np.ndarray) -> float:
    if not np.abs(ref).max() > 0:          # window covers every key: all scores are defined as 0
        return float(np.abs(got).max())
    denom = np.maximum(np.abs(ref), SCORE_FLOOR * np.abs(ref).max())
    return float((np.abs(got - ref) / denom).max())


def check_index_sets(idx_gpu: np.ndarray, idx_ref: np.ndarray, s_ref: np.ndarray, kth: np.ndarray, wl, hk, ck, window):
    """idx_* [H_kv, K_tot]; s_ref [H_kv, T] oracle scores; kth [H_kv, n_req].  Sets must be equal except
    for keys whose oracle score is within INDEX_RTOL (relative) of the h-th value."""
    cu = wl.batch.cu_seqlens
    n_mismatch = 0
    for g in range(idx_ref.shape[0]):
        for r in range(wl.batch.n_req):
            h = int(hk[r])
            a = idx_gpu[g, ck[r]:ck[r + 1]]
            b = idx_ref[g, ck[r]:ck[r + 1]]
            l = wl.batch.seq_lens[r]
            w = min(window, l)
            assert np.array_equal(a[h:], np.arange(l - w, l)), "window positions"
            assert (np.diff(a[:h]) > 0).all(), "selected positions must ascend"
            assert h == 0 or (a[0] >= 0 and a[h - 1] < l - w)
            diff = np.setxor1d(a[:h], b[:h])
            n_mismatch += len(diff)
            for j in diff:
                sc = s_ref[g, cu[r] + j]
                assert abs(sc - kth[g, r]) <= INDEX_RTOL * abs(kth[g, r]), \
                    f"key {j} (score {sc}) differs but is not within {INDEX_RTOL} of the h-th score {kth[g, r]}"
    return n_mismatch
