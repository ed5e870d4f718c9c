"""Pins for the oracle's masked attention (Eq. 1 restricted to the kept keys)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs


def small_workload(ns=5, F=3, gh=3, gw=4, nt=6, H=4, Hkv=2, d=16, n_req=1, seed=7, **mask_kw):
    batch = inputs.make_batch([ns] * n_req, [F + r for r in range(n_req)], [nt + 2 * r for r in range(n_req)], gh, gw)
    return inputs.Workload("small", seed, "fp32", H, Hkv, d, 1, (0,), (0,), batch,
                           inputs.STMask(gh, gw, **mask_kw), min(nt, 4), 0.5)


def matrix_attention(q, k, v, mask, scale):
    """Brute force: full score matrix, explicit mask matrix, two-pass softmax (one head)."""
    s = (q.astype(np.float64) @ k.astype(np.float64).T) * scale
    s = np.where(mask, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return (e / z) @ v.astype(np.float64), (m + np.log(z))[:, 0], e / z


@pytest.mark.parametrize("mask_kw", [{}, dict(anchor_frames=2, spatial_radius=1, temporal_depth=2, temporal_radius=1),
                                     dict(dense_causal=True)])
def test_against_matrix_brute_force(mask_kw):
    wl = small_workload(n_req=2, **mask_kw)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    mp = po.mask_params(wl.mask)
    out, lse = po.prefill(x["q"], x["k"], x["v"], b.cu_seqlens, b.n_prefix, b.n_frames, mp)
    G = wl.n_q_heads // wl.n_kv_heads
    cu = b.cu_seqlens
    for r in range(b.n_req):
        lo, hi = cu[r], cu[r + 1]
        mm = po.mask_matrix(mp, hi - lo, b.n_prefix[r], b.n_frames[r])
        for h in range(wl.n_q_heads):
            o, l, p = matrix_attention(x["q"][lo:hi, h], x["k"][lo:hi, h // G], x["v"][lo:hi, h // G], mm,
                                       1.0 / np.sqrt(wl.head_dim))
            assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
            np.testing.assert_allclose(out[lo:hi, h], o, rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(lse[h, lo:hi], l, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("dense", [True, False])
def test_against_torch_sdpa_float64(dense):
    wl = small_workload(ns=4, F=4, gh=4, gw=4, nt=8, H=6, Hkv=2, d=32, dense_causal=dense)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    mp = po.mask_params(wl.mask)
    out, _ = po.prefill(x["q"], x["k"], x["v"], b.cu_seqlens, b.n_prefix, b.n_frames, mp)
    G = wl.n_q_heads // wl.n_kv_heads
    tq = torch.from_numpy(x["q"]).double().permute(1, 0, 2)[None]
    tk = torch.from_numpy(x["k"]).double().permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    tv = torch.from_numpy(x["v"]).double().permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    if dense:
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    else:
        mm = torch.from_numpy(po.mask_matrix(mp, b.seq_lens[0], b.n_prefix[0], b.n_frames[0]))
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mm)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_closed_forms_and_invariants():
    wl = small_workload(ns=3, F=4, gh=3, gw=3, nt=5, H=2, Hkv=1, d=8)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    mp = po.mask_params(wl.mask)
    l = b.seq_lens[0]
    mm = po.mask_matrix(mp, l, b.n_prefix[0], b.n_frames[0])
    args = (b.cu_seqlens, b.n_prefix, b.n_frames, mp)
    out, lse = po.prefill(x["q"], x["k"], x["v"], *args)
    # row 0 keeps one key: returns v_0, LSE = its logit
    np.testing.assert_allclose(out[0, 0], x["v"][0, 0].astype(np.float64), rtol=1e-15)
    s00 = float(np.dot(x["q"][0, 0].astype(np.float64), x["k"][0, 0].astype(np.float64)) / np.sqrt(8))
    assert abs(lse[0, 0] - s00) < 1e-13
    # convex hull: per-coordinate bounds of the kept values
    for i in range(l):
        kept = x["v"][mm[i], 0].astype(np.float64)
        assert (out[i, 0] <= kept.max(axis=0) + 1e-12).all() and (out[i, 0] >= kept.min(axis=0) - 1e-12).all()
    # constant V gives constant output
    vc = np.full_like(x["v"], 1.25)
    oc, _ = po.prefill(x["q"], x["k"], vc, *args)
    np.testing.assert_allclose(oc, 1.25, rtol=1e-14)
    # zero queries: uniform weights over the kept keys, LSE = ln(count)
    oz, lz = po.prefill(np.zeros_like(x["q"]), x["k"], x["v"], *args)
    cnt = mm.sum(axis=1)
    np.testing.assert_allclose(lz[1], np.log(cnt), rtol=1e-13)
    for i in range(l):
        np.testing.assert_allclose(oz[i, 1], x["v"][mm[i], 0].astype(np.float64).mean(axis=0), rtol=1e-12, atol=1e-14)
    # explicit scale
    o2, _ = po.prefill(x["q"] * 2.0, x["k"], x["v"], *args, scale=0.5 / np.sqrt(8))
    np.testing.assert_allclose(o2, out, rtol=1e-12, atol=1e-14)


def test_row_and_head_subsets_agree_with_full():
    wl = small_workload(n_req=3, H=4, Hkv=2)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    mp = po.mask_params(wl.mask)
    args = (b.cu_seqlens, b.n_prefix, b.n_frames, mp)
    full, lse = po.prefill(x["q"], x["k"], x["v"], *args)
    rows = [0, 5, int(b.cu_seqlens[1]), int(b.cu_seqlens[2]) + 7, b.total_tokens - 1]
    heads = [3, 1]
    sub, lsub = po.prefill(x["q"], x["k"], x["v"], *args, rows=rows, heads=heads)
    np.testing.assert_array_equal(sub, full[rows][:, heads])
    np.testing.assert_array_equal(lsub, lse[heads][:, rows])
