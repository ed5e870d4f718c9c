"""GPU parity at the full sizes of workloads 1-4, through the same calls and launch configuration the benchmark times
(plans scheduled for one CTA per SM, whole batch per call).  The oracle is too slow for every output at these
sizes, so: attention is checked on a seeded sample of rows (all heads of the sample; rows are independent, so
each sampled row is checked exactly), scores on whole KV groups, selection and compaction on a few layers in full."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc

pytestmark = pytest.mark.gpu
POOL = ThreadPoolExecutor(len(os.sched_getaffinity(0)))


def sample_rows(wl, n_random, rng):
    """Rows that stress the mask: first and last rows of every request, rows next to frame and tile borders, the
    first visual and first suffix rows, plus a random draw."""
    b = wl.batch
    cu = b.cu_seqlens
    n = b.grid_h * b.grid_w
    rows = set()
    for r in range(b.n_req):
        l, base = b.seq_lens[r], int(cu[r])
        vis0, vis1 = b.n_prefix[r], b.n_prefix[r] + b.n_frames[r] * n
        marks = [0, l - 1, vis0, vis1 - 1, vis1, vis0 + n - 1, vis0 + n, vis0 + 2 * n, 127, 128, l - 129, l - 128]
        rows.update(base + m for m in marks if 0 <= m < l)
    rows.update(int(x) for x in rng.choice(b.total_tokens, size=n_random, replace=False))
    return np.array(sorted(rows), dtype=np.int64)


def check_prefill_sampled(wl, x, mask, rows):
    P = gc.pk()
    out, lse, plan = gc.gpu_prefill(wl, x, mask=mask)
    b = wl.batch
    ref, ref_lse = po.prefill(x["q"], x["k"], x["v"], b.cu_seqlens, b.n_prefix, b.n_frames, po.mask_params(mask), rows=rows)
    got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    got_lse = lse[:, torch.from_numpy(rows).cuda()].cpu().numpy()
    assert torch.isfinite(out.float()).all().item(), "unwritten or non-finite outputs"
    err = float(np.abs(got - ref).max())
    lerr = float(np.abs(got_lse - ref_lse).max())
    assert err <= gc.ATTN_TOL["bf16"], f"attention max abs err {err}"
    assert lerr <= 2e-3, f"lse max abs err {lerr}"
    return plan


def check_scores_selection_compaction(wl, x0, layers_x, groups=None):
    """x0: the scored layer's tensors; layers_x: a few compacted layers' tensors.  groups: KV groups whose scores the
    oracle computes (None = all)."""
    P = gc.pk()
    b = wl.batch
    cu = b.cu_seqlens
    db = gc.device_batch(wl)
    bud = P.Budget(db, wl.window, wl.keep_ratio)
    G = wl.n_q_heads // wl.n_kv_heads
    q0, k0 = gc.upload(x0, "q", "bf16"), gc.upload(x0, "k", "bf16")
    c = P.purekv_lowlayer_score(q0, k0, db, wl.window)
    if wl.window % 8 == 0 and all(l >= wl.window or l % 8 == 0 for l in b.seq_lens):
        # the one-pass tensor-core scores from the dense prefill's log-sum-exp must give the same selection input
        dense = inputs.STMask(b.grid_h, b.grid_w, tile=wl.mask.tile, dense_causal=True)
        plan = P.purekv_plan_build(db, P.st_params(dense), P.BF16, wl.head_dim, wl.n_q_heads, wl.n_kv_heads)
        lse = torch.empty((wl.n_q_heads, db.total_tokens), dtype=torch.float32, device="cuda")
        P.purekv_st_sparse_prefill(q0, k0, gc.upload(x0, "v", "bf16"), db, plan, lse=lse)
        c_two_pass = c
        c = P.purekv_lowlayer_score_lse(q0, k0, lse, db, wl.window)
        assert gc.score_error(c.cpu().numpy(), c_two_pass.cpu().numpy().astype(np.float64)) <= gc.SCORE_RTOL
    vs = torch.stack([gc.upload(x, "v", "bf16") for x in layers_x])
    ks = torch.stack([gc.upload(x, "k", "bf16") for x in layers_x])
    s = torch.empty((len(layers_x), wl.n_kv_heads, db.total_tokens), dtype=torch.float32, device="cuda")
    idx = P.purekv_select_topk(c, vs, db, bud, s_out=s)
    kc, vc = P.purekv_compact_kv(ks, vs, idx, db, bud)
    idx_f, kc_f, vc_f = P.purekv_select_compact(c, ks, vs, db, bud)      # one call: the same indices and bytes
    torch.cuda.synchronize()
    assert torch.equal(idx_f, idx) and torch.equal(kc_f.view(torch.int16), kc.view(torch.int16))
    assert torch.equal(vc_f.view(torch.int16), vc.view(torch.int16))
    c_gpu = c.cpu().numpy()
    hk, ck = po.budgets(b.seq_lens, wl.window, wl.keep_ratio)
    assert np.array_equal(hk, bud.h_keep) and np.array_equal(ck, bud.h_cu_kept)
    groups = list(range(wl.n_kv_heads)) if groups is None else groups
    for g in groups:                                       # oracle scores of whole KV groups
        c_ref = po.lowlayer_score(x0["q"][:, g * G:(g + 1) * G], x0["k"][:, g:g + 1], cu, wl.window)
        assert gc.score_error(c_gpu[g:g + 1], c_ref) <= gc.SCORE_RTOL
        for l, xl in enumerate(layers_x):
            s_ref = po.vnorm_scores(c_ref, xl["v"][:, g:g + 1])
            s_gpu = s[l, g:g + 1].cpu().numpy()
            assert gc.score_error(s_gpu, s_ref) <= gc.SCORE_RTOL
            idx_ref, kth = po.select(s_ref, cu, wl.window, hk, ck)
            gc.check_index_sets(idx[l, g:g + 1].cpu().numpy(), idx_ref, s_ref, kth, wl, hk, ck, wl.window)
    for l, xl in enumerate(layers_x):                      # selection and compaction of every group, exactly
        s_gpu = s[l].cpu().numpy().astype(np.float64)
        idx_gpu = idx[l].cpu().numpy()
        idx_self, _ = po.select(s_gpu, cu, wl.window, hk, ck)
        assert np.array_equal(idx_gpu, idx_self)
        view = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(view(kc[l]), po.compact(xl["k_bits"], idx_gpu, cu, ck))
        assert np.array_equal(view(vc[l]), po.compact(xl["v_bits"], idx_gpu, cu, ck))


@pytest.mark.parametrize("cfg", [1, 2, 4])
def test_workload_full_size(cfg):
    wl = inputs.workload(cfg)
    rng = np.random.default_rng(wl.seed)
    x0 = inputs.make_qkv(wl, 0, pool=POOL)
    first = wl.compacted_layers[0]
    layers_x = [inputs.make_qkv(wl, l, pool=POOL) for l in (first, wl.compacted_layers[-1])]
    dense = inputs.STMask(wl.mask.grid_h, wl.mask.grid_w, tile=wl.mask.tile, dense_causal=True)
    rows = sample_rows(wl, 48, rng)
    check_prefill_sampled(wl, x0, dense, rows)                                  # the scored (dense causal) layer
    st = layers_x[-1] if "q" in layers_x[-1] else x0
    plan = check_prefill_sampled(wl, st, wl.mask, rows)                         # an ST-SpAttn layer
    expect = {1: (184, 380, 783264), 2: (434, 2145, 4148800)}
    if cfg in expect:
        assert (plan.info.tiles_kept, plan.info.tiles_causal, plan.info.pairs_kept) == expect[cfg]
    check_scores_selection_compaction(wl, x0, layers_x, groups=None if cfg == 1 else [0, wl.n_kv_heads - 1])


def test_workload_long_video_sweep():
    wl = inputs.workload(3)
    rng = np.random.default_rng(wl.seed)
    x0 = inputs.make_qkv(wl, 0, pool=POOL)
    rows = sample_rows(wl, 40, rng)
    g = wl.mask.grid_h
    masks = [wl.mask,                                                           # the paper's mask
             inputs.STMask(g, g, 1, -1, 4, 1, -1, tile=128),                    # whole-frame links, 4 frames back
             inputs.STMask(g, g, 1, 4, -1, 5, 0, tile=128)]                     # narrow spatial window, every 5th frame
    for n, m in enumerate(masks):
        plan = check_prefill_sampled(wl, x0, m, rows)
        assert 0 < plan.info.tiles_kept < plan.info.tiles_causal
        if n == 0:
            assert plan.info.pairs_kept == 41042944                             # closed form of the paper's mask
    for keep in (0.1, 0.5):
        check_scores_selection_compaction(inputs.workload(3, keep_ratio=keep), x0, [x0], groups=[1])


def test_workload_named_mask_variants_at_full_size():
    """App. A.3 / Table 7: each named variant on the VideoLLaMA2-shaped prompt (sampled rows against the oracle)."""
    wl = inputs.workload(1)
    rng = np.random.default_rng(wl.seed + 1)
    x0 = inputs.make_qkv(wl, 0, pool=POOL)
    rows = sample_rows(wl, 32, rng)
    g = wl.mask.grid_h
    for name, kw in (("spatial", {}), ("temporal", {}), ("local", dict(local_window=256)), ("atrous", dict(atrous_dilation=4))):
        plan = check_prefill_sampled(wl, x0, inputs.mask_variant(name, g, g, tile=64, **kw), rows)
        assert 0 < plan.info.tiles_kept <= plan.info.tiles_causal
