"""GPU parity: the CUDA path (through the C-ABI binding) against the fp64 oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc

pytestmark = pytest.mark.gpu


def make_wl(dtype, H, Hkv, d, n_prefix, n_frames, n_suffix, gh, gw, tile, window=8, keep=0.3, seed=11, **mask_kw):
    batch = inputs.make_batch(n_prefix, n_frames, n_suffix, gh, gw)
    return inputs.Workload("t", seed, dtype, H, Hkv, d, 1, (0,), (0,), batch, inputs.STMask(gh, gw, tile=tile, **mask_kw),
                           window, keep)


# ---------------------------------------------------------------- prefill ---------------
@pytest.mark.parametrize("mask_kw", [{}, dict(dense_causal=True),
                                     dict(anchor_frames=2, spatial_radius=1, temporal_depth=2, temporal_stride=2, temporal_radius=1)])
@pytest.mark.parametrize("dtype,d,tile", [("fp32", 64, 16), ("fp32", 32, 32), ("bf16", 64, 64), ("fp32", 128, 64)])
def test_prefill_cuda_core_kernel(dtype, d, tile, mask_kw):
    wl = make_wl(dtype, 4, 2, d, [5, 0, 9], [4, 3, 0], [7, 33, 3], 5, 6, tile, **mask_kw)
    gc.check_prefill(wl, inputs.make_qkv(wl, 0))


@pytest.mark.parametrize("mask_kw", [{}, dict(dense_causal=True),
                                     dict(anchor_frames=0, spatial_radius=2, temporal_depth=-1, temporal_stride=2, temporal_radius=-1),
                                     dict(anchor_frames=2, spatial_radius=-1, temporal_depth=3, temporal_radius=1)])
@pytest.mark.parametrize("tile", [64, 128])
def test_prefill_tensor_core_kernel(tile, mask_kw):
    # several requests, lengths that are not multiples of the tile, frames that straddle tiles
    wl = make_wl("bf16", 4, 2, 128, [37, 0, 5, 1], [5, 3, 1, 0], [29, 140, 0, 2], 9, 11, tile, **mask_kw)
    gc.check_prefill(wl, inputs.make_qkv(wl, 0))


VARIANTS = [("spatial", {}), ("temporal", {}), ("local", dict(local_window=40)), ("atrous", dict(atrous_dilation=3))]


@pytest.mark.parametrize("coarse", [False, True])
@pytest.mark.parametrize("name,kw", VARIANTS + [("st", {})])
def test_prefill_named_mask_variants(name, kw, coarse):
    """The sparse-attention variants of App. A.3 / Table 7 and their block-level widening, on both kernels."""
    if name == "st" and not coarse:
        pytest.skip("the paper's token-exact mask is covered by the tests above")
    for dtype, d, tile in (("bf16", 128, 64), ("bf16", 128, 128), ("fp32", 64, 16)):
        batch = inputs.make_batch([37, 0, 5], [5, 3, 1], [29, 140, 0], 9, 11)
        wl = inputs.Workload("t", 19, dtype, 4, 2, d, 1, (0,), (0,), batch,
                             inputs.mask_variant(name, 9, 11, tile=tile, coarse=coarse, **kw), 8, 0.3)
        gc.check_prefill(wl, inputs.make_qkv(wl, 0))


@pytest.mark.parametrize("tile", [64, 128])
@pytest.mark.parametrize("H,Hkv,n_ctas", [(3, 1, 0), (7, 1, 5), (4, 2, 600), (5, 1, 300), (2, 2, 1)])
def test_prefill_tensor_core_schedules(tile, H, Hkv, n_ctas):
    # odd groups (a single-head unit per group), key lists split into chunks that are merged through the
    # workspace (many CTAs, little work each), everything on one CTA
    # (with many CTAs the planner cuts lists only where that pays under its cost model: a long request)
    wl = make_wl("bf16", H, Hkv, 128, [37, 0, 5], [5, 3, 1], [29, 2100 if n_ctas >= 300 else 300, 0], 9, 11, tile)
    x = inputs.make_qkv(wl, 0)
    for mask in (wl.mask, inputs.STMask(9, 11, tile=tile, dense_causal=True)):
        err, plan = gc.check_prefill(wl, x, mask=mask, n_ctas=n_ctas)
        if n_ctas >= 300:
            assert plan.info.max_chunks > 1 and plan.info.ws_bytes > 0


def test_prefill_plan_is_reusable_after_split_merges():
    # the merge counters in the plan return to zero: the same plan gives the same bits launch after launch
    P = gc.pk()
    wl = make_wl("bf16", 4, 2, 128, [10], [6], [1800], 8, 8, 64)
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    plan = P.purekv_plan_build(db, P.st_params(wl.mask), P.BF16, 128, 4, 2, n_ctas=500)
    assert plan.info.max_chunks > 1
    outs = [P.purekv_st_sparse_prefill(q, k, v, db, plan).clone() for _ in range(3)]
    torch.cuda.synchronize()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    assert torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))


@pytest.mark.parametrize("tile", [64, 128])
@pytest.mark.parametrize("kind", ["huge", "very_negative", "rising", "falling"])
def test_prefill_tensor_core_extreme_logits(tile, kind):
    # The kernel takes exponentials against a reference that only moves when a tile would overflow exp2 or when all
    # kept terms have underflowed; these inputs force both moves (and the rescaling of O that goes with them).
    wl = make_wl("bf16", 4, 2, 128, [20, 3], [4, 2], [1500, 40], 6, 7, tile)
    x = inputs.make_qkv(wl, 0)
    T = wl.batch.total_tokens
    u = np.zeros(128, dtype=np.float32)
    u[:4] = 0.5                                              # unit vector, exactly representable
    ramp = np.linspace(0.0, 1.0, T, dtype=np.float32)[:, None, None]
    if kind == "huge":                                       # logits of several hundred either way
        x["q"] = x["q"] * 40.0
    elif kind == "very_negative":                            # every logit near -115 (log2 units)
        x["k"] = x["k"] * 0.25 + 30.0 * u
        x["q"] = x["q"] * 0.25 - 30.0 * u
    elif kind == "rising":                                   # later keys score ever higher: the reference must move up often
        x["k"] = x["k"] + 60.0 * ramp * u
        x["q"] = x["q"] + 40.0 * u
    else:                                                    # later keys score ever lower
        x["k"] = x["k"] - 60.0 * ramp * u
        x["q"] = x["q"] + 40.0 * u
    # These logits make attention nearly one-hot, so outputs are single V rows; halved, they stay below 4, where the
    # bf16 output's own rounding step (2^-6 from 4 upwards) would use up most of the absolute tolerance by itself.
    x["v"] = x["v"] * 0.5
    for n in "qkv":
        bits = inputs.f32_to_bf16_bits(x[n])
        x[n + "_bits"], x[n] = bits, inputs.bf16_bits_to_f32(bits)
    gc.check_prefill(wl, x)
    err, plan = gc.check_prefill(wl, x, mask=inputs.STMask(6, 7, tile=tile, dense_causal=True), n_ctas=300)
    assert plan.info.max_chunks > 1                          # the merge of split lists sees these values too


def test_prefill_refuses_to_run_on_a_raised_status_word():
    # A bounded wait that expires raises the device status word; every later CTA and launch that is given the same
    # word returns at once instead of working on a context that may be inconsistent, and the host sees the code.
    P = gc.pk()
    wl = make_wl("bf16", 4, 2, 128, [10], [6], [50], 8, 8, 128)
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    plan = P.purekv_plan_build(db, P.st_params(wl.mask), P.BF16, 128, 4, 2)
    out = torch.full_like(q, 7.0)
    status = torch.full((1,), P.ERR_TIMEOUT, dtype=torch.int32, device="cuda")     # as a timed-out CTA would leave it
    P.purekv_st_sparse_prefill(q, k, v, db, plan, out=out, status=status)
    with pytest.raises(P.PureKVError) as e:
        P.purekv_poll_status(status)
    assert e.value.status == P.ERR_TIMEOUT
    assert (out == 7.0).all()                                                       # nothing was computed
    status.zero_()                                                                  # the context is still usable
    P.purekv_st_sparse_prefill(q, k, v, db, plan, out=out, status=status)
    assert P.purekv_poll_status(status) == 0 and torch.isfinite(out.float()).all()


def test_prefill_tensor_core_single_token_and_tiny_requests():
    wl = make_wl("bf16", 2, 1, 128, [1, 0, 3], [0, 1, 0], [0, 0, 126], 1, 1, 128)
    gc.check_prefill(wl, inputs.make_qkv(wl, 0))


def test_prefill_cfg0():
    wl = inputs.workload(0)
    err, plan = gc.check_prefill(wl, inputs.make_qkv(wl, 0))
    assert (plan.info.tiles_kept, plan.info.tiles_causal) == (131, 171)


def test_prefill_is_deterministic():
    wl = make_wl("bf16", 4, 2, 128, [10], [6], [50], 8, 8, 128)
    x = inputs.make_qkv(wl, 0)
    a, la, _ = gc.gpu_prefill(wl, x)
    b, lb, _ = gc.gpu_prefill(wl, x)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16)) and torch.equal(la, lb)


# ------------------------------------------------- score / select / compact -------------
def run_compress(wl, layers_x, window, keep):
    """layers_x: list of per-layer dicts; layer 0 is the scored layer.  Returns everything needed."""
    P = gc.pk()
    db = gc.device_batch(wl)
    bud = P.Budget(db, window, keep)
    q0, k0 = gc.upload(layers_x[0], "q", wl.dtype), gc.upload(layers_x[0], "k", wl.dtype)
    c = P.purekv_lowlayer_score(q0, k0, db, window)
    ks = torch.stack([gc.upload(x, "k", wl.dtype) for x in layers_x])
    vs = torch.stack([gc.upload(x, "v", wl.dtype) for x in layers_x])
    s = torch.empty((len(layers_x), wl.n_kv_heads, db.total_tokens), dtype=torch.float32, device="cuda")
    idx = P.purekv_select_topk(c, vs, db, bud, s_out=s)
    idx_ws = P.purekv_select_topk(c, vs, db, bud)          # workspace path must agree
    assert torch.equal(idx, idx_ws)
    kc, vc = P.purekv_compact_kv(ks, vs, idx, db, bud)
    # selection and compaction in one call: the same indices and the same bytes (checked against the oracle below
    # through kc / vc), with guard bands around the outputs
    pad = 64
    kf = torch.full((len(layers_x), bud.total_kept + 2 * pad, wl.n_kv_heads, wl.head_dim), 3.0, dtype=ks.dtype, device="cuda")
    vf = torch.full_like(kf, 3.0)
    idx_f, kc_f, vc_f = P.purekv_select_compact(c, ks, vs, db, bud, k_out=kf[:, pad:pad + bud.total_kept],
                                                v_out=vf[:, pad:pad + bud.total_kept])
    torch.cuda.synchronize()
    as_bits = lambda t: t.contiguous().view(torch.int16 if t.element_size() == 2 else torch.int32)
    assert torch.equal(idx_f, idx) and torch.equal(as_bits(kc_f), as_bits(kc)) and torch.equal(as_bits(vc_f), as_bits(vc))
    for t in (kf, vf):
        assert (t[:, :pad] == 3.0).all() and (t[:, pad + bud.total_kept:] == 3.0).all(), "guard bands"
    return c, s, idx, kc, vc, bud


def check_compress(wl, n_layers, window, keep):
    layers_x = [inputs.make_qkv(wl, l) for l in range(n_layers)]
    c, s, idx, kc, vc, bud = run_compress(wl, layers_x, window, keep)
    b = wl.batch
    cu = b.cu_seqlens
    c_ref = po.lowlayer_score(layers_x[0]["q"], layers_x[0]["k"], cu, window)
    assert gc.score_error(c.cpu().numpy(), c_ref) <= gc.SCORE_RTOL
    hk, ck = po.budgets(b.seq_lens, window, keep)
    assert np.array_equal(hk, bud.h_keep) and np.array_equal(ck, bud.h_cu_kept)
    for l in range(n_layers):
        x = layers_x[l]
        s_ref = po.vnorm_scores(c_ref, x["v"])
        s_gpu = s[l].cpu().numpy()
        assert gc.score_error(s_gpu, s_ref) <= gc.SCORE_RTOL
        idx_ref, kth = po.select(s_ref, cu, window, hk, ck)
        idx_gpu = idx[l].cpu().numpy()
        gc.check_index_sets(idx_gpu, idx_ref, s_ref, kth, wl, hk, ck, window)
        # selection alone, on the GPU's own fp32 scores: bit-exact against the oracle's selection rule
        idx_self, _ = po.select(s_gpu.astype(np.float64), cu, window, hk, ck)
        assert np.array_equal(idx_gpu, idx_self)
        # compaction: bit-exact against the oracle's gather driven by the GPU's indices
        bits = "k_bits" if wl.dtype == "bf16" else "k"
        vbits = "v_bits" if wl.dtype == "bf16" else "v"
        view = (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)) if wl.dtype == "bf16" else (lambda t: t.cpu().numpy())
        assert np.array_equal(view(kc[l]), po.compact(x[bits], idx_gpu, cu, ck))
        assert np.array_equal(view(vc[l]), po.compact(x[vbits], idx_gpu, cu, ck))


@pytest.mark.parametrize("dtype,d", [("fp32", 64), ("bf16", 128), ("bf16", 64)])
@pytest.mark.parametrize("window,keep", [(8, 0.3), (1, 0.1), (40, 0.5), (8, 1.0), (500, 0.2)])
def test_compress_small(dtype, d, window, keep):
    wl = make_wl(dtype, 6, 2, d, [5, 0, 9], [4, 3, 0], [17, 45, 30], 5, 6, 64)
    check_compress(wl, 3, window, keep)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64)])
@pytest.mark.parametrize("window,keep", [(8, 0.3), (40, 0.05), (8, 1.0)])
def test_compress_many_segments(dtype, d, window, keep):
    # 3 requests x 4 KV heads x 25 layers = 300 segments of 256-byte rows: the selection kernel streams V itself
    wl = make_wl(dtype, 8, 4, d, [5, 0, 9], [4, 3, 0], [17, 45, 30], 5, 6, 64)
    check_compress(wl, 25, window, keep)


@pytest.mark.parametrize("window", [8, 64, 200, 1000])
@pytest.mark.parametrize("H,Hkv", [(8, 2), (7, 1), (2, 2)])
def test_scores_from_prefill_lse(window, H, Hkv):
    # the one-pass tensor-core scores, fed with the log-sum-exp of the dense causal prefill of the same layer
    P = gc.pk()
    wl = make_wl("bf16", H, Hkv, 128, [5, 0, 9, 0], [4, 3, 0, 0], [27, 45, 30, 16], 5, 6, 64)      # lengths 152, 135, 39, 16
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    dense = inputs.STMask(5, 6, tile=64, dense_causal=True)
    plan = P.purekv_plan_build(db, P.st_params(dense), P.BF16, 128, H, Hkv)
    lse = torch.empty((H, db.total_tokens), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.purekv_st_sparse_prefill(q, k, v, db, plan, lse=lse, status=status)
    if any(l < window and l % 8 for l in wl.batch.seq_lens):
        with pytest.raises(P.PureKVError) as e:                      # a clipped window that is not a multiple of 8
            P.purekv_lowlayer_score_lse(q, k, lse, db, window)
        assert e.value.status == P.ERR_UNSUPPORTED
        return
    c = torch.full((Hkv, db.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    P.purekv_lowlayer_score_lse(q, k, lse, db, window, c_out=c, status=status)
    assert P.purekv_poll_status(status) == 0
    c_two_pass = P.purekv_lowlayer_score(q, k, db, window)
    torch.cuda.synchronize()
    c_ref = po.lowlayer_score(x["q"], x["k"], wl.batch.cu_seqlens, window)
    assert np.isfinite(c.cpu().numpy()).all()
    assert gc.score_error(c.cpu().numpy(), c_ref) <= gc.SCORE_RTOL
    assert gc.score_error(c.cpu().numpy(), c_two_pass.cpu().numpy().astype(np.float64)) <= gc.SCORE_RTOL


@pytest.mark.parametrize("window", [16, 64])
def test_scores_from_prefill_lse_many_requests(window):
    # 99 requests, some empty, some shorter than the window, some of several key blocks -- 660 key blocks over the 4 KV
    # heads, one block of rows each: enough items of few rows for the persistent form of the one-pass kernel, which
    # numbers its items through a table of the requests' running block counts (scanned 32 requests at a time) and
    # carries its pipeline from item to item
    P = gc.pk()
    H, Hkv = 8, 4
    pre = [(0, 8, 10, 24, 30, 0, 16, 40, 40)[i % 9] for i in range(99)]
    frames = [(0, 0, 5, 0, 9, 0, 0, 22, 0)[i % 9] for i in range(99)]
    suf = [(0, 0, 0, 0, 0, 0, 0, 0, 0)[i % 9] for i in range(99)]         # lengths 0, 8, 160, 24, 300, 0, 16, 700, 40
    wl = make_wl("bf16", H, Hkv, 128, pre, frames, suf, 5, 6, 64)
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    dense = inputs.STMask(5, 6, tile=64, dense_causal=True)
    plan = P.purekv_plan_build(db, P.st_params(dense), P.BF16, 128, H, Hkv)
    lse = torch.empty((H, db.total_tokens), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    P.purekv_st_sparse_prefill(q, k, v, db, plan, lse=lse, status=status)
    c = torch.full((Hkv, db.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):                                               # twice: nothing is left behind between calls
        P.purekv_lowlayer_score_lse(q, k, lse, db, window, c_out=c, status=status)
    assert P.purekv_poll_status(status) == 0
    c_ref = po.lowlayer_score(x["q"], x["k"], wl.batch.cu_seqlens, window)
    assert np.isfinite(c.cpu().numpy()).all()
    assert gc.score_error(c.cpu().numpy(), c_ref) <= gc.SCORE_RTOL


def test_compress_cfg0():
    wl = inputs.workload(0)
    check_compress(wl, 1, wl.window, wl.keep_ratio)


def test_select_with_ties_picks_lowest_positions():
    P = gc.pk()
    db = P.Batch([4100], [0], [0])
    bud = P.Budget(db, 100, 0.5)
    T = 4100
    c = torch.ones((1, T), dtype=torch.float32, device="cuda")
    v = torch.ones((1, T, 1, 8), dtype=torch.float32, device="cuda")          # every score equal
    idx = P.purekv_select_topk(c, v, db, bud).cpu().numpy()[0, 0]
    h = int(bud.h_keep[0])
    assert np.array_equal(idx[:h], np.arange(h)) and np.array_equal(idx[h:], np.arange(4000, 4100))
    c[0, 3000:3010] = 2.0
    c[0, 5] = 0.5
    idx = P.purekv_select_topk(c, v, db, bud).cpu().numpy()[0, 0]
    ties = np.setdiff1d(np.arange(0, h - 10 + 1), [5])           # the h-10 lowest positions among the ties
    want = np.sort(np.concatenate([np.arange(3000, 3010), ties]))
    assert np.array_equal(idx[:h], want)


def test_compact_keep_all_is_identity_and_guard_bands_survive():
    P = gc.pk()
    wl = make_wl("bf16", 2, 2, 128, [3, 1], [2, 1], [9, 4], 4, 4, 64)
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    bud = P.Budget(db, 4, 1.0)
    k = gc.upload(x, "k", "bf16")[None].contiguous()
    v = gc.upload(x, "v", "bf16")[None].contiguous()
    c = P.purekv_lowlayer_score(gc.upload(x, "q", "bf16"), k[0], db, 4)
    idx = P.purekv_select_topk(c, v, db, bud)
    n = k.numel()
    guard = torch.full((2, n + 512), 0x7B7B, dtype=torch.int16, device="cuda")
    ko = guard[0, 256:256 + n].view(torch.bfloat16).view(k.shape)
    vo = guard[1, 256:256 + n].view(torch.bfloat16).view(k.shape)
    P.purekv_compact_kv(k, v, idx, db, bud, k_out=ko, v_out=vo)
    torch.cuda.synchronize()
    assert torch.equal(ko.view(torch.int16), k.view(torch.int16)) and torch.equal(vo.view(torch.int16), v.view(torch.int16))
    assert (guard[:, :256] == 0x7B7B).all() and (guard[:, 256 + n:] == 0x7B7B).all()


def test_empty_inputs_and_bad_arguments():
    P = gc.pk()
    db = P.Batch([], [], [])
    bud = P.Budget(db, 4, 0.5)
    z = torch.empty((0, 2, 128), dtype=torch.bfloat16, device="cuda")
    plan = P.purekv_plan_build(db, P.st_params(inputs.STMask(4, 4, tile=64)), P.BF16, 128, 2, 2)
    P.purekv_st_sparse_prefill(z, z, z, db, plan)
    c = P.purekv_lowlayer_score(z, z, db, 4)
    idx = P.purekv_select_topk(c, z[None], db, bud)
    P.purekv_compact_kv(z[None], z[None], idx, db, bud)
    torch.cuda.synchronize()
    db = P.Batch([40], [0], [0])
    q = torch.zeros((40, 3, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((40, 2, 128), dtype=torch.bfloat16, device="cuda")
    plan = P.purekv_plan_build(db, P.st_params(inputs.STMask(4, 4, tile=64)), P.BF16, 128, 2, 2)
    with pytest.raises(P.PureKVError) as e:
        P.purekv_st_sparse_prefill(q, kv, kv, db, plan)          # 3 query heads, 2 KV heads
    assert e.value.status == P.ERR_INVALID_ARG
    with pytest.raises(P.PureKVError) as e:
        P.purekv_lowlayer_score(q[:, :2].contiguous(), kv, db, 4, ws=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert e.value.status == P.ERR_WORKSPACE
