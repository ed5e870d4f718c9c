"""GPU parity of the other score reductions and of the score-free policy (App. A.1 / Table 6) against the oracle,
and each policy carried through V-norm weighting, selection and compaction."""
import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc
from tests.test_gpu_parity import make_wl

pytestmark = pytest.mark.gpu

REDUCTIONS = [("accumulated attention (all rows)", -1, 1), ("observation window 16 + pooling 7", 16, 7),
              ("observation window = recent window (Eq. 2)", None, 1), ("observation window 3", 3, 1),
              ("observation longer than the recent window", 40, 5), ("all rows + pooling", 100000, 3)]


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64), ("bf16", 40)])
@pytest.mark.parametrize("name,obs,pool", REDUCTIONS)
def test_score_reductions_match_the_oracle(name, obs, pool, dtype, d):
    P = gc.pk()
    wl = make_wl(dtype, 6, 2, d, [5, 0, 9, 0], [4, 3, 0, 0], [27, 45, 30, 7], 5, 6, 64, window=8)
    obs = wl.window if obs is None else obs
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k = gc.upload(x, "q", wl.dtype), gc.upload(x, "k", wl.dtype)
    got = P.purekv_lowlayer_score_ex(q, k, db, wl.window, obs, pool).cpu().numpy()
    ref = po.lowlayer_score_ex(x["q"], x["k"], wl.batch.cu_seqlens, wl.window, obs, pool)
    assert np.isfinite(got).all()
    assert gc.score_error(got, ref) <= gc.SCORE_RTOL, name
    if obs == wl.window and pool == 1:                   # the same kernels as the plain entry point: same bits
        assert np.array_equal(got, P.purekv_lowlayer_score(q, k, db, wl.window).cpu().numpy())


def test_score_reductions_refuse_bad_arguments():
    P = gc.pk()
    wl = make_wl("bf16", 4, 2, 128, [3], [2], [20], 5, 6, 64, window=8)
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k = gc.upload(x, "q", "bf16"), gc.upload(x, "k", "bf16")
    with pytest.raises(P.PureKVError) as e:
        P.purekv_lowlayer_score_ex(q, k, db, wl.window, -1, 4)                  # even pool
    assert e.value.status == P.ERR_INVALID_ARG
    with pytest.raises(P.PureKVError) as e:
        P.purekv_lowlayer_score_ex(q, k, db, wl.window, -1, 1, ws=torch.empty(512, dtype=torch.uint8, device="cuda"))
    assert e.value.status == P.ERR_WORKSPACE


@pytest.mark.parametrize("policy", ["accumulated", "pooled window", "sink + recent"])
def test_policies_through_selection_and_compaction(policy):
    """CLIE with another policy's scores (Eq. 4 with that policy's C), then top-h and the gather: index sets against the
    oracle within the tie band, selection bit-exact on the GPU's own scores, compaction bit-exact."""
    P = gc.pk()
    wl = make_wl("bf16", 8, 2, 128, [5, 0], [4, 3], [37, 45], 5, 6, 64, window=8, keep=0.3)
    b = wl.batch
    cu = b.cu_seqlens
    x0, x1 = inputs.make_qkv(wl, 0), inputs.make_qkv(wl, 1)
    db = gc.device_batch(wl)
    bud = P.Budget(db, wl.window, wl.keep_ratio)
    hk, ck = po.budgets(b.seq_lens, wl.window, wl.keep_ratio)
    k1, v1 = gc.upload(x1, "k", "bf16")[None].contiguous(), gc.upload(x1, "v", "bf16")[None].contiguous()
    if policy == "sink + recent":
        idx = P.purekv_select_sink_recent(db, bud, 1, wl.n_kv_heads)
        assert np.array_equal(idx[0].cpu().numpy(), po.select_sink_recent(cu, wl.window, hk, ck, wl.n_kv_heads))
    else:
        obs, pool = (-1, 1) if policy == "accumulated" else (16, 5)
        c = P.purekv_lowlayer_score_ex(gc.upload(x0, "q", "bf16"), gc.upload(x0, "k", "bf16"), db, wl.window, obs, pool)
        s = torch.empty((1, wl.n_kv_heads, db.total_tokens), dtype=torch.float32, device="cuda")
        idx = P.purekv_select_topk(c, v1, db, bud, s_out=s)
        s_ref = po.vnorm_scores(po.lowlayer_score_ex(x0["q"], x0["k"], cu, wl.window, obs, pool), x1["v"])
        idx_ref, kth = po.select(s_ref, cu, wl.window, hk, ck)
        gc.check_index_sets(idx[0].cpu().numpy(), idx_ref, s_ref, kth, wl, hk, ck, wl.window)
        idx_self, _ = po.select(s[0].cpu().numpy().astype(np.float64), cu, wl.window, hk, ck)
        assert np.array_equal(idx[0].cpu().numpy(), idx_self)
    kc, vc = P.purekv_compact_kv(k1, v1, idx, db, bud)
    view = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(view(kc[0]), po.compact(x1["k_bits"], idx[0].cpu().numpy(), cu, ck))
    assert np.array_equal(view(vc[0]), po.compact(x1["v_bits"], idx[0].cpu().numpy(), cu, ck))
