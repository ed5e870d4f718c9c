"""Pins for the oracle's decode step (one new query per request over the compacted cache; the stage
Table 3 reports as decode latency): a library attention routine, closed forms, invariances, and the
keep-ratio-1.0 relation to the dense prefill's last row."""
import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs


def draw(seed, kept, H, Hkv, d):
    rng = np.random.default_rng(seed)
    ck = np.concatenate([[0], np.cumsum(kept)]).astype(np.int32)
    q = rng.standard_normal((len(kept), H, d)).astype(np.float32)
    kc = rng.standard_normal((int(ck[-1]), Hkv, d)).astype(np.float32)
    vc = rng.standard_normal((int(ck[-1]), Hkv, d)).astype(np.float32)
    return q, kc, vc, ck


@pytest.mark.parametrize("H,Hkv,d", [(4, 2, 16), (7, 1, 8), (6, 6, 32)])
def test_decode_matches_library_attention(H, Hkv, d):
    q, kc, vc, ck = draw(1, [5, 1, 40, 17], H, Hkv, d)
    out, lse = po.decode(q, kc, vc, ck)
    G = H // Hkv
    for r in range(len(ck) - 1):
        for h in range(H):
            kk = torch.from_numpy(kc[ck[r]:ck[r + 1], h // G]).double()[None]
            vv = torch.from_numpy(vc[ck[r]:ck[r + 1], h // G]).double()[None]
            qq = torch.from_numpy(q[r, h]).double()[None, None]
            ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv)[0, 0].numpy()
            np.testing.assert_allclose(out[r, h], ref, rtol=1e-11, atol=1e-13)
            logits = (kk[0] @ qq[0, 0]) / np.sqrt(d)
            np.testing.assert_allclose(lse[r, h], float(torch.logsumexp(logits, 0)), rtol=1e-12)


def test_decode_closed_forms():
    q, kc, vc, ck = draw(2, [9, 30], 4, 2, 8)
    # a zero query weighs every kept key alike: the output is the mean of the request's V rows, lse = log n
    out, lse = po.decode(np.zeros_like(q), kc, vc, ck)
    for r in range(2):
        for h in range(4):
            np.testing.assert_allclose(out[r, h], vc[ck[r]:ck[r + 1], h // 2].astype(np.float64).mean(0), rtol=1e-13)
            np.testing.assert_allclose(lse[r, h], np.log(ck[r + 1] - ck[r]), rtol=1e-13)
    # one key aligned with the query and far longer than the rest takes all the weight
    kc2 = kc.copy()
    kc2[ck[1] + 7, 1] = 200.0 * q[1, 2] / np.linalg.norm(q[1, 2])
    out2, _ = po.decode(q, kc2, vc, ck)
    np.testing.assert_allclose(out2[1, 2], vc[ck[1] + 7, 1], rtol=0, atol=1e-12)
    # identical keys: uniform weights whatever the query
    kc3 = np.broadcast_to(kc[:1], kc.shape).copy()
    out3, _ = po.decode(q, kc3, vc, ck)
    np.testing.assert_allclose(out3[0, 1], vc[:9, 0].astype(np.float64).mean(0), rtol=1e-12)


def test_decode_invariances():
    q, kc, vc, ck = draw(3, [12, 25], 6, 2, 16)
    out, lse = po.decode(q, kc, vc, ck)
    # attention over a set: the order of a request's cache rows does not matter
    perm = np.concatenate([np.random.default_rng(0).permutation(12), 12 + np.random.default_rng(1).permutation(25)])
    out_p, lse_p = po.decode(q, kc[perm], vc[perm], ck)
    np.testing.assert_allclose(out_p, out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse_p, lse, rtol=1e-13)
    # a key shift along a direction orthogonal to nothing in particular moves every logit of a row alike
    shift = np.float32(0.5) * np.ones((1, 1, 16), dtype=np.float32)
    out_s, lse_s = po.decode(q, kc + shift, vc, ck)
    np.testing.assert_allclose(out_s, out, rtol=1e-5, atol=1e-6)          # fp32 rounding of the shifted keys only
    # the explicit scale equals the default 1/sqrt(d); another scale equals a rescaled query
    out_e, _ = po.decode(q, kc, vc, ck, scale=0.25)
    np.testing.assert_allclose(out_e, out, rtol=1e-13)
    out_2, _ = po.decode(q, kc, vc, ck, scale=0.5)
    out_q, _ = po.decode(2.0 * q, kc, vc, ck)
    np.testing.assert_allclose(out_2, out_q, rtol=1e-12)
    # requests do not see one another's rows
    out_a, _ = po.decode(q[:1], kc[:12], vc[:12], ck[:2])
    np.testing.assert_allclose(out_a[0], out[0], rtol=1e-13)


def test_decode_empty_request_and_single_key():
    q, kc, vc, ck = draw(4, [0, 1, 3], 2, 1, 8)
    out, lse = po.decode(q, kc, vc, ck)
    assert np.all(out[0] == 0.0) and np.all(np.isneginf(lse[0]))
    np.testing.assert_allclose(out[1, 0], vc[0, 0], rtol=1e-15)           # a single key: its V row exactly


def test_decode_at_keep_one_is_the_dense_prefill_last_row():
    """With every key kept, the step that would follow the prompt's last token repeats that token's row of the
    dense causal prefill (same query, same keys): the invariant that ties compaction and decode to Eq. 1."""
    b = inputs.make_batch([3, 0], [2, 1], [6, 9], 3, 2)
    rng = np.random.default_rng(5)
    T, H, Hkv, d = b.total_tokens, 4, 2, 8
    q = rng.standard_normal((T, H, d)).astype(np.float32)
    k = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    v = rng.standard_normal((T, Hkv, d)).astype(np.float32)
    cu = b.cu_seqlens
    dense = inputs.STMask(3, 2, tile=16, dense_causal=True)
    last = [int(cu[r + 1]) - 1 for r in range(2)]
    ref, ref_lse = po.prefill(q, k, v, cu, b.n_prefix, b.n_frames, po.mask_params(dense), rows=last)
    w = 2
    hk, ck = po.budgets(b.seq_lens, w, 1.0)
    s = po.vnorm_scores(po.lowlayer_score(q, k, cu, w), v)
    idx, _ = po.select(s, cu, w, hk, ck)
    kc, vc = po.compact(k, idx, cu, ck), po.compact(v, idx, cu, ck)
    out, lse = po.decode(q[last], kc, vc, ck)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse, ref_lse.T, rtol=1e-12)
