"""Pins for the oracle's window scores (Eq. 1-2), V-norm scores (Eq. 3-4), top-h
selection, compaction, and the keep-ratio-1.0 invariant."""
import numpy as np
import pytest

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests.test_oracle_attention import matrix_attention, small_workload


def full_matrix_scores(q, k, cu, w, G):
    """C from the full l x l dense causal attention matrix of every head (brute force)."""
    T, H, d = q.shape
    Hkv = k.shape[1]
    c = np.zeros((Hkv, T))
    for r in range(len(cu) - 1):
        lo, hi = cu[r], cu[r + 1]
        l = hi - lo
        ww = min(w, l)
        tril = np.tril(np.ones((l, l), dtype=bool))
        for h in range(H):
            _, _, p = matrix_attention(q[lo:hi, h], k[lo:hi, h // G], k[lo:hi, h // G], tril, 1.0 / np.sqrt(d))
            c[h // G, lo:lo + l - ww] += p[l - ww:, :l - ww].sum(axis=0) / G
    return c


@pytest.mark.parametrize("w", [1, 4, 11, 1000])
def test_scores_against_full_matrix(w):
    wl = small_workload(n_req=3, H=6, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    cu = wl.batch.cu_seqlens
    c = po.lowlayer_score(x["q"], x["k"], cu, w)
    np.testing.assert_allclose(c, full_matrix_scores(x["q"], x["k"], cu, w, 3), rtol=1e-11, atol=1e-14)


def test_scores_mass_conservation_and_bounds():
    wl = small_workload(H=4, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    l, w, G = b.seq_lens[0], 5, 2
    c = po.lowlayer_score(x["q"], x["k"], b.cu_seqlens, w)
    assert (c >= 0).all() and (c <= w).all() and (c[:, l - w:] == 0).all()
    # every window row sums to 1 over j <= i, so C's mass is w minus the mass the
    # window rows put on window keys; that part from the dense-causal attention rows:
    tril = np.tril(np.ones((l, l), dtype=bool))
    for g in range(2):
        inside = 0.0
        for h in range(g * G, (g + 1) * G):
            _, _, p = matrix_attention(x["q"][:, h], x["k"][:, g], x["k"][:, g], tril, 0.25)
            inside += p[l - w:, l - w:].sum() / G
        assert abs(c[g].sum() + inside - w) < 1e-12


def test_scores_zero_queries_harmonic_closed_form():
    wl = small_workload(H=2, Hkv=1, d=8)
    x = inputs.make_qkv(wl, 0)
    l, w = wl.batch.seq_lens[0], 6
    c = po.lowlayer_score(np.zeros_like(x["q"]), x["k"], wl.batch.cu_seqlens, w)
    # row i is uniform 1/(i+1): C_j = sum_{i=l-w}^{l-1} 1/(i+1) = H_l - H_{l-w}
    want = sum(1.0 / n for n in range(l - w + 1, l + 1))
    np.testing.assert_allclose(c[0, :l - w], want, rtol=1e-13)


def test_scores_window_one_is_last_row_and_lse_matches_prefill():
    wl = small_workload(H=2, Hkv=2, d=8, dense_causal=True)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    l = b.seq_lens[0]
    c = po.lowlayer_score(x["q"], x["k"], b.cu_seqlens, 1)
    _, lse = po.prefill(x["q"], x["k"], x["v"], b.cu_seqlens, b.n_prefix, b.n_frames, po.mask_params(wl.mask))
    for h in range(2):
        logits = (x["k"][: l - 1, h].astype(np.float64) @ x["q"][l - 1, h].astype(np.float64)) / np.sqrt(8)
        np.testing.assert_allclose(c[h, : l - 1], np.exp(logits - lse[h, l - 1]), rtol=1e-12)


def numpy_select(s_row, h):
    order = np.lexsort((np.arange(len(s_row)), -s_row))      # score descending, then position ascending
    return np.sort(order[:h])


def test_vnorm_scores_and_select_against_full_sort():
    wl = small_workload(n_req=3, H=4, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    cu, w = b.cu_seqlens, 4
    c = po.lowlayer_score(x["q"], x["k"], cu, w)
    s = po.vnorm_scores(c, x["v"])
    np.testing.assert_allclose(s, c * np.linalg.norm(x["v"].astype(np.float64), axis=2).T, rtol=1e-14)
    hk, ck = po.budgets(b.seq_lens, w, 0.4)
    idx, kth = po.select(s, cu, w, hk, ck)
    for g in range(2):
        for r in range(3):
            l = b.seq_lens[r]
            seg = idx[g, ck[r]:ck[r + 1]]
            want = numpy_select(s[g, cu[r]:cu[r] + l - w], hk[r])
            assert np.array_equal(seg[:hk[r]], want)
            assert np.array_equal(seg[hk[r]:], np.arange(l - w, l))
            assert kth[g, r] == np.sort(s[g, cu[r]:cu[r] + l - w])[::-1][hk[r] - 1]


def test_select_ties_extremes_and_permutation():
    cu = np.array([0, 12], dtype=np.int32)
    s = np.array([[1.0, 3.0, 3.0, 0.5, 3.0, 2.0, 2.0, 2.0, 9.0, 9.0, 9.0, 9.0]])   # window = last 4
    ck = lambda k: np.array([0, k], dtype=np.int32)
    idx, _ = po.select(s, cu, 4, [2], ck(6))
    assert idx[0].tolist() == [1, 2, 8, 9, 10, 11]          # ties: lowest positions win
    idx, _ = po.select(s, cu, 4, [5], ck(9))
    assert idx[0].tolist() == [1, 2, 4, 5, 6, 8, 9, 10, 11]
    idx, _ = po.select(s, cu, 4, [0], ck(4))
    assert idx[0].tolist() == [8, 9, 10, 11]                 # h = 0: window only
    idx, _ = po.select(s, cu, 4, [8], ck(12))
    assert idx[0].tolist() == list(range(12))                # h = l - w: identity
    # permuting the non-recent keys permutes the selection
    rng = np.random.default_rng(3)
    s2 = rng.random((1, 40))
    cu2 = np.array([0, 40], dtype=np.int32)
    base, _ = po.select(s2, cu2, 5, [9], ck(14))
    perm = rng.permutation(35)
    sp = s2.copy()
    sp[0, :35] = s2[0, perm]
    got, _ = po.select(sp, cu2, 5, [9], ck(14))
    assert set(perm[got[0, :9]].tolist()) == set(base[0, :9].tolist())


def test_zero_queries_select_by_vnorm():
    wl = small_workload(H=2, Hkv=1, d=8)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    l, w = b.seq_lens[0], 4
    c = po.lowlayer_score(np.zeros_like(x["q"]), x["k"], b.cu_seqlens, w)
    s = po.vnorm_scores(c, x["v"])
    idx, _ = po.select(s, b.cu_seqlens, w, [7], [0, 11])
    norms = np.linalg.norm(x["v"][: l - w, 0].astype(np.float64), axis=1)
    assert np.array_equal(idx[0, :7], np.sort(np.argsort(-norms)[:7]))


def test_compact_and_keep_all_identity():
    wl = small_workload(n_req=2, H=4, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    cu, w = b.cu_seqlens, 4
    c = po.lowlayer_score(x["q"], x["k"], cu, w)
    s = po.vnorm_scores(c, x["v"])
    hk, ck = po.budgets(b.seq_lens, w, 1.0)
    idx, _ = po.select(s, cu, w, hk, ck)
    assert np.array_equal(ck, cu)
    kc = po.compact(x["k"], idx, cu, ck)
    assert np.array_equal(kc, x["k"])                         # keep ratio 1.0: the cache is unchanged
    hk, ck = po.budgets(b.seq_lens, w, 0.3)
    idx, _ = po.select(s, cu, w, hk, ck)
    vc = po.compact(x["v"], idx, cu, ck)
    bits = po.compact(x["v"].view(np.uint32), idx, cu, ck)    # byte copy, dtype-agnostic
    assert np.array_equal(vc.view(np.uint32), bits)
    for r in range(2):
        for g in range(2):
            for t in range(ck[r], ck[r + 1]):
                assert np.array_equal(vc[t, g], x["v"][cu[r] + idx[g, t], g])


def test_keep_ratio_one_reproduces_dense_attention_for_the_last_query():
    """Decode-style attention of the last query over the compacted cache at keep 1.0
    equals the last row of dense causal prefill."""
    wl = small_workload(H=2, Hkv=1, d=8, dense_causal=True)
    x = inputs.make_qkv(wl, 0)
    b = wl.batch
    cu, w, l = b.cu_seqlens, 4, b.seq_lens[0]
    out, _ = po.prefill(x["q"], x["k"], x["v"], cu, b.n_prefix, b.n_frames, po.mask_params(wl.mask))
    s = po.vnorm_scores(po.lowlayer_score(x["q"], x["k"], cu, w), x["v"])
    hk, ck = po.budgets(b.seq_lens, w, 1.0)
    idx, _ = po.select(s, cu, w, hk, ck)
    kc, vc = po.compact(x["k"], idx, cu, ck), po.compact(x["v"], idx, cu, ck)
    for h in range(2):
        o, _, _ = matrix_attention(x["q"][l - 1:l, h], kc[:, 0], vc[:, 0], np.ones((1, l), dtype=bool), 1 / np.sqrt(8))
        np.testing.assert_allclose(o[0], out[l - 1, h], rtol=1e-12, atol=1e-14)


def test_select_refuses_a_budget_that_does_not_fit_the_request():
    """h beyond the non-recent keys, or a kept count other than h + w, is an error, not an out-of-range read."""
    cu = np.array([0, 10], dtype=np.int32)
    s = np.arange(10, dtype=np.float64)[None]
    for hk, ck in (([7], [0, 11]), ([3], [0, 8]), ([-1], [0, 3])):        # w = 4: at most 6 non-recent keys
        with pytest.raises(ValueError):
            po.select(s, cu, 4, hk, ck)
    idx, _ = po.select(s, cu, 4, [6], [0, 10])
    assert np.array_equal(idx[0], np.arange(10))
