"""Pins for the oracle's other score reductions (the policies of App. A.1 / Table 6), the score-free
sink + recent selection, and Spearman's rank correlation (Sec. 3.3, Eq. 5-7)."""
import numpy as np
import pytest
import scipy.stats
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests.test_oracle_attention import matrix_attention, small_workload


def matrix_reduction(q, k, cu, w, obs, pool, G):
    """Brute force: the full l x l dense causal attention matrix of every head, the last `obs` rows summed per
    column (all rows if obs < 0), mean over the group's heads, non-recent keys only, then pooling by convolution."""
    T, H, d = q.shape
    Hkv = k.shape[1]
    c = np.zeros((Hkv, T))
    for r in range(len(cu) - 1):
        lo, hi = cu[r], cu[r + 1]
        l = hi - lo
        ww = min(w, l)
        wo = l if obs < 0 or obs > l else obs
        tril = np.tril(np.ones((l, l), dtype=bool))
        for h in range(H):
            _, _, p = matrix_attention(q[lo:hi, h], k[lo:hi, h // G], k[lo:hi, h // G], tril, 1.0 / np.sqrt(d))
            c[h // G, lo:lo + l - ww] += p[l - wo:, :l - ww].sum(axis=0) / G        # p is 0 above the diagonal
        if pool > 1 and l - ww > 0:
            for g in range(Hkv):
                seg = c[g, lo:lo + l - ww]
                c[g, lo:lo + l - ww] = np.convolve(seg, np.ones(pool) / pool, mode="same")
    return c


@pytest.mark.parametrize("w,obs,pool", [(4, -1, 1), (4, 4, 1), (4, 9, 1), (11, 3, 1), (5, 8, 3), (2, -1, 7), (1000, -1, 1),
                                        (3, 1000, 5)])
def test_reductions_against_the_full_matrix(w, obs, pool):
    wl = small_workload(n_req=3, H=6, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    cu = wl.batch.cu_seqlens
    c = po.lowlayer_score_ex(x["q"], x["k"], cu, w, obs, pool)
    np.testing.assert_allclose(c, matrix_reduction(x["q"], x["k"], cu, w, obs, pool, 3), rtol=1e-11, atol=1e-14)


def test_observation_window_equal_to_the_recent_window_is_eq_2():
    wl = small_workload(n_req=2, H=4, Hkv=2, d=16)
    x = inputs.make_qkv(wl, 0)
    cu = wl.batch.cu_seqlens
    for w in (1, 6, 50):
        assert np.array_equal(po.lowlayer_score_ex(x["q"], x["k"], cu, w, w, 1), po.lowlayer_score(x["q"], x["k"], cu, w))


def test_accumulated_scores_zero_queries_harmonic_tail_and_mass():
    """Q = 0: row i is uniform 1/(i+1), so summing every row gives C_j = H_l - H_j, the bias toward early keys
    that Sec. 3.1 describes; and the columns of all rows together hold one unit of mass per row."""
    wl = small_workload(H=2, Hkv=1, d=8)
    x = inputs.make_qkv(wl, 0)
    l, w = wl.batch.seq_lens[0], 6
    c = po.lowlayer_score_ex(np.zeros_like(x["q"]), x["k"], wl.batch.cu_seqlens, w, -1, 1)
    harm = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, l + 1))])
    np.testing.assert_allclose(c[0, :l - w], harm[l] - harm[np.arange(l - w)], rtol=1e-12)
    assert (np.diff(c[0, :l - w]) < 0).all() and (c[0, l - w:] == 0).all()
    # with real queries: all l rows hold l units of mass; the non-recent columns hold l minus what falls on the window
    cq = po.lowlayer_score_ex(x["q"], x["k"], wl.batch.cu_seqlens, w, -1, 1)
    tril = np.tril(np.ones((l, l), dtype=bool))
    on_window = 0.0
    for h in range(2):
        _, _, p = matrix_attention(x["q"][:, h], x["k"][:, 0], x["k"][:, 0], tril, 1.0 / np.sqrt(8))
        on_window += p[:, l - w:].sum() / 2
    assert abs(cq[0].sum() + on_window - l) < 1e-10


def test_pooling_is_the_library_average_pool():
    wl = small_workload(H=2, Hkv=2, d=8)
    x = inputs.make_qkv(wl, 0)
    l, w = wl.batch.seq_lens[0], 5
    raw = po.lowlayer_score_ex(x["q"], x["k"], wl.batch.cu_seqlens, w, 7, 1)
    for pool in (3, 5, 9):
        got = po.lowlayer_score_ex(x["q"], x["k"], wl.batch.cu_seqlens, w, 7, pool)
        want = torch.nn.functional.avg_pool1d(torch.from_numpy(raw[:, None, :l - w]), pool, stride=1, padding=pool // 2)
        np.testing.assert_allclose(got[:, :l - w], want[:, 0].numpy(), rtol=1e-13, atol=1e-16)
        assert (got[:, l - w:] == 0).all()


def test_sink_recent_selection_by_construction():
    cu = np.array([0, 10, 14, 30], dtype=np.int32)
    hk, ck = [3, 0, 5], [0, 7, 11, 20]                   # w = 4: kept 3+4, 0+4, 5+4
    idx = po.select_sink_recent(cu, 4, hk, ck, 2)
    want = [0, 1, 2, 6, 7, 8, 9] + [0, 1, 2, 3] + [0, 1, 2, 3, 4, 12, 13, 14, 15]
    assert np.array_equal(idx, np.array([want, want]))
    with pytest.raises(ValueError):
        po.select_sink_recent(cu, 4, [7, 0, 5], [0, 11, 15, 24], 2)          # only 6 non-recent keys in request 0


def test_spearman_against_scipy_and_closed_forms():
    rng = np.random.default_rng(5)
    for n in (2, 3, 17, 400):
        a, b = rng.standard_normal(n), rng.standard_normal(n)
        assert abs(po.spearman(a, b) - scipy.stats.spearmanr(a, b).statistic) < 1e-12       # no ties: same statistic
        assert po.spearman(a, a) == 1.0 and abs(po.spearman(a, -a) + 1.0) < 1e-15
        assert abs(po.spearman(a, np.exp(a)) - 1.0) < 1e-15                                  # monotone maps keep ranks
    # a hand case: ranks (1,2,3,4) against (2,1,4,3): sum d^2 = 4, rho = 1 - 24 / 60
    assert abs(po.spearman([4.0, 3.0, 2.0, 1.0], [3.0, 4.0, 1.0, 2.0]) - 0.6) < 1e-15
    # rank-and-correlate brute force (Pearson on ranks) on data without ties
    a, b = rng.permutation(50).astype(float), rng.permutation(50).astype(float)
    ra, rb = scipy.stats.rankdata(-a), scipy.stats.rankdata(-b)
    assert abs(po.spearman(a, b) - np.corrcoef(ra, rb)[0, 1]) < 1e-12
    # ties share the mean rank: (1.5, 1.5, 3) against (1, 2, 3): d^2 = 0.5, rho = 1 - 3 / 24
    assert abs(po.spearman([5.0, 5.0, 1.0], [9.0, 8.0, 7.0]) - 0.875) < 1e-15
    assert np.isnan(po.spearman([1.0], [2.0]))


def test_rank_agreement_tool_is_one_when_the_high_layer_is_the_low_layer():
    """Sec. 3.3's study on one layer pair: with the same layer on both sides the estimate (Eq. 4) is the ground truth
    (Eq. 6), so rho = 1; with unrelated synthetic layers it is some value in [-1, 1]."""
    wl = small_workload(n_req=2, H=4, Hkv=2, d=16)
    x0, x1 = inputs.make_qkv(wl, 0), inputs.make_qkv(wl, 1)
    cu = wl.batch.cu_seqlens
    same = po.clie_rank_agreement(x0["q"], x0["k"], x0["q"], x0["k"], x0["v"], cu, 4)
    assert same.shape == (2, 2) and np.allclose(same, 1.0)
    other = po.clie_rank_agreement(x0["q"], x0["k"], x1["q"], x1["k"], x1["v"], cu, 4)
    assert ((other >= -1) & (other <= 1)).all()
