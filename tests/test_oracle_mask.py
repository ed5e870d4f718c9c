"""Pins for the oracle's ST-SpAttn mask predicate (Sec. 3.2) and the budget rule.

The mask is checked against (i) a second construction that follows the two
sentences of Sec. 3.2 as loops over (frame, cell) and fills an l x l matrix,
(ii) a vectorised numpy construction for the generalised parameters, (iii) the
closed-form pair count of the paper's mask, (iv) special cases."""
import numpy as np
import pytest

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs


def sentence_mask(n_prefix, n_frames, gh, gw, n_suffix):
    """Paper mask built from the sentences: every visual token attends the first frame
    and its own frame (spatial path) and its own cell in the previous frame (temporal
    path); all of it causal; prefix keys visible to all; text rows dense causal."""
    n = gh * gw
    l = n_prefix + n_frames * n + n_suffix
    m = np.zeros((l, l), dtype=bool)
    pos = lambda f, c: n_prefix + f * n + c
    for i in range(n_prefix):                      # prefix text rows
        m[i, :i + 1] = True
    for f in range(n_frames):
        for c in range(n):
            i = pos(f, c)
            m[i, :n_prefix] = True
            for c2 in range(n):
                m[i, pos(0, c2)] = True            # first frame
                m[i, pos(f, c2)] = True            # current frame
            if f >= 1:
                m[i, pos(f - 1, c)] = True         # corresponding token, previous frame
    for i in range(n_prefix + n_frames * n, l):    # suffix text rows
        m[i, :] = True
    return m & np.tril(np.ones((l, l), dtype=bool))


def numpy_general_mask(n_prefix, n_frames, gh, gw, n_suffix, A, rs, D, st, rt):
    n = gh * gw
    l = n_prefix + n_frames * n + n_suffix
    t = np.arange(l)
    vis = (t >= n_prefix) & (t < n_prefix + n_frames * n)
    v = np.clip(t - n_prefix, 0, None)
    f, p = v // n, v % n
    y, x = p // gw, p % gw
    I, J = np.meshgrid(t, t, indexing="ij")
    cheb = np.maximum(np.abs(y[I] - y[J]), np.abs(x[I] - x[J]))
    df = f[I] - f[J]
    vv = vis[I] & vis[J]
    anchor = f[J] < A
    spat = (df == 0) & ((rs < 0) | (cheb <= rs))
    temp = (df >= 1) & (df % st == 0) & ((D < 0) | (df <= D * st)) & ((rt < 0) | (cheb <= rt))
    keep = ~vis[I] | (~vis[J]) | (vv & (anchor | spat | temp))
    return keep & (J <= I)


def closed_form_pairs(ns, F, N, nt):
    tri = lambda a: a * (a + 1) // 2
    tot = tri(ns)
    if F >= 1:
        tot += N * ns + tri(N)
    if F >= 2:
        tot += N * (ns + N) + tri(N)
    tot += max(F - 2, 0) * (N * (ns + N + 1) + tri(N))
    tot += nt * (ns + F * N) + tri(nt)
    return tot


SHAPES = [(16, 4, 8, 8, 16), (0, 3, 2, 3, 5), (3, 1, 4, 4, 2), (2, 5, 1, 1, 3), (5, 0, 3, 3, 4), (0, 6, 3, 2, 0)]


@pytest.mark.parametrize("ns,F,gh,gw,nt", SHAPES)
def test_paper_mask_matches_sentence_construction(ns, F, gh, gw, nt):
    mp = po.mask_params(inputs.STMask(gh, gw))
    l = ns + F * gh * gw + nt
    got = po.mask_matrix(mp, l, ns, F)
    want = sentence_mask(ns, F, gh, gw, nt)
    assert np.array_equal(got, want)
    assert got.sum() == closed_form_pairs(ns, F, gh * gw, nt)
    assert got.diagonal().all()                      # no empty row


@pytest.mark.parametrize("cfg,pairs", [(0, 29456), (1, 783264), (2, 4148800)])
def test_pair_counts_of_workloads(cfg, pairs):
    wl = inputs.workload(cfg)
    b = wl.batch
    n = b.grid_h * b.grid_w
    assert closed_form_pairs(b.n_prefix[0], b.n_frames[0], n, b.n_suffix(0)) == pairs
    got = po.mask_matrix(po.mask_params(wl.mask), b.seq_lens[0], b.n_prefix[0], b.n_frames[0])
    assert int(got.sum()) == pairs


@pytest.mark.parametrize("A,rs,D,st,rt", [(1, -1, 1, 1, 0), (2, 1, 2, 1, 1), (0, 0, -1, 2, -1), (1, 2, 3, 2, 0),
                                          (1, -1, -1, 1, -1), (3, 1, 0, 1, 0), (1, -1, 2, 3, 2)])
def test_general_mask_matches_numpy_construction(A, rs, D, st, rt):
    ns, F, gh, gw, nt = 5, 7, 4, 5, 6
    m = inputs.STMask(gh, gw, A, rs, D, st, rt)
    l = ns + F * gh * gw + nt
    got = po.mask_matrix(po.mask_params(m), l, ns, F)
    want = numpy_general_mask(ns, F, gh, gw, nt, A, rs, D, st, rt)
    assert np.array_equal(got, want)


def test_special_cases():
    tril = lambda l: np.tril(np.ones((l, l), dtype=bool))
    # one frame: dense causal
    mp = po.mask_params(inputs.STMask(4, 4))
    assert np.array_equal(po.mask_matrix(mp, 3 + 16 + 2, 3, 1), tril(21))
    # all earlier frames, whole frames: dense causal
    mp = po.mask_params(inputs.STMask(3, 3, 1, -1, -1, 1, -1))
    assert np.array_equal(po.mask_matrix(mp, 2 + 45 + 3, 2, 5), tril(50))
    # dense flag
    mp = po.mask_params(inputs.STMask(3, 3, dense_causal=True))
    assert np.array_equal(po.mask_matrix(mp, 50, 2, 5), tril(50))
    # one token per frame: {prefix, frame 0, self, previous}
    mp = po.mask_params(inputs.STMask(1, 1))
    got = po.mask_matrix(mp, 2 + 6 + 0, 2, 6)
    for f in range(6):
        want = np.zeros(8, dtype=bool)
        want[[0, 1, 2, 2 + f]] = True
        if f >= 1:
            want[2 + f - 1] = True
        assert np.array_equal(got[2 + f], want)
    # out-of-range and anti-causal pairs
    assert not po.mask(mp, 8, 2, 6, 3, 4)
    assert not po.mask(mp, 8, 2, 6, 8, 0)
    assert not po.mask(mp, 8, 2, 6, 2, -1)


def test_budget_rule():
    assert po.budget(288, 16, 0.2) == (41, 57)
    assert po.budget(2432, 64, 0.2) == (422, 486)
    assert po.budget(8320, 64, 0.2) == (1600, 1664)
    assert po.budget(37120, 256, 0.1) == (3456, 3712)
    assert po.budget(37120, 256, 0.5) == (18304, 18560)
    assert po.budget(100, 32, 0.1) == (0, 32)        # budget below the window: window only
    assert po.budget(10, 32, 0.5) == (0, 10)         # window clipped to the sequence
    assert po.budget(50, 8, 1.0) == (42, 50)         # keep everything


# ---- the comparison masks of App. A.3 / Table 7, each from its own sentence ------------------------------------------
def variant_sentence_mask(name, n_prefix, n_frames, gh, gw, n_suffix, local_window=0, dilation=0):
    """A second construction, by loops over (frame, cell): what each name keeps for a visual query; prefix keys
    stay visible and text rows dense causal as in the paper's mask; everything causal."""
    n = gh * gw
    l = n_prefix + n_frames * n + n_suffix
    m = np.zeros((l, l), dtype=bool)
    pos = lambda f, c: n_prefix + f * n + c
    for i in range(n_prefix):
        m[i, :i + 1] = True
    for f in range(n_frames):
        for c in range(n):
            i = pos(f, c)
            m[i, :n_prefix] = True
            m[i, i] = True
            if name in ("spatial", "temporal"):
                for c2 in range(n):
                    m[i, pos(0, c2)] = True                    # the first frame anchors both paths
            if name == "spatial":
                for c2 in range(n):
                    m[i, pos(f, c2)] = True                    # the current frame
            if name == "temporal" and f >= 1:
                m[i, pos(f - 1, c)] = True                     # the corresponding token of the previous frame
            if name == "local":
                for j in range(max(n_prefix, i - local_window + 1), i + 1):
                    m[i, j] = True                             # the most recent positions
            if name == "atrous":
                for j in range(i, n_prefix - 1, -dilation):
                    m[i, j] = True                             # every dilation-th position counted back
    for i in range(n_prefix + n_frames * n, l):
        m[i, :] = True
    return m & np.tril(np.ones((l, l), dtype=bool))


def variant_pairs(name, ns, F, N, nt, local_window=0, dilation=0):
    """Kept pairs of a variant in closed form (prefix rows, visual rows frame by frame, suffix rows)."""
    tri = lambda a: a * (a + 1) // 2
    tot = tri(ns) + nt * (ns + F * N) + tri(nt)
    for f in range(F):
        if name == "spatial":        # prefix + first frame + causal part of the own frame (frame 0: the two coincide)
            tot += N * ns + tri(N) + (N * N if f >= 1 else 0)
        elif name == "temporal":     # prefix + first frame + previous cell + self (they coincide for f = 0 and f = 1)
            tot += N * ns + (tri(N) if f == 0 else N * N + N * (1 if f == 1 else 2))
        elif name == "local":        # prefix + the window clipped at the first visual position
            tot += sum(ns + min(local_window, f * N + c + 1) for c in range(N))
        elif name == "atrous":       # prefix + every dilation-th position back to the first visual one
            tot += sum(ns + (f * N + c) // dilation + 1 for c in range(N))
    return tot


VARIANT_SHAPES = [(4, 5, 3, 4, 6), (0, 3, 2, 3, 5), (3, 1, 4, 4, 2), (2, 6, 1, 1, 0)]


@pytest.mark.parametrize("ns,F,gh,gw,nt", VARIANT_SHAPES)
@pytest.mark.parametrize("name,kw", [("spatial", {}), ("temporal", {}), ("local", dict(local_window=7)),
                                     ("local", dict(local_window=1)), ("atrous", dict(atrous_dilation=3)),
                                     ("atrous", dict(atrous_dilation=1))])
def test_named_variants_match_their_sentences_and_pair_counts(name, kw, ns, F, gh, gw, nt):
    m = inputs.mask_variant(name, gh, gw, **kw)
    l = ns + F * gh * gw + nt
    got = po.mask_matrix(po.mask_params(m), l, ns, F)
    lw, dil = kw.get("local_window", 0), kw.get("atrous_dilation", 0)
    assert np.array_equal(got, variant_sentence_mask(name, ns, F, gh, gw, nt, lw, dil))
    assert int(got.sum()) == variant_pairs(name, ns, F, gh * gw, nt, lw, dil)
    assert got.diagonal().all()


def test_variants_relate_to_the_paper_mask_and_to_dense_attention():
    ns, F, gh, gw, nt = 3, 5, 3, 4, 4
    l = ns + F * gh * gw + nt
    mat = lambda m: po.mask_matrix(po.mask_params(m), l, ns, F)
    st, sp, tp = (mat(inputs.mask_variant(n, gh, gw)) for n in ("st", "spatial", "temporal"))
    assert np.array_equal(st, sp | tp)                    # the paper's mask is the union of its two paths
    tril = np.tril(np.ones((l, l), dtype=bool))
    assert np.array_equal(mat(inputs.mask_variant("local", gh, gw, local_window=l)), tril)
    assert np.array_equal(mat(inputs.mask_variant("atrous", gh, gw, atrous_dilation=1)), tril)
    assert np.array_equal(mat(inputs.mask_variant("st", gh, gw)), mat(inputs.STMask(gh, gw)))


@pytest.mark.parametrize("name,kw", [("st", {}), ("temporal", {}), ("local", dict(local_window=5)),
                                     ("atrous", dict(atrous_dilation=7))])
@pytest.mark.parametrize("block", [4, 16])
def test_block_level_widening_keeps_whole_blocks_under_causality(name, kw, block):
    """coarse: a block pair is kept whole (its causal part) exactly when the token-level mask keeps any pair in it."""
    ns, F, gh, gw, nt = 5, 4, 3, 3, 7
    l = ns + F * gh * gw + nt
    fine = po.mask_matrix(po.mask_params(inputs.mask_variant(name, gh, gw, tile=block, **kw)), l, ns, F)
    got = po.mask_matrix(po.mask_params(inputs.mask_variant(name, gh, gw, tile=block, coarse=True, **kw)), l, ns, F)
    nb = (l + block - 1) // block
    pad = np.zeros((nb * block, nb * block), dtype=bool)
    pad[:l, :l] = fine
    blocks = pad.reshape(nb, block, nb, block).any(axis=(1, 3))
    want = np.repeat(np.repeat(blocks, block, axis=0), block, axis=1)[:l, :l] & np.tril(np.ones((l, l), dtype=bool))
    assert np.array_equal(got, want)
    assert (got | ~fine).all()                            # widening never drops a pair
