"""CPU tests of the C-ABI library's host side: it loads, exports what include/purekv.h
declares, validates arguments, and its plan builder agrees with the oracle's mask."""
import ctypes as C
import os
import re
import struct

import numpy as np
import pytest

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import binding as pk
from paper_2510_25600_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "purekv.h")).read()
    declared = set(re.findall(r"\b(purekv_[a-z_0-9]+)\s*\(", text))
    assert declared == set(pk.EXPORTS)
    lib = C.CDLL(pk.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in pk.purekv_version()


def test_budget_matches_oracle_rule():
    for length in [0, 1, 7, 57, 288, 2432, 8320, 37120, 12393]:
        for window in [1, 16, 64, 256, 100000]:
            for keep in [0.0, 0.05, 0.1, 0.2, 0.35, 0.5, 0.999, 1.0]:
                assert pk.purekv_budget(length, window, keep) == po.budget(length, window, keep)


def parse_plan(buf: np.ndarray):
    raw = buf.tobytes()
    (magic, tq, tk, nq, T, ne, nm, oq, oo, oe, om, wpr, n_ctas, n_units, n_counters, o_units, o_counters, H, Hkv,
     part_slots) = struct.unpack_from("<Iiiiqqqqqqqiiiiqqiiq", raw, 0)
    assert magic == 0x504B5636
    qt = np.frombuffer(raw, dtype=np.int32, count=nq * 8, offset=oq).reshape(nq, 8)
    order = np.frombuffer(raw, dtype=np.int32, count=nq, offset=oo)
    entries = np.frombuffer(raw, dtype=np.int32, count=2 * ne, offset=oe).reshape(ne, 2)
    masks = np.frombuffer(raw, dtype=np.uint32, count=nm, offset=om)
    units = np.frombuffer(raw, dtype=np.int32, count=16 * n_units, offset=o_units).reshape(n_units, 16)
    counters = np.frombuffer(raw, dtype=np.int32, count=n_counters, offset=o_counters)
    sched = np.frombuffer(raw, dtype=np.int32, count=2 if n_units else 0, offset=o_counters + 4 * n_counters)
    return dict(tq=tq, tk=tk, nq=nq, T=T, qt=qt, order=order, entries=entries, masks=masks, wpr=wpr, n_ctas=n_ctas,
                sched=sched, units=units, counters=counters, H=H, Hkv=Hkv, part_slots=part_slots)


def check_schedule(p, info, H, Hkv, n_ctas):
    """The persistent kernel's schedule: every (query tile, head pair, list entry) is covered exactly once, chunks
    of a split list are contiguous and complete, workspace slots and merge counters do not collide, the units
    come in order of decreasing cost, and handing them out in that order to whichever CTA is free first leaves no CTA
    with much more than its share.  A twin unit (two consecutive query tiles sharing the unit of a group's odd
    head) carries the union of the two tiles' lists as entry pairs: each tile's own entries in order, and the
    "none" class with no halves where a tile does not keep the key tile."""
    G = H // Hkv
    ppg = (G + 1) // 2
    n_pairs = Hkv * ppg
    units = p["units"]
    ent = p["entries"]
    assert p["n_ctas"] == n_ctas == info.n_ctas and len(units) == info.n_units
    assert (p["counters"] == 0).all() and (p["sched"] == 0).all()
    by_start = {int(r[0]): r for r in p["qt"]}
    n_own = int(p["qt"][:, 5].sum())                      # the tiles' own lists come first in the entries section
    covered = {}
    chunks = {}
    n_twin = 0
    for u in units:
        q_start, q_rows, req_start, eb, ec, pair, chunk, nch, part_base, counter_base, q_start1, q_rows1 = (int(x) for x in u[:12])
        assert (u[14:] == 0).all()
        qt = by_start[q_start]
        assert q_rows == qt[1] and req_start == qt[2] and 0 <= pair < n_pairs and 0 <= chunk < nch and ec >= 1
        if q_rows1 == 0:
            assert q_start1 == 0 and u[12] == -1 and u[13] == -1
            assert qt[4] <= eb and eb + ec <= qt[4] + qt[5]
            for e in range(eb, eb + ec):
                assert (q_start, pair, e) not in covered
                covered[(q_start, pair, e)] = chunk
            chunks.setdefault((q_start, pair), []).append((chunk, eb, ec, nch, part_base, counter_base))
            continue
        n_twin += 1
        part_base1, counter_base1 = int(u[12]), int(u[13])
        qt1 = by_start[q_start1]
        assert G % 2 == 1 and pair % ppg == ppg - 1
        assert q_rows1 == qt1[1] and req_start == qt1[2] and q_start1 == q_start + q_rows    # the next tile of the request
        assert eb >= n_own and eb + 2 * ec <= len(ent)
        pairs = ent[eb:eb + 2 * ec].reshape(ec, 2, 2)
        kts = pairs[:, 0, 0] >> 4
        assert (kts == pairs[:, 1, 0] >> 4).all() and (np.diff(kts) > 0).all()
        both = set()
        for s, (t, pb, cb) in enumerate(((qt, part_base, counter_base), (qt1, part_base1, counter_base1))):
            first = int(t[4]) + int(t[5]) * chunk // nch                                   # chunk number `chunk` of its own list
            last = int(t[4]) + int(t[5]) * (chunk + 1) // nch
            own = ent[first:last]
            mine = pairs[:, s]
            kept = (mine[:, 0] & 3) != 3
            assert last > first and np.array_equal(mine[kept], own)                        # its own chunk, in order
            assert ((mine[~kept, 0] & 15) == 3).all() and (mine[~kept, 1] == -1).all()     # none: no class, no halves
            for e in range(first, last):
                assert (int(t[0]), pair, e) not in covered
                covered[(int(t[0]), pair, e)] = chunk
            chunks.setdefault((int(t[0]), pair), []).append((chunk, first, last - first, nch, pb, cb))
            both |= set((own[:, 0] >> 4).tolist())
        assert set(kts.tolist()) == both
    assert len(covered) == n_pairs * n_own
    if G % 2 == 0:
        assert n_twin == 0 and len(ent) == n_own
    slots_used, counters_used = set(), set()
    bases = {}
    for (q_start, pair), lst in chunks.items():
        bases.setdefault(q_start, set()).update((c[4], c[5]) for c in lst)
    assert all(len(v) == 1 for v in bases.values())       # every head pair of a tile uses the tile's slots and counters
    for (q_start, pair), lst in chunks.items():
        lst.sort()
        qt = by_start[q_start]
        nch = lst[0][3]
        assert [c[0] for c in lst] == list(range(nch)) and all(c[3] == nch for c in lst)
        assert lst[0][1] == qt[4] and lst[-1][1] + lst[-1][2] == qt[4] + qt[5]
        assert all(a[1] + a[2] == b[1] for a, b in zip(lst, lst[1:]))          # contiguous, in order
        if nch == 1:
            assert lst[0][4] == -1 and lst[0][5] == -1
        else:
            assert len({c[4] for c in lst}) == 1 and len({c[5] for c in lst}) == 1
            if pair == 0:
                for c in range(nch):
                    for hq in range(H):
                        slot = (lst[0][4] + c) * H + hq
                        assert slot not in slots_used and 0 <= slot < p["part_slots"]
                        slots_used.add(slot)
                for hq in range(H):
                    cnt = lst[0][5] + hq
                    assert cnt not in counters_used and 0 <= cnt < len(p["counters"])
                    counters_used.add(cnt)
    assert len(slots_used) == p["part_slots"] and len(counters_used) == len(p["counters"])
    assert info.ws_bytes == p["part_slots"] * (128 * 128 + 256) * 4
    def cost(u):                                          # the scheduler's cost model
        if u[11] == 0:
            e = ent[u[3]:u[3] + u[4], 0]
            both = ((e >> 2) & 3) == 3
            bits = (e & 3) == 2
        else:                                             # a twin unit: the halves and bit masks of either tile
            e = ent[u[3]:u[3] + 2 * u[4], 0].reshape(-1, 2)
            both = (((e[:, 0] | e[:, 1]) >> 2) & 3) == 3
            bits = ((e[:, 0] & 3) == 2) | ((e[:, 1] & 3) == 2)
        c = np.where(both, 2, 1) * np.where(bits, 5, 4)
        return int(c.sum()) + 6 + (14 if u[7] > 1 else 0)
    costs = [cost(u) for u in units]
    assert all(a >= b for a, b in zip(costs, costs[1:]))
    load = np.zeros(n_ctas, dtype=np.int64)               # each unit goes to the CTA that is free first
    for c in costs:
        load[int(load.argmin())] += c
    if len(units) >= 4 * n_ctas:
        assert load.max() <= 1.25 * load.mean() + 40
    return load


def check_plan(batch: inputs.Batch, mask: inputs.STMask, dtype, head_dim, H=4, Hkv=2, n_ctas=0):
    b = pk.Batch(batch.seq_lens, batch.n_prefix, batch.n_frames, device=None)
    buf, info = pk.purekv_plan_build_host(b, pk.st_params(mask), dtype, head_dim, H, Hkv, n_ctas)
    assert pk.purekv_plan_bytes(b, pk.st_params(mask), dtype, head_dim, H, Hkv, n_ctas) == info.bytes_used == len(buf)
    p = parse_plan(buf)
    if info.tile_q == 128:
        check_schedule(p, info, H, Hkv, n_ctas or 148)
    else:
        assert info.n_ctas == 0 and info.n_units == 0 and info.ws_bytes == 0
    tq, tk, wpr = p["tq"], p["tk"], p["wpr"]
    gk = info.tile_k                                  # skip granularity; tk = keys per list entry
    assert tq == info.tile_q and gk == mask.tile and wpr == max(1, tk // 32)
    assert tk == (128 if tq == 128 else gk)
    mp = po.mask_params(mask)
    cu = batch.cu_seqlens
    pairs = kept = full = diag = gen = causal_tiles = 0
    qi = 0
    for r in range(batch.n_req):
        l = batch.seq_lens[r]
        mm = po.mask_matrix(mp, l, batch.n_prefix[r], batch.n_frames[r])
        tril = np.tril(np.ones((l, l), dtype=bool))
        pairs += int(mm.sum())
        for q0 in range(0, l, tq):
            q1 = min(l, q0 + tq)
            row = p["qt"][qi]
            qi += 1
            assert row[0] == cu[r] + q0 and row[1] == q1 - q0 and row[2] == cu[r] and row[3] == l
            ents = p["entries"][row[4]:row[4] + row[5]]
            listed = {int(e[0]) >> 4: ((int(e[0]) >> 2) & 3, int(e[0]) & 3, int(e[1])) for e in ents}
            assert len(listed) == len(ents) and list(listed) == sorted(listed)
            causal_tiles += (q1 - 1) // gk + 1
            for kt in range((q1 - 1) // tk + 1):
                j0, j1 = kt * tk, min(l, kt * tk + tk)
                sub = mm[q0:q1, j0:j1]
                cnt = int(sub.sum())
                # blocks of the skip granularity inside this entry that hold a kept pair
                present = [int(mm[q0:q1, j0 + h * gk:min(l, j0 + (h + 1) * gk)].sum()) > 0 for h in range(tk // gk)]
                kept += sum(present)
                if cnt == 0:
                    assert kt not in listed
                    continue
                hm, cls, at = listed[kt]
                assert hm == (3 if tk == gk else sum(1 << h for h, pr in enumerate(present) if pr))
                if cnt == (q1 - q0) * tk:
                    assert cls == 0 and at == -1
                    full += 1
                elif cnt == int(tril[q0:q1, j0:j1].sum()):
                    assert cls == 1 and at == -1
                    diag += 1
                else:
                    assert cls == 2 and at >= 0
                    gen += 1
                    words = p["masks"][at:at + tq * wpr].reshape(tq, wpr)
                    bits = ((words[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(tq, wpr * 32)[:, :tk].astype(bool)
                    want = np.zeros((tq, tk), dtype=bool)
                    want[:q1 - q0, :j1 - j0] = sub
                    assert np.array_equal(bits, want)           # the mask of Sec. 3.2, bit for bit
    assert qi == p["nq"] == info.n_qtiles
    assert (info.pairs_kept, info.tiles_kept, info.tiles_causal) == (pairs, kept, causal_tiles)
    assert (info.tiles_full, info.tiles_diag, info.tiles_general) == (full, diag, gen)
    order = p["order"]
    assert sorted(order.tolist()) == list(range(p["nq"]))
    counts = p["qt"][order, 5]
    assert (np.diff(counts) <= 0).all()
    return info


@pytest.mark.parametrize("tile", [16, 64])
@pytest.mark.parametrize("mask_kw", [{}, dict(dense_causal=True), dict(anchor_frames=2, spatial_radius=1, temporal_depth=2,
                                                                       temporal_stride=2, temporal_radius=1),
                                     dict(anchor_frames=0, spatial_radius=0, temporal_depth=-1, temporal_radius=-1),
                                     dict(temporal_depth=-1, temporal_stride=3, temporal_radius=0)])
def test_plan_matches_oracle_mask(tile, mask_kw):
    batch = inputs.make_batch([5, 0, 20], [6, 3, 0], [9, 40, 3], 5, 7)
    check_plan(batch, inputs.STMask(5, 7, tile=tile, **mask_kw), pk.FP32, 64)


@pytest.mark.parametrize("tile", [16, 64])
@pytest.mark.parametrize("coarse", [False, True])
@pytest.mark.parametrize("name,kw", [("st", {}), ("spatial", {}), ("temporal", {}), ("local", dict(local_window=9)),
                                     ("atrous", dict(atrous_dilation=5))])
def test_plan_matches_oracle_for_the_named_variants_and_their_block_level_widening(name, kw, coarse, tile):
    """App. A.3 / Table 7 variants: lists, classes and bit masks of the plan against the oracle's mask matrix, for
    the CUDA-core planner shapes and (tile 64) the tensor-core ones."""
    batch = inputs.make_batch([5, 0, 20], [6, 3, 0], [9, 40, 3], 5, 7)
    check_plan(batch, inputs.mask_variant(name, 5, 7, tile=tile, coarse=coarse, **kw), pk.FP32, 64)
    if tile == 64:
        check_plan(batch, inputs.mask_variant(name, 5, 7, tile=tile, coarse=coarse, **kw), pk.BF16, 128, 4, 2, 7)


def test_plan_for_tensor_core_shapes_and_workload_counts():
    batch = inputs.make_batch([64, 3], [5, 2], [64, 130], 12, 12)
    for tile in (64, 128):
        for H, Hkv, n_ctas in ((4, 2, 0), (7, 1, 5), (6, 2, 3), (2, 2, 400), (3, 3, 4), (9, 3, 0)):
            for dense in (False, True):
                info = check_plan(batch, inputs.STMask(12, 12, tile=tile, dense_causal=dense), pk.BF16, 128, H, Hkv, n_ctas)
                assert info.tile_q == 128 and info.tile_k == tile
    # an odd group size: the odd head of consecutive unsplit query tiles shares twin units (none with an even one)
    b = pk.Batch(batch.seq_lens, batch.n_prefix, batch.n_frames, device=None)
    for H, Hkv, want in ((7, 1, True), (3, 3, True), (6, 2, True), (8, 2, False)):
        buf, info = pk.purekv_plan_build_host(b, pk.st_params(inputs.STMask(12, 12, tile=64)), pk.BF16, 128, H, Hkv, 0)
        assert bool((parse_plan(buf)["units"][:, 11] > 0).any()) == want
    # many CTAs and one long request: its lists (text rows see every key) are cut into chunks
    long_batch = inputs.make_batch([4], [40], [20], 12, 12)
    for n_ctas in (0, 400):
        info = check_plan(long_batch, inputs.STMask(12, 12, tile=64), pk.BF16, 128, 2, 2, n_ctas)
        assert info.max_chunks > 1 and info.ws_bytes > 0
    # cfg 0: pair count of the paper's mask (closed form) and the block density quoted for 16-tiles
    wl = inputs.workload(0)
    info = check_plan(wl.batch, wl.mask, pk.FP32, 64)
    assert info.pairs_kept == 29456 and (info.tiles_kept, info.tiles_causal) == (131, 171)


def test_plan_pair_counts_on_the_large_workloads():
    # pairs kept = closed-form pair count of the paper's mask (derived in tests/test_oracle_mask.py)
    for cfg, pairs in [(1, 783264), (2, 4148800), (3, 41042944)]:
        wl = inputs.workload(cfg)
        b = pk.Batch(wl.batch.seq_lens, wl.batch.n_prefix, wl.batch.n_frames, device=None)
        buf, info = pk.purekv_plan_build_host(b, pk.st_params(wl.mask), pk.BF16, 128, wl.n_q_heads, wl.n_kv_heads)
        assert info.pairs_kept == pairs
        assert info.tile_q == 128 and 0 < info.tiles_kept < info.tiles_causal
        load = check_schedule(parse_plan(buf), info, wl.n_q_heads, wl.n_kv_heads, 148)
        assert load.max() <= 1.2 * load.mean() + 40


def test_argument_errors():
    b = pk.Batch([10], [2], [1], device=None)
    with pytest.raises(pk.PureKVError) as e:
        pk.purekv_plan_build_host(b, pk.st_params(inputs.STMask(4, 4)), pk.FP32, 64, 2, 1)     # 2 + 16 > 10
    assert e.value.status == pk.ERR_INVALID_ARG
    b = pk.Batch([30], [2], [1], device=None)
    with pytest.raises(pk.PureKVError) as e:
        pk.purekv_plan_build_host(b, pk.st_params(inputs.STMask(4, 4, tile=48)), pk.FP32, 64, 2, 1)
    assert e.value.status == pk.ERR_UNSUPPORTED
    with pytest.raises(pk.PureKVError):
        pk.purekv_budget(-1, 4, 0.5)


def test_decode_workspace_rule():
    """The decode step needs a workspace exactly when a (request, KV head) is cut into several chunks: never for
    512 kept rows or fewer with a large batch, always for one long request; its size is the chunks' partial results."""
    assert pk.purekv_decode_ws_bytes(300, 512, 8, 2, 128) == 0            # 600 CTAs already, one chunk each
    assert pk.purekv_decode_ws_bytes(300, 513, 8, 2, 128) > 0             # a chunk holds at most 512 rows
    one = pk.purekv_decode_ws_bytes(1, 20000, 28, 4, 128)
    assert one > 0 and (one - 256) % (28 * (128 + 2) * 4) == 0            # n_splits x heads x (d + 2) floats
    n_splits = (one - 256) // (28 * (128 + 2) * 4)
    assert 20000 / 512 <= n_splits <= 20000 / 64 + 1                      # chunks of 64 .. 512 rows
    assert pk.purekv_decode_ws_bytes(1, 20000, 56, 8, 128) <= 2 * one + 256   # more KV heads: fewer chunks each
    for bad in ((0, 10, 8, 2, 128), (4, 0, 8, 2, 128), (4, 10, 0, 2, 128)):
        assert pk.purekv_decode_ws_bytes(*bad) == 0
