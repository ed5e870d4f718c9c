"""GPU parity of purekv_decode_attention (one decode step over the compacted cache) against the oracle, element by
element, over group sizes, ragged and empty requests, one and many chunks per request, both row formats; plus the
keep-ratio-1.0 relation to the dense prefill's last row, taken entirely through the CUDA path."""
import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs

from tests import gpu_common as gc

pytestmark = pytest.mark.gpu


class Kept:
    """The part of a budget the decode call reads: offsets of the kept rows on host and device."""

    def __init__(self, kept):
        self.h_cu_kept = np.concatenate([[0], np.cumsum(kept)]).astype(np.int32)
        self.cu_kept = torch.from_numpy(self.h_cu_kept.copy()).cuda()
        self.total_kept = int(self.h_cu_kept[-1])


def draw(seed, kept, H, Hkv, d, dtype):
    rng = np.random.default_rng(seed)
    k_tot = int(np.sum(kept))
    x = {"q": rng.standard_normal((len(kept), H, d)).astype(np.float32) * 1.5,
         "k": rng.standard_normal((max(k_tot, 1), Hkv, d)).astype(np.float32),
         "v": rng.standard_normal((max(k_tot, 1), Hkv, d)).astype(np.float32)}
    if dtype == "bf16":
        for n in "qkv":
            bits = inputs.f32_to_bf16_bits(x[n])
            x[n + "_bits"], x[n] = bits, inputs.bf16_bits_to_f32(bits)
    return x


def run_and_check(kept, H, Hkv, d, dtype, seed=0):
    P = gc.pk()
    x = draw(seed, kept, H, Hkv, d, dtype)
    kb = Kept(kept)
    q, kc, vc = (gc.upload(x, n, dtype) for n in "qkv")
    lse = torch.full((len(kept), H), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.full_like(q, float("nan"))
    P.purekv_decode_attention(q, kc, vc, kb, out=out, lse=lse)
    torch.cuda.synchronize()
    ref, ref_lse = po.decode(x["q"], x["k"], x["v"], kb.h_cu_kept)
    got, got_lse = gc.to_numpy_f32(out), lse.cpu().numpy()
    assert np.isfinite(got).all()
    err = float(np.abs(got - ref).max()) if got.size else 0.0
    assert err <= gc.ATTN_TOL[dtype], f"decode max abs err {err}"
    has = np.diff(kb.h_cu_kept) > 0
    assert np.all(np.isneginf(got_lse[~has])) and np.all(got[~has] == 0.0)
    if has.any():
        assert float(np.abs(got_lse[has] - ref_lse[has]).max()) <= (2e-3 if dtype == "bf16" else 1e-4)
    return err


@pytest.mark.parametrize("H,Hkv", [(4, 4), (8, 4), (32, 8), (28, 4), (8, 1), (3, 1), (16, 1), (12, 1)])
def test_decode_group_sizes_bf16(H, Hkv):
    run_and_check([0, 1, 5, 64, 130, 700, 2000, 3], H, Hkv, 128, "bf16", seed=H)


def test_decode_fp32_rows():
    run_and_check([9, 0, 257, 1500], 4, 2, 64, "fp32", seed=3)
    run_and_check([33], 7, 1, 64, "fp32", seed=4)


def test_decode_one_long_request_many_chunks():
    # a single request: the kept rows are cut into many chunks and merged by the second kernel
    run_and_check([20011], 28, 4, 128, "bf16", seed=5)


def test_decode_many_requests_one_chunk_each():
    rng = np.random.default_rng(6)
    run_and_check(list(rng.integers(0, 400, size=300)), 8, 2, 128, "bf16", seed=6)


def test_decode_workload_budgets():
    # the kept counts of the benchmark workloads' budgets (one layer of their compact cache)
    for cfg in (1, 2, 4):
        wl = inputs.workload(cfg)
        kept = [po.budget(int(l), wl.window, wl.keep_ratio)[1] for l in wl.batch.seq_lens]
        run_and_check(kept, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, seed=10 + cfg)


def test_decode_extreme_logits():
    # logits of several hundred either way: the chunk maxima and the merge must carry the range
    P = gc.pk()
    x = draw(7, [900, 40], 8, 2, 128, "bf16")
    x["q"] = x["q"] * 30.0
    bits = inputs.f32_to_bf16_bits(x["q"])
    x["q_bits"], x["q"] = bits, inputs.bf16_bits_to_f32(bits)
    x["v"] = x["v"] * 0.5          # nearly one-hot weights: keep the outputs below 4, where bf16 steps are 2^-6
    bits = inputs.f32_to_bf16_bits(x["v"])
    x["v_bits"], x["v"] = bits, inputs.bf16_bits_to_f32(bits)
    kb = Kept([900, 40])
    q, kc, vc = (gc.upload(x, n, "bf16") for n in "qkv")
    out = P.purekv_decode_attention(q, kc, vc, kb)
    ref, _ = po.decode(x["q"], x["k"], x["v"], kb.h_cu_kept)
    assert float(np.abs(gc.to_numpy_f32(out) - ref).max()) <= gc.ATTN_TOL["bf16"]


def test_decode_at_keep_one_repeats_the_dense_prefill_last_row():
    """Prefill (dense causal), scores, selection at keep ratio 1.0, compaction and the decode step, all on the GPU:
    the step's output for each request's last query equals that query's row of the prefill."""
    P = gc.pk()
    b = inputs.make_batch([5, 0, 9], [3, 2, 1], [40, 130, 7], 6, 7)
    H, Hkv, d, w = 8, 2, 128, 16
    wl = inputs.Workload("t", 0, "bf16", H, Hkv, d, 1, (0,), (0,), b, inputs.STMask(6, 7, tile=64, dense_causal=True), w, 1.0)
    x = inputs.make_qkv(wl, 0)
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    db = gc.device_batch(wl)
    plan = P.purekv_plan_build(db, P.st_params(wl.mask), P.BF16, d, H, Hkv)
    o = P.purekv_st_sparse_prefill(q, k, v, db, plan)
    bud = P.Budget(db, w, 1.0)
    c = P.purekv_lowlayer_score(q, k, db, w)
    idx = P.purekv_select_topk(c, v[None], db, bud)
    kc, vc = P.purekv_compact_kv(k[None], v[None], idx, db, bud)
    last = torch.tensor([int(e) - 1 for e in b.cu_seqlens[1:]], device="cuda")
    step = P.purekv_decode_attention(q[last].contiguous(), kc[0], vc[0], bud)
    torch.cuda.synchronize()
    assert bud.total_kept == b.total_tokens
    diff = (step.float() - o[last].float()).abs().max().item()
    assert diff <= 2 * gc.ATTN_TOL["bf16"], diff          # two bf16 paths against each other
    ref, _ = po.decode(x["q"][last.cpu().numpy()], x["k"], x["v"], bud.h_cu_kept)   # and against the oracle
    assert float(np.abs(gc.to_numpy_f32(step) - ref).max()) <= gc.ATTN_TOL["bf16"]


def test_decode_rejects_unsupported_shapes():
    P = gc.pk()
    kb = Kept([4])
    q = torch.zeros((1, 17, 128), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((4, 1, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.PureKVError):                      # 17 query heads per KV head
        P.purekv_decode_attention(q, kc, kc, kb)
    q = torch.zeros((1, 2, 64), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((4, 1, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.PureKVError):                      # 128-byte rows
        P.purekv_decode_attention(q, kc, kc, kb)
    q = torch.zeros((1, 3, 128), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((4, 2, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.PureKVError):                      # heads not a multiple of KV heads
        P.purekv_decode_attention(q, kc, kc, kb)
    assert P.purekv_decode_ws_bytes(0, 0, 8, 2, 128) == 0
