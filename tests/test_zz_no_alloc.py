"""purekv_lowlayer_score_noalloc: the score entry point for callers that cannot allocate device memory (all of HBM
already handed to a cache pool, or an allocation would stall the device).  Its scratch is an array inside the
library, shared by every call, so the things to check are that it gives what purekv_lowlayer_score gives -- and what
the CPU oracle gives --, that a second call is not disturbed by what the first one left in the scratch, that it
really allocates nothing, and that problems beyond the scratch are refused before anything is launched.
Collected last (file name) so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from oracle import purekv_oracle as po
from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc

pytestmark = pytest.mark.gpu


def _workload(seed, n_prefix, n_frames, n_suffix, dtype="bf16", heads=(8, 2), d=128, window=24):
    batch = inputs.make_batch(n_prefix, n_frames, n_suffix, 5, 6)
    return inputs.Workload("noalloc", seed, dtype, heads[0], heads[1], d, 1, (0,), (0,), batch,
                           inputs.STMask(5, 6, tile=64), window, 0.3)


def _check(P, wl):
    """The no-allocation call against the workspace call (same kernels, so bit-equal is expected but only the
    score tolerance is required) and against the fp64 oracle; the output tensor is made beforehand and device
    memory is measured around the call."""
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    q, k = gc.upload(x, "q", wl.dtype), gc.upload(x, "k", wl.dtype)
    want = P.purekv_lowlayer_score(q, k, db, wl.window)
    got = torch.full_like(want, float("nan"))
    torch.cuda.synchronize()
    held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
    P.purekv_lowlayer_score_noalloc(q, k, db, wl.window, got)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == held, "the wrapper allocated through torch"
    assert torch.cuda.mem_get_info()[0] == free, "device memory was taken during the call"
    g, w = got.cpu().numpy(), want.cpu().numpy()
    assert np.isfinite(g).all()
    assert gc.score_error(g, w.astype(np.float64)) <= gc.SCORE_RTOL
    ref = po.lowlayer_score(x["q"], x["k"], wl.batch.cu_seqlens, wl.window)
    assert gc.score_error(g, ref) <= gc.SCORE_RTOL, "no-allocation scores against the oracle (Eq. 1-2)"


def test_noalloc_score_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    P = gc.pk()
    # the first call on a device looks up the scratch address (and may load the module lazily): keep it out of the
    # memory measurements below
    warm = _workload(4, [1], [1], [9])
    xw = inputs.make_qkv(warm, 0)
    P.purekv_lowlayer_score_noalloc(gc.upload(xw, "q", "bf16"), gc.upload(xw, "k", "bf16"), gc.device_batch(warm),
                                    warm.window, torch.empty((2, 40), dtype=torch.float32, device="cuda"))
    # two different problems back to back: the second is smaller, so stale entries of the first stay in the scratch
    for seed, shape in ((5, ([7, 0, 3], [6, 4, 1], [40, 29, 70])), (6, ([2, 9], [3, 0], [31, 12]))):
        _check(P, _workload(seed, *shape))


def test_noalloc_score_fp32_rows_on_the_cuda_core_kernels():
    P = gc.pk()
    _check(P, _workload(7, [3, 0], [2, 1], [21, 50], dtype="fp32", heads=(4, 2), d=64, window=16))


def test_noalloc_score_takes_a_whole_prompt_of_the_videollama2_shape():
    """2432 tokens, 32 / 8 heads, window 64: 157 696 scratch values, inside the 262 144 the library holds."""
    P = gc.pk()
    wl = inputs.workload(1)
    assert P.purekv_score_ws_bytes(gc.device_batch(wl), wl.window, wl.n_q_heads) == 157696 * 4 + 256
    _check(P, wl)


def test_noalloc_score_limit_is_exact_and_refusals_launch_nothing():
    P = gc.pk()
    h, w = 8, 64                                   # rows = 512: need = 512 + 1024 * ceil(l / 64) values
    for length, fits in ((255 * 64, True), (255 * 64 + 1, False)):      # 261 632 <= 262 144 < 262 656
        db = P.Batch([length], [0], [0])
        need = (P.purekv_score_ws_bytes(db, w, h) - 256) // 4
        assert (need <= P.NOALLOC_SCORE_MAX_ROWS) == fits
        q = torch.randn((length, h, 64), device="cuda").to(torch.bfloat16)
        k = torch.randn((length, 1, 64), device="cuda").to(torch.bfloat16)
        c = torch.full((1, length), 7.0, dtype=torch.float32, device="cuda")
        if fits:
            P.purekv_lowlayer_score_noalloc(q, k, db, w, c)
            want = P.purekv_lowlayer_score(q, k, db, w)
            torch.cuda.synchronize()
            assert gc.score_error(c.cpu().numpy(), want.cpu().numpy().astype(np.float64)) <= gc.SCORE_RTOL
        else:
            with pytest.raises(P.PureKVError) as e:
                P.purekv_lowlayer_score_noalloc(q, k, db, w, c)
            assert e.value.status == P.ERR_WORKSPACE and str(P.NOALLOC_SCORE_MAX_ROWS) in str(e.value)
            torch.cuda.synchronize()
            assert (c == 7.0).all()                # refused before any launch


def test_noalloc_score_accepts_an_empty_batch_whatever_the_other_arguments():
    P = gc.pk()
    db = P.Batch([], [], [])
    q = torch.zeros((0, 8, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((0, 2, 128), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((2, 0), dtype=torch.float32, device="cuda")
    P.purekv_lowlayer_score_noalloc(q, k, db, 0, c)      # window 0 would be refused for a batch with tokens
