"""purekv_lowlayer_score_noalloc: the score entry point for callers that cannot allocate device memory (all of HBM
already handed to a cache pool, or an allocation would stall the device).  Its scratch is an array inside the
library, shared by every call, so the things to check are that it gives what purekv_lowlayer_score gives, that a
second call is not disturbed by what the first one left in the scratch, and that oversized problems are refused.
Collected last (file name) so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc

pytestmark = pytest.mark.gpu


def _workload(seed, n_prefix, n_frames, n_suffix):
    batch = inputs.make_batch(n_prefix, n_frames, n_suffix, 5, 6)
    return inputs.Workload("noalloc", seed, "bf16", 8, 2, 128, 1, (0,), (0,), batch, inputs.STMask(5, 6, tile=64), 24, 0.3)


def test_noalloc_score_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    P = gc.pk()
    # two different problems back to back: the second is smaller, so stale entries of the first stay in the scratch
    for seed, shape in ((5, ([7, 0, 3], [6, 4, 1], [40, 29, 70])), (6, ([2, 9], [3, 0], [31, 12]))):
        wl = _workload(seed, *shape)
        x = inputs.make_qkv(wl, 0)
        db = gc.device_batch(wl)
        q, k = gc.upload(x, "q", "bf16"), gc.upload(x, "k", "bf16")
        want = P.purekv_lowlayer_score(q, k, db, wl.window)
        got = torch.full_like(want, float("nan"))
        P.purekv_lowlayer_score_noalloc(q, k, db, wl.window, got)
        torch.cuda.synchronize()
        g, w = got.cpu().numpy(), want.cpu().numpy()
        assert np.isfinite(g).all()
        assert gc.score_error(g, w.astype(np.float64)) <= gc.SCORE_RTOL


def test_noalloc_score_refuses_problems_beyond_its_scratch():
    P = gc.pk()
    db = P.Batch([600], [0], [0])
    q = torch.zeros((600, 256, 64), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((600, 1, 64), dtype=torch.bfloat16, device="cuda")
    c = torch.full((1, 600), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(P.PureKVError) as e:                     # 1 * 256 * 512 rows > 65536
        P.purekv_lowlayer_score_noalloc(q, k, db, 512, c)
    assert e.value.status == P.ERR_WORKSPACE and "65536" in str(e.value)
    torch.cuda.synchronize()
    assert (c == 7.0).all()                                      # refused before any launch
