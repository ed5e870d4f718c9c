"""Failure detection of the tensor-core prefill, in the forms that cannot fault a GPU: a plan that fails the
kernel's own checks is refused with a status code and nothing is read through its bad field, and a wait whose
event never comes gives up at the limit, the CTA drains and the context stays usable."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2510_25600_b200 import inputs
from tests import gpu_common as gc

pytestmark = pytest.mark.gpu


def _workload():
    batch = inputs.make_batch([20, 0], [5, 3], [70, 150], 12, 12)
    return inputs.Workload("failure", 77, "bf16", 8, 2, 128, 1, (0,), (0,), batch, inputs.STMask(12, 12, tile=64), 16, 0.25)


def _host_plan(P, wl, db):
    buf, info = P.purekv_plan_build_host(db, P.st_params(wl.mask), P.BF16, wl.head_dim, wl.n_q_heads, wl.n_kv_heads)
    return np.array(buf, copy=True), info


def _launch(P, wl, db, x, h_plan, info, status, fill=7.0):
    q, k, v = (gc.upload(x, n, "bf16") for n in "qkv")
    out = torch.full_like(q, fill)
    plan = P.Plan(torch.from_numpy(h_plan).cuda(), info)
    P.purekv_st_sparse_prefill(q, k, v, db, plan, out=out, status=status)
    return out


def _header(h_plan):
    return gc.pk().PlanHeaderView.from_buffer(h_plan)


def test_kernel_refuses_a_plan_whose_header_is_wrong_and_leaves_the_output_alone():
    P = gc.pk()
    wl = _workload()
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    good, info = _host_plan(P, wl, db)

    def bad_magic(h):
        _header(h).magic ^= 0x10

    def entries_past_the_end(h):
        _header(h).off_entries = info.bytes_used + 4096

    def more_units_than_there_are(h):
        _header(h).n_units = 1 << 28

    def other_head_count(h):
        _header(h).n_q_heads += 2

    for spoil in (bad_magic, entries_past_the_end, more_units_than_there_are, other_head_count):
        h = good.copy()
        spoil(h)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = _launch(P, wl, db, x, h, info, status)
        with pytest.raises(P.PureKVError) as e:
            P.purekv_poll_status(status)
        assert e.value.status == P.ERR_BAD_PLAN, spoil.__name__
        assert (out.float() == 7.0).all(), "a refused plan must not produce output"
    gc.check_prefill(wl, x)            # the context is intact: a fresh plan runs and matches the oracle


def test_kernel_refuses_units_and_entries_that_point_outside_the_plan():
    P = gc.pk()
    wl = _workload()
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    good, info = _host_plan(P, wl, db)
    hdr = _header(good.copy())
    units = lambda h: h[hdr.off_units:hdr.off_units + hdr.n_units * 4 * P.UNIT_INT32S].view(np.int32).reshape(-1, P.UNIT_INT32S)
    entries = lambda h: h[hdr.off_entries:hdr.off_entries + hdr.n_entries * 8].view(np.int32).reshape(-1, 2)
    general = np.nonzero((entries(good)[:, 0] & 3) == 2)[0]
    assert len(general) > 0, "the workload should have bit-mask tiles"

    def list_beyond_the_entries(h):
        units(h)[0, 3] = hdr.n_entries - 1          # ent_begin; with ent_count >= 1 kept, begin + count may pass the end
        units(h)[0, 4] = 5

    def rows_beyond_the_batch(h):
        units(h)[1, 0] = db.total_tokens            # q_start

    def mask_offset_beyond_the_table(h):
        entries(h)[general[0], 1] = hdr.n_mask_words   # entry.y

    def negative_mask_offset(h):
        entries(h)[general[-1], 1] = -512

    def no_half_present(h):
        entries(h)[0, 0] &= ~0xC

    for spoil in (list_beyond_the_entries, rows_beyond_the_batch, mask_offset_beyond_the_table, negative_mask_offset,
                  no_half_present):
        h = good.copy()
        spoil(h)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        _launch(P, wl, db, x, h, info, status)
        with pytest.raises(P.PureKVError) as e:
            P.purekv_poll_status(status)
        assert e.value.status == P.ERR_BAD_PLAN, spoil.__name__
    gc.check_prefill(wl, x)


def test_a_wait_that_cannot_end_gives_up_at_the_limit_and_the_next_launch_works():
    """A host copy of a good plan gets the test flag that makes every CTA's producer withhold its first K copy: the
    issuing thread's wait for that tile runs into the limit (2 ms here), every role of the CTA leaves, tensor memory
    is freed and the status word says so.  Nothing was in flight for the missing tile, so nothing is left behind."""
    P = gc.pk()
    wl = _workload()
    x = inputs.make_qkv(wl, 0)
    db = gc.device_batch(wl)
    h, info = _host_plan(P, wl, db)
    _header(h).test_flags = 1
    P.purekv_set_wait_limit_ns(2_000_000)
    try:
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        _launch(P, wl, db, x, h, info, status)
        t1.record()
        with pytest.raises(P.PureKVError) as e:
            P.purekv_poll_status(status)
        assert e.value.status == P.ERR_TIMEOUT
        assert t0.elapsed_time(t1) < 1000.0, "the kernel should have given up after a few limits, not hung"
        # the same through the library's own status word (status = NULL): raised, reported once, then clear again
        _launch(P, wl, db, x, h, info, None)
        with pytest.raises(P.PureKVError) as e:
            P.purekv_poll_status(None)
        assert e.value.status == P.ERR_TIMEOUT
        assert P.purekv_poll_status(None) == 0
    finally:
        P.purekv_set_wait_limit_ns(0)
    good, info = _host_plan(P, wl, db)
    out = _launch(P, wl, db, x, good, info, None)          # NULL status again: the word was cleared by the poll
    assert P.purekv_poll_status(None) == 0
    assert torch.isfinite(out.float()).all()
    gc.check_prefill(wl, x)
