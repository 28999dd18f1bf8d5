"""The give-up paths of the bounded device-side waits, and recovery with mw_reset.

Nothing here faults, traps or hangs a GPU: a test hook makes a wait look for something nobody provides (predecessor
records of another epoch, one grid-barrier arrival more than there are blocks, sixteen bytes more than a load delivers)
and the context is created with wait limits of about a millisecond, so the wait simply runs out.  Expected every time:
MW_ERR_TIMEOUT in the accounting, the kernels that follow skip their work (outputs and guard bands keep their
sentinel), the context refuses further work, and after mw_reset the same context plans and dispatches bit for bit again.
"""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

from gpu_util import Guarded, SENTINEL, assert_plan_equal, torch_mod

pytestmark = pytest.mark.gpu


def setup(T=1500, H=72, R=64, E=256, K=8):
    torch = torch_mod()
    inp = wl.make_random_dispatch(7, T=T, K=K, E=E, R=R, H=H, pad_fraction=0.05)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, inp.shape.row_bytes)
    ids = torch.from_numpy(inp.topk_ids).cuda()
    e2r = torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    return inp, p, ids, e2r, x


def dispatch_and_check(ctx, inp, p, ids, e2r, x):
    """A whole plan + pack + deliver on the context, compared with the oracle."""
    B = inp.shape.row_bytes
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    ctx.mw_plan(ids, e2r, inp.T)
    send, recv = Guarded(Tn * B), Guarded(SD * B)
    ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)
    ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, SD)
    tot = ctx.mw_get_totals()
    assert_plan_equal(ctx.plan_arrays(inp.T), p, tot)
    want_send = mwo.pack_mw(p, inp.x)
    assert np.array_equal(send.host().reshape(-1, B), want_send)
    assert np.array_equal(recv.host(), mwo.deliver_mw(p, want_send))
    assert send.guards_intact() and recv.guards_intact()


def untouched(buf: Guarded) -> bool:
    return bool((buf.body == SENTINEL).all()) and buf.guards_intact()


@pytest.mark.parametrize("what,flags", [(mw.MW_TEST_SKEW_LOOKBACK, 0), (mw.MW_TEST_SKEW_BARRIER, 0),
                                        (mw.MW_TEST_SKEW_LOOKBACK, mw.MW_FLAG_PLAN_MULTIPASS)])
def test_plan_wait_runs_out_then_reset_recovers(what, flags):
    torch = torch_mod()
    inp, p, ids, e2r, x = setup()
    B = inp.shape.row_bytes
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    with mw.Context(64, 256, 8, 2000, B, flags=flags | mw.MW_FLAG_SHORT_WAITS) as ctx:
        dispatch_and_check(ctx, inp, p, ids, e2r, x)                       # a good plan first: the scratch is in use
        ctx.mw_test_skew_waits(what)
        ctx.mw_plan(ids, e2r, inp.T)                                       # six tiles; every wait of this plan runs out
        send, recv, y = Guarded(Tn * B), Guarded(SD * B), Guarded(inp.T * B)
        ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)            # issued before the host has seen the status:
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, SD)   # the kernels themselves must skip the work
        ctx.mw_combine(recv.ptr(), 0, None, y.ptr())
        ctx.mw_plan(ids, e2r, inp.T)                                       # a later plan refuses on the device as well
        ctx.mw_dispatch(x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn, recv.ptr(), 0, SD)
        tot = ctx.mw_get_totals()
        assert tot["status"] == mw.MW_ERR_TIMEOUT
        assert untouched(send) and untouched(recv) and untouched(y)
        # from here on the context refuses work until it is reset
        assert ctx.mw_plan(ids, e2r, inp.T, check=False) == mw.MW_ERR_TIMEOUT
        assert ctx.mw_plan_next(ids, e2r, inp.T, check=False) == mw.MW_ERR_TIMEOUT
        assert ctx.mw_pack(x, 0, send.ptr(), Tn, check=False) == mw.MW_ERR_TIMEOUT
        assert ctx.mw_deliver(0, send.ptr(), recv.ptr(), 0, SD, check=False) == mw.MW_ERR_TIMEOUT
        assert ctx.mw_combine(recv.ptr(), 0, None, y.ptr(), check=False) == mw.MW_ERR_TIMEOUT
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_TIMEOUT           # still readable
        ctx.mw_reset()
        assert ctx.mw_pack(x, 0, send.ptr(), Tn, check=False) == mw.MW_ERR_NO_PLAN    # no plan survives a reset
        for _ in range(2):
            dispatch_and_check(ctx, inp, p, ids, e2r, x)
        # and the plan-ahead pair works on the reset context too
        ctx.mw_plan_next(ids, e2r, inp.T)
        ctx.mw_plan_swap()
        assert_plan_equal(ctx.plan_arrays(inp.T), p, ctx.mw_get_totals())


def test_plan_ahead_wait_runs_out_current_batch_unharmed():
    """The plan made ahead gives up; the batch in flight (other slot) is delivered correctly, the swapped-in plan reports it."""
    inp, p, ids, e2r, x = setup()
    B = inp.shape.row_bytes
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    with mw.Context(64, 256, 8, 2000, B, flags=mw.MW_FLAG_SHORT_WAITS) as ctx:
        ctx.mw_plan(ids, e2r, inp.T)
        ctx.mw_test_skew_waits(mw.MW_TEST_SKEW_BARRIER)
        ctx.mw_plan_next(ids, e2r, inp.T)
        send, recv = Guarded(Tn * B), Guarded(SD * B)
        ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, SD)
        assert ctx.mw_get_totals()["status"] == 0
        assert np.array_equal(recv.host(), mwo.deliver_mw(p, mwo.pack_mw(p, inp.x))) and recv.guards_intact()
        ctx.mw_plan_swap()
        recv2 = Guarded(SD * B)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv2.ptr(), 0, SD)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_TIMEOUT
        assert untouched(recv2)
        ctx.mw_reset()
        dispatch_and_check(ctx, inp, p, ids, e2r, x)


def test_bulk_copy_wait_runs_out_then_reset_recovers():
    inp, p, ids, e2r, x = setup(T=1200, H=520)
    B = inp.shape.row_bytes
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    with mw.Context(64, 256, 8, 2000, B, flags=mw.MW_FLAG_COPY_BULK | mw.MW_FLAG_SHORT_WAITS) as ctx:
        dispatch_and_check(ctx, inp, p, ids, e2r, x)
        send, recv = Guarded(Tn * B), Guarded(SD * B)
        ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)
        ctx.mw_test_skew_waits(mw.MW_TEST_SKEW_BULK_LOAD)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, SD)       # no stage of any pipeline completes
        recv2 = Guarded(SD * B)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv2.ptr(), 0, SD)      # skipped: the status is already set
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_TIMEOUT
        assert untouched(recv) and untouched(recv2)
        assert np.array_equal(send.host().reshape(-1, B), mwo.pack_mw(p, inp.x))      # the pack before it was not affected
        assert ctx.mw_deliver(0, send.ptr(), recv.ptr(), 0, SD, check=False) == mw.MW_ERR_TIMEOUT
        ctx.mw_reset()
        dispatch_and_check(ctx, inp, p, ids, e2r, x)


def test_group_major_wait_runs_out_then_reset_recovers():
    inp, p, ids, e2r, x = setup()
    B = inp.shape.row_bytes
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    gdr, gdo, gm = mwo.group_major(p)
    with mw.Context(64, 256, 8, 2000, B, flags=mw.MW_FLAG_SHORT_WAITS) as ctx:
        ctx.mw_plan(ids, e2r, inp.T)
        _, view = ctx.mw_group_major()
        got = ctx.group_major_arrays(inp.T, p.totals["G"], view)
        assert np.array_equal(got["group_dest_offset"], gdo) and np.array_equal(got["dest_pos_gm"], gm)
        ctx.mw_test_skew_waits(mw.MW_TEST_SKEW_GROUP_MAJOR)
        ctx.mw_group_major()                                                # tiles after the first wait for records nobody writes
        send, recv = Guarded(Tn * B), Guarded(SD * B)
        ctx.mw_deliver_group_major(send.ptr(), recv.ptr(), 0, SD)           # must skip
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_TIMEOUT
        assert untouched(recv)
        assert ctx.mw_group_major(check=False)[0] == mw.MW_ERR_TIMEOUT
        ctx.mw_reset()
        ctx.mw_plan(ids, e2r, inp.T)
        _, view = ctx.mw_group_major()
        got = ctx.group_major_arrays(inp.T, p.totals["G"], view)
        assert np.array_equal(got["group_dest_rank"], gdr) and np.array_equal(got["group_dest_offset"], gdo)
        assert np.array_equal(got["dest_pos_gm"], gm)
        assert ctx.mw_get_totals()["status"] == 0


def test_reset_on_a_healthy_context_and_argument_checks():
    inp, p, ids, e2r, x = setup(T=300)
    with mw.Context(64, 256, 8, 512, inp.shape.row_bytes) as ctx:
        dispatch_and_check(ctx, inp, p, ids, e2r, x)
        ctx.mw_reset()
        dispatch_and_check(ctx, inp, p, ids, e2r, x)
        with pytest.raises(mw.MwError):
            ctx.mw_test_skew_waits(0x100)
    assert mw.lib().mw_reset(None) == mw.MW_ERR_INVALID_ARG
