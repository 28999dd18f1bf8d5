"""Planning one batch ahead through one context (mw_plan_next / mw_plan_swap): two different batches are
interleaved, the plan of each is made on the library's own stream while the other is packed and delivered on
the caller's, and everything is compared with the CPU oracle bit for bit."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

from gpu_util import Guarded, assert_plan_equal, torch_mod

pytestmark = pytest.mark.gpu


class Batch:
    def __init__(self, inp, R, B):
        torch = torch_mod()
        self.inp, self.T = inp, inp.T
        self.p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
        self.want_send = mwo.pack_mw(self.p, inp.x)
        self.want_recv = mwo.deliver_mw(self.p, self.want_send)
        self.ids = torch.from_numpy(inp.topk_ids).cuda()
        self.x = torch.from_numpy(inp.x.view(np.int16)).cuda()
        self.Tn, self.SD = self.p.totals["T_nonempty"], self.p.totals["total_dest"]


def make_batches(H):
    # same domain (64 ranks, 256 experts, top-8), different routing and different sizes: one fills the context
    # (16 plan tiles), the other is ragged against the 256-token tiles
    a = wl.make_dispatch("dsv3_prefill", 100, H=H)
    b = wl.make_dispatch("dsv3_prefill", 101, T=2909, H=H)
    s = a.shape
    e2r = torch_mod().from_numpy(a.expert_to_rank).cuda()
    assert np.array_equal(a.expert_to_rank, b.expert_to_rank)
    return s, e2r, [Batch(a, s.R, s.row_bytes), Batch(b, s.R, s.row_bytes)]


@pytest.mark.parametrize("H,prefetch", [(264, False), (264, True), (7168, True)])
def test_two_batches_interleaved_through_one_context(H, prefetch):
    torch = torch_mod()
    s, e2r, batches = make_batches(H)
    B = s.row_bytes
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        assert ctx.mw_plan_swap(check=False) == mw.MW_ERR_NO_PLAN            # nothing outstanding yet
        first = batches[0]
        ctx.mw_plan_next(first.ids, e2r, first.T, first.x if prefetch else None)
        # phase 1: every iteration is checked before the next one is issued
        for i in range(4):
            cur, nxt = batches[i % 2], batches[(i + 1) % 2]
            ctx.mw_plan_swap()
            ctx.mw_plan_next(nxt.ids, e2r, nxt.T, nxt.x if prefetch else None)
            send, recv = Guarded(cur.Tn * B), Guarded(cur.SD * B)
            ctx.mw_pack(cur.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), cur.Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, cur.SD)
            tot = ctx.mw_get_totals()
            assert_plan_equal(ctx.plan_arrays(cur.T), cur.p, tot)
            assert np.array_equal(send.host().reshape(-1, B), cur.want_send)
            assert np.array_equal(recv.host(), cur.want_recv)
            assert send.guards_intact() and recv.guards_intact()
        # phase 2: ten iterations back to back, no host synchronisation in between; outputs checked at the end
        outs = []
        for i in range(4, 14):
            cur, nxt = batches[i % 2], batches[(i + 1) % 2]
            ctx.mw_plan_swap()
            ctx.mw_plan_next(nxt.ids, e2r, nxt.T, nxt.x if prefetch else None)
            send, recv = Guarded(cur.Tn * B), Guarded(cur.SD * B)
            ctx.mw_pack(cur.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), cur.Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, cur.SD)
            outs.append((cur, send, recv))
            if H > 1000 and len(outs) == 3:           # full-size rows: keep the memory bounded
                torch.cuda.synchronize()
                for c, sb, rb in outs:
                    assert torch.equal(sb.body.cpu(), torch.from_numpy(c.want_send).reshape(-1))
                    assert torch.equal(rb.body.cpu(), torch.from_numpy(c.want_recv).reshape(-1))
                    assert sb.guards_intact() and rb.guards_intact()
                outs = []
        torch.cuda.synchronize()
        for c, sb, rb in outs:
            assert np.array_equal(sb.host().reshape(-1, B), c.want_send)
            assert np.array_equal(rb.host(), c.want_recv)
            assert sb.guards_intact() and rb.guards_intact()
        tot = ctx.mw_get_totals()
        assert_plan_equal(ctx.plan_arrays(batches[13 % 2].T), batches[13 % 2].p, tot)
        # the plan still outstanding belongs to the other batch
        ctx.mw_plan_swap()
        assert_plan_equal(ctx.plan_arrays(batches[0].T), batches[0].p, ctx.mw_get_totals())


def test_plan_ahead_mixes_with_the_other_plan_calls():
    """mw_plan / mw_plan_dispatch write the current slot and leave an outstanding mw_plan_next alone; the unicast layout,
    the one-pass dispatch and the group-major arrays follow the slot that is current."""
    torch = torch_mod()
    s, e2r, (a, b) = make_batches(40)
    B = s.row_bytes
    small = wl.make_dispatch("dsv3_prefill", 102, T=200, H=40)
    sm = Batch(small, s.R, B)
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        ctx.mw_plan_next(b.ids, e2r, b.T)
        ctx.mw_plan(a.ids, e2r, a.T)                                       # current slot: a
        assert_plan_equal(ctx.plan_arrays(a.T), a.p, ctx.mw_get_totals())
        send, recv = Guarded(sm.Tn * B), Guarded(sm.SD * B)                # one launch for a small batch, current slot
        ctx.mw_plan_dispatch(sm.ids, e2r, sm.T, sm.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), sm.Tn, recv.ptr(), 0, sm.SD)
        assert_plan_equal(ctx.plan_arrays(sm.T), sm.p, ctx.mw_get_totals())
        assert np.array_equal(recv.host(), sm.want_recv) and recv.guards_intact() and send.guards_intact()
        ctx.mw_plan_swap()                                                 # current slot: b, planned before both of them
        assert_plan_equal(ctx.plan_arrays(b.T), b.p, ctx.mw_get_totals())
        ctx.mw_plan_next(a.ids, e2r, a.T)
        # unicast layout and one-pass dispatch on b while a is being planned
        want_uc = mwo.pack_uc(b.p, b.inp.x)
        send, recv = Guarded(b.SD * B), Guarded(b.SD * B)
        ctx.mw_dispatch(b.x, mw.MW_LAYOUT_UNICAST, send.ptr(), b.SD, recv.ptr(), 0, b.SD)
        assert np.array_equal(send.host().reshape(-1, B), want_uc)
        assert np.array_equal(recv.host(), b.want_recv)
        # group-major arrays belong to the plan they were made from
        _, gview = ctx.mw_group_major()
        gdr, gdo, gm = mwo.group_major(b.p)
        got = ctx.group_major_arrays(b.T, b.p.totals["G"], gview)
        assert np.array_equal(got["group_dest_rank"], gdr) and np.array_equal(got["group_dest_offset"], gdo)
        assert np.array_equal(got["dest_pos_gm"], gm)
        ctx.mw_plan_swap()                                                 # current: a; the arrays above are b's
        buf = torch.zeros(64, dtype=torch.uint8, device="cuda")
        assert ctx.mw_deliver_group_major(buf, buf, 0, 1, check=False) == mw.MW_ERR_NO_PLAN
        assert_plan_equal(ctx.plan_arrays(a.T), a.p, ctx.mw_get_totals())
        # a second mw_plan_next before the swap replaces the outstanding plan
        ctx.mw_plan_next(b.ids, e2r, b.T)
        ctx.mw_plan_next(sm.ids, e2r, sm.T)
        ctx.mw_plan_swap()
        assert_plan_equal(ctx.plan_arrays(sm.T), sm.p, ctx.mw_get_totals())
        assert ctx.mw_plan_swap(check=False) == mw.MW_ERR_NO_PLAN


def test_plan_ahead_large_ep_shape_two_words():
    """128 ranks (two bitmap words), 8192 tokens: 32 plan tiles on the side stream while the copies run."""
    torch = torch_mod()
    a = wl.make_dispatch("large_ep", 100, H=136)
    b = wl.make_dispatch("large_ep", 101, T=5000, H=136)
    s = a.shape
    B = s.row_bytes
    e2r = torch.from_numpy(a.expert_to_rank).cuda()
    batches = [Batch(a, s.R, B), Batch(b, s.R, B)]
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        ctx.mw_plan_next(batches[0].ids, e2r, batches[0].T, batches[0].x)
        outs = []
        for i in range(6):
            cur, nxt = batches[i % 2], batches[(i + 1) % 2]
            ctx.mw_plan_swap()
            ctx.mw_plan_next(nxt.ids, e2r, nxt.T, nxt.x)
            send, recv = Guarded(cur.Tn * B), Guarded(cur.SD * B)
            ctx.mw_pack(cur.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), cur.Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, cur.SD)
            outs.append((cur, send, recv))
        torch.cuda.synchronize()
        for c, sb, rb in outs:
            assert np.array_equal(sb.host().reshape(-1, B), c.want_send)
            assert np.array_equal(rb.host(), c.want_recv)
            assert sb.guards_intact() and rb.guards_intact()
        assert_plan_equal(ctx.plan_arrays(batches[1].T), batches[1].p, ctx.mw_get_totals())


@pytest.mark.parametrize("flags", [mw.MW_FLAG_PLAN_MULTIPASS, mw.MW_FLAG_COPY_BULK | mw.MW_FLAG_NO_OVERLAP])
def test_plan_ahead_with_the_multi_kernel_plan_and_the_bulk_copy_engine(flags):
    torch = torch_mod()
    s, e2r, batches = make_batches(72)
    B = s.row_bytes
    with mw.Context(s.R, s.E, s.K, s.T, B, flags=flags) as ctx:
        ctx.mw_plan_next(batches[0].ids, e2r, batches[0].T)
        outs = []
        for i in range(5):
            cur, nxt = batches[i % 2], batches[(i + 1) % 2]
            ctx.mw_plan_swap()
            ctx.mw_plan_next(nxt.ids, e2r, nxt.T)
            send, recv = Guarded(cur.Tn * B), Guarded(cur.SD * B)
            ctx.mw_pack(cur.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), cur.Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, cur.SD)
            outs.append((cur, send, recv))
        torch.cuda.synchronize()
        for c, sb, rb in outs:
            assert np.array_equal(sb.host().reshape(-1, B), c.want_send)
            assert np.array_equal(rb.host(), c.want_recv)
            assert sb.guards_intact() and rb.guards_intact()
        assert_plan_equal(ctx.plan_arrays(batches[0].T), batches[0].p, ctx.mw_get_totals())


def test_plan_ahead_with_an_empty_batch_and_a_reset_in_between():
    torch = torch_mod()
    s, e2r, (a, b) = make_batches(24)
    B = s.row_bytes
    none = torch.zeros((0, s.K), dtype=torch.int32, device="cuda")
    buf = torch.zeros(1 << 12, dtype=torch.uint8, device="cuda")
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        ctx.mw_plan_next(a.ids, e2r, a.T)
        ctx.mw_plan_swap()
        ctx.mw_plan_next(none, e2r, 0)                                    # an empty batch is a plan like any other
        send, recv = Guarded(a.Tn * B), Guarded(a.SD * B)
        ctx.mw_pack(a.x, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), a.Tn)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, a.SD)
        assert np.array_equal(recv.host(), a.want_recv) and recv.guards_intact()
        ctx.mw_plan_swap()
        tot = ctx.mw_get_totals()
        assert tot["T_nonempty"] == 0 and tot["total_dest"] == 0 and tot["G"] == 0 and tot["status"] == 0
        ctx.mw_pack(buf, mw.MW_LAYOUT_MULTIWRITE, buf, 0)                   # nothing to move
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, buf, buf, 0, 0)
        assert not buf.any()
        # a reset drops an outstanding plan as well
        ctx.mw_plan_next(b.ids, e2r, b.T)
        ctx.mw_reset()
        assert ctx.mw_plan_swap(check=False) == mw.MW_ERR_NO_PLAN
        ctx.mw_plan_next(b.ids, e2r, b.T)
        ctx.mw_plan_swap()
        assert_plan_equal(ctx.plan_arrays(b.T), b.p, ctx.mw_get_totals())
