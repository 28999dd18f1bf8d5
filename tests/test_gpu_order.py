"""GPU parity of the group-major receive order (Sections 4.3.1, 4.3.2) and of the expert index (Section 2.3.2)
against the oracle: every array and every delivered byte, bit for bit."""
import numpy as np
import pytest

from gpu_util import Guarded, SENTINEL, torch_mod
from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_order(inp, src_rank=-1, max_tokens=None, flags=0):
    torch = torch_mod()
    s = inp.shape
    T, B = inp.T, s.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B, src_rank)
    G, Tn, SD = p.totals["G"], p.totals["T_nonempty"], p.totals["total_dest"]
    gdr, gdo, gm = mwo.group_major(p)
    off, tok, slot, pairs = mwo.expert_index(p, inp.topk_ids, inp.expert_to_rank)
    ids_d = torch.from_numpy(inp.topk_ids).cuda() if T else torch.zeros((0, s.K), dtype=torch.int32, device="cuda")
    e2r_d = torch.from_numpy(inp.expert_to_rank).cuda()
    with mw.Context(s.R, s.E, s.K, max_tokens or max(T, 1), B, src_rank=src_rank, flags=flags) as ctx:
        ctx.mw_plan(ids_d, e2r_d, T)
        rc, view = ctx.mw_group_major()
        got = ctx.group_major_arrays(T, G, view)
        assert np.array_equal(got["group_dest_rank"], gdr)
        assert np.array_equal(got["group_dest_offset"], gdo)
        assert np.array_equal(got["dest_pos_gm"], gm)
        # expert index
        off_d = torch.full((s.E + 1,), -7, dtype=torch.int32, device="cuda")
        tok_d = Guarded(max(T * s.K, 1) * 4)
        slot_d = Guarded(max(T * s.K, 1) * 4)
        ctx.mw_expert_index(ids_d, e2r_d, off_d, tok_d.ptr(), slot_d.ptr())
        torch.cuda.synchronize()
        assert np.array_equal(off_d.cpu().numpy(), off)
        assert np.array_equal(tok_d.host().view(np.int32)[:T * s.K], tok)
        assert np.array_equal(slot_d.host().view(np.int32)[:T * s.K], slot)
        assert tok_d.guards_intact() and slot_d.guards_intact()
        if T == 0 or SD == 0:
            return
        # delivered bytes in group-major order, compact and strided
        x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
        want_send = mwo.pack_mw(p, inp.x)
        counts = np.diff(p.rank_offsets)
        for mode in ("compact", "strided"):
            cap = int(counts.max()) + 1 if mode == "strided" else SD
            stride = cap * B if mode == "strided" else 0
            want = mwo.deliver_group_major(p, want_send, gdr, gdo, stride, SENTINEL)
            send, recv = Guarded(Tn * B), Guarded(len(want))
            ctx.mw_pack(x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)
            ctx.mw_deliver_group_major(send.ptr(), recv.ptr(), stride, cap)
            torch.cuda.synchronize()
            assert ctx.mw_get_totals()["status"] == p.totals["status"]
            assert np.array_equal(recv.host(), want), mode
            assert recv.guards_intact()


@pytest.mark.parametrize("cfg", ["tiny", "decode"])
def test_small_configurations(cfg):
    run_order(wl.make_dispatch(cfg))


@pytest.mark.parametrize("cfg", ["dsv3_prefill", "large_ep"])
def test_large_configurations_reduced_hidden(cfg):
    run_order(wl.make_dispatch(cfg, H=264))


@pytest.mark.parametrize("flags", [0, mw.MW_FLAG_COPY_BULK])
def test_prefill_shape_full_size(flags):
    run_order(wl.make_dispatch("dsv3_prefill"), flags=flags)


@pytest.mark.parametrize("T", [0, 1, 255, 256, 257, 1025])
def test_token_counts_around_tile_edges(T):
    run_order(wl.make_random_dispatch(T + 5, T=T, K=3, E=40, R=10, H=40, pad_fraction=0.1), max_tokens=1100)


@pytest.mark.parametrize("R,E", [(1, 4), (63, 126), (65, 130), (300, 600), (1024, 2048)])
def test_rank_word_boundaries(R, E):
    run_order(wl.make_random_dispatch(R, T=700, K=4, E=E, R=R, H=16))


def test_maximum_top_k():
    run_order(wl.make_random_dispatch(64, T=600, K=64, E=256, R=128, H=16, pad_fraction=0.05))       # 64 destinations per token


def test_more_tokens_than_one_resident_grid_holds():
    run_order(wl.make_random_dispatch(17, T=40000, K=4, E=64, R=16, H=16, pad_fraction=0.05))


def test_few_large_groups_duplicates_invalid_entries_and_source_rank():
    run_order(wl.make_random_dispatch(5, T=3000, K=1, E=12, R=6, H=16))
    run_order(wl.make_random_dispatch(11, T=2000, K=2, E=4, R=4, H=8, contiguous_map=True))
    inp = wl.make_random_dispatch(7, T=600, K=4, E=24, R=7, H=16, pad_fraction=0.35, distinct=False)
    ids = inp.topk_ids.copy()
    ids[4, 0], ids[5, 1], ids[500, 2] = 24, -2, 1 << 30
    inp.topk_ids = ids
    e2r = inp.expert_to_rank.copy()
    e2r[2], e2r[3] = 7, -1
    inp.expert_to_rank = e2r
    run_order(inp)
    run_order(wl.make_random_dispatch(9, T=500, K=3, E=32, R=8, H=16, contiguous_map=True), src_rank=3)


def test_context_reuse_and_errors():
    torch = torch_mod()
    a = wl.make_random_dispatch(1, T=900, K=3, E=32, R=8, H=16)
    b = wl.make_random_dispatch(2, T=300, K=3, E=32, R=8, H=16, pad_fraction=0.5)
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with mw.Context(8, 32, 3, 900, 32) as ctx:
        assert ctx.mw_group_major(check=False)[0] == mw.MW_ERR_NO_PLAN
        assert ctx.mw_expert_index(buf, buf, buf, buf, buf, check=False) == mw.MW_ERR_NO_PLAN
        for inp in (a, b, a):
            p = mwo.plan(inp.topk_ids, inp.expert_to_rank, 8, 32)
            ids_d, e2r_d = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
            ctx.mw_plan(ids_d, e2r_d, inp.T)
            # a deliver in group-major order needs the arrays of THIS plan
            assert ctx.mw_deliver_group_major(buf, buf, 0, 10, check=False) == mw.MW_ERR_NO_PLAN
            rc, view = ctx.mw_group_major()
            got = ctx.group_major_arrays(inp.T, p.totals["G"], view)
            gdr, gdo, gm = mwo.group_major(p)
            assert np.array_equal(got["group_dest_offset"], gdo) and np.array_equal(got["dest_pos_gm"], gm)
        assert ctx.mw_deliver_group_major(buf.data_ptr() + 8, buf, 0, 10, check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_deliver_group_major(buf, buf, 64, 3, check=False) == mw.MW_ERR_CAPACITY
        assert ctx.mw_expert_index(None, e2r_d, buf, buf, buf, check=False) == mw.MW_ERR_INVALID_ARG
    with mw.Context(8, 20000, 3, 64, 32) as ctx:      # 32 bytes of shared memory per expert: too many experts
        ids = torch.zeros((4, 3), dtype=torch.int32, device="cuda")
        e2r = torch.zeros(20000, dtype=torch.int32, device="cuda")
        ctx.mw_plan(ids, e2r, 4)
        assert ctx.mw_expert_index(ids, e2r, buf, buf, buf, check=False) == mw.MW_ERR_CAPACITY
