"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit.

Metadata arrays are compared whole (including their -1 / 0 tails), payload buffers byte by byte,
with sentinel guard bands around every output buffer.  Integer and data-movement work only, so the
tolerance is zero everywhere.
"""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

from gpu_util import Guarded, SENTINEL, assert_plan_equal, run_dispatch, torch_mod

pytestmark = pytest.mark.gpu


# ---- the four dispatch configurations ----------------------------------------------------------
@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
@pytest.mark.parametrize("seed", [None, 100, 101])
def test_plan_parity_full_configurations(cfg, seed):
    inp = wl.make_dispatch(cfg, seed, payload=False)
    run_dispatch(inp, check_payload=False, repeats=2)


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("cfg", [0, 3])
def test_dispatch_parity_small_configurations_full_size(cfg, separate):
    run_dispatch(wl.make_dispatch(cfg), separate=separate)


@pytest.mark.parametrize("flags,separate", [(0, False), (0, True), (mw.MW_FLAG_COPY_BULK, False)])
@pytest.mark.parametrize("cfg", [1, 2])
def test_dispatch_parity_large_configurations_full_size(cfg, flags, separate):
    # full T and full hidden size, the shapes the benchmark times; compact MultiWrite + strided unicast
    inp = wl.make_dispatch(cfg)
    run_dispatch(inp, layouts=(mw.MW_LAYOUT_MULTIWRITE,), strides=("compact",), flags=flags, separate=separate)
    run_dispatch(inp, layouts=(mw.MW_LAYOUT_UNICAST,), strides=("strided",), flags=flags, separate=separate)


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("cfg", [1, 2])
@pytest.mark.parametrize("seed", [100, 101])
def test_dispatch_parity_large_configurations_reduced_hidden(cfg, seed, separate):
    run_dispatch(wl.make_dispatch(cfg, seed, H=264), separate=separate)          # 528-byte rows: ragged against every tile size


@pytest.mark.parametrize("flags", [mw.MW_FLAG_PLAN_MULTIPASS, mw.MW_FLAG_NO_OVERLAP, mw.MW_FLAG_COPY_BULK, mw.MW_FLAG_SHORT_WAITS,
                                   mw.MW_FLAG_PLAN_MULTIPASS | mw.MW_FLAG_COPY_BULK | mw.MW_FLAG_NO_OVERLAP])
def test_launch_and_plan_variants_match(flags):
    """The multi-pass plan, the non-overlapped launches, the bulk-copy engine and the short wait limits give the
    same bits as the defaults."""
    run_dispatch(wl.make_random_dispatch(41, T=3000, K=1, E=12, R=6, H=16), flags=flags)       # large groups
    run_dispatch(wl.make_dispatch("large_ep", 100, H=264), flags=flags, repeats=2)
    run_dispatch(wl.make_random_dispatch(31, T=1025, K=2, E=12, R=6, H=24, pad_fraction=0.1), flags=flags)
    run_dispatch(wl.make_dispatch("decode", H=64), flags=flags)


def test_maximum_top_k():
    """K = 64 expert slots per token, the largest the library accepts: 64 destinations per token on 128 ranks, and heavy
    per-rank dedup on 8 ranks; fused and multi-kernel plan, separate calls and the one-pass dispatch."""
    assert mw.lib() is not None
    wide = wl.make_random_dispatch(64, T=700, K=64, E=256, R=128, H=24, pad_fraction=0.05)
    run_dispatch(wide, separate=True)
    run_dispatch(wide, flags=mw.MW_FLAG_PLAN_MULTIPASS)
    run_dispatch(wl.make_random_dispatch(65, T=900, K=64, E=64, R=8, H=24, distinct=False), one_call=True)


# ---- edge cases ------------------------------------------------------------------------------------
@pytest.mark.parametrize("R", [1, 2, 63, 64, 65, 128, 129, 256, 1000, 1024])
def test_rank_word_boundaries(R):
    E = R if R > 8 else 8 * R
    inp = wl.make_random_dispatch(R, T=300, K=min(6, R), E=E, R=R, H=24, pad_fraction=0.1)
    ids = inp.topk_ids.copy()
    e2r = inp.expert_to_rank.copy()
    e2r[0], e2r[1] = 0, R - 1
    ids[0, 0], ids[0, -1] = 0, 1                                   # first and last rank in one token
    inp.topk_ids, inp.expert_to_rank = ids, e2r
    run_dispatch(inp)


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("T", [0, 1, 31, 255, 256, 257, 1000, 1025])
def test_token_counts_around_tile_edges(T, separate):
    inp = wl.make_random_dispatch(T + 3, T=T, K=3, E=40, R=10, H=40)
    run_dispatch(inp, max_tokens=1100, separate=separate)


def test_more_tokens_than_one_resident_grid_holds():
    # 40000 tokens = 157 tiles, more than the SMs of a B200: the plan takes its three-kernel route by itself
    inp = wl.make_random_dispatch(17, T=40000, K=4, E=64, R=16, H=16, pad_fraction=0.05)
    p, tot = run_dispatch(inp)
    assert tot["T_nonempty"] > 39000 and tot["G"] > 1000
    run_dispatch(inp, layouts=(mw.MW_LAYOUT_MULTIWRITE,), strides=("compact",), separate=True)


def test_top1_and_few_large_groups():
    # every token in a large group: exercises member ranking inside groups across tiles
    inp = wl.make_random_dispatch(5, T=3000, K=1, E=12, R=6, H=16)
    p, tot = run_dispatch(inp)
    assert tot["G"] <= 6 and tot["mw_bytes"] == tot["unicast_bytes"]
    inp = wl.make_random_dispatch(6, T=2500, K=2, E=8, R=4, H=16)
    p, tot = run_dispatch(inp)
    assert tot["G"] <= 10


def test_all_tokens_identical_and_all_distinct():
    T, R = 700, 70
    e2r = np.arange(R, dtype=np.int32)
    same = wl.make_random_dispatch(1, T=T, K=3, E=R, R=R, H=16)
    same.expert_to_rank = e2r
    same.topk_ids = np.tile(np.array([[3, 66, 9]], np.int32), (T, 1))
    p, tot = run_dispatch(same)
    assert tot["G"] == 1
    dist = wl.make_random_dispatch(2, T=R, K=2, E=R, R=R, H=16)
    dist.expert_to_rank = e2r
    dist.topk_ids = np.stack([np.arange(R), (np.arange(R) + 1) % R], 1).astype(np.int32)
    p, tot = run_dispatch(dist)
    assert tot["G"] == R


def test_padding_empty_tokens_duplicates_and_invalid_ids():
    inp = wl.make_random_dispatch(7, T=600, K=4, E=24, R=7, H=16, pad_fraction=0.35, distinct=False)
    ids = inp.topk_ids.copy()
    ids[3, :] = -1
    ids[299, :] = -1
    ids[6, :] = ids[6, 0]
    inp.topk_ids = ids
    p, tot = run_dispatch(inp)
    assert tot["status"] == 0 and tot["T_nonempty"] < 600
    ids[4, 0] = 24                 # == E
    ids[5, 1] = -2                 # negative, not the padding value
    ids[500, 2] = 1 << 30
    inp.topk_ids = ids
    p, tot = run_dispatch(inp)
    assert tot["status"] == mw.MW_ERR_BAD_INDEX
    e2r = inp.expert_to_rank.copy()
    e2r[2] = 7                     # == R
    e2r[3] = -1
    inp.expert_to_rank = e2r
    p, tot = run_dispatch(inp)
    assert tot["status"] == mw.MW_ERR_BAD_INDEX


def test_all_padding_batch():
    inp = wl.make_random_dispatch(9, T=300, K=4, E=16, R=4, H=16)
    inp.topk_ids = np.full_like(inp.topk_ids, -1)
    p, tot = run_dispatch(inp)
    assert tot["G"] == 0 and tot["total_dest"] == 0 and tot["mw_bytes"] == 0


def test_source_rank_inside_domain():
    inp = wl.make_random_dispatch(11, T=500, K=3, E=16, R=6, H=16)
    p, tot = run_dispatch(inp, src_rank=2)
    q = mwo.plan(inp.topk_ids, inp.expert_to_rank, 6, 32, -1)
    assert tot["unicast_bytes"] < q.totals["unicast_bytes"]


def test_context_reuse_with_changing_batches_is_stateless():
    """One context, many plans of different sizes: each result depends only on its own inputs."""
    torch = torch_mod()
    R, E, K, H = 16, 64, 4, 16
    with mw.Context(R, E, K, 2048, 2 * H) as ctx:
        for seed, T in [(1, 2048), (2, 5), (3, 777), (4, 0), (5, 2047), (1, 2048)]:
            inp = wl.make_random_dispatch(seed, T=T, K=K, E=E, R=R, H=H, contiguous_map=True)
            p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, 2 * H)
            ids_d = torch.from_numpy(inp.topk_ids).cuda()
            e2r_d = torch.from_numpy(inp.expert_to_rank).cuda()
            ctx.mw_plan(ids_d, e2r_d, T)
            assert_plan_equal(ctx.plan_arrays(T), p, ctx.mw_get_totals())


def test_two_runs_give_identical_bytes():
    torch = torch_mod()
    inp = wl.make_dispatch("tiny")
    s = inp.shape
    outs = []
    for _ in range(2):
        with mw.Context(s.R, s.E, s.K, s.T, s.row_bytes) as ctx:
            ids_d, e2r_d = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
            x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
            ctx.mw_plan(ids_d, e2r_d, s.T)
            tot = ctx.mw_get_totals()
            send = torch.zeros(tot["T_nonempty"] * s.row_bytes, dtype=torch.uint8, device="cuda")
            recv = torch.zeros(tot["total_dest"] * s.row_bytes, dtype=torch.uint8, device="cuda")
            ctx.mw_dispatch(x_d, mw.MW_LAYOUT_MULTIWRITE, send, tot["T_nonempty"], recv, 0, tot["total_dest"])
            torch.cuda.synchronize()
            outs.append((send.cpu().numpy(), recv.cpu().numpy(), ctx.plan_arrays(s.T)))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    for k in outs[0][2]:
        assert np.array_equal(outs[0][2][k], outs[1][2][k])


def test_nan_and_negative_zero_payload_round_trips():
    inp = wl.make_random_dispatch(3, T=64, K=2, E=8, R=4, H=16)
    x = inp.x.copy()
    x[0, :] = 0x7FC1      # NaN with payload
    x[1, :] = 0x8000      # -0
    x[2, :] = 0xFFFF
    inp.x = x
    run_dispatch(inp)


def test_large_batch_with_many_empty_tokens():
    """9000 tokens of 8 KB rows (a send buffer beyond half of L2), more than half of the expert slots padding: the
    number of send rows is far below the host-side bound the launches are sized from."""
    inp = wl.make_random_dispatch(77, T=9000, K=4, E=64, R=32, H=4096, pad_fraction=0.55)
    run_dispatch(inp, layouts=(mw.MW_LAYOUT_MULTIWRITE,), strides=("compact", "strided"))


# ---- planning with the hidden rows prefetched into L2 -------------------------------------------------
@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
def test_plan_prefetch_gives_the_same_plan_and_payload(cfg):
    # full size: the large_ep rows (117 MB) exceed the half of L2 the prefetch is limited to
    run_dispatch(wl.make_dispatch(cfg), layouts=(mw.MW_LAYOUT_MULTIWRITE,), strides=("compact",), separate=True, prefetch=True,
                 repeats=2)


@pytest.mark.parametrize("T", [0, 1, 255, 257, 1025])
def test_plan_prefetch_token_counts(T):
    inp = wl.make_random_dispatch(T + 3, T=T, K=3, E=40, R=10, H=40, pad_fraction=0.1)
    run_dispatch(inp, max_tokens=1100, prefetch=True)


def test_plan_prefetch_argument_errors():
    torch = torch_mod()
    inp = wl.make_random_dispatch(5, T=64, K=2, E=8, R=4, H=16)
    ids = torch.from_numpy(inp.topk_ids).cuda()
    e2r = torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    with mw.Context(4, 8, 2, 64, 32) as ctx:
        assert ctx.mw_plan_prefetch(ids, e2r, 64, None, check=False) == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_plan_prefetch(ids, e2r, 64, x.data_ptr() + 8, check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_plan_prefetch(ids, e2r, 65, x, check=False) == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_plan_prefetch(ids, e2r, 64, x, check=False) == mw.MW_OK
        torch.cuda.synchronize()


# ---- plan + dispatch in one call (single-launch path for small batches) ----------------------------
@pytest.mark.parametrize("cfg,H", [("decode", None), ("tiny", None), ("decode", 72)])
def test_one_call_small_batches_match(cfg, H):
    run_dispatch(wl.make_dispatch(cfg, H=H), one_call=True, repeats=1)
    run_dispatch(wl.make_dispatch(cfg, 100, H=H), one_call=True)


@pytest.mark.parametrize("T", [0, 1, 31, 128, 129, 255, 256, 257, 600, 1023, 1024, 1025, 1500])
def test_one_call_token_counts(T):
    # up to 128 tokens the single launch with 256 threads per block, up to 1024 tokens the one with 1024 threads,
    # beyond that the three-kernel route: same results
    inp = wl.make_random_dispatch(T + 11, T=T, K=3, E=40, R=10, H=40, pad_fraction=0.1)
    run_dispatch(inp, one_call=True, max_tokens=1600)


@pytest.mark.parametrize("cfg,T,H", [("dsv3_prefill", 1024, 72), ("dsv3_prefill", 700, None), ("large_ep", 1000, 40), ("decode", 1024, 24)])
def test_one_call_wide_variant_on_the_configurations_routing(cfg, T, H):
    # one bitmap word (64 ranks), two (128) and four (256); 700 tokens of full-size rows
    run_dispatch(wl.make_dispatch(cfg, 100, T=T, H=H), one_call=True)


def test_one_call_wide_variant_groups_and_sixteen_destinations():
    run_dispatch(wl.make_random_dispatch(21, T=1000, K=2, E=8, R=4, H=16), one_call=True)                 # few groups of hundreds
    run_dispatch(wl.make_random_dispatch(22, T=900, K=16, E=64, R=32, H=16, pad_fraction=0.2), one_call=True, src_rank=5)


def test_one_call_groups_padding_invalid_ids_and_source_rank():
    same = wl.make_random_dispatch(1, T=200, K=2, E=8, R=4, H=16)            # few, large groups
    run_dispatch(same, one_call=True)
    inp = wl.make_random_dispatch(7, T=250, K=4, E=24, R=7, H=16, pad_fraction=0.35, distinct=False)
    ids = inp.topk_ids.copy()
    ids[3, :] = -1
    ids[4, 0] = 24
    ids[5, 1] = -2
    inp.topk_ids = ids
    p, tot = run_dispatch(inp, one_call=True)
    assert tot["status"] == mw.MW_ERR_BAD_INDEX
    run_dispatch(wl.make_random_dispatch(11, T=180, K=3, E=16, R=6, H=16), one_call=True, src_rank=2)
    wide = wl.make_random_dispatch(12, T=256, K=8, E=512, R=256, H=24)       # four bitmap words
    run_dispatch(wide, one_call=True)
    big_k = wl.make_random_dispatch(13, T=100, K=20, E=64, R=64, H=16)       # more than 16 destinations: falls back
    run_dispatch(big_k, one_call=True)


def test_one_call_replays_from_a_cuda_graph():
    """The single-launch path keeps no host-side state, so a captured call can be replayed: the same graph is run
    on two different batches written into the same device buffers and checked against the oracle both times."""
    torch = torch_mod()
    a, b = wl.make_dispatch("decode"), wl.make_dispatch("decode", 100)
    s = a.shape
    T, B = a.T, s.row_bytes
    ids_d = torch.from_numpy(a.topk_ids).cuda()
    e2r_d = torch.from_numpy(a.expert_to_rank).cuda()
    x_d = torch.from_numpy(a.x.view(np.int16)).cuda()
    plans = [mwo.plan(i.topk_ids, i.expert_to_rank, s.R, B) for i in (a, b)]
    Tn = max(p.totals["T_nonempty"] for p in plans)
    SD = max(p.totals["total_dest"] for p in plans)
    send, recv = Guarded(Tn * B), Guarded(SD * B)
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan_dispatch(ids_d, e2r_d, T, x_d.data_ptr(), mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn, recv.ptr(), 0, SD)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.mw_plan_dispatch(ids_d, e2r_d, T, x_d.data_ptr(), mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn, recv.ptr(), 0, SD)
        for inp, p in ((a, plans[0]), (b, plans[1]), (a, plans[0])):
            ids_d.copy_(torch.from_numpy(inp.topk_ids))
            x_d.copy_(torch.from_numpy(inp.x.view(np.int16)))
            send.body.fill_(SENTINEL)
            recv.body.fill_(SENTINEL)
            graph.replay()
            torch.cuda.synchronize()
            assert_plan_equal(ctx.plan_arrays(T), p, ctx.mw_get_totals())
            want_send = mwo.pack_mw(p, inp.x)
            n_send, n_recv = p.totals["T_nonempty"] * B, p.totals["total_dest"] * B
            assert np.array_equal(send.host()[:n_send].reshape(-1, B), want_send)
            assert np.array_equal(recv.host()[:n_recv], mwo.deliver_mw(p, want_send, 0, SENTINEL))
            assert (send.host()[n_send:] == SENTINEL).all() and (recv.host()[n_recv:] == SENTINEL).all()
            assert send.guards_intact() and recv.guards_intact()


@pytest.mark.parametrize("flags,prefetch", [(0, True), (0, False), (mw.MW_FLAG_PLAN_MULTIPASS, False)])
def test_three_call_step_replays_from_a_cuda_graph(flags, prefetch):
    """The tiled plan keeps its running counts (epoch of the look-back records, barrier arrivals, tile tickets) on the
    device, so a captured plan + pack + deliver can be replayed: one graph, three different batches in the same buffers,
    ordinary calls in between."""
    torch = torch_mod()
    batches = [wl.make_dispatch("dsv3_prefill", seed, T=1500, H=72) for seed in (100, 101, 102)]
    s = batches[0].shape
    T, B = 1500, s.row_bytes
    ids_d = torch.from_numpy(batches[0].topk_ids).cuda()
    e2r_d = torch.from_numpy(batches[0].expert_to_rank).cuda()
    x_d = torch.from_numpy(batches[0].x.view(np.int16)).cuda()
    plans = [mwo.plan(i.topk_ids, i.expert_to_rank, s.R, B) for i in batches]
    Tn = max(p.totals["T_nonempty"] for p in plans)
    SD = max(p.totals["total_dest"] for p in plans)
    send, recv = Guarded(Tn * B), Guarded(SD * B)

    def step(ctx):
        if prefetch:
            ctx.mw_plan_prefetch(ids_d, e2r_d, T, x_d)
        else:
            ctx.mw_plan(ids_d, e2r_d, T)
        ctx.mw_pack(x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, SD)

    with mw.Context(s.R, s.E, s.K, 2000, B, flags=flags) as ctx:
        step(ctx)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(ctx)
        for k, (inp, p) in enumerate(zip(batches + batches[:1], plans + plans[:1])):
            ids_d.copy_(torch.from_numpy(inp.topk_ids))
            x_d.copy_(torch.from_numpy(inp.x.view(np.int16)))
            send.body.fill_(SENTINEL)
            recv.body.fill_(SENTINEL)
            if k == 2:
                step(ctx)                     # an ordinary call between two replays
            graph.replay()
            graph.replay()                    # twice in a row: the counts advance on the device
            torch.cuda.synchronize()
            assert_plan_equal(ctx.plan_arrays(T), p, ctx.mw_get_totals())
            want_send = mwo.pack_mw(p, inp.x)
            n_send, n_recv = p.totals["T_nonempty"] * B, p.totals["total_dest"] * B
            assert np.array_equal(send.host()[:n_send].reshape(-1, B), want_send)
            assert np.array_equal(recv.host()[:n_recv], mwo.deliver_mw(p, want_send, 0, SENTINEL))
            assert (send.host()[n_send:] == SENTINEL).all() and (recv.host()[n_recv:] == SENTINEL).all()
            assert send.guards_intact() and recv.guards_intact()


def test_one_call_capacity_overflow_is_reported_and_contained():
    torch = torch_mod()
    inp = wl.make_random_dispatch(21, T=200, K=3, E=32, R=8, H=16, contiguous_map=True)
    s = inp.shape
    B = s.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B)
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    ids_d, e2r_d = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
    want_send = mwo.pack_mw(p, inp.x)
    want_recv = mwo.deliver_mw(p, want_send)
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        send, recv = Guarded((Tn - 1) * B), Guarded((SD - 10) * B)
        ctx.mw_plan_dispatch(ids_d, e2r_d, s.T, x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn - 1, recv.ptr(), 0, SD - 10)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_CAPACITY
        assert send.guards_intact() and recv.guards_intact()
        assert np.array_equal(send.host().reshape(-1, B), want_send[:Tn - 1])
        assert np.array_equal(recv.host(), want_recv[:(SD - 10) * B])
        send, recv = Guarded(Tn * B), Guarded(SD * B)
        ctx.mw_plan_dispatch(ids_d, e2r_d, s.T, x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn, recv.ptr(), 0, SD)
        assert ctx.mw_get_totals()["status"] == 0
        assert np.array_equal(recv.host(), want_recv)
        # the plan left behind serves a later separate dispatch
        recv2 = Guarded(SD * B)
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv2.ptr(), 0, SD)
        assert np.array_equal(recv2.host(), want_recv)
        assert ctx.mw_plan_dispatch(ids_d, e2r_d, s.T, x_d.data_ptr() + 8, 0, send.ptr(), Tn, recv.ptr(), 0, SD,
                                    check=False) == mw.MW_ERR_ALIGNMENT


# ---- capacity and argument errors ----------------------------------------------------------------
def test_capacity_overflow_is_reported_and_contained():
    torch = torch_mod()
    inp = wl.make_random_dispatch(21, T=400, K=3, E=32, R=8, H=16, contiguous_map=True)
    s = inp.shape
    B = s.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B)
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    ids_d, e2r_d = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        # send buffer one row short
        ctx.mw_plan(ids_d, e2r_d, s.T)
        send, recv = Guarded((Tn - 1) * B), Guarded(SD * B)
        ctx.mw_pack(x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn - 1)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_CAPACITY
        assert send.guards_intact()
        assert np.array_equal(send.host().reshape(-1, B), mwo.pack_mw(p, inp.x)[:Tn - 1])
        # compact receive area ten rows short: the rows that fit are right, nothing is written past the end
        ctx.mw_plan(ids_d, e2r_d, s.T)
        send = Guarded(Tn * B)
        recv = Guarded((SD - 10) * B)
        ctx.mw_dispatch(x_d, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), Tn, recv.ptr(), 0, SD - 10)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_CAPACITY
        assert recv.guards_intact()
        want = mwo.deliver_mw(p, mwo.pack_mw(p, inp.x))
        assert np.array_equal(recv.host(), want[:(SD - 10) * B])
        # strided regions smaller than the fullest region
        ctx.mw_plan(ids_d, e2r_d, s.T)
        cap = int(np.diff(p.rank_offsets).max()) - 1
        recv = Guarded(s.R * cap * B)
        send_uc = Guarded(SD * B)
        ctx.mw_dispatch(x_d, mw.MW_LAYOUT_UNICAST, send_uc.ptr(), SD, recv.ptr(), cap * B, cap)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_CAPACITY
        assert recv.guards_intact()
        # a fresh plan clears the status
        ctx.mw_plan(ids_d, e2r_d, s.T)
        assert ctx.mw_get_totals()["status"] == 0


def test_host_side_argument_errors():
    torch = torch_mod()
    with pytest.raises(mw.MwError):
        mw.Context(0, 8, 2, 16, 32)
    with pytest.raises(mw.MwError):
        mw.Context(2000, 8, 2, 16, 32)
    with pytest.raises(mw.MwError) as e:
        mw.Context(8, 8, 2, 16, 24)                       # row size not a multiple of 16
    assert e.value.code == mw.MW_ERR_ALIGNMENT
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    ids = torch.zeros((16, 2), dtype=torch.int32, device="cuda")
    e2r = torch.zeros(8, dtype=torch.int32, device="cuda")
    with mw.Context(8, 8, 2, 16, 32) as ctx:
        assert ctx.mw_pack(buf, 0, buf, 16, check=False) == mw.MW_ERR_NO_PLAN
        assert ctx.mw_plan(ids, e2r, 17, check=False) == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_plan(None, e2r, 4, check=False) == mw.MW_ERR_INVALID_ARG
        ctx.mw_plan(ids, e2r, 16)
        assert ctx.mw_pack(buf.data_ptr() + 8, 0, buf, 16, check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_pack(buf, 5, buf, 16, check=False) == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_deliver(0, buf, buf.data_ptr() + 4, 0, 16, check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_deliver(0, buf, buf, 40, 1, check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_deliver(0, buf, buf, 64, 3, check=False) == mw.MW_ERR_CAPACITY
        assert ctx.mw_deliver(0, None, buf, 0, 16, check=False) == mw.MW_ERR_INVALID_ARG
        rc, _ = ctx.mw_allgather_pack(buf, 24, 0, buf, buf, check=False)
        assert rc == mw.MW_ERR_ALIGNMENT
        rc, _ = ctx.mw_allgather_pack(buf, 32, 0, buf, buf, 0, 6, 4, check=False)
        assert rc == mw.MW_ERR_INVALID_ARG
        rc, _ = ctx.mw_dispatch_host(ids, e2r, buf, 4, 0, buf, 16, e2r, check=False)
        assert rc == mw.MW_ERR_INVALID_ARG               # context was created without host staging
    assert mw.strerror(mw.MW_ERR_TIMEOUT) and mw.strerror(12345) == "unknown error code"


# ---- deliver into regions named by an array of addresses (Section 4.3.2) ------------------------------------
@pytest.mark.parametrize("flags", [0, mw.MW_FLAG_COPY_BULK])
@pytest.mark.parametrize("layout", [mw.MW_LAYOUT_MULTIWRITE, mw.MW_LAYOUT_UNICAST])
def test_deliver_to_an_array_of_region_addresses(layout, flags):
    torch = torch_mod()
    for inp in (wl.make_random_dispatch(61, T=700, K=4, E=32, R=16, H=24, pad_fraction=0.1), wl.make_dispatch("dsv3_prefill", 100, T=1500, H=264)):
        s = inp.shape
        B, R = s.row_bytes, s.R
        p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
        counts = np.diff(p.rank_offsets)
        cap = int(counts.max()) + 1
        send_want = mwo.pack_mw(p, inp.x) if layout == mw.MW_LAYOUT_MULTIWRITE else mwo.pack_uc(p, inp.x)
        strided = (mwo.deliver_mw if layout == mw.MW_LAYOUT_MULTIWRITE else mwo.deliver_uc)(p, send_want, cap * B, SENTINEL)
        # regions scattered over one buffer in a shuffled order with uneven 16-byte gaps
        rng = np.random.default_rng(5)
        order, offs, at = rng.permutation(R), np.zeros(R, np.int64), 0
        for r in order:
            at += 16 * int(rng.integers(0, 9))
            offs[r] = at
            at += cap * B
        area = Guarded(at + 64)
        want = np.full(at + 64, SENTINEL, np.uint8)
        for r in range(R):
            want[offs[r]:offs[r] + counts[r] * B] = strided[r * cap * B:r * cap * B + counts[r] * B]
        ptrs = torch.from_numpy(offs + area.ptr()).cuda()
        ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
        x = torch.from_numpy(inp.x.view(np.int16)).cuda()
        send = Guarded(len(send_want.reshape(-1)))
        with mw.Context(R, s.E, s.K, inp.T, B, flags=flags) as ctx:
            ctx.mw_plan(ids, e2r, inp.T)
            ctx.mw_pack(x, layout, send.ptr(), len(send_want))
            ctx.mw_deliver_ptrs(layout, send.ptr(), ptrs, cap)
            assert ctx.mw_get_totals()["status"] == 0
            assert np.array_equal(area.host(), want)
            assert area.guards_intact() and send.guards_intact()


def test_deliver_ptrs_reports_bad_addresses_and_capacity():
    torch = torch_mod()
    inp = wl.make_random_dispatch(62, T=300, K=3, E=12, R=6, H=8)
    s = inp.shape
    B, R = s.row_bytes, s.R
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    cap = int(np.diff(p.rank_offsets).max())
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    area = Guarded(R * cap * B)
    good = np.arange(R, dtype=np.int64) * cap * B + area.ptr()
    with mw.Context(R, s.E, s.K, inp.T, B) as ctx:
        send = torch.empty(p.totals["T_nonempty"] * B, dtype=torch.uint8, device="cuda")
        for bad, code in ((0, mw.MW_ERR_INVALID_ARG), (good[2] + 8, mw.MW_ERR_ALIGNMENT)):
            ptrs = good.copy()
            ptrs[2] = bad
            ctx.mw_plan(ids, e2r, inp.T)
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, p.totals["T_nonempty"])
            ctx.mw_deliver_ptrs(mw.MW_LAYOUT_MULTIWRITE, send, torch.from_numpy(ptrs).cuda(), cap)
            assert ctx.mw_get_totals()["status"] == code
            got = area.host().reshape(R, cap * B)
            assert (got[2] == SENTINEL).all()                     # the region with the bad address is left alone
            area.body.fill_(SENTINEL)
        ctx.mw_plan(ids, e2r, inp.T)
        ctx.mw_deliver_ptrs(mw.MW_LAYOUT_MULTIWRITE, send, torch.from_numpy(good).cuda(), cap - 1)
        assert ctx.mw_get_totals()["status"] == mw.MW_ERR_CAPACITY
        assert area.guards_intact()
        assert ctx.mw_deliver_ptrs(mw.MW_LAYOUT_MULTIWRITE, send, None, cap, check=False) == mw.MW_ERR_INVALID_ARG
        assert ctx.mw_deliver_ptrs(7, send, torch.from_numpy(good).cuda(), cap, check=False) == mw.MW_ERR_INVALID_ARG


# ---- seeded sweep over shapes -------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(30))
def test_random_shapes(seed):
    """Shapes drawn from a seeded generator (ranks across the bitmap-word boundaries, top-k from 1 to 12, batches across
    the tile, small-batch and wide-variant limits, padding, repeated ids, a source inside the domain), each through one of
    the call chains: three calls, three calls with the prefetching plan, or the single call."""
    rng = np.random.default_rng(9000 + seed)
    R = int(rng.choice([1, 2, 7, 16, 63, 64, 65, 100, 128, 129, 200, 256, 300]))
    E = R * int(rng.integers(1, 4))
    K = int(rng.integers(1, 13))
    T = int(rng.choice([0, 1, 33, 127, 128, 129, 256, 257, 700, 1024, 1025, 1300]))
    H = int(rng.choice([8, 24, 40, 520]))
    inp = wl.make_random_dispatch(seed, T=T, K=K, E=E, R=R, H=H, pad_fraction=float(rng.choice([0.0, 0.1, 0.5])),
                                  distinct=bool(rng.integers(0, 2)))
    src = int(rng.integers(0, R)) if rng.integers(0, 3) == 0 else -1
    chain = seed % 3
    run_dispatch(inp, src_rank=src, max_tokens=1400, one_call=chain == 0, prefetch=chain == 1, separate=bool(seed % 2))


# ---- AllGather ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, mw.MW_FLAG_COPY_BULK])
@pytest.mark.parametrize("layout", [mw.MW_LAYOUT_MULTIWRITE, mw.MW_LAYOUT_UNICAST])
@pytest.mark.parametrize("R,S,begin,count,strided", [
    (8, 48, 0, 8, False), (5, 4112, 1, 3, True), (64, 4096, 0, 64, False), (64, 16384, 0, 64, False),
    (64, 65536, 0, 64, True), (64, 1 << 18, 0, 64, False), (64, 1 << 20, 16, 16, False),
    (64, 4 << 20, 60, 4, False), (64, 16 << 20, 63, 1, False), (1, 64, 0, 1, False), (3, 16, 2, 0, False),
    (128, 4096, 0, 128, False), (65, 4112, 60, 5, True), (1024, 4096, 1000, 3, False)])   # beyond 64 ranks the bitmap costs payload bytes
def test_allgather_parity(layout, R, S, begin, count, strided, flags):
    torch = torch_mod()
    sh = wl.make_allgather_shards(R, S, seed=4)
    stride = R * S + 4096 if strided else 0
    want_send, want_recv, want_tot, ret = mwo.allgather(sh, layout, begin, count, stride, SENTINEL)
    assert ret == 0
    sh_d = torch.from_numpy(sh).cuda()
    send, recv = Guarded(len(want_send)), Guarded(max(len(want_recv), 16))
    with mw.Context(R, 8, 2, 16, 32, flags=flags) as ctx:
        rc, tot = ctx.mw_allgather_pack(sh_d, S, layout, send.ptr(), recv.ptr(), stride, begin, count)
        torch.cuda.synchronize()
    assert tot == want_tot
    assert np.array_equal(send.host(), want_send)
    assert np.array_equal(recv.host()[:len(want_recv)], want_recv)
    assert send.guards_intact() and recv.guards_intact()


def test_allgather_largest_shard_of_the_sweep():
    """64 ranks x 64 MB shards (4 GB of shards), the top of the size sweep; one destination region is materialised."""
    torch = torch_mod()
    R, S = 64, 64 << 20
    sh = wl.make_allgather_shards(R, S, seed=4)
    want_send, want_recv, want_tot, ret = mwo.allgather(sh, mw.MW_LAYOUT_MULTIWRITE, 5, 1, 0, SENTINEL)
    assert ret == 0
    sh_d = torch.from_numpy(sh).cuda()
    send, recv = Guarded(len(want_send)), Guarded(len(want_recv))
    with mw.Context(R, 8, 2, 16, 32) as ctx:
        rc, tot = ctx.mw_allgather_pack(sh_d, S, mw.MW_LAYOUT_MULTIWRITE, send.ptr(), recv.ptr(), 0, 5, 1)
        torch.cuda.synchronize()
    assert tot == want_tot
    assert torch.equal(send.body.cpu(), torch.from_numpy(want_send))
    assert torch.equal(recv.body.cpu(), torch.from_numpy(want_recv))
    assert send.guards_intact() and recv.guards_intact()


# ---- the host-buffer entry point ---------------------------------------------------------------------
@pytest.mark.parametrize("layout", [mw.MW_LAYOUT_MULTIWRITE, mw.MW_LAYOUT_UNICAST])
def test_dispatch_from_host_buffers(layout):
    torch = torch_mod()
    inp = wl.make_dispatch("dsv3_prefill", 100, T=1500, H=520)
    s = inp.shape
    B = s.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B)
    want = mwo.deliver_definition(p, inp.x, inp.topk_ids, inp.expert_to_rank)
    SD = p.totals["total_dest"]
    recv_h = torch.full((SD * B + 64,), SENTINEL, dtype=torch.uint8).pin_memory()
    ro_h = torch.zeros(s.R + 1, dtype=torch.int32).pin_memory()
    x_h = torch.from_numpy(inp.x.view(np.int16)).pin_memory()
    ids_h = torch.from_numpy(inp.topk_ids).pin_memory()
    e2r_h = torch.from_numpy(inp.expert_to_rank)
    with mw.Context(s.R, s.E, s.K, 2000, B, flags=mw.MW_FLAG_HOST_STAGING) as ctx:
        for _ in range(2):
            rc, tot = ctx.mw_dispatch_host(ids_h, e2r_h, x_h, s.T, layout, recv_h, SD, ro_h)
            assert tot == p.totals
            assert np.array_equal(ro_h.numpy(), p.rank_offsets)
            assert np.array_equal(recv_h.numpy()[:SD * B], want)
            assert (recv_h.numpy()[SD * B:] == SENTINEL).all()
        rc, _ = ctx.mw_dispatch_host(ids_h, e2r_h, x_h, s.T, layout, recv_h, SD - 1, ro_h, check=False)
        assert rc == mw.MW_ERR_CAPACITY
