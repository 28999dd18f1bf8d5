"""mw_group_tokens_static: the allocation-free entry point, checked against the CPU oracle and against mw_plan.

The entry point exists for hosts that cannot allocate device memory themselves (a serving process
whose framework pool already owns the GPU, or a caller that must not trigger the synchronisation an
allocation can imply); it keeps its scratch in a fixed array inside the library.  Here it is called
through the C ABI twice in a row, with different batches, and everything it returns is compared
with what the CPU oracle's plan gives for the same inputs (bitmaps and destination counts directly,
the group leader as the first member of the token's group, the group size from the group offsets)
and with the ordinary plan entry point, mw_plan.  Exact equality (integer work).
The second call also shows that the shared scratch left by the first call does no harm.
"""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _both_ways(inp):
    import torch
    s = inp.shape
    T, W = inp.T, (s.R + 63) // 64
    ids = torch.from_numpy(inp.topk_ids).cuda()
    e2r = torch.from_numpy(inp.expert_to_rank).cuda()
    # every output below is caller-owned memory; the call itself allocates nothing
    mask = torch.full((T, W), -1, dtype=torch.int64, device="cuda")
    ndest = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    leader = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    gsize = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    rc = mw.mw_group_tokens_static(ids, e2r, T, s.K, s.E, s.R, mask, ndest, leader, gsize, status)
    assert rc == mw.MW_OK
    torch.cuda.synchronize()
    got = {"mask": mask.cpu().numpy().view(np.uint64), "ndest": ndest.cpu().numpy(), "leader": leader.cpu().numpy(),
           "size": gsize.cpu().numpy()}

    def leaders_and_sizes(token_group, mw_row_token, group_offsets, G):
        nonempty = token_group >= 0
        want_leader = np.full(T, -1, np.int32)
        want_size = np.zeros(T, np.int32)
        want_leader[nonempty] = mw_row_token[group_offsets[token_group[nonempty]]]       # first member of the group
        want_size[nonempty] = np.diff(group_offsets[:G + 1])[token_group[nonempty]]
        return want_leader, want_size

    # the CPU oracle (sequential C, no code shared with the CUDA library)
    o = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, s.row_bytes)
    assert int(status.item()) == o.totals["status"]
    assert np.array_equal(got["mask"], o.token_mask)
    assert np.array_equal(got["ndest"], o.token_ndest)
    want_leader, want_size = leaders_and_sizes(o.token_group, o.mw_row_token, o.group_offsets, o.totals["G"])
    assert np.array_equal(got["leader"], want_leader)
    assert np.array_equal(got["size"], want_size)
    # the ordinary entry point, which takes its scratch from the workspace mw_create allocated
    with mw.Context(s.R, s.E, s.K, max(T, 1), s.row_bytes) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        p = ctx.plan_arrays(T)
    assert int(status.item()) == tot["status"]
    assert np.array_equal(got["mask"], p["token_mask"])
    assert np.array_equal(got["ndest"], p["token_ndest"])
    want_leader, want_size = leaders_and_sizes(p["token_group"], p["mw_row_token"], p["group_offsets"], tot["G"])
    assert np.array_equal(got["leader"], want_leader)
    assert np.array_equal(got["size"], want_size)
    return tot


def test_static_grouping_matches_oracle_and_plan_on_two_calls_in_a_row():
    first = wl.make_dispatch("tiny", payload=False)                     # many multi-member groups
    tot1 = _both_ways(first)
    assert 1 < tot1["G"] < first.T
    second = wl.make_random_dispatch(77, T=3001, K=6, E=300, R=150, H=8, pad_fraction=0.2)
    second.topk_ids[5, 0] = 300                                         # an invalid id: status must say so
    tot2 = _both_ways(second)
    assert tot2["status"] == mw.MW_ERR_BAD_INDEX
    _both_ways(first)                                                   # and back again: no residue from the larger batch


def test_static_grouping_rejects_oversized_batches():
    import torch
    buf = torch.zeros(64, dtype=torch.int32, device="cuda")
    rc = mw.mw_group_tokens_static(buf, buf, mw.MW_STATIC_MAX_TOKENS + 1, 2, 8, 8, buf, buf, buf, buf, buf)
    assert rc == mw.MW_ERR_CAPACITY
    assert mw.mw_group_tokens_static(buf, buf, 4, 2, 8, 8, buf, buf, buf, buf, None) == mw.MW_ERR_INVALID_ARG
    assert mw.mw_group_tokens_static(buf, buf, 0, 2, 8, 8, None, None, None, None, buf) == mw.MW_OK
