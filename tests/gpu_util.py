"""Helpers for the GPU parity tests: run the CUDA path through the C ABI binding on seeded inputs,
with sentinel guard bands around every output buffer, and compare with the CPU oracle bit for bit."""
from __future__ import annotations

import numpy as np

from oracle import mwo
from paper_2605_22428_b200 import binding as mw

GUARD = 4096          # bytes of sentinel before and after every output buffer
SENTINEL = 0xA5


def torch_mod():
    import torch
    return torch


class Guarded:
    """A device byte buffer with sentinel bands on both sides."""

    def __init__(self, nbytes: int, fill: int = SENTINEL):
        torch = torch_mod()
        self.nbytes = int(nbytes)
        self.raw = torch.full((self.nbytes + 2 * GUARD,), fill, dtype=torch.uint8, device="cuda")
        self.fill = fill

    @property
    def body(self):
        return self.raw[GUARD:GUARD + self.nbytes]

    def ptr(self) -> int:
        return self.raw.data_ptr() + GUARD

    def host(self) -> np.ndarray:
        return self.body.cpu().numpy()

    def guards_intact(self) -> bool:
        torch = torch_mod()
        lo, hi = self.raw[:GUARD], self.raw[GUARD + self.nbytes:]
        return bool(torch.all(lo == self.fill)) and bool(torch.all(hi == self.fill))


PLAN_KEYS = ("token_mask", "token_ndest", "token_group", "token_mw_row", "mw_row_token", "group_offsets",
             "group_mask", "rank_offsets", "rank_tokens", "dest_rank", "dest_pos")


def assert_plan_equal(got: dict, p: mwo.Plan, totals: dict):
    for k in PLAN_KEYS:
        want = getattr(p, k)
        assert got[k].shape == want.shape, k
        if not np.array_equal(got[k], want):
            bad = np.argwhere(got[k] != want)[:5]
            raise AssertionError(f"plan array {k} differs at {bad.tolist()}: got {got[k][tuple(bad[0])]}, want {want[tuple(bad[0])]}")
    assert totals == p.totals, (totals, p.totals)


def run_dispatch(inp, *, layouts=(mw.MW_LAYOUT_MULTIWRITE, mw.MW_LAYOUT_UNICAST), strides=("compact", "strided"),
                 flags: int = 0, src_rank: int = -1, max_tokens: int | None = None, check_payload: bool = True,
                 repeats: int = 1, one_call: bool = False, separate: bool = False, prefetch: bool = False):
    """Plans and dispatches `inp` on the GPU, checks everything against the oracle, returns (plan, totals)."""
    torch = torch_mod()
    s = inp.shape
    T, B = inp.T, s.row_bytes
    ids_d = torch.from_numpy(inp.topk_ids).cuda() if T else torch.zeros((0, s.K), dtype=torch.int32, device="cuda")
    e2r_d = torch.from_numpy(inp.expert_to_rank).cuda()
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B, src_rank)
    assert p.ret == 0
    x_early = torch.from_numpy(inp.x.view(np.int16)).cuda() if prefetch else None
    with mw.Context(s.R, s.E, s.K, max_tokens or max(T, 1), B, src_rank=src_rank, flags=flags) as ctx:
        for _ in range(repeats):
            if prefetch:
                # the same plan; the launch also asks L2 for the hidden rows
                ctx.mw_plan_prefetch(ids_d, e2r_d, T, x_early)
            else:
                ctx.mw_plan(ids_d, e2r_d, T)
            totals = ctx.mw_get_totals()
            got = ctx.plan_arrays(T)
            assert_plan_equal(got, p, totals)
        if not check_payload or T == 0:
            return p, totals
        x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
        Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
        want_send = {mw.MW_LAYOUT_MULTIWRITE: mwo.pack_mw(p, inp.x), mw.MW_LAYOUT_UNICAST: mwo.pack_uc(p, inp.x)}
        counts = np.diff(p.rank_offsets)
        for layout in layouts:
            nsend = Tn if layout == mw.MW_LAYOUT_MULTIWRITE else SD
            for mode in strides:
                cap = int(counts.max()) + 1 if mode == "strided" else SD
                stride = cap * B if mode == "strided" else 0
                want_recv = (mwo.deliver_mw(p, want_send[layout], stride, SENTINEL) if layout == mw.MW_LAYOUT_MULTIWRITE
                             else mwo.deliver_uc(p, want_send[layout], stride, SENTINEL))
                send = Guarded(nsend * B)
                recv = Guarded(len(want_recv))
                if one_call:
                    # plan + dispatch through the single entry point; the plan it leaves behind must be the same
                    ctx.mw_plan_dispatch(ids_d, e2r_d, T, x_d.data_ptr(), layout, send.ptr(), nsend, recv.ptr(), stride, cap)
                    tot2 = ctx.mw_get_totals()
                    assert_plan_equal(ctx.plan_arrays(T), p, tot2)
                elif separate:
                    # the two steps as calls of their own (mw_dispatch does both in one pass over the rows)
                    ctx.mw_pack(x_d.data_ptr(), layout, send.ptr(), nsend)
                    ctx.mw_deliver(layout, send.ptr(), recv.ptr(), stride, cap)
                    tot2 = ctx.mw_get_totals()
                else:
                    ctx.mw_dispatch(x_d.data_ptr(), layout, send.ptr(), nsend, recv.ptr(), stride, cap)
                    tot2 = ctx.mw_get_totals()
                assert tot2["status"] == p.totals["status"], tot2
                assert np.array_equal(send.host().reshape(-1, B), want_send[layout]), ("send", layout, mode)
                assert np.array_equal(recv.host(), want_recv), ("recv", layout, mode)
                assert send.guards_intact() and recv.guards_intact()
    return p, totals
