"""GPU parity of the two-level (relayed) dispatch against the oracle: both plans, the per-link byte
accounting, the send buffer, the hop area and the final receive regions, bit for bit."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads as wl

from gpu_util import Guarded, SENTINEL, assert_plan_equal, torch_mod

pytestmark = pytest.mark.gpu


def run_relay(inp, P, src, strided=False, flags=0, max_tokens=None):
    torch = torch_mod()
    s = inp.shape
    T, B, R = inp.T, s.row_bytes, s.R
    # the receive buffer is the relay buffer: only copies held by pure relays are staged in the hop area
    hp, fp, want_send, want_hop, _, want_tot = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x, 0, SENTINEL, in_place=True)
    counts = np.diff(fp.rank_offsets)
    cap = int(counts.max()) + 1 if strided else fp.totals["total_dest"]
    stride = cap * B if strided else 0
    _, _, _, _, want_recv, _ = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x, stride, SENTINEL, in_place=True)
    # the relayed route must end in the regions of the flat dispatch (the definitional two-buffer form agrees)
    assert np.array_equal(want_recv, mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x, stride, SENTINEL)[4])
    ids_d = torch.from_numpy(inp.topk_ids).cuda()
    e2r_d = torch.from_numpy(inp.expert_to_rank).cuda()
    x_d = torch.from_numpy(inp.x.view(np.int16)).cuda()
    with mw.Relay(R, s.E, s.K, max_tokens or max(T, 1), B, src, P, flags=flags) as relay:
        for _ in range(2):
            relay.mw_relay_plan(ids_d, e2r_d, T)
            tot = relay.mw_relay_get_totals()
            assert tot == want_tot, (tot, want_tot)
            assert_plan_equal(relay.hop.plan_arrays(T), hp, relay.hop.mw_get_totals())
            assert_plan_equal(relay.flat.plan_arrays(T), fp, relay.flat.mw_get_totals())
        if T == 0:
            return tot
        send = Guarded(len(want_send) * B)
        hop = Guarded(len(want_hop))
        recv = Guarded(len(want_recv))
        relay.mw_relay_dispatch(x_d, send.ptr(), len(want_send), hop.ptr(), len(want_hop) // B, recv.ptr(), stride, cap)
        assert relay.mw_relay_get_totals()["status"] == want_tot["status"]
        assert np.array_equal(send.host().reshape(-1, B), want_send)
        assert np.array_equal(hop.host(), want_hop)
        assert np.array_equal(recv.host(), want_recv)
        assert send.guards_intact() and hop.guards_intact() and recv.guards_intact()
    return tot


@pytest.mark.parametrize("R,P,src,E,K,T", [(16, 8, 0, 64, 8, 1500), (8, 4, 5, 16, 3, 700), (12, 3, 7, 24, 4, 300),
                                           (6, 6, 2, 12, 3, 257), (5, 1, 3, 10, 2, 64), (128, 8, 77, 256, 8, 2000),
                                           (64, 8, 13, 128, 12, 900), (64, 4, 62, 128, 20, 515),    # 12 and 20 destinations per token
                                           (128, 16, 5, 256, 64, 300)])                             # the largest top-k
def test_relay_parity_random(R, P, src, E, K, T):
    inp = wl.make_random_dispatch(R + T, T=T, K=K, E=E, R=R, H=40, pad_fraction=0.1, contiguous_map=(E % R == 0))
    run_relay(inp, P, src)
    run_relay(inp, P, src, strided=True)


def test_relay_dsv3_shape_eight_servers():
    # the DeepSeek-V3-shaped routing on 8 servers of 8 ranks, reduced hidden size
    inp = wl.make_dispatch("dsv3_prefill", H=264)
    tot = run_relay(inp, 8, 0)
    assert tot["inter_multiwrite_bytes"] < tot["inter_unicast_bytes"]
    assert tot["direct_bytes"] + tot["inter_unicast_bytes"] <= tot["delivered_rows"] * inp.shape.row_bytes


def test_relay_dsv3_shape_full_size_rows():
    # the same routing with the full 14336-byte rows (the shape the benchmark times): 8 servers of 8 ranks
    inp = wl.make_dispatch("dsv3_prefill")
    assert inp.shape.row_bytes == 14336
    tot = run_relay(inp, 8, 0)
    assert tot["hop_rows"] < tot["delivered_rows"]


def test_relay_small_batches_and_invalid_ids():
    inp = wl.make_random_dispatch(3, T=40, K=4, E=32, R=16, H=16, pad_fraction=0.3)
    ids = inp.topk_ids.copy()
    ids[3, :] = -1
    ids[4, 0] = 32
    inp.topk_ids = ids
    tot = run_relay(inp, 4, 9, max_tokens=64)
    assert tot["status"] == mw.MW_ERR_BAD_INDEX
    run_relay(wl.make_random_dispatch(4, T=0, K=4, E=32, R=16, H=16), 4, 9)
    run_relay(wl.make_dispatch("decode", H=64), 8, 200)


def test_relay_errors():
    torch = torch_mod()
    with pytest.raises(mw.MwError):
        mw.Relay(16, 32, 4, 64, 32, -1, 8)                 # the source must be a member of the domain
    with pytest.raises(mw.MwError):
        mw.Relay(16, 32, 4, 64, 32, 0, 5)                  # ranks per server must divide R
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    ids = torch.zeros((16, 4), dtype=torch.int32, device="cuda")
    e2r = torch.full((32,), 9, dtype=torch.int32, device="cuda")   # every token goes to rank 9: rank 8 relays without being a destination
    with mw.Relay(16, 32, 4, 64, 32, 0, 8) as relay:
        assert relay.mw_relay_dispatch(buf, buf, 64, buf, 64, buf, 0, 64, check=False) == mw.MW_ERR_NO_PLAN
        assert relay.mw_relay_plan(ids, e2r, 65, check=False) == mw.MW_ERR_INVALID_ARG
        relay.mw_relay_plan(ids, e2r, 16)
        assert relay.mw_relay_dispatch(buf, buf, 64, buf.data_ptr() + 8, 64, buf, 0, 64, check=False) == mw.MW_ERR_ALIGNMENT
        # hop area one row short: reported, nothing written past it
        hop = Guarded(15 * 32)
        relay.mw_relay_dispatch(buf, buf, 64, hop.ptr(), 15, buf, 0, 64)
        tot = relay.mw_relay_get_totals()
        assert tot["status"] == mw.MW_ERR_CAPACITY and tot["staged_rows"] == 16
        assert hop.guards_intact()
