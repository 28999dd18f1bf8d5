"""Pins for the oracle's two-level (relayed) MultiWrite: brute force with Python sets, the paper's
worked example, closed forms for uniform routing, and degenerate topologies."""
import math

import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import workloads as wl
from test_oracle_pins import load_paper_constants


def brute_relay(ids, e2r, R, P, src, rows):
    T, K = ids.shape
    E = len(e2r)
    server = lambda r: r // P
    relay_of = lambda s: s * P + src % P
    dest = []
    for t in range(T):
        s = set()
        for k in range(K):
            e = int(ids[t, k])
            if 0 <= e < E and 0 <= int(e2r[e]) < R:
                s.add(int(e2r[e]))
        dest.append(sorted(s))
    hops = [sorted({r if server(r) == server(src) else relay_of(server(r)) for r in d}) for d in dest]
    hop_rows = sum(len(h) for h in hops)
    direct = sum(1 for d in dest for r in d if server(r) == server(src) and r != src)
    inter_uc = sum(1 for d in dest for r in d if server(r) != server(src))
    inter_mw = sum(len({server(r) for r in d if server(r) != server(src)}) for d in dest)
    forward = sum(1 for d in dest for r in d if server(r) != server(src) and r != relay_of(server(r)))
    recv = [[rows[t] for t in range(T) if r in dest[t]] for r in range(R)]
    hop_recv = [[rows[t] for t in range(T) if h in hops[t]] for h in range(R)]
    # with the receive buffer as relay buffer only a pure relay (a next hop that is not a destination) stages its copy
    staged = [[rows[t] if h not in dest[t] else None for t in range(T) if h in hops[t]] for h in range(R)]
    return dict(staged=staged, hop_rows=hop_rows, direct=direct, inter_uc=inter_uc, inter_mw=inter_mw, forward=forward, recv=recv,
                hop_recv=hop_recv, delivered=sum(len(d) for d in dest))


@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("R,P,src,E,K", [(8, 4, 1, 16, 3), (16, 8, 0, 64, 8), (12, 3, 7, 24, 4), (6, 6, 2, 12, 3), (5, 1, 3, 10, 2)])
def test_relay_brute_force(seed, R, P, src, E, K):
    inp = wl.make_random_dispatch(seed, T=37, K=K, E=E, R=R, H=8, pad_fraction=0.1 if seed % 2 else 0.0,
                                  contiguous_map=(seed % 2 == 0))
    B = 16
    xb = inp.x.view(np.uint8).reshape(inp.T, B)
    bf = brute_relay(inp.topk_ids, inp.expert_to_rank, R, P, src, [xb[t].tobytes() for t in range(inp.T)])
    hp, fp, send, hop_buf, recv, tot = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x)
    assert tot["hop_rows"] == bf["hop_rows"] == hp.totals["total_dest"] == len(hop_buf) // B
    assert tot["delivered_rows"] == bf["delivered"] == fp.totals["total_dest"]
    assert tot["direct_bytes"] == bf["direct"] * B
    assert tot["inter_unicast_bytes"] == bf["inter_uc"] * B
    assert tot["inter_multiwrite_bytes"] == bf["inter_mw"] * B
    assert tot["forward_bytes"] == bf["forward"] * B
    assert hop_buf.tobytes() == b"".join(b"".join(rows) for rows in bf["hop_recv"])
    assert recv.tobytes() == b"".join(b"".join(rows) for rows in bf["recv"])
    # the relayed route ends in exactly the same receive regions as the flat one
    assert np.array_equal(recv, mwo.deliver_definition(fp, inp.x, inp.topk_ids, inp.expert_to_rank))
    # each row is packed once per group of identical next-hop set
    assert len(send) == hp.totals["T_nonempty"]
    assert tot["staged_rows"] == sum(1 for rows in bf["staged"] for r in rows if r is not None)
    # Section 6.4: with the receive buffer as the relay buffer the regions come out the same, the accounting too, and
    # only the copies held by pure relays appear in the hop area
    for stride in (0, (int(np.diff(fp.rank_offsets).max()) + 1) * B):
        _, _, send2, hop2, recv2, tot2 = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x, stride, 0xEE, in_place=True)
        _, _, _, _, recv_ref, _ = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, B, src, P, inp.x, stride, 0xEE)
        assert tot2 == tot and np.array_equal(send2, send)
        assert np.array_equal(recv2, recv_ref)
        want_hop = b"".join(b"".join(r if r is not None else b"\xEE" * B for r in rows) for rows in bf["staged"])
        assert hop2.tobytes() == want_hop


def test_paper_example_four_local_four_remote():
    """Section 3.2: NPU0 of Server0 sends a token to eight experts, four in each of two 8-NPU servers."""
    c = load_paper_constants()
    R, P, src = 16, 8, 0
    e2r = np.arange(R, dtype=np.int32)                       # one expert per NPU
    ids = np.array([[1, 2, 3, 4, 9, 10, 11, 12]], np.int32)
    hp, fp, _, _, _, tot = mwo.relay(ids, e2r, R, 16, src, P)
    assert tot["inter_unicast_bytes"] // 16 == c["relay_example_remote_copies_unicast"]
    assert tot["inter_multiwrite_bytes"] // 16 == c["relay_example_remote_copies_multiwrite"]
    assert tot["direct_bytes"] // 16 == 4 and tot["forward_bytes"] // 16 == 4
    assert tot["staged_rows"] == 1                          # NPU8 relays for 9..12 without being a destination itself
    hops = [int(r) for r in hp.dest_rank[0] if r >= 0]
    assert hops == [1, 2, 3, 4, c["relay_example_relay_rank"]]
    assert mwo.next_hop(12, src, P) == c["relay_example_relay_rank"] and mwo.next_hop(3, src, P) == 3


def test_uniform_routing_closed_forms_two_servers():
    """2 servers x 8 NPUs, 64 experts (4 per NPU), top-8, uniform: expected distinct remote ranks per token
    8 (1 - C(60,8)/C(64,8)) = 3.375; a remote copy is needed with probability 1 - C(32,8)/C(64,8) = 0.9976."""
    R, P, E, K, T = 16, 8, 64, 8, 20000
    remote_ranks = 8 * (1 - math.comb(60, 8) / math.comb(64, 8))
    need_relay = 1 - math.comb(32, 8) / math.comb(64, 8)
    assert abs(remote_ranks - 3.375) < 0.001 and abs(need_relay - 0.9976) < 0.0001
    inp = wl.make_random_dispatch(3, T=T, K=K, E=E, R=R, H=8, contiguous_map=True)
    _, _, _, _, _, tot = mwo.relay(inp.topk_ids, inp.expert_to_rank, R, 16, 0, P)
    assert abs(tot["inter_unicast_bytes"] / 16 / T - remote_ranks) / remote_ranks < 0.01
    assert abs(tot["inter_multiwrite_bytes"] / 16 / T - need_relay) / need_relay < 0.005
    ratio = tot["inter_unicast_bytes"] / tot["inter_multiwrite_bytes"]
    assert abs(ratio - remote_ranks / need_relay) < 0.05            # about 3.38: the cross-server bytes MultiWrite removes
    # relays forward everything except the copies addressed to themselves (1 of 8 remote ranks is the relay)
    assert abs(tot["forward_bytes"] / tot["inter_unicast_bytes"] - 7 / 8) < 0.01


def test_degenerate_topologies():
    inp = wl.make_random_dispatch(9, T=300, K=4, E=32, R=8, H=8)
    one_server = mwo.relay(inp.topk_ids, inp.expert_to_rank, 8, 16, 2, 8)      # everything is local
    hp, fp, _, _, _, tot = one_server
    assert tot["inter_unicast_bytes"] == tot["inter_multiwrite_bytes"] == tot["forward_bytes"] == 0
    assert np.array_equal(hp.rank_tokens, fp.rank_tokens) and tot["hop_rows"] == tot["delivered_rows"]
    assert tot["direct_bytes"] == fp.totals["unicast_bytes"]
    hp, fp, _, _, _, tot = mwo.relay(inp.topk_ids, inp.expert_to_rank, 8, 16, 2, 1)   # every rank its own server
    assert tot["inter_unicast_bytes"] == tot["inter_multiwrite_bytes"] == fp.totals["unicast_bytes"]
    assert tot["forward_bytes"] == 0 and tot["direct_bytes"] == 0
