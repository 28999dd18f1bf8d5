"""Pins for the oracle's paired-relay AllGather (Sections 3.1 and 5.2): library concatenate, brute force on
the link loads, and the latencies the paper derives."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import workloads as wl
from test_oracle_pins import load_paper_constants


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("R,S,direct", [(8, 64, 32), (8, 4096, 3072), (8, 64, 0), (8, 64, 64), (4, 48, 16), (2, 32, 16), (16, 160, 96)])
def test_every_rank_gets_its_domain_in_order(layout, R, S, direct):
    sh = wl.make_allgather_shards(R, S, seed=4)
    relay_buf, recv, tot, ret = mwo.paired_allgather(sh, direct, layout, fill=0xEE)
    assert ret == 0
    n = R // 2
    recv = recv.reshape(R, n * S)
    for r in range(R):
        dom = r // n
        assert np.array_equal(recv[r], np.concatenate([sh[dom * n + q] for q in range(n)]))
    copies = 1 if layout == 0 else n - 1
    rb = relay_buf.reshape(R, copies, S - direct) if S > direct and copies else None
    if rb is not None:
        for p in range(R):
            for c in range(copies):
                assert np.array_equal(rb[p, c], sh[(p + n) % R][direct:])      # a relay holds its partner's segment
    # link loads by enumeration of (source, link) pairs
    links = {}
    for r in range(R):
        dom, partner = r // n, (r + n) % R
        peers = [dom * n + q for q in range(n) if dom * n + q != r]
        for d in peers:
            links[(r, d)] = links.get((r, d), 0) + direct
            links[(partner, d)] = links.get((partner, d), 0) + (S - direct)
        if peers:
            links[(r, partner)] = links.get((r, partner), 0) + copies * (S - direct)
    assert tot["max_link_bytes"] == max(links.values(), default=0)
    assert tot["total_bytes"] == sum(links.values())
    if n > 1:
        assert tot["pair_link_bytes"] == links[(0, n)] and tot["direct_link_bytes"] == links[(0, 1)]


def test_paper_latencies_full_mesh_tp4():
    """Section 3.1 with link bandwidth w and shard size s: s/w, 3s/(4w), s/(2w); -50 % and -33 %."""
    c = load_paper_constants()
    S, R = 1 << 20, 8
    sh = np.zeros((R, S), np.uint8)
    t_direct = mwo.paired_allgather(sh, S, 0)[2]["max_link_bytes"] / S
    d_uc = mwo.balanced_direct_bytes(S, 4, 1)
    d_mw = mwo.balanced_direct_bytes(S, 4, 0)
    t_uc = mwo.paired_allgather(sh, d_uc, 1)[2]["max_link_bytes"] / S
    t_mw = mwo.paired_allgather(sh, d_mw, 0)[2]["max_link_bytes"] / S
    assert t_direct == c["pair_time_direct_only"]
    assert t_uc == c["pair_time_unicast_relay"] and d_uc == 3 * S // 4
    assert t_mw == c["pair_time_multicast_relay"] and d_mw == S // 2
    assert round(100 * (1 - t_mw / t_direct)) == c["pair_gain_vs_direct_percent"]
    assert round(100 * (1 - t_mw / t_uc)) == c["pair_gain_vs_unicast_relay_percent"]
    # the unicast relay puts three copies on the pair link, MultiWrite one (relay_link_copies_* above)
    assert mwo.paired_allgather(sh, d_mw, 1)[2]["pair_link_bytes"] == c["relay_link_copies_unicast"] * (S - d_mw)
    assert mwo.paired_allgather(sh, d_mw, 0)[2]["pair_link_bytes"] == c["relay_link_copies_multicast"] * (S - d_mw)
    # any other split is slower than the balanced one
    for d in (d_mw - 4096, d_mw + 4096):
        assert mwo.paired_allgather(sh, d, 0)[2]["max_link_bytes"] > t_mw * S


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("S,n,w_direct,w_pair", [(1 << 20, 4, 56.0, 56.0), (1 << 20, 4, 56.0, 25.0), (16 << 20, 4, 56.0, 112.0),
                                                 (4096, 2, 3.0, 1.0), (4096 + 16, 8, 1.0, 7.0), (1 << 24, 4, 450.0, 50.0)])
def test_split_by_bandwidth_ratio_lets_both_link_classes_finish_together(layout, S, n, w_direct, w_pair):
    """Section 5.2 step 1.  Enumerate every split that is a multiple of 16 bytes: with exact fractions, the one the
    oracle returns is the largest for which a direct link is done no later than the pair link."""
    from fractions import Fraction
    c = 1 if layout == 0 else n - 1
    d = mwo.split_direct_bytes(S, n, layout, w_direct, w_pair)
    assert d % 16 == 0 and 0 <= d <= S

    def t_direct(x):
        return Fraction(x) / Fraction(w_direct)

    def t_pair(x):
        return c * Fraction(S - x) / Fraction(w_pair)

    best = max(x for x in range(0, S + 1, 16) if t_direct(x) <= t_pair(x)) if S <= 8192 else None
    if best is not None:
        assert d == best
    assert t_direct(d) <= t_pair(d)
    assert d + 16 > S or t_direct(d + 16) > t_pair(d + 16)
    # the oracle's link loads, weighted by the two bandwidths, agree: the slower class decides the transfer time
    tot = mwo.paired_allgather(np.zeros((2 * n, S), np.uint8), d, layout)[2]
    assert Fraction(tot["direct_link_bytes"]) / Fraction(w_direct) <= Fraction(tot["pair_link_bytes"]) / Fraction(w_pair)
    assert tot["forward_link_bytes"] <= tot["pair_link_bytes"]


def test_split_with_equal_bandwidths_is_the_papers_split():
    """Section 3.1: equal links give s/2 direct with MultiWrite (latency s/2w) and 3s/4 with the unicast relay (3s/4w)."""
    for S in (1 << 20, 16 << 20, 4096, 48):
        for n in (2, 4, 8):
            for layout in (0, 1):
                assert mwo.split_direct_bytes(S, n, layout, 56.0, 56.0) == mwo.balanced_direct_bytes(S, n, layout)
    assert mwo.split_direct_bytes(1 << 20, 4, 0, 1.0, 1.0) == (1 << 20) // 2
    assert mwo.split_direct_bytes(1 << 20, 4, 1, 1.0, 1.0) == 3 * (1 << 20) // 4
    # degenerate inputs: a single-rank domain, or no usable bandwidth figure, sends everything direct
    assert mwo.split_direct_bytes(4096, 1, 0, 1.0, 1.0) == 4096
    assert mwo.split_direct_bytes(4096, 4, 0, 0.0, 1.0) == 4096
    assert mwo.split_direct_bytes(4096, 4, 0, 1.0, -1.0) == 4096
    # a pair link twice as fast takes two thirds of the shard with MultiWrite
    assert mwo.split_direct_bytes(3 << 20, 4, 0, 1.0, 2.0) == 1 << 20


def test_invalid_arguments():
    sh = np.zeros((8, 64), np.uint8)
    assert mwo.paired_allgather(sh, 80, 0)[3] == mwo.MWO_ERR_INVALID_ARG
    assert mwo.paired_allgather(sh, 16, 2)[3] == mwo.MWO_ERR_INVALID_ARG
    assert mwo.paired_allgather(np.zeros((7, 64), np.uint8), 16, 0)[3] == mwo.MWO_ERR_INVALID_ARG
