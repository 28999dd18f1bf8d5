"""Pins for the oracle's group-major receive order (Section 4.3.1: one MultiWrite = one source buffer into one
target buffer per destination; Section 4.3.2: an array of remote buffer addresses) and for its expert index
(Section 2.3.2: tokens go to the nodes that host their experts).  Expected values come from brute force written
here with Python sets and lists, from numpy library routines, or from special cases with a known answer; none
of them calls the functions under test to make its expectation."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import workloads as wl


def dest_sets(ids, e2r, R):
    E = len(e2r)
    return [sorted({int(e2r[e]) for e in row if 0 <= e < E and 0 <= e2r[e] < R}) for row in ids]


def brute_groups(sets):
    """Groups in order of first occurrence: list of (destination ranks, member tokens)."""
    index, groups = {}, []
    for t, s in enumerate(sets):
        if not s:
            continue
        key = tuple(s)
        if key not in index:
            index[key] = len(groups)
            groups.append((s, []))
        groups[index[key]][1].append(t)
    return groups


def brute_group_major_regions(sets, R):
    groups = brute_groups(sets)
    regions = [[] for _ in range(R)]
    starts = []
    for s, members in groups:
        starts.append([len(regions[r]) for r in s])
        for r in s:
            regions[r].extend(members)
    return groups, starts, regions


def tagged_rows(T, B):
    """Row t holds its own index in every 4-byte word."""
    return np.repeat(np.arange(1, T + 1, dtype=np.uint32)[:, None], B // 4, axis=1).view(np.uint8).reshape(T, B)


def check_group_major(inp, R):
    ids, e2r = inp.topk_ids, inp.expert_to_rank
    B = 16
    p = mwo.plan(ids, e2r, R, B)
    gdr, gdo, gm = mwo.group_major(p)
    sets = dest_sets(ids, e2r, R)
    groups, starts, regions = brute_group_major_regions(sets, R)
    assert len(groups) == p.totals["G"]
    for g, ((s, members), st) in enumerate(zip(groups, starts)):
        assert list(gdr[g][:len(s)]) == s and all(v == -1 for v in gdr[g][len(s):])
        assert list(gdo[g][:len(s)]) == st and all(v == -1 for v in gdo[g][len(s):])
    for t, s in enumerate(sets):
        want = [regions[r].index(t) for r in s]
        assert list(gm[t][:len(s)]) == want and all(v == -1 for v in gm[t][len(s):])
    # delivered bytes: region r holds the rows of brute-force region r, in that order
    x = tagged_rows(inp.T, B)
    send = mwo.pack_mw(p, x)
    recv = mwo.deliver_group_major(p, send, gdr, gdo, 0, 0xEE).reshape(-1, B)
    at = 0
    for r in range(R):
        for t in regions[r]:
            assert np.array_equal(recv[at], x[t]), (r, t)
            at += 1
    assert at == p.totals["total_dest"] == len(recv)
    # strided regions hold the same rows
    cap = max(len(q) for q in regions) + 2
    rs = mwo.deliver_group_major(p, send, gdr, gdo, cap * B, 0xEE).reshape(R, cap, B)
    for r in range(R):
        assert np.array_equal(rs[r, :len(regions[r])], x[regions[r]].reshape(-1, B))
        assert (rs[r, len(regions[r]):] == 0xEE).all()


@pytest.mark.parametrize("seed,R,E,K,pad", [(0, 3, 6, 2, 0.0), (1, 8, 32, 4, 0.2), (2, 9, 9, 3, 0.0), (3, 65, 130, 4, 0.1),
                                            (4, 2, 8, 5, 0.3), (5, 130, 260, 6, 0.0)])
def test_group_major_brute_force(seed, R, E, K, pad):
    check_group_major(wl.make_random_dispatch(seed, T=37, K=K, E=E, R=R, H=8, pad_fraction=pad), R)


def test_group_major_with_few_large_groups():
    # 4 ranks, top-2 of 4 experts: at most 6 destination sets over 200 tokens, so blocks are long
    check_group_major(wl.make_random_dispatch(11, T=200, K=2, E=4, R=4, H=8, contiguous_map=True), 4)


def test_top1_group_major_equals_token_major():
    # one destination per token: a group is a rank, each region is one block, both orders coincide
    inp = wl.make_random_dispatch(6, T=300, K=1, E=16, R=8, H=8, contiguous_map=True)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, 8, 16)
    gdr, gdo, gm = mwo.group_major(p)
    assert (gdo[:, 0] == 0).all() and np.array_equal(gm, p.dest_pos)
    send = mwo.pack_mw(p, inp.x)
    assert np.array_equal(mwo.deliver_group_major(p, send, gdr, gdo), mwo.deliver_mw(p, send))


def test_blocks_tile_every_region_on_the_prefill_shape():
    inp = wl.make_dispatch("dsv3_prefill", T=1024, H=8)
    R = inp.shape.R
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, 16)
    gdr, gdo, gm = mwo.group_major(p)
    size = np.diff(p.group_offsets[:p.totals["G"] + 1])
    counts = np.diff(p.rank_offsets)
    for r in range(R):
        g, i = np.nonzero(gdr == r)
        iv = sorted((int(gdo[a, b]), int(size[a])) for a, b in zip(g, i))
        end = 0
        for start, n in iv:
            assert start == end
            end += n
        assert end == counts[r]
        # same tokens as the token-major region, in another order
        sel = p.dest_rank == r
        assert sorted(gm[sel]) == list(range(counts[r])) and sorted(p.dest_pos[sel]) == list(range(counts[r]))


# ---- expert index ---------------------------------------------------------------------------------------
def check_expert_index(inp, R):
    ids, e2r = inp.topk_ids, inp.expert_to_rank
    E, T, K = len(e2r), inp.T, ids.shape[1]
    p = mwo.plan(ids, e2r, R, 16)
    off, tok, slot, n = mwo.expert_index(p, ids, e2r)
    sets = dest_sets(ids, e2r, R)
    region = [[t for t in range(T) if r in sets[t]] for r in range(R)]         # token-major regions
    at = 0
    for e in range(E):
        assert off[e] == at
        if not 0 <= e2r[e] < R:
            continue
        for t in range(T):
            if e in ids[t]:
                assert tok[at] == t and slot[at] == region[e2r[e]].index(t)
                at += 1
    assert off[E] == at == n
    assert (tok[at:] == -1).all() and (slot[at:] == -1).all()


@pytest.mark.parametrize("seed,R,E,K,pad,distinct", [(0, 3, 6, 2, 0.0, True), (1, 8, 32, 4, 0.2, True), (2, 9, 9, 3, 0.0, False),
                                                     (3, 65, 130, 4, 0.1, True), (4, 2, 8, 5, 0.3, False)])
def test_expert_index_brute_force(seed, R, E, K, pad, distinct):
    check_expert_index(wl.make_random_dispatch(seed, T=41, K=K, E=E, R=R, H=8, pad_fraction=pad, distinct=distinct), R)


def test_expert_index_ignores_invalid_table_entries_and_ids():
    inp = wl.make_random_dispatch(8, T=50, K=3, E=12, R=4, H=8)
    e2r = inp.expert_to_rank.copy()
    e2r[2], e2r[7] = -1, 4
    inp.expert_to_rank = e2r
    ids = inp.topk_ids.copy()
    ids[5, 0], ids[6, 1] = 12, -7
    inp.topk_ids = ids
    check_expert_index(inp, 4)
    p = mwo.plan(ids, e2r, 4, 16)
    off, *_ = mwo.expert_index(p, ids, e2r)
    assert off[3] == off[2] and off[8] == off[7]


def test_expert_counts_are_a_bincount_and_top1_is_a_stable_sort():
    inp = wl.make_dispatch("tiny")
    s = inp.shape
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, 16)
    off, tok, slot, n = mwo.expert_index(p, inp.topk_ids, inp.expert_to_rank)
    assert np.array_equal(np.diff(off), np.bincount(inp.topk_ids.ravel(), minlength=s.E)) and n == s.T * s.K
    one = wl.make_random_dispatch(3, T=500, K=1, E=16, R=8, H=8, contiguous_map=True)
    p = mwo.plan(one.topk_ids, one.expert_to_rank, 8, 16)
    off, tok, slot, n = mwo.expert_index(p, one.topk_ids, one.expert_to_rank)
    assert np.array_equal(tok, np.argsort(one.topk_ids[:, 0], kind="stable"))
    # the slot leads to the token's row in the delivered region
    x = tagged_rows(one.T, 16)
    recv = mwo.deliver_mw(p, mwo.pack_mw(p, x)).reshape(-1, 16)
    for e in range(16):
        r = one.expert_to_rank[e]
        for i in range(off[e], off[e + 1]):
            assert np.array_equal(recv[p.rank_offsets[r] + slot[i]], x[tok[i]])
