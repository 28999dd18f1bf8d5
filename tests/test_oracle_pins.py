"""Pins for the CPU oracle: everything here is independent of oracle/mwo.c.

The checks are (a) a brute-force enumeration of (token, rank) pairs written with
Python sets and lists on tiny inputs, (b) invariants that hold at every size,
(c) special cases that reduce to library routines (stable counting sort,
bincount, concatenate), (d) closed forms and the constants the paper prints.
"""
import math
import os

import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import workloads as wl


# ----------------------------------------------------------------------------------------------
# (a) brute force, written from the definition with Python containers
# ----------------------------------------------------------------------------------------------
def brute_force(ids, e2r, R, x_rows):
    """Returns the whole plan and all buffers as Python lists, by enumeration."""
    T, K = ids.shape
    E = len(e2r)
    dest = []          # D_t as a sorted list of ranks
    bad = False
    valid = 0
    for t in range(T):
        s = set()
        for k in range(K):
            e = int(ids[t, k])
            if e == -1:
                continue
            if not 0 <= e < E or not 0 <= int(e2r[e]) < R:
                bad = True
                continue
            valid += 1
            s.add(int(e2r[e]))
        dest.append(sorted(s))
    first_seen = {}    # frozenset -> group id in order of first occurrence
    token_group = []
    for t in range(T):
        if not dest[t]:
            token_group.append(-1)
            continue
        key = frozenset(dest[t])
        if key not in first_seen:
            first_seen[key] = len(first_seen)
        token_group.append(first_seen[key])
    G = len(first_seen)
    members = [[t for t in range(T) if token_group[t] == g] for g in range(G)]
    mw_row_token = [t for g in range(G) for t in members[g]]
    group_offsets = [0]
    for g in range(G):
        group_offsets.append(group_offsets[-1] + len(members[g]))
    recv_tokens = [[t for t in range(T) if r in dest[t]] for r in range(R)]
    recv = [[x_rows[t] for t in recv_tokens[r]] for r in range(R)]
    return dict(dest=dest, token_group=token_group, G=G, mw_row_token=mw_row_token, group_offsets=group_offsets,
                recv_tokens=recv_tokens, recv=recv, bad=bad, valid=valid,
                group_sets=[sorted(k) for k, _ in sorted(first_seen.items(), key=lambda kv: kv[1])])


def mask_to_ranks(words):
    out = []
    for w, v in enumerate(words):
        v = int(v)
        for b in range(64):
            if v >> b & 1:
                out.append(64 * w + b)
    return out


def check_against_brute_force(inp, R, src_rank=-1):
    ids, e2r, x = inp.topk_ids, inp.expert_to_rank, inp.x
    B = x.shape[1] * 2
    T, K = ids.shape
    xb = x.view(np.uint8).reshape(T, B)
    bf = brute_force(ids, e2r, R, [xb[t].tobytes() for t in range(T)])
    p = mwo.plan(ids, e2r, R, B, src_rank)
    assert p.ret == 0
    Kd = min(K, R)
    # masks and counts
    for t in range(T):
        assert mask_to_ranks(p.token_mask[t]) == bf["dest"][t]
        assert p.token_ndest[t] == len(bf["dest"][t])
        assert list(p.dest_rank[t, :len(bf["dest"][t])]) == bf["dest"][t]
        assert all(v == -1 for v in p.dest_rank[t, len(bf["dest"][t]):])
        assert all(v == -1 for v in p.dest_pos[t, len(bf["dest"][t]):])
        for i, r in enumerate(bf["dest"][t]):
            assert p.dest_pos[t, i] == bf["recv_tokens"][r].index(t)
    # groups
    assert list(p.token_group) == bf["token_group"]
    assert p.totals["G"] == bf["G"]
    Tn = len(bf["mw_row_token"])
    assert p.totals["T_nonempty"] == Tn
    assert list(p.mw_row_token[:Tn]) == bf["mw_row_token"]
    assert all(v == -1 for v in p.mw_row_token[Tn:])
    assert list(p.group_offsets[:bf["G"] + 1]) == bf["group_offsets"]
    for g in range(bf["G"]):
        assert mask_to_ranks(p.group_mask[g]) == bf["group_sets"][g]
    for t in range(T):
        assert p.token_mw_row[t] == (bf["mw_row_token"].index(t) if bf["dest"][t] else -1)
    # ranks
    counts = [len(v) for v in bf["recv_tokens"]]
    assert list(np.diff(p.rank_offsets)) == counts and p.rank_offsets[0] == 0
    flat = [t for r in range(R) for t in bf["recv_tokens"][r]]
    assert list(p.rank_tokens[:len(flat)]) == flat
    assert all(v == -1 for v in p.rank_tokens[len(flat):])
    assert p.totals["total_dest"] == len(flat)
    # byte accounting
    sent = [[r for r in d if r != src_rank] for d in bf["dest"]]
    assert p.totals["mw_bytes"] == sum(1 for d in sent if d) * B
    assert p.totals["unicast_bytes"] == sum(len(d) for d in sent) * B
    assert p.totals["unicast_per_expert_bytes"] == bf["valid"] * B
    assert p.totals["status"] == (mwo.MWO_ERR_BAD_INDEX if bf["bad"] else 0)
    # buffers
    send_mw = mwo.pack_mw(p, x)
    assert [send_mw[j].tobytes() for j in range(Tn)] == [xb[t].tobytes() for t in bf["mw_row_token"]]
    send_uc = mwo.pack_uc(p, x)
    assert [send_uc[i].tobytes() for i in range(len(flat))] == [xb[t].tobytes() for t in flat]
    want_compact = b"".join(b"".join(rows) for rows in bf["recv"])
    for recv in (mwo.deliver_mw(p, send_mw), mwo.deliver_uc(p, send_uc), mwo.deliver_definition(p, x, ids, e2r)):
        assert recv.tobytes() == want_compact
    # strided regions with a sentinel fill: rows land where they should, nothing else is touched
    stride = (max(counts) + 1) * B if counts else B
    want = bytearray(b"\xAB" * (R * stride))
    for r in range(R):
        blob = b"".join(bf["recv"][r])
        want[r * stride:r * stride + len(blob)] = blob
    for recv in (mwo.deliver_mw(p, send_mw, stride, 0xAB), mwo.deliver_uc(p, send_uc, stride, 0xAB),
                 mwo.deliver_definition(p, x, ids, e2r, stride, 0xAB)):
        assert recv.tobytes() == bytes(want)
    return p, bf


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("R,E,K", [(3, 6, 2), (8, 32, 4), (9, 9, 3), (65, 130, 4), (2, 8, 5)])
def test_brute_force_tiny(seed, R, E, K):
    inp = wl.make_random_dispatch(seed, T=29, K=K, E=E, R=R, H=8, pad_fraction=0.15 if seed % 2 else 0.0,
                                  contiguous_map=(seed % 3 == 0))
    check_against_brute_force(inp, R)


def test_brute_force_with_padding_duplicates_and_invalid_ids():
    inp = wl.make_random_dispatch(7, T=31, K=4, E=12, R=5, H=8, pad_fraction=0.3, distinct=False)
    ids = inp.topk_ids.copy()
    ids[3, :] = -1            # a token with no destination at all
    ids[4, 0] = 12            # id == E: invalid
    ids[5, 1] = -2            # negative but not the padding value: invalid
    ids[6, :] = ids[6, 0]     # the same expert four times
    inp.topk_ids = ids
    p, bf = check_against_brute_force(inp, 5)
    assert bf["bad"] and p.token_group[3] == -1 and p.token_mw_row[3] == -1
    e2r = inp.expert_to_rank.copy()
    e2r[2] = 5                # table entry == R: invalid
    inp.expert_to_rank = e2r
    check_against_brute_force(inp, 5)


def test_groups_differing_only_in_a_high_word():
    """Tokens that share the first 64 ranks' bits but differ above rank 63 are different groups."""
    R = 130
    inp = wl.make_random_dispatch(1, T=12, K=2, E=R, R=R, H=8)
    inp.expert_to_rank = np.arange(R, dtype=np.int32)
    inp.topk_ids = np.array([[0, 64], [0, 65], [0, 64], [0, 129], [0, 128], [0, 0], [0, 129], [5, 64], [0, 65],
                             [64, 0], [128, 0], [0, -1]], np.int32)
    p, bf = check_against_brute_force(inp, R)
    assert bf["G"] == 6 and list(p.token_group) == [0, 1, 0, 2, 3, 4, 2, 5, 1, 0, 3, 4]


def test_brute_force_source_inside_domain():
    inp = wl.make_random_dispatch(11, T=40, K=3, E=16, R=6, H=8)
    p, _ = check_against_brute_force(inp, 6, src_rank=2)
    q = mwo.plan(inp.topk_ids, inp.expert_to_rank, 6, 16, -1)
    assert q.totals["unicast_bytes"] - p.totals["unicast_bytes"] == int(np.diff(q.rank_offsets)[2]) * 16


def test_tiny_configuration_brute_force():
    inp = wl.make_dispatch("tiny", H=16)
    p, bf = check_against_brute_force(inp, 8)
    # at most 4 of 8 ranks per token: the number of possible destination sets bounds G
    assert bf["G"] <= sum(math.comb(8, j) for j in range(1, 5)) == 162


# ----------------------------------------------------------------------------------------------
# (b) invariants at configuration sizes
# ----------------------------------------------------------------------------------------------
def check_invariants(p, ids, e2r):
    T, K, R, Kd, B = p.T, p.K, p.R, p.Kd, p.row_bytes
    tot = p.totals
    Tn, G, SD = tot["T_nonempty"], tot["G"], tot["total_dest"]
    # library bincount over the per-token deduplicated rank lists
    ranks = e2r[np.clip(ids, 0, len(e2r) - 1)].astype(np.int64)
    ranks[ids < 0] = -1
    onehot = np.zeros((T, R), bool)
    tt, kk = np.nonzero(ranks >= 0)
    onehot[tt, ranks[tt, kk]] = True
    counts = onehot.sum(0)
    assert np.array_equal(np.diff(p.rank_offsets), counts) and p.rank_offsets[0] == 0 and p.rank_offsets[R] == SD
    assert np.array_equal(p.token_ndest, onehot.sum(1))
    assert SD == p.token_ndest.sum() and (p.token_ndest <= Kd).all()
    # the bitmaps, bit by bit (rank r = bit r mod 64 of word r div 64), and nothing beyond rank R - 1
    bits = ((p.token_mask[:, np.arange(R) // 64] >> (np.arange(R) % 64).astype(np.uint64)) & np.uint64(1)).astype(bool)
    assert np.array_equal(bits, onehot)
    assert sum(int(v).bit_count() for v in p.token_mask.reshape(-1)) == SD
    # a token's destination list: its ranks ascending, then -1
    want_ranks = np.where(onehot, np.arange(R)[None, :], R + 1)
    want_ranks.sort(axis=1)
    want_ranks = np.where(want_ranks[:, :Kd] > R, -1, want_ranks[:, :Kd])
    assert np.array_equal(p.dest_rank, want_ranks)
    assert np.array_equal(p.dest_pos < 0, p.dest_rank < 0)
    assert np.array_equal(p.token_group < 0, p.token_ndest == 0) and np.array_equal(p.token_mw_row < 0, p.token_ndest == 0)
    # offsets monotone, summing to totals
    go = p.group_offsets[:G + 1]
    assert go[0] == 0 and (np.diff(go) >= 1).all() and go[G] == Tn
    assert (p.group_offsets[G + 1:] == -1).all()
    # mw_row_token is a bijection onto the non-empty tokens and inverts token_mw_row
    nonempty = np.nonzero(p.token_ndest > 0)[0]
    assert np.array_equal(np.sort(p.mw_row_token[:Tn]), nonempty)
    assert np.array_equal(p.token_mw_row[p.mw_row_token[:Tn]], np.arange(Tn))
    # groups: equal mask <=> equal group, numbered by first occurrence, members ascending
    g_of_row = p.token_group[p.mw_row_token[:Tn]]
    assert (np.diff(g_of_row) >= 0).all()
    same = np.diff(g_of_row) == 0
    assert (np.diff(p.mw_row_token[:Tn])[same] > 0).all()
    leaders = p.mw_row_token[:Tn][go[:-1]]
    assert (np.diff(leaders) > 0).all()
    assert np.array_equal(p.group_mask[g_of_row], p.token_mask[p.mw_row_token[:Tn]])
    assert len(np.unique(p.group_mask[:G], axis=0)) == G
    # rank_tokens strictly ascending inside each segment; dest_pos is the running count
    for r in range(R):
        seg = p.rank_tokens[p.rank_offsets[r]:p.rank_offsets[r + 1]]
        assert (np.diff(seg) > 0).all()
        assert np.array_equal(seg, np.nonzero(onehot[:, r])[0])
    running = np.cumsum(onehot, axis=0) - onehot
    tt, ii = np.nonzero(p.dest_rank >= 0)
    assert np.array_equal(p.dest_pos[tt, ii], running[tt, p.dest_rank[tt, ii]])
    assert np.array_equal(np.sort(np.stack([tt, p.dest_rank[tt, ii]], 1), axis=0),
                          np.sort(np.stack(np.nonzero(onehot), 1), axis=0))
    # bytes
    assert tot["mw_bytes"] == Tn * B == int(np.diff(go).sum()) * B
    assert tot["unicast_bytes"] == SD * B
    assert tot["unicast_per_expert_bytes"] == int((ranks >= 0).sum()) * B
    return onehot


@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
@pytest.mark.parametrize("seed", [None, 100])
def test_configuration_invariants_and_exactly_once(cfg, seed):
    H = 8  # payload rows are tagged, not drawn: 16 bytes carrying (token, checksum)
    inp = wl.make_dispatch(cfg, seed, payload=False)
    s = inp.shape
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, 2 * H)
    assert p.ret == 0 and p.totals["status"] == 0
    onehot = check_invariants(p, inp.topk_ids, inp.expert_to_rank)
    # exactly-once delivery: tag every row with its token index and read the tags back from recv
    x = np.zeros((s.T, H), np.uint16)
    x.view(np.int32).reshape(s.T, -1)[:, 0] = np.arange(s.T)
    x.view(np.int32).reshape(s.T, -1)[:, 1] = np.arange(s.T) * 7 + 1
    send_mw, send_uc = mwo.pack_mw(p, x), mwo.pack_uc(p, x)
    a = mwo.deliver_mw(p, send_mw)
    b = mwo.deliver_uc(p, send_uc)
    c = mwo.deliver_definition(p, x, inp.topk_ids, inp.expert_to_rank)
    assert np.array_equal(a, b) and np.array_equal(a, c)
    assert np.array_equal(send_uc.reshape(-1), a)          # unicast send buffer == compact receive area
    tags = a.view(np.int32).reshape(-1, 4)[:, 0]
    pairs = set()
    for r in range(s.R):
        for t in tags[p.rank_offsets[r]:p.rank_offsets[r + 1]]:
            assert (int(t), r) not in pairs
            pairs.add((int(t), r))
    assert pairs == set(zip(*map(lambda v: v.tolist(), np.nonzero(onehot))))


def test_decode_configuration_closed_form():
    inp = wl.make_dispatch("decode", payload=False)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, 256, 14336)
    assert (p.token_ndest == 8).all()                       # one expert per rank, distinct experts
    assert p.totals["total_dest"] == 64 * 8 and p.W == 4
    assert p.totals["mw_bytes"] * 8 == p.totals["unicast_bytes"]      # saved = 1 - 1/8 exactly
    assert p.totals["unicast_per_expert_bytes"] == p.totals["unicast_bytes"]


@pytest.mark.parametrize("R,E,K,want", [(64, 256, 8, 7.68), (128, 256, 8, 7.89)])
def test_uniform_routing_expected_destinations(R, E, K, want):
    """E|D_t| = R (1 - C(E - E/R, K) / C(E, K)) for K distinct uniform experts."""
    closed = R * (1 - math.comb(E - E // R, K) / math.comb(E, K))
    assert abs(closed - want) < 0.006
    inp = wl.make_random_dispatch(5, T=4096, K=K, E=E, R=R, H=8, contiguous_map=True)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, 16)
    assert abs(p.totals["total_dest"] / 4096 - closed) / closed < 0.01
    saved = 1 - p.totals["mw_bytes"] / p.totals["unicast_bytes"]
    assert abs(saved - (1 - 1 / closed)) < 0.01


# ----------------------------------------------------------------------------------------------
# (c) special cases that reduce to library routines
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("R", [5, 64, 100])
def test_top1_is_a_stable_counting_sort(R):
    rng = np.random.default_rng(R)
    T, E = 777, 2 * R
    ids = rng.integers(0, E, size=(T, 1), dtype=np.int32)
    e2r = rng.integers(0, R, size=E, dtype=np.int32)
    x = wl.normal_bf16(rng, (T, 8))
    p = mwo.plan(ids, e2r, R, 16)
    key = e2r[ids[:, 0]]
    order = np.argsort(key, kind="stable")
    assert np.array_equal(p.rank_tokens[:T], order)
    assert np.array_equal(np.diff(p.rank_offsets), np.bincount(key, minlength=R))
    xb = x.view(np.uint8).reshape(T, 16)
    assert np.array_equal(mwo.pack_uc(p, x), xb[order])
    # groups are the ranks present, numbered by first occurrence
    _, first = np.unique(key, return_index=True)
    ranks_by_first = key[np.sort(first)]
    assert p.totals["G"] == len(ranks_by_first)
    for g, r in enumerate(ranks_by_first):
        assert mask_to_ranks(p.group_mask[g]) == [int(r)]
    gid = np.empty(R, np.int64)
    gid[ranks_by_first] = np.arange(len(ranks_by_first))
    assert np.array_equal(p.mw_row_token[:T], np.argsort(gid[key], kind="stable"))
    assert p.totals["mw_bytes"] == p.totals["unicast_bytes"]          # nothing to save with one destination


def test_identical_and_all_distinct_tokens():
    T, R, E = 50, 70, 70
    e2r = np.arange(E, dtype=np.int32)
    same = np.tile(np.array([[3, 66, 9]], np.int32), (T, 1))
    p = mwo.plan(same, e2r, R, 32)
    assert p.totals["G"] == 1 and np.array_equal(p.mw_row_token, np.arange(T)) and (p.token_group == 0).all()
    assert list(p.group_offsets[:2]) == [0, T]
    distinct = np.stack([np.arange(T), (np.arange(T) + 1) % E], 1).astype(np.int32)  # {t, t+1}: all different
    p = mwo.plan(distinct, e2r, R, 32)
    assert p.totals["G"] == T and np.array_equal(p.mw_row_token, np.arange(T))
    assert np.array_equal(p.token_group, np.arange(T)) and np.array_equal(p.group_offsets, np.arange(T + 1))
    one = np.full((T, 4), 5, np.int32)                                                # all ids equal: a single bit
    p = mwo.plan(one, e2r, R, 32)
    assert (p.token_ndest == 1).all() and mask_to_ranks(p.group_mask[0]) == [5]
    assert p.totals["unicast_per_expert_bytes"] == 4 * p.totals["unicast_bytes"]


@pytest.mark.parametrize("R", [1, 63, 64, 65, 128, 129, 256, 1024])
def test_word_boundaries(R):
    E = R
    e2r = np.arange(E, dtype=np.int32)
    ids = np.array([[0, R - 1], [R - 1, R - 1], [max(R - 2, 0), 0]], np.int32)
    p = mwo.plan(ids, e2r, R, 16)
    assert p.W == (R + 63) // 64 and p.token_mask.shape == (3, p.W)
    assert mask_to_ranks(p.token_mask[0]) == sorted({0, R - 1})
    assert mask_to_ranks(p.token_mask[1]) == [R - 1]
    # bits at or above R are never set
    full = np.arange(R, dtype=np.int32)[None, :]
    q = mwo.plan(full, e2r, R, 16)
    assert mask_to_ranks(q.token_mask[0]) == list(range(R)) and q.token_ndest[0] == R
    if R % 64:
        assert int(q.token_mask[0, -1]) >> (R % 64) == 0


def test_empty_batch():
    p = mwo.plan(np.zeros((0, 4), np.int32), np.zeros(8, np.int32), 4, 16)
    assert p.ret == 0 and p.totals["G"] == 0 and p.totals["total_dest"] == 0
    assert list(p.rank_offsets) == [0] * 5 and list(p.group_offsets) == [0]


def test_invalid_arguments():
    ids = np.zeros((2, 2), np.int32)
    assert mwo.plan(ids, np.zeros(4, np.int32), 0, 16).ret == mwo.MWO_ERR_INVALID_ARG
    assert mwo.plan(ids, np.zeros(4, np.int32), 4, 0).ret == mwo.MWO_ERR_INVALID_ARG
    assert mwo.plan(ids, np.zeros(4, np.int32), 4, 16, src_rank=4).ret == mwo.MWO_ERR_INVALID_ARG


# ----------------------------------------------------------------------------------------------
# AllGather
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("layout", [mwo.LAYOUT_MULTIWRITE, mwo.LAYOUT_UNICAST])
@pytest.mark.parametrize("R,S,begin,count", [(8, 64, 0, 8), (5, 48, 1, 3), (64, 4096, 0, 64), (4, 16, 3, 1), (1, 32, 0, 1)])
def test_allgather_is_concatenate(layout, R, S, begin, count):
    sh = wl.make_allgather_shards(R, S, seed=4)
    send, recv, tot, ret = mwo.allgather(sh, layout, begin, count, fill=0xCD)
    assert ret == 0
    want = np.concatenate([sh[i] for i in range(R)])
    assert np.array_equal(recv.reshape(count, R * S), np.broadcast_to(want, (count, R * S)))
    if layout == mwo.LAYOUT_MULTIWRITE:
        assert np.array_equal(send.reshape(R, S), sh)
    else:
        s3 = send.reshape(R, count, S)
        for i in range(R):
            for d in range(count):
                if begin + d == i:
                    assert (s3[i, d] == 0xCD).all()        # the self copy is never transmitted
                else:
                    assert np.array_equal(s3[i, d], sh[i])
    assert tot["mw_bytes"] == (R * S if R > 1 else 0) and tot["unicast_bytes"] == R * (R - 1) * S
    # strided regions leave the gaps untouched
    stride = R * S + 32
    _, recv2, _, _ = mwo.allgather(sh, layout, begin, count, recv_stride_bytes=stride, fill=0xEE)
    r2 = recv2.reshape(count, stride)
    assert np.array_equal(r2[:, :R * S], recv.reshape(count, R * S)) and (r2[:, R * S:] == 0xEE).all()


def test_allgather_saved_closed_form_and_paper_example():
    consts = load_paper_constants()
    sh = wl.make_allgather_shards(8, 32)
    _, _, tot, _ = mwo.allgather(sh, mwo.LAYOUT_MULTIWRITE)
    # Section 2.3.1: in an 8-node domain each source transmits its partition seven times
    assert tot["unicast_bytes"] // tot["mw_bytes"] == consts["allgather_8_nodes_unicast_copies_per_source"] == 7
    sh = wl.make_allgather_shards(64, 4096)
    _, _, tot, _ = mwo.allgather(sh, mwo.LAYOUT_MULTIWRITE, 0, 2)
    assert abs((1 - tot["mw_bytes"] / tot["unicast_bytes"]) - (1 - 1 / 63)) < 1e-12
    assert mwo.allgather(sh, 2)[3] == mwo.MWO_ERR_INVALID_ARG
    assert mwo.allgather(sh, 0, 60, 8)[3] == mwo.MWO_ERR_INVALID_ARG


def test_allgather_bitmap_overhead_beyond_64_ranks():
    """Section 6.4: up to 64 ranks the bitmap rides in the 64-bit immediate field (no payload bytes); beyond
    that it is carried in the payload, one bitmap of one bit per rank with every 4096-byte packet."""
    c = load_paper_constants()
    P = c["meta_payload_bytes"]
    # 64 ranks: nothing; 65 ranks: two words although one bit would do (whole 64-bit words travel)
    assert mwo.allgather(wl.make_allgather_shards(64, 64), mwo.LAYOUT_MULTIWRITE, 0, 1)[2]["meta_bytes"] == 0
    assert mwo.allgather(wl.make_allgather_shards(65, 64), mwo.LAYOUT_MULTIWRITE, 0, 1)[2]["meta_bytes"] == 65 * 1 * 16
    # 128 ranks, one packet per shard: 128 shards x 1 packet x 128 bits
    sh = wl.make_allgather_shards(128, P)
    for layout in (mwo.LAYOUT_MULTIWRITE, mwo.LAYOUT_UNICAST):
        tot = mwo.allgather(sh, layout, 0, 1)[2]
        assert tot["meta_bytes"] == 128 * 1 * (128 // 8)
    # a shard one byte-vector longer than a packet needs a second bitmap
    assert mwo.allgather(wl.make_allgather_shards(128, P + 16), mwo.LAYOUT_MULTIWRITE, 0, 1)[2]["meta_bytes"] == 128 * 2 * 16
    # 1024 ranks: 1024 bits per 4096-byte packet = the paper's 3.13 % of the transmitted payload
    tot = mwo.allgather(wl.make_allgather_shards(1024, P), mwo.LAYOUT_MULTIWRITE, 0, 1)[2]
    assert tot["meta_bytes"] * 8 == 1024 * c["meta_bits_1024_ranks"]
    assert 100 * tot["meta_bytes"] / tot["mw_bytes"] == 3.125
    assert math.floor(100 * 3.125 + 0.5) / 100 == c["meta_overhead_percent_1024_ranks"]


def test_large_shard_generator_marks_every_page():
    sh = wl.make_allgather_shards(3, 4 << 20)
    pages = sh.view(np.uint64).reshape(3, -1, 512)[:, :, 0]
    assert len(np.unique(pages)) == pages.size


# ----------------------------------------------------------------------------------------------
# (d) constants printed in the paper
# ----------------------------------------------------------------------------------------------
def load_paper_constants():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = [s.strip() for s in line.split("=")]
            out[k] = float(v) if "." in v else int(v)
    return out


def test_paper_constants():
    c = load_paper_constants()
    # Section 2.3.2: the destination-set space at EP = 64, top-8
    assert math.comb(64, 8) == 4426165368 > c["group_space_ep64_top8_exceeds"]
    # Section 4.1: an address list for 8 destinations is 128 bytes; the bitmap for <= 64 ranks is 8 bytes
    assert 8 * c["eid_bits"] // 8 == c["eid_list_bytes_8_dests"]
    e2r = np.arange(64, dtype=np.int32)
    p = mwo.plan(np.arange(8, dtype=np.int32)[None, :], e2r, 64, 4096)
    assert p.token_mask.nbytes == c["bitmap_bits_small_domain"] // 8 and p.totals["meta_bytes"] == 0
    # Section 6.4: 1024 ranks, 4096-byte payload: 1024 bits of bitmap per packet = 3.13 %
    e2r = np.arange(1024, dtype=np.int32)
    p = mwo.plan(np.array([[0, 1023], [5, 6]], np.int32), e2r, 1024, c["meta_payload_bytes"])
    per_row = p.totals["meta_bytes"] / 2
    assert per_row * 8 == c["meta_bits_1024_ranks"]
    assert 100 * per_row / c["meta_payload_bytes"] == 3.125           # printed rounded half-up as 3.13
    assert math.floor(100 * 3.125 + 0.5) / 100 == c["meta_overhead_percent_1024_ranks"]
    # two packets per row when the row is 8192 bytes
    p = mwo.plan(np.array([[0, 1023]], np.int32), e2r, 1024, 8192)
    assert p.totals["meta_bytes"] == 2 * 128
    # Section 3.1: the relayed segment crosses the pair link 3 times (unicast) vs once (MultiWrite):
    # a 4-destination set {5,6,7,8}\{5}... modelled as one token bound for 3 ranks
    p = mwo.plan(np.array([[1, 2, 3]], np.int32), np.arange(8, dtype=np.int32), 8, 16)
    assert p.totals["unicast_bytes"] // p.totals["mw_bytes"] == c["relay_link_copies_unicast"]
    assert p.totals["mw_bytes"] // 16 == c["relay_link_copies_multicast"]
