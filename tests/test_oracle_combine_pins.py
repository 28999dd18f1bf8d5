"""Pins for the oracle's combine (reverse of dispatch): cases whose result is exact and known
independently of the oracle, plus the bf16 rounding helper against exhaustive enumeration."""
import numpy as np
import pytest

from oracle import mwo
from paper_2605_22428_b200 import workloads as wl


def bf16_to_f32(bits):
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def dest_sets(inp, R):
    out = []
    for t in range(inp.T):
        s = set()
        for e in inp.topk_ids[t]:
            if 0 <= e < len(inp.expert_to_rank) and 0 <= inp.expert_to_rank[e] < R:
                s.add(int(inp.expert_to_rank[e]))
        out.append(sorted(s))
    return out


def test_combine_of_dispatch_with_one_destination_is_identity():
    inp = wl.make_random_dispatch(3, T=200, K=1, E=16, R=8, H=24)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, 8, 48)
    z = mwo.deliver_definition(p, inp.x, inp.topk_ids, inp.expert_to_rank)
    assert np.array_equal(mwo.combine(p, z), inp.x)


@pytest.mark.parametrize("strided", [False, True])
def test_one_hot_weights_select_one_destination(strided):
    """w = unit vector e_i returns exactly the row the i-th destination sent back: checks every (token, i) slot."""
    R, B = 12, 32
    inp = wl.make_random_dispatch(5, T=90, K=4, E=36, R=R, H=B // 2, pad_fraction=0.15)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    D = dest_sets(inp, R)
    counts = np.diff(p.rank_offsets)
    stride = (int(counts.max()) + 2) * B if strided else 0
    # each rank answers with rows tagged (rank, slot): z[r][i] is filled with the bf16 value 1 + r + (i mod 8) / 8 (exact)
    nbytes = R * stride if strided else int(p.rank_offsets[R]) * B
    z = np.zeros(nbytes // 2, np.uint16)
    tag = {}
    for r in range(R):
        for i in range(int(counts[r])):
            val = np.float32(1 + r + (i % 8) / 8.0)
            bits = wl.f32_to_bf16_bits(np.array([val], np.float32))[0]
            assert bf16_to_f32(np.array([bits], np.uint16))[0] == val
            start = (r * stride if strided else int(p.rank_offsets[r]) * B) // 2 + i * (B // 2)
            z[start:start + B // 2] = bits
            tag[(r, i)] = bits
    for i_sel in range(p.Kd):
        w = np.zeros((inp.T, p.Kd), np.float32)
        w[:, i_sel] = 1.0
        y = mwo.combine(p, z.view(np.uint8), w, stride)
        for t in range(inp.T):
            if i_sel < len(D[t]):
                r = D[t][i_sel]
                slot = sum(1 for u in range(t) if r in D[u])
                assert (y[t] == tag[(r, slot)]).all(), (t, i_sel)
            else:
                assert (y[t] == 0).all()


def test_unit_weights_sum_small_integers_exactly():
    """Rank r answers with the constant r + 1; y[t] = sum of (r + 1) over the destinations of t (exact in bf16)."""
    R, B = 16, 32
    inp = wl.make_random_dispatch(8, T=300, K=6, E=64, R=R, H=B // 2, contiguous_map=True)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    D = dest_sets(inp, R)
    z = np.zeros((int(p.rank_offsets[R]), B // 2), np.uint16)
    for r in range(R):
        z[p.rank_offsets[r]:p.rank_offsets[r + 1]] = wl.f32_to_bf16_bits(np.array([r + 1], np.float32))[0]
    y = bf16_to_f32(mwo.combine(p, z.view(np.uint8)))
    for t in range(inp.T):
        assert (y[t] == float(sum(r + 1 for r in D[t]))).all()
    # weights scale linearly: w = 0.5 halves every exact sum
    w = np.full((inp.T, p.Kd), 0.5, np.float32)
    y2 = bf16_to_f32(mwo.combine(p, z.view(np.uint8), w))
    assert np.array_equal(y2, y / 2)


def test_rounding_is_nearest_even_with_a_single_rounding():
    """Two destinations answer a and b; y must be the bf16 nearest to the real a + b, ties to even.
    Checked against exact rational arithmetic over many bf16 pairs, including ties and carries."""
    from fractions import Fraction
    rng = np.random.default_rng(0)
    R, B, T = 2, 32, 1
    ids = np.array([[0, 1]], np.int32)
    e2r = np.array([0, 1], np.int32)
    p = mwo.plan(ids, e2r, R, B)
    a_bits = np.concatenate([rng.integers(0x3800, 0x4800, 4000), rng.integers(0xB800, 0xC800, 4000),
                             np.array([0x3F80, 0x3F81, 0x3F83, 0x7F7F, 0x0001, 0x0080])]).astype(np.uint16)
    b_bits = np.concatenate([rng.integers(0x3800, 0x4800, 4000), rng.integers(0x3000, 0x4000, 4000),
                             np.array([0x3B80, 0x3B80, 0x3B80, 0x7F7F, 0x0001, 0x8001])]).astype(np.uint16)
    n = len(a_bits)
    out = np.zeros(n, np.uint16)
    for k0 in range(0, n, B // 2):
        k1 = min(n, k0 + B // 2)
        z = np.zeros((2, B // 2), np.uint16)
        z[0, :k1 - k0], z[1, :k1 - k0] = a_bits[k0:k1], b_bits[k0:k1]
        out[k0:k1] = mwo.combine(p, z.view(np.uint8))[0, :k1 - k0]
    for k in range(n):
        exact = Fraction(float(bf16_to_f32(a_bits[k:k + 1])[0])) + Fraction(float(bf16_to_f32(b_bits[k:k + 1])[0]))
        got = out[k]
        if abs(exact) >= Fraction(2) ** 128:
            assert got & 0x7FFF == 0x7F80
            continue
        gv = Fraction(float(bf16_to_f32(np.array([got], np.uint16))[0]))
        # neighbours of the result in bf16
        lo = Fraction(float(bf16_to_f32(np.array([got - 1 if got & 0x7FFF else got], np.uint16))[0]))
        hi = Fraction(float(bf16_to_f32(np.array([got + 1], np.uint16))[0])) if (got & 0x7FFF) < 0x7F7F else None
        err = abs(exact - gv)
        for nb in (lo, hi):
            if nb is not None:
                assert err <= abs(exact - nb), (k, hex(int(a_bits[k])), hex(int(b_bits[k])), hex(int(got)))
                if err == abs(exact - nb) and nb != gv:
                    assert got & 1 == 0, "ties go to the even significand"
