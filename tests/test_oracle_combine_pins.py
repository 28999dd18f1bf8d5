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


# ----------------------------------------------------------------------------------------------
# The binary32 mode: every step is correctly rounded, so exact rational arithmetic pins it bit for bit
# ----------------------------------------------------------------------------------------------
def round_nearest_even(x, frac_bits, min_exp=-126):
    """The binary floating-point value with `frac_bits` fraction bits nearest to the rational x (ties to even)."""
    from fractions import Fraction
    if x == 0:
        return Fraction(0)
    sign, a = (-1 if x < 0 else 1), abs(x)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    ulp = Fraction(2) ** (max(e, min_exp) - frac_bits)
    q = a / ulp
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * ulp


def test_round_helper_against_numpy_float32():
    from fractions import Fraction
    rng = np.random.default_rng(3)
    for v in np.concatenate([rng.standard_normal(300), rng.standard_normal(50) * 1e-30, [1 + 2.0 ** -24, 1 + 3 * 2.0 ** -24]]):
        assert round_nearest_even(Fraction(float(v)), 23) == Fraction(float(np.float32(v)))     # numpy rounds binary64 -> binary32 to nearest even


@pytest.mark.parametrize("seed,K", [(0, 8), (1, 3), (2, 5)])
def test_f32_mode_is_fused_multiply_add_in_rank_order_with_one_rounding(seed, K):
    """acc_0 = 0; acc_i = RN32(w_i * z_i + acc_{i-1}) over ascending ranks; y = RN_bf16(acc_last): redone with fractions."""
    from fractions import Fraction
    rng = np.random.default_rng(seed)
    R, H = 16, 16
    inp = wl.make_random_dispatch(20 + seed, T=24, K=K, E=48, R=R, H=H, pad_fraction=0.1)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, 2 * H)
    D = dest_sets(inp, R)
    rows = int(p.rank_offsets[R])
    zf = (rng.standard_normal((rows, H)) * np.exp2(rng.integers(-3, 4, (rows, H)))).astype(np.float32)
    z = wl.f32_to_bf16_bits(zf)
    w = (rng.standard_normal((inp.T, p.Kd)) * 1.7).astype(np.float32)
    y = mwo.combine(p, z.view(np.uint8), w, 0, precision="f32")
    zval = bf16_to_f32(z)
    differs_from_unfused = 0
    for t in range(inp.T):
        for c in range(H):
            acc, acc_unfused = Fraction(0), Fraction(0)
            for i, r in enumerate(D[t]):
                slot = sum(1 for u in range(t) if r in D[u])
                term = Fraction(float(w[t, i])) * Fraction(float(zval[int(p.rank_offsets[r]) + slot, c]))
                acc = round_nearest_even(term + acc, 23)
                acc_unfused = round_nearest_even(round_nearest_even(term, 23) + acc_unfused, 23)
            want = round_nearest_even(acc, 7)
            got = Fraction(float(bf16_to_f32(y[t, c:c + 1])[0]))
            assert got == want, (t, c, got, want)
            differs_from_unfused += acc != acc_unfused
    assert differs_from_unfused > 0        # the data can tell a fused multiply-add from a rounded product


def test_f32_mode_equals_f64_mode_where_every_partial_sum_is_exact():
    R, B = 16, 32
    inp = wl.make_random_dispatch(8, T=300, K=6, E=64, R=R, H=B // 2, contiguous_map=True)
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    z = np.zeros((int(p.rank_offsets[R]), B // 2), np.uint16)
    for r in range(R):
        z[p.rank_offsets[r]:p.rank_offsets[r + 1]] = wl.f32_to_bf16_bits(np.array([r + 1.125], np.float32))[0]
    for w in (None, np.full((inp.T, p.Kd), 0.5, np.float32)):
        assert np.array_equal(mwo.combine(p, z.view(np.uint8), w, precision="f32"), mwo.combine(p, z.view(np.uint8), w))
    one = wl.make_random_dispatch(3, T=200, K=1, E=16, R=8, H=24)
    p1 = mwo.plan(one.topk_ids, one.expert_to_rank, 8, 48)
    z1 = mwo.deliver_definition(p1, one.x, one.topk_ids, one.expert_to_rank)
    assert np.array_equal(mwo.combine(p1, z1, precision="f32"), one.x)


def test_f32_mode_stays_within_the_accumulation_bound_of_the_f64_mode():
    """|y32 - y64| <= one bf16 unit in the last place + Kd * 2^-23 * sum |w z| (the binary32 rounding of each partial sum)."""
    rng = np.random.default_rng(9)
    inp = wl.make_dispatch("tiny", seed=11)
    R, B = inp.shape.R, inp.shape.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    rows = int(p.rank_offsets[R])
    z = wl.f32_to_bf16_bits(rng.standard_normal((rows, B // 2)).astype(np.float32))
    w = rng.random((inp.T, p.Kd), dtype=np.float32)
    a = bf16_to_f32(mwo.combine(p, z.view(np.uint8), w, precision="f32")).astype(np.float64)
    b = bf16_to_f32(mwo.combine(p, z.view(np.uint8), w)).astype(np.float64)
    absum = np.zeros_like(b)
    zv = np.abs(bf16_to_f32(z).astype(np.float64))
    for t in range(inp.T):
        for i in range(int(p.token_ndest[t])):
            absum[t] += abs(float(w[t, i])) * zv[int(p.rank_offsets[p.dest_rank[t, i]]) + int(p.dest_pos[t, i])]
    assert np.all(np.abs(a - b) <= 2.0 ** -7 * np.abs(b) + p.Kd * 2.0 ** -23 * absum)
    assert np.mean(a == b) > 0.99


def test_f32_mode_does_not_round_the_product_before_the_addition():
    """Two destinations per token; the first returns 1.0 with weight -RN32(w2 * z2), so the sum is exactly the
    part of the product w2 * z2 that binary32 cannot hold: a fused multiply-add keeps it, a rounded product gives 0."""
    from fractions import Fraction
    rng = np.random.default_rng(4)
    T, H = 64, 16
    ids = np.tile(np.array([[0, 1]], np.int32), (T, 1))
    p = mwo.plan(ids, np.array([0, 1], np.int32), 2, 2 * H)
    assert np.array_equal(p.rank_offsets, [0, T, 2 * T]) and np.array_equal(p.dest_pos[:, 0], np.arange(T))
    z = np.zeros((2 * T, H), np.uint16)
    z[:T] = 0x3F80                                                                  # rank 0 answers 1.0 everywhere
    z[T:] = wl.f32_to_bf16_bits((1 + rng.random((T, H))).astype(np.float32))        # rank 1: values in [1, 2)
    w = np.zeros((T, 2), np.float32)
    w[:, 1] = (1 + rng.random(T)).astype(np.float32)
    for t in range(T):
        prod = Fraction(float(w[t, 1])) * Fraction(float(bf16_to_f32(z[T + t, :1])[0]))
        w[t, 0] = np.float32(float(-round_nearest_even(prod, 23)))
    y = mwo.combine(p, z.view(np.uint8), w, 0, precision="f32")
    nonzero = 0
    for t in range(T):
        for c in range(H):
            acc = round_nearest_even(Fraction(float(w[t, 0])) * 1 + 0, 23)
            acc = round_nearest_even(Fraction(float(w[t, 1])) * Fraction(float(bf16_to_f32(z[T + t, c:c + 1])[0])) + acc, 23)
            assert Fraction(float(bf16_to_f32(y[t, c:c + 1])[0])) == round_nearest_even(acc, 7), (t, c)
        nonzero += int(y[t, 0] & 0x7FFF != 0)
    assert nonzero > T // 2          # the residual of the product survives in most tokens
