"""GPU parity of mw_combine (Section 2.3.2: results return to the sender) against the oracle's combine.

The kernel's contract is stated step by step: binary32 fused multiply-adds over the destinations in ascending
rank order, one rounding to bf16.  The oracle's binary32 mode performs exactly those correctly rounded steps in
plain C, so the comparison is bit for bit, on random weights and data too.  The oracle's binary64 mode stays the
accuracy reference: the kernel is within one bf16 unit in the last place plus the binary32 accumulation error,
Kd * 2^-23 * sum |w z|, of it.
"""
import numpy as np
import pytest

from gpu_util import Guarded, torch_mod
from oracle import mwo
from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import workloads

pytestmark = pytest.mark.gpu


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 values that are exactly representable in bf16 -> their 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert not (u & 0xFFFF).any()
    return (u >> 16).astype(np.uint16)


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def random_bf16(rng, shape) -> np.ndarray:
    u = rng.standard_normal(shape, dtype=np.float32).view(np.uint32) & 0xFFFF0000
    return (u >> 16).astype(np.uint16)


def gpu_combine(inp, z_bits_of, weights, mode, src_rank=-1):
    """Plans inp on the GPU, fills z (built from the oracle's plan by z_bits_of) and combines.  Returns (plan, y, z, stride)."""
    torch = torch_mod()
    s = inp.shape
    T, B = inp.T, s.row_bytes
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, s.R, B, src_rank)
    counts = np.diff(p.rank_offsets)
    SD = p.totals["total_dest"]
    cap = int(counts.max()) + 1 if mode == "strided" else SD
    stride = cap * B if mode == "strided" else 0
    rows = s.R * cap if mode == "strided" else SD
    z = z_bits_of(p, rows, cap if mode == "strided" else 0)                  # uint16 [rows, B/2]
    ids_d = torch.from_numpy(inp.topk_ids).cuda()
    e2r_d = torch.from_numpy(inp.expert_to_rank).cuda()
    z_d = torch.from_numpy(z.view(np.int16)).cuda()
    w_d = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights, dtype=np.float32)).cuda()
    y = Guarded(T * B)
    with mw.Context(s.R, s.E, s.K, max(T, 1), B, src_rank=src_rank) as ctx:
        ctx.mw_plan(ids_d, e2r_d, T)
        ctx.mw_combine(z_d.data_ptr(), stride, None if w_d is None else w_d.data_ptr(), y.ptr())
        torch.cuda.synchronize()
        assert ctx.mw_get_totals()["status"] == 0
    assert y.guards_intact()
    got = y.host().view(np.uint16).reshape(T, B // 2)
    return p, got, z, stride


def slot_row(p, r, pos, cap):
    return r * cap + pos if cap else int(p.rank_offsets[r]) + pos


@pytest.mark.parametrize("mode", ["compact", "strided"])
@pytest.mark.parametrize("cfg", ["tiny", "decode"])
def test_random_data_bit_exact_in_stated_order_and_within_one_ulp_of_fp64(cfg, mode):
    inp = workloads.make_dispatch(cfg, seed=11)
    rng = np.random.default_rng(5)
    Kd = min(inp.shape.K, inp.shape.R)
    w = rng.random((inp.T, Kd), dtype=np.float32)
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, inp.shape.row_bytes // 2)), w, mode)
    assert np.array_equal(got, mwo.combine(p, z, w, stride, precision="f32"))          # the stated order: bit for bit
    want = mwo.combine(p, z, w, stride)
    a, b = bf16_to_f64(got), bf16_to_f64(want)
    # bound: one bf16 ulp of the result (2^-7 relative covers the ulp of either neighbour) + fp32 accumulation error
    cap = stride // inp.shape.row_bytes
    absum = np.zeros_like(b)
    for t in range(inp.T):
        for i in range(int(p.token_ndest[t])):
            r, pos = int(p.dest_rank[t, i]), int(p.dest_pos[t, i])
            absum[t] += abs(float(w[t, i])) * np.abs(bf16_to_f64(z[slot_row(p, r, pos, cap)]))
    assert np.all(np.abs(a - b) <= 2.0 ** -7 * np.abs(b) + Kd * 2.0 ** -23 * absum)
    assert np.mean(got == want) > 0.99, np.mean(got == want)


@pytest.mark.parametrize("mode", ["compact", "strided"])
@pytest.mark.parametrize("K,pad", [(6, 0.1), (2, 0.5)])
def test_random_weights_and_rows_bit_exact(mode, K, pad):
    inp = workloads.make_random_dispatch(21, T=900, R=130, E=260, K=K, H=1032, pad_fraction=pad)
    rng = np.random.default_rng(K)
    Kd = min(inp.shape.K, inp.shape.R)
    w = (rng.standard_normal((inp.T, Kd)) * 1.5).astype(np.float32)
    for weights in (w, None):
        p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, 1032)), weights, mode)
        assert np.array_equal(got, mwo.combine(p, z, weights, stride, precision="f32"))


def test_maximum_top_k_bit_exact():
    inp = workloads.make_random_dispatch(64, T=400, R=128, E=256, K=64, H=264, pad_fraction=0.05)     # up to 64 addends per element
    rng = np.random.default_rng(64)
    w = (rng.standard_normal((inp.T, 64)) * 0.7).astype(np.float32)
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, 264)), w, "strided")
    assert np.array_equal(got, mwo.combine(p, z, w, stride, precision="f32"))


def test_prefill_shape_full_size_bit_exact():
    """The shape the benchmark times (4096 tokens, 64 ranks, 14336-byte rows), random weights and rows."""
    inp = workloads.make_dispatch("dsv3_prefill", payload=False)
    rng = np.random.default_rng(12)
    H = inp.shape.row_bytes // 2
    w = rng.random((inp.T, 8), dtype=np.float32)
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, H)), w, "compact")
    want = mwo.combine(p, z, w, stride, precision="f32")
    assert np.array_equal(got, want)


@pytest.mark.parametrize("mode", ["compact", "strided"])
@pytest.mark.parametrize("K,pad", [(6, 0.1), (2, 0.5)])
def test_small_integers_sum_exactly(mode, K, pad):
    # every partial sum is a small integer or a multiple of 1/8: exact in fp32 and in bf16, so bit-exact
    inp = workloads.make_random_dispatch(3, T=700, R=16, E=64, K=K, H=528, pad_fraction=pad)
    H = inp.shape.row_bytes // 2

    def zfill(p, rows, cap):
        z = np.zeros((rows, H), np.float32)
        for t in range(inp.T):
            for i in range(int(p.token_ndest[t])):
                r, pos = int(p.dest_rank[t, i]), int(p.dest_pos[t, i])
                z[slot_row(p, r, pos, cap)] = 1 + (r % 4) + ((t + np.arange(H)) % 8) / 8.0
        return bf16_bits(z)

    p, got, z, stride = gpu_combine(inp, zfill, None, mode)
    assert np.array_equal(got, mwo.combine(p, z, None, stride))
    half = np.full((inp.T, min(inp.shape.K, inp.shape.R)), 0.5, np.float32)
    p, got, z, stride = gpu_combine(inp, zfill, half, mode)
    assert np.array_equal(got, mwo.combine(p, z, half, stride))
    empty = np.flatnonzero(p.token_ndest == 0)
    assert (len(empty) > 0) == (K == 2) and not got[empty].any()


def test_one_destination_is_identity():
    inp = workloads.make_random_dispatch(9, T=300, R=8, E=8, K=1, H=3584)
    rng = np.random.default_rng(1)
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, 3584)), None, "compact")
    assert np.array_equal(got, mwo.combine(p, z, None, stride))
    for t in range(0, inp.T, 17):
        if p.token_ndest[t]:
            assert np.array_equal(got[t], z[slot_row(p, int(p.dest_rank[t, 0]), int(p.dest_pos[t, 0]), 0)])


def test_one_hot_weights_select_a_row():
    inp = workloads.make_random_dispatch(4, T=257, R=32, E=64, K=8, H=2056)
    rng = np.random.default_rng(2)
    Kd = 8
    w = np.zeros((inp.T, Kd), np.float32)
    p0 = mwo.plan(inp.topk_ids, inp.expert_to_rank, 32, 4112, -1)
    pick = np.array([rng.integers(0, max(int(n), 1)) for n in p0.token_ndest])
    w[np.arange(inp.T), pick] = 1.0
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, 2056)), w, "strided")
    assert np.array_equal(got, mwo.combine(p, z, w, stride))


def test_source_rank_excluded_and_errors():
    torch = torch_mod()
    inp = workloads.make_random_dispatch(6, T=64, R=4, E=8, K=2, H=32)
    rng = np.random.default_rng(3)
    p, got, z, stride = gpu_combine(inp, lambda p, rows, cap: random_bf16(rng, (rows, 32)), None, "compact", src_rank=1)
    assert np.array_equal(got, mwo.combine(p, z, None, stride, precision="f32"))
    want = mwo.combine(p, z, None, stride)
    # at most two addends: the fp32 sum is exact or off by 2^-24 of the larger one, so the result is within one ulp
    assert np.all(np.abs(bf16_to_f64(got) - bf16_to_f64(want)) <= 2.0 ** -7 * np.abs(bf16_to_f64(want)))
    assert np.mean(got == want) > 0.99
    assert not got[p.token_ndest == 0].any()
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with mw.Context(4, 8, 2, 64, 64) as ctx:
        assert ctx.mw_combine(buf.data_ptr(), 0, None, buf.data_ptr(), check=False) == mw.MW_ERR_NO_PLAN
        ctx.mw_plan(torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda(), 64)
        assert ctx.mw_combine(buf.data_ptr() + 8, 0, None, buf.data_ptr(), check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_combine(buf.data_ptr(), 24, None, buf.data_ptr(), check=False) == mw.MW_ERR_ALIGNMENT
        assert ctx.mw_combine(0, 0, None, buf.data_ptr(), check=False) == mw.MW_ERR_INVALID_ARG
