"""Seeded synthetic inputs for the MultiWrite dispatch / AllGather path.

This module only *draws inputs* (router choices, the expert->rank table, hidden
rows, AllGather shards).  It holds none of the method's arithmetic: no masks,
no grouping, no offsets, no packing.  Both the CPU oracle's tests and the CUDA
library's tests / benchmark take their arrays from here, so the two sides never
have to reproduce a random-number generator in two languages.

The paper describes its workloads by shape only (Section 6.1: 64 experts,
top-8, batches of 64 / 128 / 1k / 2k tokens; Section 6.2: 16 MB AllGather
messages; Section 6.3: a 256 KB - 200 MB sweep).  The five named
configurations below scale those shapes to DeepSeek-V3-like sizes.

All arrays are numpy, host side:
  topk_ids        int32  [T, K]   expert ids chosen per token (distinct)
  expert_to_rank  int32  [E]      contiguous blocks: expert e lives on rank e // (E // R)
  x               uint16 [T, H]   bf16 bit patterns of N(0,1) draws (opaque payload)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    """N(0,1) float32 draws rounded to bf16 bit patterns (uint16)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    step = 1 << 22
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = f32_to_bf16_bits(rng.standard_normal(hi - lo, dtype=np.float32))
    return out.reshape(shape)


def contiguous_expert_map(E: int, R: int) -> np.ndarray:
    """expert e -> rank e // (E // R): equal contiguous blocks of experts per rank."""
    assert E % R == 0
    return (np.arange(E, dtype=np.int64) // (E // R)).astype(np.int32)


def topk_desc(scores: np.ndarray, K: int) -> np.ndarray:
    """Indices of the K largest scores per row, best first; ties go to the lower index."""
    order = np.argsort(-scores, axis=1, kind="stable")
    return np.ascontiguousarray(order[:, :K]).astype(np.int32)


@dataclass(frozen=True)
class DispatchShape:
    name: str
    R: int
    E: int
    K: int
    T: int
    H: int
    router: str  # "normal" | "normal_bias" | "zipf" | "uniform"

    @property
    def row_bytes(self) -> int:
        return 2 * self.H


# The dispatch configurations (index = configuration number - 1).
DISPATCH_SHAPES = (
    DispatchShape("tiny", R=8, E=32, K=4, T=256, H=1024, router="normal"),
    DispatchShape("dsv3_prefill", R=64, E=256, K=8, T=4096, H=7168, router="normal_bias"),
    DispatchShape("large_ep", R=128, E=256, K=8, T=8192, H=7168, router="zipf"),
    DispatchShape("decode", R=256, E=256, K=8, T=64, H=7168, router="uniform"),
)
SHAPE_BY_NAME = {s.name: s for s in DISPATCH_SHAPES}

# AllGather sweep: R = 64 ranks, shard sizes 4 KB .. 64 MB in powers of 4.
ALLGATHER_R = 64
ALLGATHER_SHARD_BYTES = tuple(4096 * 4 ** i for i in range(8))


def draw_router(shape: DispatchShape, rng: np.random.Generator, T: int | None = None) -> np.ndarray:
    """topk_ids int32 [T, K] for one configuration's router model."""
    T = shape.T if T is None else T
    E, K = shape.E, shape.K
    if shape.router == "normal":
        scores = rng.standard_normal((T, E))
    elif shape.router == "normal_bias":
        # per-token logits N(0,1) plus a per-expert bias N(0, sd=0.5) that skews the load
        scores = rng.standard_normal((T, E))
        scores = scores + 0.5 * rng.standard_normal(E)[None, :]
    elif shape.router == "zipf":
        # popularity p ~ rank^-1.2 laid over a seeded permutation of the experts; K distinct
        # experts per token sampled without replacement (top-K of log p + Gumbel noise)
        perm = rng.permutation(E)
        p = np.empty(E, dtype=np.float64)
        p[perm] = np.arange(1, E + 1, dtype=np.float64) ** -1.2
        p /= p.sum()
        scores = np.log(p)[None, :] + rng.gumbel(size=(T, E))
    elif shape.router == "uniform":
        scores = rng.random((T, E))
    else:  # pragma: no cover
        raise ValueError(shape.router)
    return topk_desc(scores, K)


@dataclass
class DispatchInputs:
    shape: DispatchShape
    seed: int
    topk_ids: np.ndarray        # int32 [T, K]
    expert_to_rank: np.ndarray  # int32 [E]
    x: np.ndarray | None        # uint16 [T, H] (bf16 bits) or None when payload was not requested

    @property
    def T(self) -> int:
        return int(self.topk_ids.shape[0])


def make_dispatch(name_or_index, seed: int | None = None, *, T: int | None = None,
                  H: int | None = None, payload: bool = True) -> DispatchInputs:
    """Inputs of a named dispatch configuration.

    Draw order is fixed: router first, then the hidden rows.  `seed` defaults to the
    configuration index (configuration 1 -> seed 0).  `T` / `H` override the shape for
    reduced-size parity cases that keep the configuration's routing structure.
    """
    if isinstance(name_or_index, int):
        shape = DISPATCH_SHAPES[name_or_index]
    else:
        shape = SHAPE_BY_NAME[name_or_index]
    if seed is None:
        seed = DISPATCH_SHAPES.index(shape)
    if T is not None or H is not None:
        shape = DispatchShape(shape.name, shape.R, shape.E, shape.K,
                              shape.T if T is None else T, shape.H if H is None else H, shape.router)
    rng = np.random.default_rng(seed)
    ids = draw_router(shape, rng)
    e2r = contiguous_expert_map(shape.E, shape.R)
    x = normal_bf16(rng, (shape.T, shape.H)) if payload else None
    return DispatchInputs(shape, seed, ids, e2r, x)


def make_random_dispatch(seed: int, *, T: int, K: int, E: int, R: int, H: int,
                         pad_fraction: float = 0.0, contiguous_map: bool = False,
                         distinct: bool = True) -> DispatchInputs:
    """Free-form dispatch inputs for edge-case tests: arbitrary expert->rank table,
    optional -1 padding slots, optional repeated expert ids inside a token."""
    rng = np.random.default_rng(seed)
    if distinct and K <= E:
        ids = topk_desc(rng.random((T, E)), K) if T > 0 else np.zeros((0, K), np.int32)
    else:
        ids = rng.integers(0, E, size=(T, K), dtype=np.int32)
    if pad_fraction > 0.0 and T > 0:
        pad = rng.random((T, K)) < pad_fraction
        ids = np.where(pad, np.int32(-1), ids).astype(np.int32)
    if contiguous_map and E % R == 0:
        e2r = contiguous_expert_map(E, R)
    else:
        e2r = rng.integers(0, R, size=E, dtype=np.int32)
    x = normal_bf16(rng, (T, H))
    shape = DispatchShape("random", R, E, K, T, H, "uniform")
    return DispatchInputs(shape, seed, np.ascontiguousarray(ids, dtype=np.int32), e2r, x)


def make_allgather_shards(R: int, shard_bytes: int, seed: int = 4) -> np.ndarray:
    """uint8 [R, shard_bytes]: each rank's contiguous bf16 shard.

    Up to 1 MB per shard the values are direct N(0,1) bf16 draws.  Larger shards tile
    one seeded 1 MB block and stamp (shard index, page index) into the first 8 bytes of
    every 4 KB page, so every shard and every page stays distinguishable without
    drawing gigabytes of normals (payload content does not affect what is computed).
    """
    assert shard_bytes % 16 == 0
    rng = np.random.default_rng(seed)
    block = 1 << 20
    if shard_bytes <= block:
        return normal_bf16(rng, (R, shard_bytes // 2)).view(np.uint8).reshape(R, shard_bytes)
    base = normal_bf16(rng, (block // 2,)).view(np.uint8)
    reps = shard_bytes // block
    assert reps * block == shard_bytes
    out = np.empty((R, shard_bytes), dtype=np.uint8)
    out[:] = np.tile(base, reps)[None, :]
    pages = out.view(np.uint64).reshape(R, shard_bytes // 4096, 512)
    stamp = (np.arange(R, dtype=np.uint64)[:, None] << np.uint64(32)) | \
        np.arange(shard_bytes // 4096, dtype=np.uint64)[None, :]
    pages[:, :, 0] ^= stamp
    return out
