"""ctypes front end of the CPU oracle (oracle/mwo.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports or links this.
It marshals numpy arrays into the C functions; it does no arithmetic of its own.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mwo.c")
_LIB = os.path.join(_HERE, "libmwo.so")

MWO_OK = 0
MWO_ERR_INVALID_ARG = -1
MWO_ERR_BAD_INDEX = -5

LAYOUT_MULTIWRITE = 0
LAYOUT_UNICAST = 1


class Totals(C.Structure):
    _fields_ = [("T_nonempty", C.c_int64), ("G", C.c_int64), ("total_dest", C.c_int64),
                ("mw_bytes", C.c_int64), ("unicast_bytes", C.c_int64),
                ("unicast_per_expert_bytes", C.c_int64), ("meta_bytes", C.c_int64),
                ("status", C.c_int32), ("reserved", C.c_int32)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}


def build(force: bool = False) -> str:
    """Compile oracle/mwo.c into oracle/libmwo.so with gcc (plain C, no CUDA)."""
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.mwo_plan.restype = C.c_int
        _lib.mwo_allgather.restype = C.c_int
        for name in ("mwo_pack_mw", "mwo_pack_uc", "mwo_deliver_mw", "mwo_deliver_uc", "mwo_deliver_definition"):
            getattr(_lib, name).restype = None
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return C.c_void_p(a.ctypes.data)


@dataclass
class Plan:
    T: int
    K: int
    E: int
    R: int
    W: int
    Kd: int
    row_bytes: int
    token_mask: np.ndarray     # uint64 [T, W]
    token_ndest: np.ndarray    # int32  [T]
    token_group: np.ndarray    # int32  [T]
    token_mw_row: np.ndarray   # int32  [T]
    mw_row_token: np.ndarray   # int32  [T]      first T' defined
    group_offsets: np.ndarray  # int32  [T + 1]  first G + 1 defined
    group_mask: np.ndarray     # uint64 [T, W]   first G defined
    rank_offsets: np.ndarray   # int32  [R + 1]
    rank_tokens: np.ndarray    # int32  [T * Kd] first total_dest defined
    dest_rank: np.ndarray      # int32  [T, Kd]
    dest_pos: np.ndarray       # int32  [T, Kd]
    totals: dict
    ret: int


def plan(topk_ids: np.ndarray, expert_to_rank: np.ndarray, R: int, row_bytes: int, src_rank: int = -1) -> Plan:
    ids = np.ascontiguousarray(topk_ids, dtype=np.int32)
    e2r = np.ascontiguousarray(expert_to_rank, dtype=np.int32)
    T, K = ids.shape
    E = e2r.shape[0]
    W = (R + 63) // 64
    Kd = min(K, R)
    o = dict(
        token_mask=np.zeros((T, W), np.uint64), token_ndest=np.zeros(T, np.int32),
        token_group=np.zeros(T, np.int32), token_mw_row=np.zeros(T, np.int32),
        mw_row_token=np.zeros(T, np.int32), group_offsets=np.zeros(T + 1, np.int32),
        group_mask=np.zeros((T, W), np.uint64), rank_offsets=np.zeros(R + 1, np.int32),
        rank_tokens=np.zeros(T * Kd, np.int32), dest_rank=np.zeros((T, Kd), np.int32),
        dest_pos=np.zeros((T, Kd), np.int32))
    tot = Totals()
    ret = lib().mwo_plan(_p(ids), _p(e2r), C.c_int32(T), C.c_int32(K), C.c_int32(E), C.c_int32(R),
                         C.c_int64(row_bytes), C.c_int32(src_rank),
                         _p(o["token_mask"]), _p(o["token_ndest"]), _p(o["token_group"]), _p(o["token_mw_row"]),
                         _p(o["mw_row_token"]), _p(o["group_offsets"]), _p(o["group_mask"]), _p(o["rank_offsets"]),
                         _p(o["rank_tokens"]), _p(o["dest_rank"]), _p(o["dest_pos"]), C.byref(tot))
    return Plan(T=T, K=K, E=E, R=R, W=W, Kd=Kd, row_bytes=row_bytes, totals=tot.as_dict(), ret=ret, **o)


def _bytes2d(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.ndim == 2:
        return x.view(np.uint8).reshape(x.shape[0], x.shape[1] * x.itemsize)
    return x.view(np.uint8)


def recv_bytes_needed(p: Plan, recv_stride_bytes: int) -> int:
    if recv_stride_bytes:
        return p.R * recv_stride_bytes
    return int(p.totals["total_dest"]) * p.row_bytes


def pack_mw(p: Plan, x: np.ndarray) -> np.ndarray:
    xb = _bytes2d(x)
    Tn = p.totals["T_nonempty"]
    out = np.zeros((Tn, p.row_bytes), np.uint8)
    lib().mwo_pack_mw(_p(xb), C.c_int64(p.row_bytes), _p(p.mw_row_token), C.c_int64(Tn), _p(out))
    return out


def pack_uc(p: Plan, x: np.ndarray) -> np.ndarray:
    xb = _bytes2d(x)
    n = p.totals["total_dest"]
    out = np.zeros((n, p.row_bytes), np.uint8)
    lib().mwo_pack_uc(_p(xb), C.c_int64(p.row_bytes), _p(p.rank_tokens), C.c_int64(n), _p(out))
    return out


def deliver_mw(p: Plan, send_mw: np.ndarray, recv_stride_bytes: int = 0, fill: int = 0) -> np.ndarray:
    recv = np.full(recv_bytes_needed(p, recv_stride_bytes), fill, np.uint8)
    lib().mwo_deliver_mw(_p(send_mw), C.c_int64(p.row_bytes), C.c_int64(p.totals["T_nonempty"]), C.c_int32(p.R),
                         C.c_int32(p.K), _p(p.mw_row_token), _p(p.token_group), _p(p.group_mask), _p(p.dest_pos),
                         _p(p.rank_offsets), _p(recv), C.c_int64(recv_stride_bytes))
    return recv


def deliver_uc(p: Plan, send_uc: np.ndarray, recv_stride_bytes: int = 0, fill: int = 0) -> np.ndarray:
    recv = np.full(recv_bytes_needed(p, recv_stride_bytes), fill, np.uint8)
    lib().mwo_deliver_uc(_p(send_uc), C.c_int64(p.row_bytes), C.c_int32(p.R), _p(p.rank_offsets), _p(recv),
                         C.c_int64(recv_stride_bytes))
    return recv


def deliver_definition(p: Plan, x: np.ndarray, topk_ids: np.ndarray, expert_to_rank: np.ndarray,
                       recv_stride_bytes: int = 0, fill: int = 0) -> np.ndarray:
    xb = _bytes2d(x)
    ids = np.ascontiguousarray(topk_ids, dtype=np.int32)
    e2r = np.ascontiguousarray(expert_to_rank, dtype=np.int32)
    recv = np.full(recv_bytes_needed(p, recv_stride_bytes), fill, np.uint8)
    lib().mwo_deliver_definition(_p(xb), C.c_int64(p.row_bytes), _p(ids), _p(e2r), C.c_int32(p.T), C.c_int32(p.K),
                                 C.c_int32(p.E), C.c_int32(p.R), _p(p.rank_offsets), _p(recv),
                                 C.c_int64(recv_stride_bytes))
    return recv


class RelayTotals(C.Structure):
    _fields_ = [("hop_rows", C.c_int64), ("delivered_rows", C.c_int64), ("direct_bytes", C.c_int64),
                ("inter_multiwrite_bytes", C.c_int64), ("inter_unicast_bytes", C.c_int64),
                ("forward_bytes", C.c_int64), ("staged_rows", C.c_int64), ("status", C.c_int32), ("reserved", C.c_int32)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}


def next_hop(r: int, src_rank: int, ranks_per_server: int) -> int:
    lib().mwo_next_hop.restype = C.c_int
    return int(lib().mwo_next_hop(C.c_int32(r), C.c_int32(src_rank), C.c_int32(ranks_per_server)))


def relay(topk_ids: np.ndarray, expert_to_rank: np.ndarray, R: int, row_bytes: int, src_rank: int,
          ranks_per_server: int, x: np.ndarray | None = None, recv_stride_bytes: int = 0, fill: int = 0,
          in_place: bool = False):
    """Two-level dispatch.  Returns (hop_plan, flat_plan, send_buf, hop_buf, recv, totals); the buffers are None
    when no payload is given.  in_place: the receive buffer serves as relay buffer (a copy whose next hop is itself a
    destination goes straight to its final slot; only the other copies use the hop area, whose remaining rows keep `fill`)."""
    e2r = np.ascontiguousarray(expert_to_rank, dtype=np.int32)
    hop_tab = np.zeros_like(e2r)
    lib().mwo_relay_table.restype = None
    lib().mwo_relay_expand.restype = None
    lib().mwo_relay_table(_p(e2r), C.c_int32(len(e2r)), C.c_int32(R), C.c_int32(src_rank), C.c_int32(ranks_per_server),
                          _p(hop_tab))
    hp = plan(topk_ids, hop_tab, R, row_bytes, src_rank)
    fp = plan(topk_ids, e2r, R, row_bytes, src_rank)
    send = hop_buf = recv = None
    hop_ptr, recv_ptr = C.c_void_p(0), C.c_void_p(0)
    if x is not None:
        send = pack_mw(hp, x)                                # each row once per group of identical next-hop set
        hop_buf = deliver_mw(hp, send)                       # first level: one copy per next hop
        recv = np.full(recv_bytes_needed(fp, recv_stride_bytes), fill, np.uint8)
        hop_ptr, recv_ptr = _p(hop_buf), _p(recv)
    if in_place and x is not None:
        hop_buf = np.full(hp.totals["total_dest"] * row_bytes, fill, np.uint8)
        lib().mwo_relay_first_in_place.restype = None
        lib().mwo_relay_forward_in_place.restype = None
        lib().mwo_relay_first_in_place(_p(_bytes2d(send)), C.c_int64(row_bytes), C.c_int64(hp.totals["T_nonempty"]), C.c_int32(R),
                                       C.c_int32(fp.K), _p(hp.mw_row_token), _p(hp.dest_rank), _p(hp.dest_pos), _p(hp.rank_offsets),
                                       _p(fp.dest_rank), _p(fp.dest_pos), _p(fp.rank_offsets), _p(hop_buf), _p(recv),
                                       C.c_int64(recv_stride_bytes))
        lib().mwo_relay_forward_in_place(_p(hop_buf), C.c_int64(row_bytes), C.c_int32(R), C.c_int32(fp.K), C.c_int32(src_rank),
                                         C.c_int32(ranks_per_server), _p(hp.rank_offsets), _p(hp.rank_tokens),
                                         _p(fp.dest_rank), _p(fp.dest_pos), _p(fp.rank_offsets), _p(recv),
                                         C.c_int64(recv_stride_bytes))
        recv_ptr = C.c_void_p(0)                              # the accounting below is the same; nothing more to write
    tot = RelayTotals()
    lib().mwo_relay_expand(hop_ptr, C.c_int64(row_bytes), C.c_int32(fp.T), C.c_int32(R), C.c_int32(fp.K),
                           C.c_int32(src_rank), C.c_int32(ranks_per_server), _p(hp.rank_offsets), _p(hp.rank_tokens),
                           _p(fp.dest_rank), _p(fp.dest_pos), _p(fp.rank_offsets),
                           C.c_int32(fp.totals["status"]), recv_ptr, C.c_int64(recv_stride_bytes), C.byref(tot))
    return hp, fp, send, hop_buf, recv, tot.as_dict()


def combine(p: Plan, z: np.ndarray, weights: np.ndarray | None = None, z_stride_bytes: int = 0,
            precision: str = "f64") -> np.ndarray:
    """y uint16 [T, H] (bf16 bits).  z: the receive area (uint8), laid out like the dispatch's.
    precision "f64": binary64 sum, one rounding; "f32": binary32 fused multiply-adds in rank order, one rounding."""
    zz = np.ascontiguousarray(z).view(np.uint8).reshape(-1)
    y = np.zeros((p.T, p.row_bytes // 2), np.uint16)
    w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float32)
    fn = {"f64": lib().mwo_combine, "f32": lib().mwo_combine_f32}[precision]
    fn.restype = None
    fn(_p(zz), C.c_int64(z_stride_bytes), _p(w) if w is not None else C.c_void_p(0), C.c_int32(p.T),
                      C.c_int32(p.R), C.c_int32(p.K), C.c_int64(p.row_bytes), _p(p.dest_rank), _p(p.dest_pos),
                      _p(p.rank_offsets), _p(y))
    return y


def group_major(p: Plan):
    """Group-major receive order.  Returns (group_dest_rank [G,Kd], group_dest_offset [G,Kd], dest_pos_gm [T,Kd])."""
    G, Kd = int(p.totals["G"]), p.Kd
    gdr = np.full((max(G, 1), Kd), -1, np.int32)
    gdo = np.full((max(G, 1), Kd), -1, np.int32)
    gm = np.full((max(p.T, 1), Kd), -1, np.int32)
    lib().mwo_group_major.restype = None
    lib().mwo_group_major(C.c_int32(p.T), C.c_int32(p.R), C.c_int32(p.K), C.c_int64(G), _p(p.group_mask), _p(p.group_offsets),
                          _p(p.token_group), _p(p.token_mw_row), _p(gdr), _p(gdo), _p(gm))
    return gdr[:G], gdo[:G], gm[:p.T]


def deliver_group_major(p: Plan, send_mw: np.ndarray, gdr: np.ndarray, gdo: np.ndarray, recv_stride_bytes: int = 0,
                        fill: int = 0) -> np.ndarray:
    """Receive area (uint8, flat) after one MultiWrite per group, regions in group-major order."""
    recv = np.full(recv_bytes_needed(p, recv_stride_bytes), fill, np.uint8)
    G = int(p.totals["G"])
    if G == 0:
        return recv
    send = np.ascontiguousarray(send_mw).view(np.uint8).reshape(-1)
    a, b = np.ascontiguousarray(gdr, dtype=np.int32), np.ascontiguousarray(gdo, dtype=np.int32)
    lib().mwo_deliver_group_major.restype = None
    lib().mwo_deliver_group_major(_p(send), C.c_int64(p.row_bytes), C.c_int32(p.R), C.c_int32(p.K), C.c_int64(G),
                                  _p(p.group_offsets), _p(a), _p(b), _p(p.rank_offsets), _p(recv), C.c_int64(recv_stride_bytes))
    return recv


def expert_index(p: Plan, topk_ids: np.ndarray, expert_to_rank: np.ndarray):
    """Returns (expert_offsets [E+1], expert_token [T*K], expert_slot [T*K], pairs)."""
    ids = np.ascontiguousarray(topk_ids, dtype=np.int32).reshape(p.T, p.K)
    e2r = np.ascontiguousarray(expert_to_rank, dtype=np.int32)
    E = len(e2r)
    off = np.zeros(E + 1, np.int32)
    tok = np.full(max(p.T * p.K, 1), -1, np.int32)
    slot = np.full(max(p.T * p.K, 1), -1, np.int32)
    lib().mwo_expert_index.restype = C.c_int64
    n = lib().mwo_expert_index(_p(ids), _p(e2r), C.c_int32(p.T), C.c_int32(p.K), C.c_int32(E), C.c_int32(p.R),
                               _p(p.dest_rank), _p(p.dest_pos), _p(off), _p(tok), _p(slot))
    return off, tok[:p.T * p.K], slot[:p.T * p.K], int(n)


class PairTotals(C.Structure):
    _fields_ = [("direct_link_bytes", C.c_int64), ("pair_link_bytes", C.c_int64), ("forward_link_bytes", C.c_int64),
                ("max_link_bytes", C.c_int64), ("total_bytes", C.c_int64)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


def balanced_direct_bytes(shard_bytes: int, n: int, layout: int) -> int:
    lib().mwo_balanced_direct_bytes.restype = C.c_int64
    return int(lib().mwo_balanced_direct_bytes(C.c_int64(shard_bytes), C.c_int32(n), C.c_int(layout)))


def split_direct_bytes(shard_bytes: int, n: int, layout: int, w_direct: float, w_pair: float) -> int:
    lib().mwo_split_direct_bytes.restype = C.c_int64
    return int(lib().mwo_split_direct_bytes(C.c_int64(shard_bytes), C.c_int32(n), C.c_int(layout), C.c_double(w_direct),
                                            C.c_double(w_pair)))


def paired_allgather(shards: np.ndarray, direct_bytes: int, layout: int, fill: int = 0):
    """Returns (relay_buf, recv, totals, ret).  shards: uint8 [R, S], R = 2n."""
    sh = np.ascontiguousarray(shards).view(np.uint8)
    R, S = sh.shape
    n = R // 2
    copies = 1 if layout == LAYOUT_MULTIWRITE else max(n - 1, 0)
    relay_buf = np.full(max(R * copies * (S - direct_bytes), 0), fill, np.uint8)
    recv = np.full(R * n * S, fill, np.uint8)
    tot = PairTotals()
    lib().mwo_paired_allgather.restype = C.c_int
    ret = lib().mwo_paired_allgather(_p(sh), C.c_int32(R), C.c_int64(S), C.c_int64(direct_bytes), C.c_int(layout),
                                     _p(relay_buf), _p(recv), C.byref(tot))
    return relay_buf, recv, tot.as_dict(), ret


def allgather(shards: np.ndarray, layout: int, dst_begin: int = 0, dst_count: int | None = None,
              recv_stride_bytes: int = 0, fill: int = 0):
    """Returns (send_buf, recv, totals, ret).  shards: uint8 [R, S]."""
    sh = np.ascontiguousarray(shards).view(np.uint8)
    R, S = sh.shape
    dst_count = R if dst_count is None else dst_count
    stride = recv_stride_bytes or R * S
    send = np.full(R * S if layout == LAYOUT_MULTIWRITE else R * dst_count * S, fill, np.uint8)
    recv = np.full(max(dst_count, 0) * stride, fill, np.uint8)
    tot = Totals()
    ret = lib().mwo_allgather(_p(sh), C.c_int32(R), C.c_int64(S), C.c_int(layout), C.c_int32(dst_begin),
                              C.c_int32(dst_count), _p(send), _p(recv), C.c_int64(recv_stride_bytes), C.byref(tot))
    return send, recv, tot.as_dict(), ret
