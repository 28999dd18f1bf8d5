"""ctypes binding of libmw.so: same names as the C ABI in include/mw.h, argument marshalling only.

Device buffers are torch CUDA tensors (or raw integer device pointers); streams are torch streams.
Every step of the path runs in the library's CUDA kernels.  If the library cannot be loaded this
module raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

MW_OK = 0
MW_ERR_INVALID_ARG = -1
MW_ERR_ALIGNMENT = -2
MW_ERR_CAPACITY = -3
MW_ERR_CUDA = -4
MW_ERR_BAD_INDEX = -5
MW_ERR_TIMEOUT = -6
MW_ERR_NO_PLAN = -7

MW_LAYOUT_MULTIWRITE = 0
MW_LAYOUT_UNICAST = 1

MW_FLAG_HOST_STAGING = 0x1
MW_FLAG_PLAN_MULTIPASS = 0x2
MW_FLAG_NO_OVERLAP = 0x10
MW_FLAG_COPY_BULK = 0x40
MW_FLAG_SHORT_WAITS = 0x80

MW_TEST_SKEW_LOOKBACK = 0x1
MW_TEST_SKEW_BARRIER = 0x2
MW_TEST_SKEW_BULK_LOAD = 0x4
MW_TEST_SKEW_GROUP_MAJOR = 0x8

RELAY_EXPORTS = ("mw_relay_create", "mw_relay_destroy", "mw_relay_reset", "mw_relay_plan", "mw_relay_get_totals", "mw_relay_dispatch",
                 "mw_relay_contexts")
INT_EXPORTS = ("mw_create", "mw_destroy", "mw_reset", "mw_plan", "mw_plan_prefetch", "mw_plan_next", "mw_plan_swap",
               "mw_get_plan_view", "mw_get_totals", "mw_pack", "mw_deliver", "mw_deliver_ptrs", "mw_dispatch", "mw_plan_dispatch",
               "mw_allgather_pack", "mw_paired_allgather", "mw_combine", "mw_group_major", "mw_deliver_group_major",
               "mw_expert_index", "mw_dispatch_host", "mw_group_tokens_static", "mw_read_device", "mw_test_skew_waits") + RELAY_EXPORTS
EXPORTS = INT_EXPORTS + ("mw_kernel_launches", "mw_strerror", "mw_pair_balanced_direct_bytes", "mw_pair_split_direct_bytes")


class mw_config(C.Structure):
    _fields_ = [("R", C.c_int32), ("E", C.c_int32), ("K", C.c_int32), ("max_tokens", C.c_int32),
                ("row_bytes", C.c_int64), ("src_rank", C.c_int32), ("device", C.c_int32),
                ("flags", C.c_uint32), ("reserved", C.c_uint32)]


class mw_totals(C.Structure):
    _fields_ = [("T_nonempty", C.c_int64), ("G", C.c_int64), ("total_dest", C.c_int64),
                ("mw_bytes", C.c_int64), ("unicast_bytes", C.c_int64),
                ("unicast_per_expert_bytes", C.c_int64), ("meta_bytes", C.c_int64),
                ("status", C.c_int32), ("reserved", C.c_int32)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}


class mw_relay_totals(C.Structure):
    _fields_ = [("hop_rows", C.c_int64), ("delivered_rows", C.c_int64), ("direct_bytes", C.c_int64),
                ("inter_multiwrite_bytes", C.c_int64), ("inter_unicast_bytes", C.c_int64),
                ("forward_bytes", C.c_int64), ("staged_rows", C.c_int64), ("status", C.c_int32), ("reserved", C.c_int32)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}


class mw_pair_totals(C.Structure):
    _fields_ = [("direct_link_bytes", C.c_int64), ("pair_link_bytes", C.c_int64), ("forward_link_bytes", C.c_int64),
                ("max_link_bytes", C.c_int64), ("total_bytes", C.c_int64)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class mw_group_major_view(C.Structure):
    _fields_ = [("group_dest_rank", C.c_void_p), ("group_dest_offset", C.c_void_p), ("dest_pos_gm", C.c_void_p),
                ("Kd", C.c_int32), ("reserved", C.c_int32)]


class mw_plan_view(C.Structure):
    _fields_ = [("token_mask", C.c_void_p), ("token_ndest", C.c_void_p), ("token_group", C.c_void_p),
                ("token_mw_row", C.c_void_p), ("mw_row_token", C.c_void_p), ("group_offsets", C.c_void_p),
                ("group_mask", C.c_void_p), ("rank_offsets", C.c_void_p), ("rank_tokens", C.c_void_p),
                ("dest_rank", C.c_void_p), ("dest_pos", C.c_void_p), ("totals", C.c_void_p),
                ("T", C.c_int32), ("W", C.c_int32), ("Kd", C.c_int32), ("reserved", C.c_int32)]


class MwError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def lib():
    """Loads libmw.so (built in-tree by build.build_library); raises if it is missing."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2605_22428_b200.build` "
                               "(or __graft_entry__.build()); there is no CPU fallback")
        L = C.CDLL(path)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.mw_create.argtypes = [C.POINTER(vp), C.POINTER(mw_config)]
        L.mw_destroy.argtypes = [vp]
        L.mw_reset.argtypes = [vp]
        L.mw_test_skew_waits.argtypes = [vp, C.c_uint32]
        L.mw_plan_next.argtypes = [vp, vp, vp, i32, vp, vp]
        L.mw_plan_swap.argtypes = [vp, C.POINTER(mw_plan_view), vp]
        L.mw_plan.argtypes = [vp, vp, vp, i32, C.POINTER(mw_plan_view), vp]
        L.mw_plan_prefetch.argtypes = [vp, vp, vp, i32, vp, C.POINTER(mw_plan_view), vp]
        L.mw_get_plan_view.argtypes = [vp, C.POINTER(mw_plan_view)]
        L.mw_get_totals.argtypes = [vp, C.POINTER(mw_totals), vp]
        L.mw_pack.argtypes = [vp, vp, C.c_int, vp, i64, vp]
        L.mw_deliver.argtypes = [vp, C.c_int, vp, vp, i64, i64, vp]
        L.mw_deliver_ptrs.argtypes = [vp, C.c_int, vp, vp, i64, vp]
        L.mw_dispatch.argtypes = [vp, vp, C.c_int, vp, i64, vp, i64, i64, vp]
        L.mw_plan_dispatch.argtypes = [vp, vp, vp, i32, vp, C.c_int, vp, i64, vp, i64, i64, C.POINTER(mw_plan_view), vp]
        L.mw_allgather_pack.argtypes = [vp, vp, i64, C.c_int, vp, vp, i64, i32, i32, C.POINTER(mw_totals), vp]
        L.mw_paired_allgather.argtypes = [vp, vp, i64, i64, C.c_int, vp, vp, C.POINTER(mw_pair_totals), vp]
        L.mw_pair_balanced_direct_bytes.argtypes = [i64, i32, C.c_int]
        L.mw_pair_balanced_direct_bytes.restype = i64
        L.mw_pair_split_direct_bytes.argtypes = [i64, i32, C.c_int, C.c_double, C.c_double]
        L.mw_pair_split_direct_bytes.restype = i64
        L.mw_combine.argtypes = [vp, vp, i64, vp, vp, vp]
        L.mw_group_major.argtypes = [vp, C.POINTER(mw_group_major_view), vp]
        L.mw_deliver_group_major.argtypes = [vp, vp, vp, i64, i64, vp]
        L.mw_expert_index.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.mw_dispatch_host.argtypes = [vp, vp, vp, vp, i32, C.c_int, vp, i64, vp, C.POINTER(mw_totals), vp]
        L.mw_group_tokens_static.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.mw_read_device.argtypes = [vp, vp, vp, i64, vp]
        L.mw_kernel_launches.argtypes = [vp]
        L.mw_kernel_launches.restype = C.c_int64
        L.mw_relay_create.argtypes = [C.POINTER(vp), C.POINTER(mw_config), i32]
        L.mw_relay_destroy.argtypes = [vp]
        L.mw_relay_reset.argtypes = [vp]
        L.mw_relay_plan.argtypes = [vp, vp, vp, i32, vp]
        L.mw_relay_get_totals.argtypes = [vp, C.POINTER(mw_relay_totals), vp]
        L.mw_relay_dispatch.argtypes = [vp, vp, vp, i64, vp, i64, vp, i64, i64, vp]
        L.mw_relay_contexts.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        L.mw_strerror.argtypes = [C.c_int]
        L.mw_strerror.restype = C.c_char_p
        for name in INT_EXPORTS:
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def mw_pair_balanced_direct_bytes(shard_bytes: int, ranks_per_domain: int, layout: int) -> int:
    return int(lib().mw_pair_balanced_direct_bytes(shard_bytes, ranks_per_domain, layout))


def mw_pair_split_direct_bytes(shard_bytes: int, ranks_per_domain: int, layout: int, w_direct: float, w_pair: float) -> int:
    return int(lib().mw_pair_split_direct_bytes(shard_bytes, ranks_per_domain, layout, w_direct, w_pair))


def strerror(code: int) -> str:
    return lib().mw_strerror(int(code)).decode()


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / integer address / None, as a plain integer
    (ctypes converts it; building a c_void_p object per argument doubles the cost of a call)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


_raw_stream = None


def _stream(stream):
    """cudaStream_t of a torch stream / integer handle / None (= torch's current stream), as a plain integer."""
    global _raw_stream
    if stream is None:
        import torch
        if _raw_stream is None:
            # the raw handle without building a Stream object (a microsecond per call); falls back to the public API
            fast = getattr(torch._C, "_cuda_getCurrentRawStream", None)
            _raw_stream = fast if fast is not None else (lambda dev: torch.cuda.current_stream(dev).cuda_stream)
        return _raw_stream(torch.cuda.current_device()) or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


MW_STATIC_MAX_TOKENS = 16384


def mw_group_tokens_static(topk_ids, expert_to_rank, T: int, K: int, E: int, R: int, token_mask, token_ndest,
                           token_leader, token_group_size, status, stream=None) -> int:
    """Bitmaps and token grouping for callers that may not allocate device memory (for example a
    server whose framework pool owns the whole GPU): the library's own fixed scratch array is used,
    every buffer is the caller's.  Returns the C return code; see include/mw.h for the rules
    (T <= MW_STATIC_MAX_TOKENS, calls that overlap on the GPU race on the shared scratch)."""
    return lib().mw_group_tokens_static(_ptr(topk_ids), _ptr(expert_to_rank), T, K, E, R, _ptr(token_mask),
                                        _ptr(token_ndest), _ptr(token_leader), _ptr(token_group_size),
                                        _ptr(status), _stream(stream))


def _view_of(ctx) -> "mw_plan_view":
    view = mw_plan_view()
    rc = lib().mw_get_plan_view(ctx._h, C.byref(view))
    if rc != MW_OK:
        raise MwError(rc, "mw_get_plan_view")
    return view


class Context:
    """Owns one mw_ctx (or borrows one owned by a Relay).  Methods mirror the C entry points and return the C return code checked."""

    def __init__(self, R: int, E: int, K: int, max_tokens: int, row_bytes: int, src_rank: int = -1,
                 device: int = 0, flags: int = 0):
        self.cfg = mw_config(R, E, K, max_tokens, row_bytes, src_rank, device, flags, 0)
        self._h = C.c_void_p()
        rc = lib().mw_create(C.byref(self._h), C.byref(self.cfg))
        if rc != MW_OK:
            raise MwError(rc, "mw_create")
        self.R, self.E, self.K, self.row_bytes = R, E, K, row_bytes
        self.W = (R + 63) // 64
        self.Kd = min(K, R)
        self.device = device
        self.view = None

    @classmethod
    def borrowed(cls, handle, R: int, E: int, K: int, row_bytes: int, device: int = 0):
        """A view of a context owned elsewhere (not destroyed on close)."""
        self = cls.__new__(cls)
        self._h = C.c_void_p(handle)
        self._owned = False
        self.R, self.E, self.K, self.row_bytes = R, E, K, row_bytes
        self.W, self.Kd, self.device, self.view = (R + 63) // 64, min(K, R), device, None
        return self

    def close(self):
        if C is None:                      # interpreter shutdown: the module globals are already gone
            return
        if self._h and getattr(self, "_owned", True):
            lib().mw_destroy(self._h)
        self._h = C.c_void_p()

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- C ABI mirrors ----------------------------------------------------------------------
    def mw_plan(self, topk_ids, expert_to_rank, T: int | None = None, stream=None, check: bool = True) -> int:
        T = int(topk_ids.shape[0]) if T is None else T
        view = mw_plan_view()
        rc = lib().mw_plan(self._h, _ptr(topk_ids), _ptr(expert_to_rank), T, C.byref(view), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_plan")
        self.view = view
        return rc

    def mw_plan_prefetch(self, topk_ids, expert_to_rank, T: int | None, x, stream=None, check: bool = True) -> int:
        T = int(topk_ids.shape[0]) if T is None else T
        view = mw_plan_view()
        rc = lib().mw_plan_prefetch(self._h, _ptr(topk_ids), _ptr(expert_to_rank), T, _ptr(x), C.byref(view), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_plan_prefetch")
        self.view = view
        return rc

    def mw_plan_next(self, topk_ids, expert_to_rank, T: int | None = None, x=None, stream=None, check: bool = True) -> int:
        T = int(topk_ids.shape[0]) if T is None else T
        rc = lib().mw_plan_next(self._h, _ptr(topk_ids), _ptr(expert_to_rank), T, _ptr(x), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_plan_next")
        return rc

    def mw_plan_swap(self, stream=None, check: bool = True) -> int:
        view = mw_plan_view()
        rc = lib().mw_plan_swap(self._h, C.byref(view), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_plan_swap")
        if rc == MW_OK:
            self.view = view
        return rc

    def mw_reset(self, check: bool = True) -> int:
        rc = lib().mw_reset(self._h)
        if check and rc != MW_OK:
            raise MwError(rc, "mw_reset")
        return rc

    def mw_test_skew_waits(self, what: int) -> int:
        rc = lib().mw_test_skew_waits(self._h, what)
        if rc != MW_OK:
            raise MwError(rc, "mw_test_skew_waits")
        return rc

    def mw_get_totals(self, stream=None) -> dict:
        tot = mw_totals()
        rc = lib().mw_get_totals(self._h, C.byref(tot), _stream(stream))
        if rc != MW_OK:
            raise MwError(rc, "mw_get_totals")
        return tot.as_dict()

    def mw_pack(self, x, layout: int, send_buf, send_capacity_rows: int, stream=None, check: bool = True) -> int:
        rc = lib().mw_pack(self._h, _ptr(x), layout, _ptr(send_buf), send_capacity_rows, _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_pack")
        return rc

    def mw_deliver(self, layout: int, send_buf, recv, recv_stride_bytes: int, recv_capacity_rows: int,
                   stream=None, check: bool = True) -> int:
        rc = lib().mw_deliver(self._h, layout, _ptr(send_buf), _ptr(recv), recv_stride_bytes, recv_capacity_rows,
                              _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_deliver")
        return rc

    def mw_deliver_ptrs(self, layout: int, send_buf, recv_ptrs, recv_capacity_rows: int, stream=None, check: bool = True) -> int:
        """recv_ptrs: device int64 tensor (or address) holding the R region base addresses."""
        rc = lib().mw_deliver_ptrs(self._h, layout, _ptr(send_buf), _ptr(recv_ptrs), recv_capacity_rows, _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_deliver_ptrs")
        return rc

    def mw_dispatch(self, x, layout: int, send_buf, send_capacity_rows: int, recv, recv_stride_bytes: int,
                    recv_capacity_rows: int, stream=None, check: bool = True) -> int:
        rc = lib().mw_dispatch(self._h, _ptr(x), layout, _ptr(send_buf), send_capacity_rows, _ptr(recv),
                               recv_stride_bytes, recv_capacity_rows, _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_dispatch")
        return rc

    def mw_plan_dispatch(self, topk_ids, expert_to_rank, T: int, x, layout: int, send_buf, send_capacity_rows: int,
                         recv, recv_stride_bytes: int, recv_capacity_rows: int, stream=None, check: bool = True) -> int:
        view = mw_plan_view()
        rc = lib().mw_plan_dispatch(self._h, _ptr(topk_ids), _ptr(expert_to_rank), T, _ptr(x), layout, _ptr(send_buf),
                                    send_capacity_rows, _ptr(recv), recv_stride_bytes, recv_capacity_rows,
                                    C.byref(view), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_plan_dispatch")
        self.view = view
        return rc

    def mw_allgather_pack(self, shards, shard_bytes: int, layout: int, send_buf, recv, recv_stride_bytes: int = 0,
                          dst_rank_begin: int = 0, dst_rank_count: int | None = None, stream=None,
                          check: bool = True):
        tot = mw_totals()
        cnt = self.R if dst_rank_count is None else dst_rank_count
        rc = lib().mw_allgather_pack(self._h, _ptr(shards), shard_bytes, layout, _ptr(send_buf), _ptr(recv),
                                     recv_stride_bytes, dst_rank_begin, cnt, C.byref(tot), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_allgather_pack")
        return rc, tot.as_dict()

    def mw_paired_allgather(self, shards, shard_bytes: int, direct_bytes: int, layout: int, relay_buf, recv,
                            stream=None, check: bool = True):
        tot = mw_pair_totals()
        rc = lib().mw_paired_allgather(self._h, _ptr(shards), shard_bytes, direct_bytes, layout, _ptr(relay_buf),
                                       _ptr(recv), C.byref(tot), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_paired_allgather")
        return rc, tot.as_dict()

    def mw_combine(self, z, z_stride_bytes: int, weights, y, stream=None, check: bool = True) -> int:
        rc = lib().mw_combine(self._h, _ptr(z), z_stride_bytes, _ptr(weights), _ptr(y), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_combine")
        return rc

    def mw_group_major(self, stream=None, check: bool = True):
        """Returns (rc, view); the view's fields are device addresses of context-owned arrays."""
        view = mw_group_major_view()
        rc = lib().mw_group_major(self._h, C.byref(view), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_group_major")
        return rc, view

    def group_major_arrays(self, T: int, G: int, view) -> dict:
        """Host copies (numpy) of the arrays mw_group_major filled: first G groups, first T tokens."""
        import numpy as np
        Kd = view.Kd
        out = {}
        for name, rows in (("group_dest_rank", G), ("group_dest_offset", G), ("dest_pos_gm", T)):
            a = np.empty((rows, Kd), np.int32)
            if rows:
                rc = lib().mw_read_device(self._h, _ptr(a), C.c_void_p(getattr(view, name)), a.nbytes, None)
                if rc != MW_OK:
                    raise MwError(rc, "mw_read_device")
            out[name] = a
        return out

    def mw_deliver_group_major(self, send_buf, recv_base, recv_stride_bytes: int, recv_capacity_rows: int, stream=None,
                               check: bool = True) -> int:
        rc = lib().mw_deliver_group_major(self._h, _ptr(send_buf), _ptr(recv_base), recv_stride_bytes, recv_capacity_rows,
                                          _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_deliver_group_major")
        return rc

    def mw_expert_index(self, topk_ids, expert_to_rank, expert_offsets, expert_token, expert_slot, stream=None,
                        check: bool = True) -> int:
        rc = lib().mw_expert_index(self._h, _ptr(topk_ids), _ptr(expert_to_rank), _ptr(expert_offsets), _ptr(expert_token),
                                   _ptr(expert_slot), _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_expert_index")
        return rc

    def mw_dispatch_host(self, topk_ids_host, expert_to_rank_host, x_host, T: int, layout: int, recv_host,
                         recv_capacity_rows: int, rank_offsets_host, stream=None, check: bool = True):
        tot = mw_totals()
        rc = lib().mw_dispatch_host(self._h, _ptr(topk_ids_host), _ptr(expert_to_rank_host), _ptr(x_host), T, layout,
                                    _ptr(recv_host), recv_capacity_rows, _ptr(rank_offsets_host), C.byref(tot),
                                    _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_dispatch_host")
        return rc, tot.as_dict()

    def mw_kernel_launches(self) -> int:
        return int(lib().mw_kernel_launches(self._h))

    # -- reading the plan back (tests, diagnostics) -------------------------------------------
    def plan_arrays(self, T: int, stream=None) -> dict:
        """Copies the plan metadata of the latest mw_plan to numpy arrays (synchronises)."""
        import numpy as np
        v = self.view
        W, Kd, R = self.W, self.Kd, self.R
        spec = dict(token_mask=(np.uint64, (T, W)), token_ndest=(np.int32, (T,)), token_group=(np.int32, (T,)),
                    token_mw_row=(np.int32, (T,)), mw_row_token=(np.int32, (T,)), group_offsets=(np.int32, (T + 1,)),
                    group_mask=(np.uint64, (T, W)), rank_offsets=(np.int32, (R + 1,)),
                    rank_tokens=(np.int32, (T * Kd,)), dest_rank=(np.int32, (T, Kd)), dest_pos=(np.int32, (T, Kd)))
        out = {}
        for name, (dt, shape) in spec.items():
            a = np.empty(shape, dt)
            rc = lib().mw_read_device(self._h, _ptr(a), C.c_void_p(getattr(v, name)), a.nbytes, _stream(stream))
            if rc != MW_OK:
                raise MwError(rc, "mw_read_device")
            out[name] = a
        return out


class Relay:
    """Owns one mw_relay: two-level dispatch through same-index relays (mirrors the mw_relay_* entry points)."""

    def __init__(self, R: int, E: int, K: int, max_tokens: int, row_bytes: int, src_rank: int, ranks_per_server: int,
                 device: int = 0, flags: int = 0):
        self.cfg = mw_config(R, E, K, max_tokens, row_bytes, src_rank, device, flags, 0)
        self._h = C.c_void_p()
        rc = lib().mw_relay_create(C.byref(self._h), C.byref(self.cfg), ranks_per_server)
        if rc != MW_OK:
            raise MwError(rc, "mw_relay_create")
        hop, flat = C.c_void_p(), C.c_void_p()
        lib().mw_relay_contexts(self._h, C.byref(hop), C.byref(flat))
        self.hop = Context.borrowed(hop.value, R, E, K, row_bytes, device)
        self.flat = Context.borrowed(flat.value, R, E, K, row_bytes, device)
        self.R, self.Kd, self.row_bytes = R, min(K, R), row_bytes

    def close(self):
        if C is None:
            return
        if self._h:
            lib().mw_relay_destroy(self._h)
            self._h = C.c_void_p()

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def mw_relay_plan(self, topk_ids, expert_to_rank, T: int, stream=None, check: bool = True) -> int:
        rc = lib().mw_relay_plan(self._h, _ptr(topk_ids), _ptr(expert_to_rank), T, _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_relay_plan")
        # the inner contexts' views are fixed workspace pointers: fetch them once for plan_arrays()
        for ctx in (self.hop, self.flat) if rc == MW_OK else ():
            if ctx.view is None:
                ctx.view = _view_of(ctx)
        return rc

    def mw_relay_reset(self) -> int:
        rc = lib().mw_relay_reset(self._h)
        if rc != MW_OK:
            raise MwError(rc, "mw_relay_reset")
        return rc

    def mw_relay_get_totals(self, stream=None) -> dict:
        tot = mw_relay_totals()
        rc = lib().mw_relay_get_totals(self._h, C.byref(tot), _stream(stream))
        if rc != MW_OK:
            raise MwError(rc, "mw_relay_get_totals")
        return tot.as_dict()

    def mw_relay_dispatch(self, x, send_buf, send_capacity_rows: int, hop_buf, hop_capacity_rows: int, recv,
                          recv_stride_bytes: int, recv_capacity_rows: int, stream=None, check: bool = True) -> int:
        rc = lib().mw_relay_dispatch(self._h, _ptr(x), _ptr(send_buf), send_capacity_rows, _ptr(hop_buf),
                                     hop_capacity_rows, _ptr(recv), recv_stride_bytes, recv_capacity_rows,
                                     _stream(stream))
        if check and rc != MW_OK:
            raise MwError(rc, "mw_relay_dispatch")
        return rc
