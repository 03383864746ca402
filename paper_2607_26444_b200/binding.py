"""ctypes binding of the C-ABI library: argument marshalling only.

Every function named ``strata_*`` forwards to the C entry point of the same
name (see ``include/strata_moe.h``).  ``MoEContext`` is a small convenience
wrapper that uses torch for device memory and streams; it performs no
arithmetic of its own.  There is no CPU fallback: if the CUDA library has not
been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
# STRATA_MOE_LIB names another build of the same library (the test-hooks variant in the time-out test)
LIB_PATH = os.environ.get("STRATA_MOE_LIB") or os.path.join(_HERE, "libstrata_moe.so")

STRATA_OK = 0
STRATA_ERR_INVALID_ARG = 1
STRATA_ERR_SHAPE = 2
STRATA_ERR_ALIGNMENT = 3
STRATA_ERR_NOT_REGISTERED = 4
STRATA_ERR_CAPACITY = 5
STRATA_ERR_BAD_EXPERT_ID = 6
STRATA_ERR_WORKSPACE = 7
STRATA_ERR_CUDA = 8
STRATA_ERR_TIMEOUT = 9
STRATA_ERR_BAD_ROW = 10

STRATA_BF16 = 0
STRATA_FP8_E4M3_B128 = 1
STRATA_FLAG_ALLOW_UNROUTED = 1

EXPORTS = [
    "strata_status_string", "strata_ctx_create", "strata_ctx_destroy", "strata_moe_workspace_bytes",
    "strata_ctx_set_workspace", "strata_ctx_launch_count", "strata_pool_register", "strata_pool_is_ready",
    "strata_pool_unregister", "strata_pool_carve", "strata_pool_reset", "strata_moe_layout",
    "strata_moe_dispatch", "strata_moe_combine", "strata_moe_recv_view", "strata_device_status",
    "strata_moe_roundtrip_host", "strata_moe_layout_noalloc", "strata_ctx_set_trace",
    "strata_moe_partition_max_units", "strata_moe_partition", "strata_moe_dispatch_windows",
    "strata_moe_recv_rows",
    "strata_ctx_set_timeline", "strata_timeline_decode", "strata_ctx_set_sm_budget", "strata_moe_row_experts",
    "strata_moe_mask_ragged", "strata_moe_expert_affine_inplace", "strata_ctx_set_x_early",
    "strata_allgather", "strata_alltoall", "strata_broadcast", "strata_reducescatter", "strata_allreduce",
    "strata_p2p", "strata_alltoallv",
]


class strata_moe_shape(ctypes.Structure):
    _fields_ = [("R", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("E", ctypes.c_int32), ("K", ctypes.c_int32), ("dispatch_dtype", ctypes.c_int32),
                ("segment_align", ctypes.c_int32), ("flags", ctypes.c_int32), ("slot_capacity", ctypes.c_int32)]


class strata_moe_layout_t(ctypes.Structure):
    _fields_ = [("expert_count", ctypes.c_void_p), ("expert_offset", ctypes.c_void_p),
                ("rank_count", ctypes.c_void_p), ("rank_offset", ctypes.c_void_p),
                ("src_expert_count", ctypes.c_void_p), ("dst_row", ctypes.c_void_p),
                ("src_of_row", ctypes.c_void_p)]


class strata_moe_device_buffers(ctypes.Structure):
    _fields_ = [("ids", ctypes.c_void_p), ("x", ctypes.c_void_p), ("w", ctypes.c_void_p),
                ("recv", ctypes.c_void_p), ("out", ctypes.c_void_p), ("layout", strata_moe_layout_t)]


class strata_span(ctypes.Structure):
    _fields_ = [("cta", ctypes.c_uint32), ("kernel", ctypes.c_uint8), ("stage", ctypes.c_uint8),
                ("flags", ctypes.c_uint16), ("begin_ns", ctypes.c_uint64), ("end_ns", ctypes.c_uint64)]


class strata_tier(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_int64), ("beta", ctypes.c_int64), ("unit_rows", ctypes.c_int64),
                ("fanout_cap", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class strata_partition_policy(ctypes.Structure):
    _fields_ = [("n_tiers", ctypes.c_int32), ("g0", ctypes.c_int32), ("g1", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("tiers", strata_tier * 3)]


class strata_partition_t(ctypes.Structure):
    _fields_ = [("win_base", ctypes.c_void_p), ("unit_desc", ctypes.c_void_p), ("unit_cost", ctypes.c_void_p),
                ("n_units", ctypes.c_void_p), ("task_offset", ctypes.c_void_p), ("task_unit", ctypes.c_void_p),
                ("core_load", ctypes.c_void_p), ("scratch", ctypes.c_void_p), ("task_stripe", ctypes.c_void_p)]


def make_policy(tiers, g0: int = 1, g1: int = 1) -> strata_partition_policy:
    """tiers: list of (alpha, beta, unit_rows, fanout_cap), at most 3."""
    p = strata_partition_policy()
    p.n_tiers, p.g0, p.g1 = len(tiers), g0, g1
    for i, (a, be, ur, cap) in enumerate(tiers):
        p.tiers[i] = strata_tier(a, be, ur, cap, 0)
    return p


class StrataError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: status {self.code} ({strata_status_string(self.code)})")


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           f"`python -m paper_2607_26444_b200.build` (there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, sz, i32, u64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64
    P = ctypes.POINTER
    L.strata_status_string.restype = ctypes.c_char_p
    L.strata_status_string.argtypes = [i32]
    sigs = {
        "strata_ctx_create": [P(vp), P(strata_moe_shape), i32],
        "strata_ctx_destroy": [vp],
        "strata_moe_workspace_bytes": [P(strata_moe_shape), P(sz)],
        "strata_moe_recv_rows": [P(strata_moe_shape), P(sz)],
        "strata_ctx_set_workspace": [vp, vp, sz],
        "strata_ctx_launch_count": [vp, P(u64)],
        "strata_pool_register": [vp, vp, sz, P(u64)],
        "strata_pool_is_ready": [vp, vp, sz],
        "strata_pool_unregister": [vp, u64],
        "strata_pool_carve": [vp, u64, sz, sz, P(vp)],
        "strata_pool_reset": [vp, u64],
        "strata_moe_layout": [vp, vp, P(strata_moe_layout_t), vp],
        "strata_moe_dispatch": [vp, P(strata_moe_layout_t), vp, vp, vp, sz, vp],
        "strata_moe_combine": [vp, P(strata_moe_layout_t), vp, sz, vp, vp, vp],
        "strata_moe_recv_view": [vp, vp, i32, vp, P(vp), P(ctypes.c_int64)],
        "strata_device_status": [vp, vp, P(i32)],
        "strata_moe_roundtrip_host": [vp, P(strata_moe_device_buffers), vp, vp, vp, vp, vp],
        "strata_moe_layout_noalloc": [P(strata_moe_shape), vp, P(strata_moe_layout_t), vp, vp],
        "strata_ctx_set_trace": [vp, vp, sz],
        "strata_moe_partition_max_units": [P(strata_moe_shape), P(strata_partition_policy), P(sz)],
        "strata_moe_partition": [vp, P(strata_moe_layout_t), P(strata_partition_policy), i32,
                                 P(strata_partition_t), sz, vp],
        "strata_moe_dispatch_windows": [vp, P(strata_moe_layout_t), P(strata_partition_t), i32, vp, vp, sz, vp],
        "strata_ctx_set_sm_budget": [vp, i32],
        "strata_ctx_set_x_early": [vp, i32],
        "strata_moe_row_experts": [vp, P(strata_moe_layout_t), vp, sz, vp],
        "strata_moe_mask_ragged": [vp, vp, vp, vp],
        "strata_moe_expert_affine_inplace": [vp, P(strata_moe_layout_t), vp, sz, vp, vp, i32, vp],
        "strata_ctx_set_timeline": [vp, vp, sz, sz],
        "strata_timeline_decode": [vp, sz, sz, vp, sz, P(sz), P(sz)],
        "strata_allgather": [vp, i32, vp, vp, sz, vp],
        "strata_alltoall": [vp, i32, vp, vp, sz, vp],
        "strata_broadcast": [vp, i32, i32, vp, vp, sz, vp],
        "strata_p2p": [vp, i32, i32, i32, vp, vp, sz, vp],
        "strata_alltoallv": [vp, i32, vp, sz, vp, sz, vp, vp, vp, vp],
        "strata_reducescatter": [vp, i32, vp, vp, sz, vp],
        "strata_allreduce": [vp, i32, vp, vp, sz, vp],
    }
    for name, args in sigs.items():
        fn = getattr(L, name)
        fn.restype = i32
        fn.argtypes = args
    _lib = L
    return L


# ---- one Python function per C entry point (same names, raw pointers) -------

def strata_status_string(code: int) -> str:
    return lib().strata_status_string(int(code)).decode()


def strata_ctx_create(shape: strata_moe_shape, device: int) -> Tuple[int, Optional[int]]:
    h = ctypes.c_void_p()
    rc = lib().strata_ctx_create(ctypes.byref(h), ctypes.byref(shape), device)
    return rc, h.value


def strata_ctx_destroy(ctx) -> int:
    return lib().strata_ctx_destroy(ctx)


def strata_moe_workspace_bytes(shape: strata_moe_shape) -> Tuple[int, int]:
    n = ctypes.c_size_t()
    rc = lib().strata_moe_workspace_bytes(ctypes.byref(shape), ctypes.byref(n))
    return rc, n.value


def strata_moe_recv_rows(shape: strata_moe_shape) -> Tuple[int, int]:
    n = ctypes.c_size_t()
    rc = lib().strata_moe_recv_rows(ctypes.byref(shape), ctypes.byref(n))
    return rc, n.value


def strata_ctx_set_workspace(ctx, dptr: int, nbytes: int) -> int:
    return lib().strata_ctx_set_workspace(ctx, dptr, nbytes)


def strata_ctx_set_trace(ctx, dptr: Optional[int], capacity_ctas: int) -> int:
    return lib().strata_ctx_set_trace(ctx, dptr, capacity_ctas)


def strata_ctx_launch_count(ctx) -> Tuple[int, int]:
    n = ctypes.c_uint64()
    rc = lib().strata_ctx_launch_count(ctx, ctypes.byref(n))
    return rc, n.value


def strata_pool_register(ctx, dbase: int, nbytes: int) -> Tuple[int, int]:
    rid = ctypes.c_uint64()
    rc = lib().strata_pool_register(ctx, dbase, nbytes, ctypes.byref(rid))
    return rc, rid.value


def strata_pool_is_ready(ctx, dptr: int, nbytes: int) -> int:
    return lib().strata_pool_is_ready(ctx, dptr, nbytes)


def strata_pool_unregister(ctx, region_id: int) -> int:
    return lib().strata_pool_unregister(ctx, region_id)


def strata_pool_carve(ctx, region_id: int, nbytes: int, align: int) -> Tuple[int, Optional[int]]:
    p = ctypes.c_void_p()
    rc = lib().strata_pool_carve(ctx, region_id, nbytes, align, ctypes.byref(p))
    return rc, p.value


def strata_pool_reset(ctx, region_id: int) -> int:
    return lib().strata_pool_reset(ctx, region_id)


def strata_moe_layout(ctx, topk_ids: int, layout: strata_moe_layout_t, stream: int) -> int:
    return lib().strata_moe_layout(ctx, topk_ids, ctypes.byref(layout), stream)


def strata_moe_dispatch(ctx, layout: strata_moe_layout_t, x: int, recv: int, recv_scale: Optional[int],
                        capacity_rows: int, stream: int) -> int:
    return lib().strata_moe_dispatch(ctx, ctypes.byref(layout), x, recv, recv_scale, capacity_rows, stream)


def strata_moe_combine(ctx, layout: strata_moe_layout_t, y: int, y_rows: int, topk_w: int, out: int,
                       stream: int) -> int:
    return lib().strata_moe_combine(ctx, ctypes.byref(layout), y, y_rows, topk_w, out, stream)


def strata_moe_recv_view(ctx, h_rank_offset, rank: int, recv: int) -> Tuple[int, Optional[int], int]:
    """h_rank_offset: a host numpy int32 array [R+1]."""
    base, rows = ctypes.c_void_p(), ctypes.c_int64()
    rc = lib().strata_moe_recv_view(ctx, h_rank_offset.ctypes.data, rank, recv, ctypes.byref(base),
                                    ctypes.byref(rows))
    return rc, base.value, rows.value


def strata_device_status(ctx, stream: int) -> Tuple[int, int]:
    out = ctypes.c_int()
    rc = lib().strata_device_status(ctx, stream, ctypes.byref(out))
    return rc, out.value


def strata_moe_roundtrip_host(ctx, dev: strata_moe_device_buffers, h_ids: int, h_x: int, h_w: int, h_out: int,
                              stream: int) -> int:
    return lib().strata_moe_roundtrip_host(ctx, ctypes.byref(dev), h_ids, h_x, h_w, h_out, stream)


def strata_moe_layout_noalloc(shape: strata_moe_shape, topk_ids: int, layout: strata_moe_layout_t,
                              device_status: Optional[int], stream: int) -> int:
    """Routing layout on the current device with the library's built-in scratch: no context, no
    workspace, nothing allocated.  For callers that cannot allocate device memory (see the header)."""
    return lib().strata_moe_layout_noalloc(ctypes.byref(shape), topk_ids, ctypes.byref(layout), device_status,
                                           stream)


def strata_moe_partition_max_units(shape: strata_moe_shape, policy: strata_partition_policy) -> Tuple[int, int]:
    n = ctypes.c_size_t()
    rc = lib().strata_moe_partition_max_units(ctypes.byref(shape), ctypes.byref(policy), ctypes.byref(n))
    return rc, n.value


def strata_moe_partition(ctx, layout: strata_moe_layout_t, policy: strata_partition_policy, n_cores: int,
                         out: strata_partition_t, max_units: int, stream: int) -> int:
    return lib().strata_moe_partition(ctx, ctypes.byref(layout), ctypes.byref(policy), n_cores, ctypes.byref(out),
                                      max_units, stream)


def strata_moe_dispatch_windows(ctx, layout: strata_moe_layout_t, partition: strata_partition_t, n_cores: int,
                                x: int, recv: int, capacity_rows: int, stream: int) -> int:
    return lib().strata_moe_dispatch_windows(ctx, ctypes.byref(layout), ctypes.byref(partition), n_cores, x, recv,
                                             capacity_rows, stream)


def strata_moe_row_experts(ctx, layout: strata_moe_layout_t, row_expert: int, capacity_rows: int, stream: int) -> int:
    return lib().strata_moe_row_experts(ctx, ctypes.byref(layout), row_expert, capacity_rows, stream)


def strata_moe_mask_ragged(ctx, tokens_per_rank: int, topk_ids: int, stream: int) -> int:
    return lib().strata_moe_mask_ragged(ctx, tokens_per_rank, topk_ids, stream)


def strata_moe_expert_affine_inplace(ctx, layout: strata_moe_layout_t, recv: int, capacity_rows: int, scale: int,
                                     bias: int, tile_rows: int, stream: int) -> int:
    return lib().strata_moe_expert_affine_inplace(ctx, ctypes.byref(layout), recv, capacity_rows, scale, bias,
                                                  tile_rows, stream)


def strata_ctx_set_x_early(ctx, on: int) -> int:
    return lib().strata_ctx_set_x_early(ctx, int(on))


def strata_ctx_set_sm_budget(ctx, n_sm: int) -> int:
    return lib().strata_ctx_set_sm_budget(ctx, n_sm)


def strata_ctx_set_timeline(ctx, buf: Optional[int], n_ctas: int, events_per_cta: int) -> int:
    return lib().strata_ctx_set_timeline(ctx, buf, n_ctas, events_per_cta)


def strata_timeline_decode(host_buf: int, n_ctas: int, events_per_cta: int, spans: Optional[int],
                           max_spans: int) -> Tuple[int, int, int]:
    """Returns (status, spans found, events dropped); host_buf and spans are host addresses."""
    n, lost = ctypes.c_size_t(), ctypes.c_size_t()
    rc = lib().strata_timeline_decode(host_buf, n_ctas, events_per_cta, spans, max_spans, ctypes.byref(n),
                                      ctypes.byref(lost))
    return rc, n.value, lost.value


def strata_allgather(ctx, R: int, src: int, dst: int, bytes_per_rank: int, stream: int) -> int:
    return lib().strata_allgather(ctx, R, src, dst, bytes_per_rank, stream)


def strata_alltoall(ctx, R: int, src: int, dst: int, bytes_per_slice: int, stream: int) -> int:
    return lib().strata_alltoall(ctx, R, src, dst, bytes_per_slice, stream)


def strata_broadcast(ctx, R: int, root: int, src: int, dst: int, nbytes: int, stream: int) -> int:
    return lib().strata_broadcast(ctx, R, root, src, dst, nbytes, stream)


def strata_p2p(ctx, R: int, src_rank: int, dst_rank: int, src: int, dst: int, nbytes: int, stream: int) -> int:
    return lib().strata_p2p(ctx, R, src_rank, dst_rank, src, dst, nbytes, stream)


def strata_alltoallv(ctx, R: int, src: int, in_stride: int, dst: int, out_stride: int, send_bytes: int,
                     send_offset: int, recv_offset: int, stream: int) -> int:
    return lib().strata_alltoallv(ctx, R, src, in_stride, dst, out_stride, send_bytes, send_offset, recv_offset, stream)


def strata_reducescatter(ctx, R: int, src: int, dst: int, elems_per_slice: int, stream: int) -> int:
    return lib().strata_reducescatter(ctx, R, src, dst, elems_per_slice, stream)


def strata_allreduce(ctx, R: int, src: int, dst: int, elems: int, stream: int) -> int:
    return lib().strata_allreduce(ctx, R, src, dst, elems, stream)


# ---- convenience wrapper over torch tensors (memory + streams only) ---------

def _check(rc: int, where: str) -> None:
    if rc != STRATA_OK:
        raise StrataError(rc, where)


class Layout:
    """Device tensors holding the routing metadata, plus the C struct pointing at them."""

    def __init__(self, R: int, T: int, K: int, E: int, device, with_optional: bool = True,
                 recv_rows: Optional[int] = None):
        import torch
        i32 = dict(dtype=torch.int32, device=device)
        self.expert_count = torch.empty(E, **i32)
        self.expert_offset = torch.empty(E + 1, **i32)
        self.rank_count = torch.empty(R, **i32)
        self.rank_offset = torch.empty(R + 1, **i32)
        self.src_expert_count = torch.empty((R, E), **i32) if with_optional else None
        self.dst_row = torch.empty((R, T, K), **i32)
        self.src_of_row = torch.empty(recv_rows or R * T * K, **i32) if with_optional else None
        self.c = strata_moe_layout_t(
            self.expert_count.data_ptr(), self.expert_offset.data_ptr(), self.rank_count.data_ptr(),
            self.rank_offset.data_ptr(),
            self.src_expert_count.data_ptr() if with_optional else None,
            self.dst_row.data_ptr(),
            self.src_of_row.data_ptr() if with_optional else None)


class Partition:
    """Device tensors of a window-partitioning policy, plus the C struct pointing at them."""

    def __init__(self, R: int, E: int, n_cores: int, max_units: int, device):
        import torch
        i32 = dict(dtype=torch.int32, device=device)
        i64 = dict(dtype=torch.int64, device=device)
        self.n_cores, self.max_units = n_cores, max_units
        self.win_base = torch.zeros((R, E), **i32)
        self.unit_desc = torch.zeros((max_units, 4), **i32)
        self.unit_cost = torch.zeros(max_units, **i64)
        self.n_units = torch.zeros(1, **i32)
        self.task_offset = torch.zeros(n_cores + 1, **i32)
        self.task_unit = torch.zeros(max_units, **i32)
        self.core_load = torch.zeros(n_cores, **i64)
        self.scratch = torch.zeros(max_units * (R + 2), **i32)
        self.task_stripe = torch.zeros(max_units, **i32)
        self.c = strata_partition_t(self.win_base.data_ptr(), self.unit_desc.data_ptr(), self.unit_cost.data_ptr(),
                                    self.n_units.data_ptr(), self.task_offset.data_ptr(), self.task_unit.data_ptr(),
                                    self.core_load.data_ptr(), self.scratch.data_ptr(), self.task_stripe.data_ptr())


class MoEContext:
    """One shape on one GPU.  Owns a strata_ctx and its workspace tensor."""

    def __init__(self, R: int, T: int, H: int, E: int, K: int, dispatch_dtype: int = STRATA_BF16,
                 device: int = 0, segment_align: int = 0, allow_unrouted: bool = False,
                 slot_capacity: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("MoEContext needs a CUDA device (there is no CPU fallback)")
        self.shape = strata_moe_shape(R, T, H, E, K, dispatch_dtype, segment_align,
                                      STRATA_FLAG_ALLOW_UNROUTED if allow_unrouted else 0, slot_capacity)
        self.R, self.T, self.H, self.E, self.K = R, T, H, E, K
        self.fp8 = dispatch_dtype == STRATA_FP8_E4M3_B128
        self.n_tok, self.n_items = R * T, R * T * K
        self.device = torch.device("cuda", device)
        rc, h = strata_ctx_create(self.shape, device)
        _check(rc, "strata_ctx_create")
        self.h = h
        rc, self.recv_rows = strata_moe_recv_rows(self.shape)     # rows a receive buffer must hold
        _check(rc, "strata_moe_recv_rows")
        rc, nbytes = strata_moe_workspace_bytes(self.shape)
        _check(rc, "strata_moe_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        _check(strata_ctx_set_workspace(self.h, self.workspace.data_ptr(), nbytes), "strata_ctx_set_workspace")
        self._regions = {}

    def close(self) -> None:
        if getattr(self, "h", None):
            strata_ctx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _stream() -> int:
        import torch
        return torch.cuda.current_stream().cuda_stream

    # pool -----------------------------------------------------------------
    def register(self, tensor) -> int:
        rc, rid = strata_pool_register(self.h, tensor.data_ptr(), tensor.numel() * tensor.element_size())
        _check(rc, "strata_pool_register")
        self._regions[rid] = tensor          # keep the allocation alive while registered
        return rid

    def unregister(self, rid: int) -> None:
        _check(strata_pool_unregister(self.h, rid), "strata_pool_unregister")
        self._regions.pop(rid, None)

    def carve(self, rid: int, shape, dtype, align: int = 256):
        """A tensor view of a sub-range carved from a registered region (zero copy)."""
        import torch
        base = self._regions[rid]
        n = 1
        for d in shape:
            n *= int(d)
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        rc, p = strata_pool_carve(self.h, rid, nbytes, align)
        _check(rc, "strata_pool_carve")
        off = p - base.data_ptr()
        return base.view(torch.uint8).reshape(-1)[off:off + nbytes].view(dtype).reshape(*shape)

    def new_layout(self, with_optional: bool = True) -> Layout:
        return Layout(self.R, self.T, self.K, self.E, self.device, with_optional, self.recv_rows)

    # hot path ---------------------------------------------------------------
    def layout(self, ids, layout: Optional[Layout] = None) -> Layout:
        layout = layout or self.new_layout()
        _check(strata_moe_layout(self.h, ids.data_ptr(), layout.c, self._stream()), "strata_moe_layout")
        return layout

    def dispatch(self, layout: Layout, x, recv, recv_scale=None) -> None:
        _check(strata_moe_dispatch(self.h, layout.c, x.data_ptr(), recv.data_ptr(),
                                   recv_scale.data_ptr() if recv_scale is not None else None,
                                   recv.shape[0], self._stream()), "strata_moe_dispatch")

    def combine(self, layout: Layout, y, w, out) -> None:
        _check(strata_moe_combine(self.h, layout.c, y.data_ptr(), y.shape[0], w.data_ptr(), out.data_ptr(),
                                  self._stream()), "strata_moe_combine")

    def mask_ragged(self, tokens_per_rank, ids) -> None:
        """Marks, in place, the slots of the tokens t >= tokens_per_rank[r] as not routed (-1)."""
        _check(strata_moe_mask_ragged(self.h, tokens_per_rank.data_ptr(), ids.data_ptr(), self._stream()),
               "strata_moe_mask_ragged")

    def expert_affine_inplace(self, layout: Layout, recv, scale, bias, tile_rows: int = 1) -> None:
        """recv[row] = bf16(fma(recv[row], scale[e], bias[e])) for every occupied row, in place, tile by tile."""
        _check(strata_moe_expert_affine_inplace(self.h, layout.c, recv.data_ptr(), recv.shape[0], scale.data_ptr(),
                                                bias.data_ptr(), tile_rows, self._stream()),
               "strata_moe_expert_affine_inplace")

    def row_experts(self, layout: Layout, out=None):
        """int32 [recv_rows]: the expert of every occupied receive row, -1 for padding and empty rows."""
        import torch
        if out is None:
            out = torch.empty((self.recv_rows,), dtype=torch.int32, device=self.device)
        _check(strata_moe_row_experts(self.h, layout.c, out.data_ptr(), out.shape[0], self._stream()),
               "strata_moe_row_experts")
        return out

    def trace(self, capacity_ctas: int = 4096):
        """Turns per-CTA probes on; returns the tensor [capacity, 4] = (start_ns, end_ns, wait_in_ns, wait_out_ns)."""
        import torch
        t = torch.zeros((capacity_ctas, 4), dtype=torch.int64, device=self.device)
        _check(strata_ctx_set_trace(self.h, t.data_ptr(), capacity_ctas), "strata_ctx_set_trace")
        self._trace = t
        return t

    @staticmethod
    def trace_summary(trace) -> dict:
        """Decodes a trace tensor after a launch (see timeline.trace_summary)."""
        from .timeline import trace_summary
        return trace_summary(trace.cpu().numpy())

    def trace_off(self) -> None:
        _check(strata_ctx_set_trace(self.h, None, 0), "strata_ctx_set_trace")
        self._trace = None

    def x_early(self, on: bool = True) -> None:
        """Promise that x is complete before the call preceding each dispatch starts (see the header)."""
        _check(strata_ctx_set_x_early(self.h, 1 if on else 0), "strata_ctx_set_x_early")

    def sm_budget(self, n_sm: int) -> None:
        """Sizes the persistent grids for n_sm SMs (0: the whole GPU)."""
        _check(strata_ctx_set_sm_budget(self.h, n_sm), "strata_ctx_set_sm_budget")

    def timeline(self, n_ctas: int = 2048, events_per_cta: int = 2048, pinned: bool = False):
        """Turns the event timeline on; returns the zeroed buffer [n_ctas, 1 + events_per_cta] (int64), in
        device memory or, with pinned=True, in page-locked host memory that the kernels write in place."""
        import torch
        if pinned:
            t = torch.zeros((n_ctas, 1 + events_per_cta), dtype=torch.int64, pin_memory=True)
        else:
            t = torch.zeros((n_ctas, 1 + events_per_cta), dtype=torch.int64, device=self.device)
        torch.cuda.synchronize(self.device)
        _check(strata_ctx_set_timeline(self.h, t.data_ptr(), n_ctas, events_per_cta), "strata_ctx_set_timeline")
        self._timeline = t
        return t

    def timeline_off(self) -> None:
        _check(strata_ctx_set_timeline(self.h, None, 0, 0), "strata_ctx_set_timeline")
        self._timeline = None

    @staticmethod
    def timeline_spans(t):
        """Synchronises and decodes a timeline buffer (see timeline.decode_timeline); returns (spans, dropped)."""
        import torch
        from .timeline import decode_timeline
        torch.cuda.synchronize()
        return decode_timeline(t.cpu().numpy().view("uint64"))

    # the paper's static window partitioning, as an alternative to run-time work claiming ------------
    def partition(self, layout: Layout, policy: strata_partition_policy, n_cores: int,
                  part: Optional[Partition] = None) -> Partition:
        if part is None:
            rc, mu = strata_moe_partition_max_units(self.shape, policy)
            _check(rc, "strata_moe_partition_max_units")
            part = Partition(self.R, self.E, n_cores, mu, self.device)
        _check(strata_moe_partition(self.h, layout.c, policy, n_cores, part.c, part.max_units, self._stream()),
               "strata_moe_partition")
        return part

    def dispatch_windows(self, layout: Layout, part: Partition, x, recv) -> None:
        _check(strata_moe_dispatch_windows(self.h, layout.c, part.c, part.n_cores, x.data_ptr(), recv.data_ptr(),
                                           recv.shape[0], self._stream()), "strata_moe_dispatch_windows")

    # full-mesh collectives over emulated ranks: tensors are [R, ...] slabs, one part per rank ------
    def allgather(self, src, dst) -> None:
        """src [R, n] -> dst [R, R, n] (any dtype; moved as bytes)."""
        R = src.shape[0]
        _check(strata_allgather(self.h, R, src.data_ptr(), dst.data_ptr(), src[0].numel() * src.element_size(),
                                self._stream()), "strata_allgather")

    def alltoall(self, src, dst) -> None:
        """src [R, R, n] -> dst [R, R, n], dst[r, p] = src[p, r]."""
        R = src.shape[0]
        _check(strata_alltoall(self.h, R, src.data_ptr(), dst.data_ptr(), src[0, 0].numel() * src.element_size(),
                               self._stream()), "strata_alltoall")

    def broadcast(self, src, dst, root: int) -> None:
        """src [R, n] -> dst [R, n], dst[r] = src[root]."""
        R = src.shape[0]
        _check(strata_broadcast(self.h, R, root, src.data_ptr(), dst.data_ptr(),
                                src[0].numel() * src.element_size(), self._stream()), "strata_broadcast")

    def p2p(self, src, dst, src_rank: int, dst_rank: int) -> None:
        """src, dst [R, n]: dst[dst_rank] = src[src_rank]."""
        R = src.shape[0]
        _check(strata_p2p(self.h, R, src_rank, dst_rank, src.data_ptr(), dst.data_ptr(),
                          src[0].numel() * src.element_size(), self._stream()), "strata_p2p")

    def alltoallv(self, src, dst, send_bytes, send_offset, recv_offset) -> None:
        """src [R, in_stride] and dst [R, out_stride] uint8; the three int64 [R, R] device tensors give, per
        (sender, receiver), the byte count, the offset in the sender's part and (indexed [receiver, sender])
        the offset in the receiver's part."""
        R = src.shape[0]
        for t in (src, dst, send_bytes, send_offset, recv_offset):
            if not t.is_contiguous():
                raise ValueError("alltoallv needs contiguous tensors")
        _check(strata_alltoallv(self.h, R, src.data_ptr(), src[0].numel() * src.element_size(), dst.data_ptr(),
                                dst[0].numel() * dst.element_size(), send_bytes.data_ptr(), send_offset.data_ptr(),
                                recv_offset.data_ptr(), self._stream()), "strata_alltoallv")

    def reducescatter(self, src, dst) -> None:
        """src bf16 [R, R, n] -> dst bf16 [R, n], dst[r] = sum over p of src[p, r] (rank order, fp32)."""
        R = src.shape[0]
        _check(strata_reducescatter(self.h, R, src.data_ptr(), dst.data_ptr(), src[0, 0].numel(), self._stream()),
               "strata_reducescatter")

    def allreduce(self, src, dst) -> None:
        """src bf16 [R, n] -> dst bf16 [R, n], dst[r] = sum over p of src[p] (rank order, fp32)."""
        R = src.shape[0]
        _check(strata_allreduce(self.h, R, src.data_ptr(), dst.data_ptr(), src[0].numel(), self._stream()),
               "strata_allreduce")

    def device_status(self) -> int:
        rc, st = strata_device_status(self.h, self._stream())
        _check(rc, "strata_device_status")
        return st

    def launch_count(self) -> int:
        rc, n = strata_ctx_launch_count(self.h)
        _check(rc, "strata_ctx_launch_count")
        return n
