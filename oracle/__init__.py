"""CPU oracle (test infrastructure): ctypes access to ``strata_oracle.c``.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It never imports the CUDA binding, and the CUDA binding never
imports it.  Arrays are numpy; bf16 travels as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "strata_oracle.c")
_LIB = os.path.join(_HERE, "libstrata_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (IEEE arithmetic: no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-march=native", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
               "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", _SRC, "-o", _LIB + ".tmp", "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i32, i64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        L.oracle_layout.restype = i64
        L.oracle_layout.argtypes = [i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.oracle_dispatch_bf16.restype = None
        L.oracle_dispatch_bf16.argtypes = [i64, i32, i32, vp, vp, vp, i32]
        L.oracle_dispatch_fp8.restype = None
        L.oracle_dispatch_fp8.argtypes = [i64, i32, i32, vp, vp, vp, vp, i32]
        L.oracle_combine.restype = None
        L.oracle_combine.argtypes = [i64, i32, i32, vp, vp, vp, vp, i32]
        L.oracle_e4m3_encode.restype = ctypes.c_uint8
        L.oracle_e4m3_encode.argtypes = [ctypes.c_float]
        L.oracle_partition.restype = i64
        L.oracle_partition.argtypes = [i32, i32, i64, i32, vp, vp, vp, i32, i32, i32, i64, vp, vp, vp, vp, vp, vp, vp]
        L.oracle_dispatch_windows.restype = None
        L.oracle_dispatch_windows.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        for name in ("oracle_allgather", "oracle_alltoall", "oracle_reducescatter", "oracle_allreduce"):
            getattr(L, name).restype = None
            getattr(L, name).argtypes = [i32, i64, vp, vp]
        L.oracle_broadcast.restype = None
        L.oracle_broadcast.argtypes = [i32, i32, i64, vp, vp]
        L.oracle_expert_affine.restype = None
        L.oracle_expert_affine.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.oracle_mask_ragged.restype = None
        L.oracle_mask_ragged.argtypes = [i32, i32, i32, vp, vp]
        L.oracle_row_experts.restype = None
        L.oracle_row_experts.argtypes = [i32, i32, i32, vp, vp, vp, i64, vp]
        L.oracle_alltoallv.restype = i64
        L.oracle_alltoallv.argtypes = [i32, i64, i64, vp, vp, vp, vp, vp]
        L.oracle_p2p.restype = None
        L.oracle_p2p.argtypes = [i32, i32, i64, vp, vp]
        L.oracle_max_threads.restype = i32
        L.oracle_max_threads.argtypes = []
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def max_threads() -> int:
    return int(lib().oracle_max_threads())


class BadExpertId(ValueError):
    def __init__(self, item: int):
        super().__init__(f"expert id out of range at flat item {item}")
        self.item = item


def layout(ids: np.ndarray, E: int, segment_align: int = 1, allow_unrouted: bool = False,
           slot_capacity: int = 0) -> Dict[str, np.ndarray]:
    """Routing layout of ids int32 [R,T,K]; raises BadExpertId for an id outside [0,E) (-1 is accepted
    as "not routed" with allow_unrouted).  segment_align > 1 pads every expert segment to that many rows.
    slot_capacity > 0 selects the fixed-capacity layout [E][R][capacity]; out["dropped"] counts the items
    that did not fit."""
    ids = _c(ids, np.int32)
    R, T, K = ids.shape
    N = R * T * K
    A = max(1, int(segment_align))
    out = {
        "expert_count": np.zeros(E, np.int32),
        "expert_offset": np.zeros(E + 1, np.int32),
        "rank_count": np.zeros(R, np.int32),
        "rank_offset": np.zeros(R + 1, np.int32),
        "src_expert_count": np.zeros((R, E), np.int32),
        "dst_row": np.full((R, T, K), -1, np.int32),
        "src_of_row": np.full(E * R * slot_capacity if slot_capacity > 0 else N + E * (A - 1), -1, np.int32),
    }
    rc = lib().oracle_layout(R, T, K, E, A, int(bool(allow_unrouted)), int(slot_capacity), _p(ids),
                             _p(out["expert_count"]),
                             _p(out["expert_offset"]), _p(out["rank_count"]), _p(out["rank_offset"]),
                             _p(out["src_expert_count"]), _p(out["dst_row"]), _p(out["src_of_row"]))
    if rc < 0:
        if rc < -(1 << 40):
            raise ValueError("invalid shape (need R,K,E > 0 and E % R == 0)")
        raise BadExpertId(int(-rc - 1))
    out["src_of_row"] = out["src_of_row"][:int(out["expert_offset"][E])]
    out["dropped"] = int(rc) if slot_capacity > 0 else 0
    return out


def mask_ragged(ids: np.ndarray, tokens_per_rank) -> np.ndarray:
    """A copy of ids int32 [R,T,K] with the slots of tokens t >= tokens_per_rank[r] set to -1."""
    out = _c(ids, np.int32).copy()
    R, T, K = out.shape
    tpr = _c(tokens_per_rank, np.int32)
    assert tpr.shape == (R,)
    lib().oracle_mask_ragged(R, T, K, _p(tpr), _p(out))
    return out


def row_experts(lay: Dict[str, np.ndarray], R: int, slot_capacity: int = 0) -> np.ndarray:
    """int32 [rows of the receive buffer]: the expert of every occupied row, -1 for padding and empty rows."""
    E = lay["expert_count"].shape[0]
    n_rows = lay["src_of_row"].shape[0]
    out = np.empty(n_rows, np.int32)
    lib().oracle_row_experts(R, E, int(slot_capacity), _p(_c(lay["expert_count"], np.int32)),
                             _p(_c(lay["expert_offset"], np.int32)), _p(_c(lay["src_expert_count"], np.int32)),
                             n_rows, _p(out))
    return out


def expert_affine(lay: Dict[str, np.ndarray], recv: np.ndarray, scale: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """A copy of recv uint16 [rows,H] in which every occupied row of expert e's segment has become
    bf16(fma(f32(row), scale[e], bias[e])); padding rows keep their contents."""
    out = _c(recv, np.uint16).copy()
    E = lay["expert_count"].shape[0]
    scale, bias = _c(scale, np.float32), _c(bias, np.float32)
    assert scale.shape == (E,) and bias.shape == (E,)
    assert out.shape[0] >= int(lay["expert_offset"][E])
    lib().oracle_expert_affine(E, out.shape[1], _p(_c(lay["expert_count"], np.int32)),
                               _p(_c(lay["expert_offset"], np.int32)), _p(scale), _p(bias), _p(out))
    return out


def dispatch_bf16(dst_row: np.ndarray, x: np.ndarray, nthreads: int = 1,
                  recv: Optional[np.ndarray] = None, n_rows: Optional[int] = None) -> np.ndarray:
    """recv uint16 [n_rows,H] (default n_rows = N) with recv[dst_row[i]] = x[i // K]; rows that no item
    maps to (padding) keep 0xDEAD."""
    dst_row = _c(dst_row, np.int32)
    K = dst_row.shape[-1]
    H = x.shape[-1]
    x2 = _c(x, np.uint16).reshape(-1, H)
    n_tok = x2.shape[0]
    assert dst_row.size == n_tok * K
    if recv is None:
        recv = np.full((n_rows if n_rows is not None else n_tok * K, H), 0xDEAD, np.uint16)
    assert recv.dtype == np.uint16 and recv.flags.c_contiguous
    lib().oracle_dispatch_bf16(n_tok, K, H, _p(dst_row), _p(x2), _p(recv), nthreads)
    return recv


def dispatch_fp8(dst_row: np.ndarray, x: np.ndarray, nthreads: int = 1, n_rows: Optional[int] = None):
    """(recv_q uint8 [n_rows,H], recv_scale float32 [n_rows,H/128]); padding rows keep 0x7F / -7."""
    dst_row = _c(dst_row, np.int32)
    K = dst_row.shape[-1]
    H = x.shape[-1]
    assert H % 128 == 0
    x2 = _c(x, np.uint16).reshape(-1, H)
    n_tok = x2.shape[0]
    assert dst_row.size == n_tok * K
    rows = n_rows if n_rows is not None else n_tok * K
    q = np.full((rows, H), 0x7F, np.uint8)
    s = np.full((rows, H // 128), -7.0, np.float32)
    lib().oracle_dispatch_fp8(n_tok, K, H, _p(dst_row), _p(x2), _p(q), _p(s), nthreads)
    return q, s


def combine(dst_row: np.ndarray, y: np.ndarray, w: np.ndarray, nthreads: int = 1) -> np.ndarray:
    """out uint16 [n_tok,H] = bf16(sum_k w[n,k] * y[dst_row[n,k]]) (fp32 FMA chain, slot order)."""
    dst_row = _c(dst_row, np.int32)
    K = dst_row.shape[-1]
    y = _c(y, np.uint16)
    H = y.shape[-1]
    w2 = _c(w, np.float32).reshape(-1, K)
    n_tok = w2.shape[0]
    assert dst_row.size == n_tok * K
    out = np.empty((n_tok, H), np.uint16)
    lib().oracle_combine(n_tok, K, H, _p(dst_row), _p(y), _p(w2), _p(out), nthreads)
    return out


def e4m3_encode(v: np.ndarray) -> np.ndarray:
    """uint8 codes of a float32 array (scalar loop in C; for tests)."""
    v = _c(v, np.float32)
    f = lib().oracle_e4m3_encode
    return np.fromiter((f(float(t)) for t in v.ravel()), dtype=np.uint8, count=v.size).reshape(v.shape)


TIER_DTYPE = np.dtype([("alpha", np.int64), ("beta", np.int64), ("unit_rows", np.int64),
                       ("fanout_cap", np.int32), ("pad", np.int32)])


def make_tiers(tiers) -> np.ndarray:
    """tiers: list of (alpha, beta, unit_rows, fanout_cap)."""
    a = np.zeros(len(tiers), TIER_DTYPE)
    for i, (al, be, ur, cap) in enumerate(tiers):
        a[i] = (al, be, ur, cap, 0)
    return a


def partition(lay: Dict[str, np.ndarray], row_bytes: int, n_cores: int, tiers, g0: int = 1, g1: int = 1,
              max_units: int = 1 << 16) -> Dict[str, np.ndarray]:
    """Window partitioning + LPT-style list scheduling of dispatch (paper Sec. 6.2, App. B to D)."""
    sec = _c(lay["src_expert_count"], np.int32)
    R, E = sec.shape
    off = _c(lay["expert_offset"], np.int32)
    t = make_tiers(tiers)
    out = {
        "win_base": np.zeros((R, E), np.int32),
        "unit_desc": np.zeros((max_units, 4), np.int32),
        "unit_cost": np.zeros(max_units, np.int64),
        "task_offset": np.zeros(n_cores + 1, np.int32),
        "task_unit": np.zeros(max_units, np.int32),
        "task_stripe": np.zeros(max_units, np.int32),
        "core_load": np.zeros(n_cores, np.int64),
    }
    U = lib().oracle_partition(R, E, row_bytes, n_cores, _p(sec), _p(off), _p(t), len(t), g0, g1, max_units,
                               _p(out["win_base"]), _p(out["unit_desc"]), _p(out["unit_cost"]),
                               _p(out["task_offset"]), _p(out["task_unit"]), _p(out["task_stripe"]),
                               _p(out["core_load"]))
    if U < 0:
        raise ValueError("more units than max_units" if U == -1 else "a tier's cap, unit size or bandwidth is below 1")
    out["n_units"] = int(U)
    out["unit_desc"] = out["unit_desc"][:U]
    out["unit_cost"] = out["unit_cost"][:U]
    out["task_unit"] = out["task_unit"][:U]
    out["task_stripe"] = out["task_stripe"][:U]
    return out


def dispatch_windows(lay: Dict[str, np.ndarray], part: Dict[str, np.ndarray], x: np.ndarray, K: int) -> np.ndarray:
    sec = _c(lay["src_expert_count"], np.int32)
    R, E = sec.shape
    H = x.shape[-1]
    x2 = _c(x, np.uint16).reshape(-1, H)
    n_cores = part["task_offset"].size - 1
    recv = np.full((x2.shape[0] * K, H), 0xDEAD, np.uint16)
    lib().oracle_dispatch_windows(R, E, K, H, n_cores, _p(sec), _p(_c(part["win_base"], np.int32)),
                                  _p(_c(part["unit_desc"], np.int32)), _p(_c(part["task_offset"], np.int32)),
                                  _p(_c(part["task_unit"], np.int32)), _p(_c(lay["src_of_row"], np.int32)),
                                  _p(x2), _p(recv))
    return recv


# ---- full-mesh collectives over emulated ranks (paper Sec. 6.1) ----------------------------------

def allgather(x: np.ndarray) -> np.ndarray:
    """x uint8 [R, M] -> out uint8 [R, R, M], out[r, p] = x[p]."""
    x = _c(x, np.uint8)
    R, M = x.shape
    out = np.empty((R, R, M), np.uint8)
    lib().oracle_allgather(R, M, _p(x), _p(out))
    return out


def alltoall(x: np.ndarray) -> np.ndarray:
    """x uint8 [R, R, S] -> out uint8 [R, R, S], out[r, p] = x[p, r]."""
    x = _c(x, np.uint8)
    R, R2, S = x.shape
    assert R == R2
    out = np.empty((R, R, S), np.uint8)
    lib().oracle_alltoall(R, S, _p(x), _p(out))
    return out


def broadcast(x: np.ndarray, root: int) -> np.ndarray:
    """x uint8 [R, M] -> out uint8 [R, M], out[r] = x[root]."""
    x = _c(x, np.uint8)
    R, M = x.shape
    assert 0 <= root < R
    out = np.empty((R, M), np.uint8)
    lib().oracle_broadcast(R, root, M, _p(x), _p(out))
    return out


def reducescatter(x: np.ndarray) -> np.ndarray:
    """x bf16 bits uint16 [R, R, S] -> out uint16 [R, S], out[r] = sum over p (rank order, fp32) of x[p, r]."""
    x = _c(x, np.uint16)
    R, R2, S = x.shape
    assert R == R2
    out = np.empty((R, S), np.uint16)
    lib().oracle_reducescatter(R, S, _p(x), _p(out))
    return out


def allreduce(x: np.ndarray) -> np.ndarray:
    """x bf16 bits uint16 [R, M] -> out uint16 [R, M], out[r] = sum over p (rank order, fp32) of x[p]."""
    x = _c(x, np.uint16)
    R, M = x.shape
    out = np.empty((R, M), np.uint16)
    lib().oracle_allreduce(R, M, _p(x), _p(out))
    return out


def alltoallv(x: np.ndarray, out: np.ndarray, send_bytes, send_off, recv_off) -> int:
    """x uint8 [R, in_stride]; out uint8 [R, out_stride] is updated in place: rank p's send_bytes[p, r] bytes at
    x[p, send_off[p, r]:] land at out[r, recv_off[r, p]:].  Returns the number of pairs skipped for not fitting."""
    x = _c(x, np.uint8)
    assert out.dtype == np.uint8 and out.flags.c_contiguous
    R = x.shape[0]
    sb, so, ro = (_c(a, np.int64).reshape(R, R) for a in (send_bytes, send_off, recv_off))
    return int(lib().oracle_alltoallv(R, x.shape[1], out.shape[1], _p(x), _p(out), _p(sb), _p(so), _p(ro)))


def p2p(x: np.ndarray, out: np.ndarray, src: int, dst: int) -> None:
    """x, out uint8 [R, M]: out[dst] = x[src]; the other parts of out are left alone."""
    x = _c(x, np.uint8)
    assert out.dtype == np.uint8 and out.flags.c_contiguous and out.shape == x.shape
    lib().oracle_p2p(src, dst, x.shape[1], _p(x), _p(out))
