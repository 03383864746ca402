"""Seeded synthetic MoE routing workloads (inputs only).

This module produces the *inputs* of the dispatch/combine path: top-k expert
ids, bf16 hidden vectors, fp32 gate weights, and the stand-in for the expert
computation that sits between dispatch and combine.  It holds none of the
method's arithmetic (no layout, no scatter, no quantisation, no combine) and
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed
the very same bytes.

Shapes follow the paper's microbenchmark setting (Sec. 8.1: hidden 7168, top-8,
4096 tokens per batch) and its serving deployment (EP=16 decode); the expert
counts and the FP8/skew variants are the build's own benchmark configurations.
The paper's production routing traces are not available: uniform and Zipf
routing stand in for them.

All arrays are numpy, host resident.  bf16 tensors are carried as uint16 bit
patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

BF16 = 0
FP8_E4M3_B128 = 1


@dataclass(frozen=True)
class MoEConfig:
    name: str
    R: int            # emulated expert-parallel ranks
    T: int            # tokens per rank
    H: int            # hidden size (bf16 elements per row)
    E: int            # experts, E % R == 0, owner(e) = e // (E // R)
    K: int            # experts per token
    routing: str = "uniform"      # "uniform" | "zipf"
    zipf_s: float = 1.2
    sigma: float = 1.0            # std-dev of x
    dispatch_dtype: int = BF16
    expert: str = "identity"      # "identity" | "scale" | "affine" | "dequant"
    seed: int = 0

    @property
    def n_tok(self) -> int:
        return self.R * self.T

    @property
    def n_items(self) -> int:
        return self.R * self.T * self.K

    @property
    def e_loc(self) -> int:
        return self.E // self.R

    def dispatch_bytes(self) -> int:
        """Algorithmic bytes of one dispatch call: every source row read once,
        every receive row (and its scales) written once, ids read and dst_row
        written (8 B per item)."""
        n, nt, h = self.n_items, self.n_tok, self.H
        if self.dispatch_dtype == FP8_E4M3_B128:
            out_row = h + 4 * (h // 128)
        else:
            out_row = 2 * h
        return nt * h * 2 + n * out_row + 8 * n

    def combine_bytes(self) -> int:
        """Algorithmic bytes of one combine call: K expert-output rows read and
        one output row written per token, plus dst_row and weights (8 B/item)."""
        n, nt, h = self.n_items, self.n_tok, self.H
        return n * h * 2 + nt * h * 2 + 8 * n


CONFIGS: Dict[str, MoEConfig] = {
    "tiny": MoEConfig("tiny", R=4, T=128, H=1024, E=16, K=2, expert="scale", seed=1000),
    "decode": MoEConfig("decode", R=16, T=128, H=7168, E=256, K=8, expert="affine", seed=1001),
    "prefill": MoEConfig("prefill", R=16, T=4096, H=7168, E=256, K=8, expert="identity", seed=1002),
    "skew": MoEConfig("skew", R=32, T=512, H=4096, E=128, K=8, routing="zipf",
                      expert="identity", seed=1003),
    "fp8": MoEConfig("fp8", R=64, T=256, H=4096, E=128, K=8, sigma=2.0 ** 0.5,
                     dispatch_dtype=FP8_E4M3_B128, expert="dequant", seed=1004),
}
CONFIG_ORDER = ["tiny", "decode", "prefill", "skew", "fp8"]


def shrink(cfg: MoEConfig, **kw) -> MoEConfig:
    """A smaller or altered copy of a config (same recipe, other sizes)."""
    return replace(cfg, **kw)


# ----------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (format conversion of inputs, not method arithmetic)
# ----------------------------------------------------------------------------

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# generators
# ----------------------------------------------------------------------------

def _rng(seed: int, stream: int) -> np.random.Generator:
    # Philox is counter based: (seed, stream) fully determines the sequence.
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def gen_topk_ids(cfg: MoEConfig) -> np.ndarray:
    """int32 [R, T, K] expert ids, K distinct per token.

    uniform: a uniformly random K-subset in uniformly random order
             (the K smallest of E iid uniform keys, in key order).
    zipf:    popularity rank j in [1, E] has weight j**-s; the expert holding
             rank j is perm[j-1] with perm a seeded permutation; K successive
             draws without replacement, renormalising after each draw, slot
             order = draw order.  Sampled with the Gumbel-top-k identity, which
             has exactly that distribution.
    """
    rng = _rng(cfg.seed, 1)
    nt, E, K = cfg.n_tok, cfg.E, cfg.K
    if K > E:
        raise ValueError("K > E")
    out = np.empty((nt, K), dtype=np.int32)
    logw: Optional[np.ndarray] = None
    if cfg.routing == "zipf":
        perm = _rng(cfg.seed + 1, 7).permutation(E)
        w = np.arange(1, E + 1, dtype=np.float64) ** (-cfg.zipf_s)
        logw = np.empty(E, dtype=np.float64)
        logw[perm] = np.log(w)
    elif cfg.routing != "uniform":
        raise ValueError(cfg.routing)
    step = max(1, (1 << 22) // E)
    for lo in range(0, nt, step):
        hi = min(nt, lo + step)
        u = rng.random((hi - lo, E))
        if logw is None:
            key = u
        else:
            # Gumbel(0,1) = -log(-log(u)); order by descending log w + g
            key = -(logw[None, :] - np.log(-np.log(np.clip(u, 1e-300, 1.0 - 1e-16))))
        if K < E:
            part = np.argpartition(key, K - 1, axis=1)[:, :K]
        else:
            part = np.broadcast_to(np.arange(E), key.shape).copy()
        sub = np.take_along_axis(key, part, axis=1)
        order = np.argsort(sub, axis=1, kind="stable")
        out[lo:hi] = np.take_along_axis(part, order, axis=1).astype(np.int32)
    return out.reshape(cfg.R, cfg.T, K)


def gen_x(cfg: MoEConfig) -> np.ndarray:
    """uint16 [R, T, H]: bf16 bits of fp32 N(0, sigma^2) samples, rounded RNE."""
    rng = _rng(cfg.seed, 2)
    out = np.empty((cfg.R, cfg.T, cfg.H), dtype=np.uint16)
    for r in range(cfg.R):
        f = rng.standard_normal((cfg.T, cfg.H), dtype=np.float32)
        if cfg.sigma != 1.0:
            f *= np.float32(cfg.sigma)
        out[r] = f32_to_bf16_bits(f)
    return out


def gen_gate_weights(cfg: MoEConfig) -> np.ndarray:
    """float32 [R, T, K]: max-subtracted fp32 softmax of K N(0,1) logits."""
    rng = _rng(cfg.seed, 3)
    z = rng.standard_normal((cfg.n_tok, cfg.K), dtype=np.float32)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z, dtype=np.float32)
    p = p / p.sum(axis=1, keepdims=True, dtype=np.float32)
    return np.ascontiguousarray(p.reshape(cfg.R, cfg.T, cfg.K), dtype=np.float32)


def gen_payload(R: int, elems_per_rank: int, seed: int) -> np.ndarray:
    """uint16 [R, elems_per_rank]: every emulated rank's collective payload, bf16 bits of N(0, 1).

    The data-movement collectives treat the same array as raw bytes.
    """
    rng = _rng(seed, 7)
    out = np.empty((R, elems_per_rank), dtype=np.uint16)
    for r in range(R):
        out[r] = f32_to_bf16_bits(rng.standard_normal(elems_per_rank, dtype=np.float32))
    return out


def gen_pair_bytes(R: int, mean_bytes: int, seed: int, skew: float = 1.2, zero_frac: float = 0.1) -> np.ndarray:
    """int64 [R, R]: bytes rank p sends to rank r in an uneven all-to-all, multiples of 16.

    Receiver popularity follows a Zipf(skew) law over a seeded permutation (the shape of the MoE skew
    workload), each pair is jittered by a uniform factor in [0.5, 1.5), and a fraction of the pairs is empty."""
    rng = _rng(seed, 8)
    pop = 1.0 / np.arange(1, R + 1, dtype=np.float64) ** skew
    pop = pop[rng.permutation(R)] / pop.mean()
    size = mean_bytes * pop[None, :] * rng.uniform(0.5, 1.5, size=(R, R))
    size[rng.uniform(size=(R, R)) < zero_frac] = 0.0
    return (np.floor(size / 16.0).astype(np.int64)) * 16


def packed_offsets(pair_bytes: np.ndarray):
    """(send_off [R, R], recv_off [R, R], in_stride, out_stride) for back-to-back packing: rank p's slices lie in
    receiver order in its input, rank r's in sender order in its output."""
    send_off = np.cumsum(pair_bytes, axis=1) - pair_bytes
    recv = pair_bytes.T                                   # recv[r, p] = bytes r gets from p
    recv_off = np.cumsum(recv, axis=1) - recv
    in_stride = int(max(16, pair_bytes.sum(axis=1).max()))
    out_stride = int(max(16, recv.sum(axis=1).max()))
    return (np.ascontiguousarray(send_off, dtype=np.int64), np.ascontiguousarray(recv_off, dtype=np.int64),
            in_stride, out_stride)


def generate(cfg: MoEConfig) -> Dict[str, np.ndarray]:
    return {"ids": gen_topk_ids(cfg), "x": gen_x(cfg), "w": gen_gate_weights(cfg)}


# ----------------------------------------------------------------------------
# stand-in for the expert computation between dispatch and combine.
# Computed ONCE on the host; the same bytes are fed to both combine
# implementations, so its own rounding cannot influence a comparison.
# ----------------------------------------------------------------------------

def e4m3_value_table() -> np.ndarray:
    """float32[256]: value of each OCP e4m3 (fn) code; NaN codes map to NaN."""
    t = np.empty(256, dtype=np.float32)
    for c in range(256):
        s = -1.0 if c & 0x80 else 1.0
        ex, m = (c >> 3) & 0xF, c & 7
        if ex == 0xF and m == 7:
            v = float("nan")
        elif ex == 0:
            v = s * m * 2.0 ** -9
        else:
            v = s * (1.0 + m / 8.0) * 2.0 ** (ex - 7)
        t[c] = v
    return t


def expert_of_row(expert_offset: np.ndarray, n_rows: int) -> np.ndarray:
    """int32[n_rows]: the expert whose receive segment holds each row."""
    counts = np.diff(np.asarray(expert_offset, dtype=np.int64))
    return np.repeat(np.arange(counts.size, dtype=np.int32), counts)[:n_rows]


def expert_standin(cfg: MoEConfig, recv: np.ndarray, expert_offset: np.ndarray,
                   recv_scale: Optional[np.ndarray] = None) -> np.ndarray:
    """uint16 [N, H] bf16 bits of the "expert output" for received rows.

    identity: y is recv itself (the very same array: zero copy).
    scale:    y = bf16(f32(recv) * (1 + e/E))
    affine:   y = bf16(f32(recv) * (1 + e/E) + 0.01 e)
    dequant:  y = bf16(value(recv_q) * recv_scale[row, col // 128])
    with e the expert owning the row.
    """
    n = recv.shape[0]
    if cfg.expert == "identity":
        return recv
    y = np.empty((n, cfg.H), dtype=np.uint16)
    chunk = max(1, (1 << 24) // cfg.H)
    if cfg.expert == "dequant":
        assert recv_scale is not None and recv.dtype == np.uint8
        tab = e4m3_value_table()
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            v = tab[recv[lo:hi]]
            v = v.reshape(hi - lo, cfg.H // 128, 128) * recv_scale[lo:hi, :, None]
            y[lo:hi] = f32_to_bf16_bits(v.reshape(hi - lo, cfg.H))
        return y
    e = expert_of_row(expert_offset, n).astype(np.float32)
    mul = (np.float32(1.0) + e / np.float32(cfg.E)).astype(np.float32)
    add = (np.float32(0.01) * e).astype(np.float32) if cfg.expert == "affine" else None
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        v = bf16_bits_to_f32(recv[lo:hi]) * mul[lo:hi, None]
        if add is not None:
            v = v + add[lo:hi, None]
        y[lo:hi] = f32_to_bf16_bits(v)
    return y
