"""Pins for the oracle's full-mesh collectives over emulated ranks (paper Sec. 6.1)."""
import os

import numpy as np
import pytest

import oracle
from paper_2607_26444_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "reduce_order_example.txt")


def _golden():
    rows, out, R, M = {}, None, 0, 0
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "R":
            R = int(t[1])
        elif t[0] == "M":
            M = int(t[1])
        elif t[0].startswith("in"):
            rows[int(t[0][2:])] = [int(v, 16) for v in t[1:]]
        elif t[0] == "out":
            out = [int(v, 16) for v in t[1:]]
    x = np.array([rows[p] for p in range(R)], np.uint16)
    assert x.shape == (R, M)
    return x, np.array(out, np.uint16)


def _bytes(R, n, seed):
    return wl.gen_payload(R, (n + 1) // 2, seed).view(np.uint8)[:, :n].copy()


# ---- data movement -----------------------------------------------------------------------------

@pytest.mark.parametrize("R,M", [(1, 16), (2, 1), (4, 48), (7, 33)])
def test_allgather_counter_pattern(R, M):
    # rank p holds the bytes p*M .. p*M+M-1 of a ramp  =>  every rank ends with the whole ramp
    x = (np.arange(R * M) % 251).astype(np.uint8).reshape(R, M)
    out = oracle.allgather(x)
    for r in range(R):
        assert np.array_equal(out[r].ravel(), np.arange(R * M) % 251)


def test_allgather_random_is_a_tile():
    x = _bytes(5, 112, 3)
    assert np.array_equal(oracle.allgather(x), np.broadcast_to(x[None], (5, 5, 112)))


@pytest.mark.parametrize("R,S", [(1, 8), (2, 3), (4, 16), (6, 5)])
def test_alltoall_is_the_rank_transpose(R, S):
    x = _bytes(R, R * S, 5).reshape(R, R, S)
    out = oracle.alltoall(x)
    assert np.array_equal(out, x.transpose(1, 0, 2))
    assert np.array_equal(oracle.alltoall(out), x)             # applying it twice returns the input
    # closed form on a coded pattern: the byte names (sender, receiver, position)
    code = np.fromfunction(lambda p, r, j: (p * 49 + r * 7 + j) % 256, (R, R, S)).astype(np.uint8)
    out = oracle.alltoall(code)
    for r in range(R):
        for p in range(R):
            assert out[r, p, 0] == (p * 49 + r * 7) % 256


def test_alltoall_is_not_the_identity():
    x = _bytes(3, 3 * 4, 9).reshape(3, 3, 4)
    assert not np.array_equal(oracle.alltoall(x), x)


@pytest.mark.parametrize("root", [0, 2, 3])
def test_broadcast_reads_only_the_root(root):
    x = _bytes(4, 40, 11)
    out = oracle.broadcast(x, root)
    assert all(np.array_equal(out[r], x[root]) for r in range(4))
    y = x.copy()
    y[np.arange(4) != root] ^= 0xFF                            # the other ranks' inputs do not matter
    assert np.array_equal(oracle.broadcast(y, root), out)


def test_empty_payloads():
    assert oracle.allgather(np.zeros((3, 0), np.uint8)).shape == (3, 3, 0)
    assert oracle.allreduce(np.zeros((3, 0), np.uint16)).shape == (3, 0)


# ---- reductions --------------------------------------------------------------------------------

def test_reduction_order_worked_example():
    x, want = _golden()
    out = oracle.allreduce(x)
    assert all(np.array_equal(out[r], want) for r in range(x.shape[0]))
    # the same operands as the slices of one destination rank of a reduce-scatter
    R, M = x.shape
    xs = np.zeros((R, R, M), np.uint16)
    xs[:, 1, :] = x
    assert np.array_equal(oracle.reducescatter(xs)[1], want)
    assert np.all(oracle.reducescatter(xs)[0] == 0)


@pytest.mark.parametrize("R", [1, 2, 5, 16])
def test_small_integers_sum_exactly(R):
    # integers in [-8, 8]: every partial sum is an integer of magnitude <= 128, exact in fp32 and bf16
    rng = np.random.default_rng(R)
    v = rng.integers(-8, 9, size=(R, R, 24))
    x = wl.f32_to_bf16_bits(v.astype(np.float32)).reshape(R, R, 24)
    got = wl.bf16_bits_to_f32(oracle.reducescatter(x))
    assert np.array_equal(got.astype(np.int64), v.sum(axis=0))
    got = wl.bf16_bits_to_f32(oracle.allreduce(x.reshape(R, R * 24)))
    assert np.array_equal(got.astype(np.int64), np.broadcast_to(v.sum(axis=0).reshape(1, -1), (R, R * 24)))


def test_reduction_within_the_fp64_bound():
    R, S = 8, 64
    x = wl.gen_payload(R, R * S, 21).reshape(R, R, S)
    v = wl.bf16_bits_to_f32(x).astype(np.float64)
    exact = v.sum(axis=0)                                      # [R, S]: column sums over the peers
    got = wl.bf16_bits_to_f32(oracle.reducescatter(x)).astype(np.float64)
    # R-1 fp32 roundings of partial sums, then one bf16 rounding (half an ulp of an 8-bit significand)
    bound = np.abs(exact) * 2.0 ** -8 + R * 2.0 ** -24 * np.abs(v).sum(axis=0) + 1e-30
    assert np.all(np.abs(got - exact) <= bound)
    # and it is a real sum: far from any single operand
    assert np.abs(got - v[0]).max() > 0.5


def test_allreduce_is_reducescatter_then_allgather():
    R, S = 4, 40
    x = wl.gen_payload(R, R * S, 22)
    rs = oracle.reducescatter(x.reshape(R, R, S))             # [R, S]
    ag = oracle.allgather(rs.view(np.uint8))                   # [R, R, S*2] bytes
    assert np.array_equal(oracle.allreduce(x).view(np.uint8).reshape(R, R, S * 2), ag)


def test_single_rank_reduction_returns_the_input_as_values():
    x = wl.gen_payload(1, 64, 23)
    x[0, 0] = 0x8000                                           # +0 + (-0) = +0
    out = oracle.allreduce(x)
    assert out[0, 0] == 0 and np.array_equal(out[0, 1:], x[0, 1:])
