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


# ---- all-to-all-v and point-to-point -----------------------------------------------------------

def _v_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "alltoallv_worked_example.txt")
    d = {}
    for line in open(path):
        t = line.split()
        if t and not t[0].startswith("#"):
            d[t[0]] = [int(v) for v in t[1:]]
    return d


def test_alltoallv_worked_example():
    d = _v_golden()
    R, si, so = d["R"][0], d["in_stride"][0], d["out_stride"][0]
    x = (np.arange(R)[:, None] * 16 + np.arange(si)[None, :]).astype(np.uint8)
    out = np.full((R, so), 255, np.uint8)
    bad = oracle.alltoallv(x, out, d["send_bytes"], d["send_off"], d["recv_off"])
    assert bad == 0
    for r in range(R):
        assert out[r].tolist() == d[f"out{r}"], r


def test_alltoallv_with_equal_counts_is_alltoall():
    R, S = 5, 48
    x = _bytes(R, R * S, 31)
    sb = np.full((R, R), S, np.int64)
    off = np.tile(np.arange(R) * S, (R, 1)).astype(np.int64)
    out = np.zeros((R, R * S), np.uint8)
    assert oracle.alltoallv(x, out, sb, off, off) == 0
    assert np.array_equal(out.reshape(R, R, S), oracle.alltoall(x.reshape(R, R, S)))


def test_alltoallv_reverse_exchange_restores_the_input_and_leaves_gaps_alone():
    R = 6
    sb = wl.gen_pair_bytes(R, 160, seed=4)
    so, ro, si, st = wl.packed_offsets(sb)
    so += 16                                                   # a 16-byte gap in front of every rank's data
    ro += 32
    si, st = si + 48, st + 64
    x = _bytes(R, si, 32)
    out = np.full((R, st), 0xEE, np.uint8)
    assert oracle.alltoallv(x, out, sb, so, ro) == 0
    # conservation: every rank received exactly the bytes addressed to it, the rest is untouched
    touched = np.zeros((R, st), bool)
    for r in range(R):
        for p in range(R):
            touched[r, ro[r, p]:ro[r, p] + sb[p, r]] = True
    assert touched.sum() == sb.sum() and np.all(out[~touched] == 0xEE)
    # the reverse exchange: receivers send back what they got, from where it landed to where it came from
    back = np.full((R, si), 0x11, np.uint8)
    assert oracle.alltoallv(out, back, sb.T.copy(), ro, so) == 0
    sent = np.zeros((R, si), bool)
    for p in range(R):
        for r in range(R):
            sent[p, so[p, r]:so[p, r] + sb[p, r]] = True
    assert np.array_equal(back[sent], x[sent]) and np.all(back[~sent] == 0x11)


def test_alltoallv_skips_pairs_that_do_not_fit():
    R = 2
    x = _bytes(R, 64, 33)
    out = np.zeros((R, 64), np.uint8)
    sb = np.array([[16, 32], [0, 16]], np.int64)
    so = np.array([[0, 48], [0, 0]], np.int64)                 # 48 + 32 > 64: pair (0 -> 1) is skipped
    ro = np.array([[0, 0], [16, 0]], np.int64)
    assert oracle.alltoallv(x, out, sb, so, ro) == 1
    assert np.array_equal(out[0, :16], x[0, :16]) and np.array_equal(out[1, :16], x[1, :16])
    assert np.all(out[1, 16:] == 0)


def test_p2p_copies_one_part():
    x = _bytes(4, 80, 34)
    out = np.full((4, 80), 7, np.uint8)
    oracle.p2p(x, out, 2, 0)
    assert np.array_equal(out[0], x[2]) and np.all(out[1:] == 7)


def test_pair_bytes_recipe():
    sb = wl.gen_pair_bytes(32, 1 << 20, seed=1)
    assert sb.shape == (32, 32) and np.all(sb % 16 == 0) and (sb == 0).mean() > 0.03
    col = sb.sum(axis=0)
    assert col.max() > 5 * np.median(col)                      # a few hot receivers
    so, ro, si, st = wl.packed_offsets(sb)
    assert np.all(so[:, 0] == 0) and np.all(np.diff(so, axis=1) == sb[:, :-1])
    assert si == sb.sum(axis=1).max() and st == sb.sum(axis=0).max()
