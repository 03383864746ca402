"""Pins for the oracle's bf16 dispatch: every received row equals its source
row bit for bit, every row is written exactly once, nothing else is touched."""
import numpy as np
import pytest

import oracle
from paper_2607_26444_b200 import workloads as wl


@pytest.mark.parametrize("threads", [1, 3])
def test_rows_equal_source_rows(threads):
    cfg = wl.CONFIGS["tiny"]
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    N = cfg.n_items
    guard = 5
    buf = np.full((N + 2 * guard, cfg.H), 0xDEAD, np.uint16)
    recv = buf[guard:guard + N]
    oracle.dispatch_bf16(lay["dst_row"], inp["x"], nthreads=threads, recv=recv)
    assert np.all(buf[:guard] == 0xDEAD) and np.all(buf[guard + N:] == 0xDEAD)
    x2 = inp["x"].reshape(cfg.n_tok, cfg.H)
    d = lay["dst_row"].ravel()
    for i in range(N):
        assert np.array_equal(recv[d[i]], x2[i // cfg.K])
    # through the inverse map: row j holds the token of item src_of_row[j]
    assert np.array_equal(recv, x2[lay["src_of_row"] // cfg.K])
    # each expert segment is ordered by (rank, token, slot)
    src = lay["src_of_row"]
    for e in range(cfg.E):
        seg = src[lay["expert_offset"][e]:lay["expert_offset"][e + 1]]
        assert np.all(np.diff(seg) > 0)


def test_bit_patterns_survive():
    # NaN payloads, -0, infinities and subnormals are copied, not canonicalised
    ids = np.array([[[1, 0]], [[0, 1]]], np.int32)
    x = np.array([[[0x7FC1, 0x8000, 0x7F80, 0x0001, 0xFFFF, 0x7FA5, 0x0000, 0x8001]],
                  [[0x3F80, 0xBF80, 0x7F81, 0xFF80, 0x0080, 0x8080, 0x1234, 0xFEDC]]], np.uint16)
    lay = oracle.layout(ids, 2)
    recv = oracle.dispatch_bf16(lay["dst_row"], x)
    # expert 0 <- (r0,k1), (r1,k0); expert 1 <- (r0,k0), (r1,k1)
    assert np.array_equal(recv, np.stack([x[0, 0], x[1, 0], x[0, 0], x[1, 0]]))


def test_duplicate_ids_in_one_token():
    ids = np.array([[[1, 1, 0]]], np.int32)
    x = np.arange(8, dtype=np.uint16).reshape(1, 1, 8)
    lay = oracle.layout(ids, 2)
    assert lay["dst_row"].ravel().tolist() == [1, 2, 0]
    recv = oracle.dispatch_bf16(lay["dst_row"], x)
    assert np.all(recv == x[0, 0])
