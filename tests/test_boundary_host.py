"""Host-side behaviour of the C-ABI library, exercised without a GPU:
exported symbols, shape validation, the registration pool and every
host-detectable error code (through a host-only context, which computes nothing)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import build as strata_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    strata_build.build()


def declared_functions():
    inc = os.path.join(ROOT, "include")
    text = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(strata_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 17
    L = B.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(B.EXPORTS) == names          # the binding wraps each of them, under the same name
    for n in names:
        assert callable(getattr(B, n)), n


def test_status_strings():
    assert B.strata_status_string(B.STRATA_OK) == "ok"
    seen = {B.strata_status_string(c) for c in range(11)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert B.strata_status_string(99) == "unknown status"


def shape(R=4, T=128, H=1024, E=16, K=2, dt=B.STRATA_BF16):
    return B.strata_moe_shape(R, T, H, E, K, dt)


@pytest.mark.parametrize("kw", [dict(R=0), dict(T=0), dict(K=0), dict(E=18), dict(E=2048, R=4), dict(K=33),
                                dict(H=1020), dict(dt=7), dict(H=1032, dt=B.STRATA_FP8_E4M3_B128),
                                dict(R=64, T=1 << 20, K=32, E=64)])
def test_bad_shapes_are_rejected(kw):
    rc, _ = B.strata_moe_workspace_bytes(shape(**kw))
    assert rc == B.STRATA_ERR_SHAPE
    rc, h = B.strata_ctx_create(shape(**kw), -1)
    assert rc == B.STRATA_ERR_SHAPE and not h


def test_workspace_size():
    rc, n = B.strata_moe_workspace_bytes(shape())
    # 4 ranks x ceil(128*2/4096)=1 tile, 16 experts, 256-byte header, rounded to 256; then the pair table of
    # all-to-all-v (1028 + 1024 uint32, 2 x 1024 uint64 = 24,592 bytes, rounded to 256)
    table = 24832
    assert rc == 0 and n == 512 + table
    rc, n = B.strata_moe_workspace_bytes(shape(R=16, T=4096, H=7168, E=256, K=8))
    assert rc == 0 and n == 256 + 16 * 8 * 256 * 4 + table


@pytest.fixture
def ctx():
    rc, h = B.strata_ctx_create(shape(), -1)
    assert rc == 0 and h
    yield h
    assert B.strata_ctx_destroy(h) == 0


def test_pool_register_ready_carve_reset(ctx):
    base = 0x7F00_0000_0000
    rc, rid = B.strata_pool_register(ctx, base, 1 << 20)
    assert rc == 0 and rid > 0
    assert B.strata_pool_is_ready(ctx, base, 1 << 20) == 0
    assert B.strata_pool_is_ready(ctx, base + 4096, 100) == 0
    assert B.strata_pool_is_ready(ctx, base + 4096, 1 << 20) == B.STRATA_ERR_NOT_REGISTERED
    assert B.strata_pool_is_ready(ctx, base - 16, 32) == B.STRATA_ERR_NOT_REGISTERED
    assert B.strata_pool_is_ready(ctx, base + (1 << 20), 0) == 0          # empty range at the end
    # overlapping registration is refused, a disjoint one is fine
    rc, _ = B.strata_pool_register(ctx, base + 4096, 64)
    assert rc == B.STRATA_ERR_INVALID_ARG
    rc, rid2 = B.strata_pool_register(ctx, base + (1 << 20), 4096)
    assert rc == 0 and rid2 != rid
    rc, _ = B.strata_pool_register(ctx, base + (2 << 20) + 8, 64)
    assert rc == B.STRATA_ERR_ALIGNMENT
    # bump carving with alignment
    rc, p0 = B.strata_pool_carve(ctx, rid, 100, 256)
    rc1, p1 = B.strata_pool_carve(ctx, rid, 100, 256)
    assert rc == 0 and rc1 == 0 and p0 == base and p1 == base + 256
    rc, _ = B.strata_pool_carve(ctx, rid, 1 << 20, 16)
    assert rc == B.STRATA_ERR_CAPACITY
    rc, _ = B.strata_pool_carve(ctx, rid, 16, 3)
    assert rc == B.STRATA_ERR_INVALID_ARG
    assert B.strata_pool_reset(ctx, rid) == 0
    rc, p2 = B.strata_pool_carve(ctx, rid, 1 << 20, 16)
    assert rc == 0 and p2 == base
    rc, _ = B.strata_pool_carve(ctx, 12345, 16, 16)
    assert rc == B.STRATA_ERR_NOT_REGISTERED
    assert B.strata_pool_unregister(ctx, rid) == 0
    assert B.strata_pool_unregister(ctx, rid) == B.STRATA_ERR_NOT_REGISTERED
    assert B.strata_pool_is_ready(ctx, base, 16) == B.STRATA_ERR_NOT_REGISTERED


def _fake_layout(base=0x7E00_0000_0000):
    return B.strata_moe_layout_t(base, base + 4096, base + 8192, base + 12288, None, base + 16384, None)


def test_host_detectable_errors_before_any_launch(ctx):
    lay = _fake_layout()
    ids = x = 0x7D00_0000_0000
    recv = 0x7C00_0000_0000
    n_rows = 4 * 128 * 2
    # no workspace yet
    assert B.strata_moe_layout(ctx, ids, lay, None) == B.STRATA_ERR_WORKSPACE
    assert B.strata_ctx_set_workspace(ctx, 0x7B00_0000_0010, 1 << 16) == B.STRATA_ERR_ALIGNMENT
    assert B.strata_ctx_set_workspace(ctx, 0x7B00_0000_0000, 16) == B.STRATA_ERR_CAPACITY
    assert B.strata_ctx_set_workspace(ctx, 0x7B00_0000_0000, 1 << 16) == 0
    # NULLs
    assert B.strata_moe_layout(ctx, None, lay, None) == B.STRATA_ERR_INVALID_ARG
    bad = _fake_layout()
    bad.dst_row = None
    assert B.strata_moe_layout(ctx, ids, bad, None) == B.STRATA_ERR_INVALID_ARG
    bad = _fake_layout()
    bad.expert_offset = None
    assert B.strata_moe_layout(ctx, ids, bad, None) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_dispatch(ctx, lay, None, recv, None, n_rows, None) == B.STRATA_ERR_INVALID_ARG
    # bf16 context must not get a scale pointer
    assert B.strata_moe_dispatch(ctx, lay, x, recv, recv, n_rows, None) == B.STRATA_ERR_INVALID_ARG
    # alignment, capacity, registration -- in that order
    assert B.strata_moe_dispatch(ctx, lay, x + 8, recv, None, n_rows, None) == B.STRATA_ERR_ALIGNMENT
    assert B.strata_moe_dispatch(ctx, lay, x, recv + 2, None, n_rows, None) == B.STRATA_ERR_ALIGNMENT
    assert B.strata_moe_dispatch(ctx, lay, x, recv, None, n_rows - 1, None) == B.STRATA_ERR_CAPACITY
    assert B.strata_moe_dispatch(ctx, lay, x, recv, None, n_rows, None) == B.STRATA_ERR_NOT_REGISTERED
    rc, rid = B.strata_pool_register(ctx, recv, n_rows * 1024 * 2 - 16)      # one vector short
    assert rc == 0
    assert B.strata_moe_dispatch(ctx, lay, x, recv, None, n_rows, None) == B.STRATA_ERR_NOT_REGISTERED
    assert B.strata_pool_unregister(ctx, rid) == 0
    rc, rid = B.strata_pool_register(ctx, recv, n_rows * 1024 * 2)
    # everything valid: a host-only context stops right before the launch
    assert B.strata_moe_dispatch(ctx, lay, x, recv, None, n_rows, None) == B.STRATA_ERR_CUDA
    assert B.strata_moe_layout(ctx, ids, lay, None) == B.STRATA_ERR_CUDA
    assert B.strata_moe_combine(ctx, lay, recv, n_rows, x, x, None) == B.STRATA_ERR_CUDA
    assert B.strata_moe_combine(ctx, lay, recv + 4, n_rows, x, x, None) == B.STRATA_ERR_ALIGNMENT
    assert B.strata_moe_combine(ctx, lay, None, n_rows, x, x, None) == B.STRATA_ERR_INVALID_ARG
    rc, n = B.strata_ctx_launch_count(ctx)
    assert rc == 0 and n == 0                                              # nothing was ever launched


def test_fp8_context_needs_registered_scales():
    rc, h = B.strata_ctx_create(shape(dt=B.STRATA_FP8_E4M3_B128), -1)
    assert rc == 0
    try:
        assert B.strata_ctx_set_workspace(h, 0x7B00_0000_0000, 1 << 16) == 0
        lay = _fake_layout()
        x, recv, sc = 0x7D00_0000_0000, 0x7C00_0000_0000, 0x7A00_0000_0000
        n_rows = 1024
        assert B.strata_moe_dispatch(h, lay, x, recv, None, n_rows, None) == B.STRATA_ERR_INVALID_ARG
        B.strata_pool_register(h, recv, n_rows * 1024)
        assert B.strata_moe_dispatch(h, lay, x, recv, sc, n_rows, None) == B.STRATA_ERR_NOT_REGISTERED
        B.strata_pool_register(h, sc, n_rows * 8 * 4)
        assert B.strata_moe_dispatch(h, lay, x, recv, sc, n_rows, None) == B.STRATA_ERR_CUDA
        dev = B.strata_moe_device_buffers(x, x, x, recv, x, lay)
        assert B.strata_moe_roundtrip_host(h, dev, x, x, x, x, None) == B.STRATA_ERR_SHAPE
    finally:
        B.strata_ctx_destroy(h)


def test_recv_view(ctx):
    off = np.array([0, 10, 10, 300, 1024], np.int32)
    recv = 0x7C00_0000_0000
    rc, base, rows = B.strata_moe_recv_view(ctx, off, 2, recv)
    assert rc == 0 and base == recv + 10 * 1024 * 2 and rows == 290
    rc, base, rows = B.strata_moe_recv_view(ctx, off, 1, recv)
    assert rc == 0 and rows == 0
    rc, _, _ = B.strata_moe_recv_view(ctx, off, 4, recv)
    assert rc == B.STRATA_ERR_INVALID_ARG


def test_null_context_everywhere():
    assert B.strata_ctx_destroy(None) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_pool_is_ready(None, 16, 16) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_layout(None, 16, _fake_layout(), None) == B.STRATA_ERR_INVALID_ARG
    rc, _ = B.strata_device_status(None, None)
    assert rc == B.STRATA_ERR_INVALID_ARG


def test_collectives_reject_bad_arguments_before_any_launch():
    rc, h = B.strata_ctx_create(shape(), -1)
    assert rc == B.STRATA_OK
    try:
        fake = 1 << 20
        # no workspace yet
        assert B.strata_allgather(h, 4, fake, 2 * fake, 64, None) == B.STRATA_ERR_WORKSPACE
        assert B.strata_ctx_set_workspace(h, 256 << 10, 1 << 30) == B.STRATA_OK
        assert B.strata_allgather(h, 0, fake, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_allgather(h, 2000, fake, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_allgather(h, 4, None, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_allgather(h, 4, fake + 8, 2 * fake, 64, None) == B.STRATA_ERR_ALIGNMENT
        assert B.strata_alltoall(h, 4, fake, 2 * fake + 4, 64, None) == B.STRATA_ERR_ALIGNMENT
        assert B.strata_broadcast(h, 4, 4, fake, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_broadcast(h, 4, -1, fake, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_allgather(h, 4, fake, 2 * fake, 40, None) == B.STRATA_ERR_SHAPE
        assert B.strata_allreduce(h, 4, fake, 2 * fake, 12, None) == B.STRATA_ERR_SHAPE
        assert B.strata_reducescatter(h, 4, fake, 2 * fake, 4, None) == B.STRATA_ERR_SHAPE
        assert B.strata_allgather(h, 4, fake, 2 * fake, 0, None) == B.STRATA_OK        # nothing to move
        assert B.strata_p2p(h, 4, 4, 0, fake, 2 * fake, 64, None) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_p2p(h, 4, 0, 1, fake, 2 * fake, 64, None) == B.STRATA_ERR_CUDA
        assert B.strata_alltoallv(h, 33, fake, 64, 2 * fake, 64, fake, fake, fake, None) == B.STRATA_ERR_SHAPE
        assert B.strata_alltoallv(h, 4, fake, 0, 2 * fake, 64, fake, fake, fake, None) == B.STRATA_ERR_SHAPE
        assert B.strata_alltoallv(h, 4, fake, 64, 2 * fake, 64, fake + 4, fake, fake, None) == B.STRATA_ERR_ALIGNMENT
        assert B.strata_alltoallv(h, 4, fake, 64, 2 * fake, 64, fake, fake, fake, None) == B.STRATA_ERR_CUDA
        # a host-only context never launches
        for rc in (B.strata_allgather(h, 4, fake, 2 * fake, 64, None),
                   B.strata_alltoall(h, 4, fake, 2 * fake, 64, None),
                   B.strata_broadcast(h, 4, 1, fake, 2 * fake, 64, None),
                   B.strata_reducescatter(h, 4, fake, 2 * fake, 64, None),
                   B.strata_allreduce(h, 4, fake, 2 * fake, 64, None)):
            assert rc == B.STRATA_ERR_CUDA
        rc, n = B.strata_ctx_launch_count(h)
        assert rc == B.STRATA_OK and n == 0
    finally:
        B.strata_ctx_destroy(h)
