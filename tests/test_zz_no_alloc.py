"""The allocation-free routing layout (strata_moe_layout_noalloc).

Some users of this library run where they cannot allocate device memory: all of the GPU's memory
already belongs to a framework pool, or an allocation's implicit device synchronisation is not
acceptable in their hook, or their binding has no allocator to create a workspace with.  For them
the library carries the layout kernels' scratch in a fixed 2 MiB array of its own.  This file checks,
through the C ABI, that the entry point returns exactly what strata_moe_layout returns and what the
CPU oracle returns (layouts are integer work: the bar is bit equality), twice in a row on different
inputs, because the shared array still holds the first call's contents when the second call starts.

Collected last on purpose, so a failure here cannot hide any other test's result.  It passes both on
its own in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import build as strata_build
from paper_2607_26444_b200 import workloads as wl

FIELDS = ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row",
          "src_of_row")


def test_shapes_beyond_the_built_in_scratch_are_refused():
    """2 MiB holds 256 + n_tiles*E*4 bytes; anything larger is refused before any CUDA call."""
    strata_build.build()
    lay = B.strata_moe_layout_t(16, 32, 48, 64, None, 80, None)       # never dereferenced
    fits = B.strata_moe_shape(16, 4096, 7168, 256, 8, 0)               # prefill: 128 tiles * 256 experts
    too_big = B.strata_moe_shape(64, 16384, 7168, 1024, 8, 0)          # 2048 tiles * 1024 experts = 8 MiB
    assert B.strata_moe_layout_noalloc(too_big, 16, lay, None, None) == B.STRATA_ERR_CAPACITY
    assert "capacity" in B.strata_status_string(B.STRATA_ERR_CAPACITY)
    assert B.strata_moe_layout_noalloc(B.strata_moe_shape(3, 8, 64, 8, 2, 0), 16, lay, None, None) \
        == B.STRATA_ERR_SHAPE                                           # E % R != 0
    assert B.strata_moe_layout_noalloc(fits, None, lay, None, None) == B.STRATA_ERR_INVALID_ARG
    unknown_flag = B.strata_moe_shape(16, 4096, 7168, 256, 8, 0, 0, 0x40, 0)
    assert B.strata_moe_layout_noalloc(unknown_flag, 16, lay, None, None) == B.STRATA_ERR_SHAPE
    both = B.strata_moe_shape(16, 128, 7168, 256, 8, 0, 128, 0, 16)    # aligned segments and fixed slots together
    assert B.strata_moe_layout_noalloc(both, 16, lay, None, None) == B.STRATA_ERR_SHAPE
    rc, ws = B.strata_moe_workspace_bytes(fits)
    assert rc == 0 and ws <= 2 << 20


@pytest.mark.gpu
def test_noalloc_layout_matches_workspace_layout_twice_in_a_row():
    import torch
    dev = "cuda:0"
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    cases = [wl.CONFIGS["skew"],                                                   # 32 tiles, hot expert
             wl.shrink(wl.CONFIGS["decode"], R=4, T=300, E=64, K=5, seed=31)]       # ragged tiles, smaller E
    for cfg in cases:
        ids = torch.from_numpy(wl.gen_topk_ids(cfg)).to(dev)
        ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
        want = ctx.layout(ids)
        torch.cuda.synchronize()
        assert ctx.device_status() == B.STRATA_OK

        got = ctx.new_layout()
        for f in FIELDS:
            getattr(got, f).fill_(-12345)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        rc = B.strata_moe_layout_noalloc(ctx.shape, ids.data_ptr(), got.c, status.data_ptr(), stream)
        assert rc == B.STRATA_OK, B.strata_status_string(rc)
        torch.cuda.synchronize()
        assert status.item() == 0
        ref = oracle.layout(ids.cpu().numpy(), cfg.E)
        for f in FIELDS:
            assert torch.equal(getattr(got, f), getattr(want, f)), (cfg.name, f)
            assert np.array_equal(getattr(got, f).cpu().numpy(), ref[f]), (cfg.name, f, "oracle")
        ctx.close()

    # an id outside [0, E) is skipped and reported through the caller's status word, as in the workspace path
    cfg = cases[1]
    h_ids = wl.gen_topk_ids(cfg)
    h_ids[2, 7, 1] = cfg.E + 3
    ids = torch.from_numpy(h_ids).to(dev)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    want = ctx.layout(ids)
    assert ctx.device_status() == B.STRATA_ERR_BAD_EXPERT_ID
    got = ctx.new_layout()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    assert B.strata_moe_layout_noalloc(ctx.shape, ids.data_ptr(), got.c, status.data_ptr(), stream) == B.STRATA_OK
    torch.cuda.synchronize()
    assert status.item() == B.STRATA_ERR_BAD_EXPERT_ID
    assert got.dst_row[2, 7, 1].item() == -1
    assert torch.equal(got.dst_row, want.dst_row) and torch.equal(got.expert_offset, want.expert_offset)
    ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("cap", [40, 1000], ids=["slots_overflow", "slots_never_full"])
def test_noalloc_layout_with_fixed_capacity_slots(cap):
    """slot_capacity > 0 is honoured: rows are [E][R][capacity], and an overflowing slot is reported
    through the caller's status word as STRATA_ERR_CAPACITY, exactly as the workspace path does."""
    import torch
    dev = "cuda:0"
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    cfg = wl.shrink(wl.CONFIGS["decode"], R=4, T=1500, H=64, E=32, K=4, seed=32)    # two tiles per rank
    h_ids = wl.gen_topk_ids(cfg)
    h_ids[np.random.default_rng(5).random(h_ids.shape) < 0.1] = -1
    ref = oracle.layout(h_ids, cfg.E, allow_unrouted=True, slot_capacity=cap)
    assert bool(ref["dropped"]) == (cap == 40)
    ids = torch.from_numpy(h_ids).to(dev)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, allow_unrouted=True, slot_capacity=cap)
    want = ctx.layout(ids)
    want_status = ctx.device_status()
    for _ in range(2):
        got = ctx.new_layout()
        for f in FIELDS:
            getattr(got, f).fill_(-12345)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        assert B.strata_moe_layout_noalloc(ctx.shape, ids.data_ptr(), got.c, status.data_ptr(), stream) == B.STRATA_OK
        torch.cuda.synchronize()
        assert status.item() == want_status == (B.STRATA_ERR_CAPACITY if ref["dropped"] else B.STRATA_OK)
        for f in FIELDS:
            assert torch.equal(getattr(got, f), getattr(want, f)), f
            assert np.array_equal(getattr(got, f).cpu().numpy(), ref[f]), (f, "oracle")
    ctx.close()
