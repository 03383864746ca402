"""GPU-vs-oracle parity for the in-place consumer of the receive buffer, through the C ABI: the whole chain
layout -> dispatch -> expert stand-in -> combine runs on the device with no host step, and every buffer must be
bit-identical to the oracle's chain (the stand-in and combine mirror the oracle's fused multiply-adds)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SENTINEL16 = 0x7FC7
GUARD = 3


def to_dev(a):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(a).to(DEV)


def u16(t):
    return t.cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("kw,align,tile,frac", [
    (dict(R=4, T=128, H=1024, E=16, K=4), 128, 128, 0.0),
    (dict(R=4, T=128, H=1024, E=16, K=4), 128, 32, 0.2),             # several tiles per aligned block, unrouted slots
    (dict(R=2, T=50, H=136, E=4, K=2), 1, 1, 0.0),                   # packed segments: a tile is a row; 17 vectors per row
    (dict(R=8, T=300, H=520, E=64, K=6), 16, 16, 0.1),               # many experts, some nearly empty
    (dict(R=16, T=128, H=7168, E=256, K=8), 128, 128, 0.0),          # decode shape, GEMM-tile-aligned segments
    (dict(R=4, T=64, H=256, E=8, K=2), 64, 64, 1.0),                 # nothing routed: every tile is empty
], ids=lambda v: str(v) if not isinstance(v, dict) else "R{R}T{T}H{H}E{E}K{K}".format(**v))
def test_chain_with_the_in_place_expert_matches_the_oracle(kw, align, tile, frac):
    cfg = wl.shrink(wl.CONFIGS["decode"], seed=4242, **kw)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    if frac:
        ids[np.random.default_rng(3).random(ids.shape) < frac] = -1
    scale = (np.float32(1.0) + np.arange(cfg.E, dtype=np.float32) / np.float32(cfg.E)).astype(np.float32)
    bias = (np.float32(0.01) * np.arange(cfg.E, dtype=np.float32)).astype(np.float32)

    ref = oracle.layout(ids, cfg.E, segment_align=align, allow_unrouted=True)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, segment_align=align, allow_unrouted=True)
    n_rows = ctx.recv_rows
    want_recv = oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4, n_rows=n_rows)
    want_recv[want_recv == 0xDEAD] = SENTINEL16                     # rows no item maps to: the GPU buffer's fill
    want_y = oracle.expert_affine(ref, want_recv, scale, bias)
    want_out = oracle.combine(ref["dst_row"], want_y, inp["w"], nthreads=4)

    whole = torch.full((n_rows + 2 * GUARD, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    recv = whole[GUARD:GUARD + n_rows]
    ctx.register(whole)
    lay = ctx.layout(to_dev(ids))
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    ctx.expert_affine_inplace(lay, recv, to_dev(scale), to_dev(bias), tile_rows=tile)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, to_dev(inp["w"]), out)
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    got = u16(whole)
    assert np.array_equal(got[GUARD:GUARD + n_rows], want_y)       # occupied rows transformed, padding rows untouched
    assert np.all(got[:GUARD] == SENTINEL16) and np.all(got[GUARD + n_rows:] == SENTINEL16)
    assert np.array_equal(u16(out), want_out)
    ctx.close()


def test_host_errors():
    cfg = wl.shrink(wl.CONFIGS["tiny"], H=64)
    s = torch.cuda.current_stream().cuda_stream
    sc = torch.ones(cfg.E, dtype=torch.float32, device=DEV)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, segment_align=64)
    lay = ctx.layout(to_dev(wl.gen_topk_ids(cfg)))
    recv = torch.zeros((ctx.recv_rows, cfg.H), dtype=torch.int16, device=DEV)
    args = (recv.data_ptr(), recv.shape[0], sc.data_ptr(), sc.data_ptr())
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, *args, 64, s) == B.STRATA_ERR_NOT_REGISTERED
    ctx.register(recv)
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, *args, 48, s) == B.STRATA_ERR_SHAPE      # 64 % 48 != 0
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, *args, 0, s) == B.STRATA_ERR_SHAPE
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, recv.data_ptr(), recv.shape[0] - 1, sc.data_ptr(),
                                              sc.data_ptr(), 64, s) == B.STRATA_ERR_CAPACITY
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, recv.data_ptr(), recv.shape[0], None, sc.data_ptr(), 64, s) \
        == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_expert_affine_inplace(ctx.h, lay.c, *args, 16, s) == B.STRATA_OK
    ctx.close()
    packed = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    lay = packed.layout(to_dev(wl.gen_topk_ids(cfg)))
    packed.register(recv)
    assert B.strata_moe_expert_affine_inplace(packed.h, lay.c, *args, 2, s) == B.STRATA_ERR_SHAPE   # packed: rows only
    packed.close()
    fp8 = B.MoEContext(4, 16, 128, 16, 2, B.STRATA_FP8_E4M3_B128)
    assert B.strata_moe_expert_affine_inplace(fp8.h, lay.c, *args, 1, s) == B.STRATA_ERR_SHAPE
    fp8.close()
    torch.cuda.synchronize()
