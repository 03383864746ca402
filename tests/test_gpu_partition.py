"""GPU-vs-oracle parity for the paper's window partitioning and LPT-style policy (Sec. 6.2, App. B to D),
through the C ABI: every output array of the policy is integer work and must be bit-identical, and the
window-major dispatch must write exactly what the oracle's (and the token-major) dispatch writes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SENTINEL16 = 0x7FC7


def to_dev(a):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(a).to(DEV)


CASES = [
    # (config overrides, tiers [(alpha, beta, unit_rows, cap)], g0, g1, n_cores)
    (dict(R=4, T=128, H=1024, E=16, K=2), [(10, 64, 16, 2)], 1, 1, 8),
    (dict(R=8, T=96, H=256, E=32, K=4), [(20, 512, 24, 4), (70, 400, 16, 3), (210, 350, 8, 2)], 2, 4, 12),
    (dict(R=16, T=128, H=7168, E=256, K=8), [(200, 1024, 64, 8)], 1, 1, 296),          # decode shape
    (dict(R=32, T=512, H=4096, E=128, K=8, routing="zipf"), [(200, 1024, 128, 6), (700, 800, 96, 4)], 8, 8, 444),
    (dict(R=3, T=50, H=64, E=6, K=3), [(0, 1, 1000000, 1)], 1, 1, 5),                   # one unit per peer window, cap 1
    (dict(R=2, T=700, H=128, E=4, K=2), [(5, 16, 3, 1000)], 1, 1, 1000),                # more cores than needed
    (dict(R=16, T=128, H=7168, E=256, K=8), [(200, 1024, 64, 296)], 1, 1, 296),        # a cap that cannot bind: register-min loop
    (dict(R=32, T=512, H=4096, E=128, K=8, routing="zipf"), [(1000, 22, 64, 300), (700, 20, 96, 500)], 8, 8, 296),
    (dict(R=8, T=256, H=2048, E=32, K=4), [(900000, 1, 32, 64)], 1, 1, 64),            # loads leave the 21-bit keys mid-run
    (dict(R=4, T=128, H=1024, E=16, K=2), [(10, 64, 16, 33)], 1, 1, 33),               # 33 cores: two cores on lane 0
    (dict(R=16, T=1024, H=512, E=64, K=4), [(1000, 22, 32, 296)], 1, 1, 296),           # long runs of equal-cost units: rounds
    (dict(R=16, T=1024, H=512, E=64, K=4), [(1000, 22, 32, 100), (1, 22, 16, 100)], 4, 4, 100),   # two tiers, two long runs
    (dict(R=8, T=2048, H=256, E=32, K=2), [(7, 64, 8, 40)], 1, 1, 40),                  # many rounds on few cores
    (dict(R=16, T=1024, H=512, E=64, K=4), [(0, 1 << 40, 32, 64)], 1, 1, 64),           # every unit costs 1
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "R{R}T{T}H{H}E{E}K{K}".format(**c[0]))
def test_policy_and_window_dispatch_match_the_oracle(case):
    kw, tiers, g0, g1, n_cores = case
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=77, **kw)
    inp = wl.generate(cfg)
    ref_lay = oracle.layout(inp["ids"], cfg.E)
    ref = oracle.partition(ref_lay, cfg.H * 2, n_cores, tiers, g0=g0, g1=g1, max_units=1 << 16)
    U = ref["n_units"]

    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    lay = ctx.layout(to_dev(inp["ids"]))
    pol = B.make_policy(tiers, g0, g1)
    rc, mu = B.strata_moe_partition_max_units(ctx.shape, pol)
    assert rc == 0 and mu >= U
    part = ctx.partition(lay, pol, n_cores)
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    assert part.n_units.item() == U
    assert np.array_equal(part.win_base.cpu().numpy(), ref["win_base"])
    assert np.array_equal(part.unit_desc.cpu().numpy()[:U], ref["unit_desc"])
    assert np.array_equal(part.unit_cost.cpu().numpy()[:U], ref["unit_cost"])
    assert np.array_equal(part.task_offset.cpu().numpy(), ref["task_offset"])
    assert np.array_equal(part.task_unit.cpu().numpy()[:U], ref["task_unit"])
    assert np.array_equal(part.task_stripe.cpu().numpy()[:U], ref["task_stripe"])
    assert np.array_equal(part.core_load.cpu().numpy(), ref["core_load"])

    # window-major dispatch, with guard rows
    N = cfg.n_items
    whole = torch.full((N + 6, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    recv = whole[3:3 + N]
    ctx.register(whole)
    ctx.dispatch_windows(lay, part, to_dev(inp["x"]), recv)
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    want = oracle.dispatch_windows(ref_lay, ref, inp["x"], cfg.K)
    got = whole.cpu().numpy().view(np.uint16)
    assert np.array_equal(got[3:3 + N], want)
    assert np.array_equal(want, oracle.dispatch_bf16(ref_lay["dst_row"], inp["x"], nthreads=4))
    assert np.all(got[:3] == SENTINEL16) and np.all(got[3 + N:] == SENTINEL16)
    ctx.close()


def test_too_many_units_is_reported_on_the_device():
    cfg = wl.shrink(wl.CONFIGS["tiny"], R=4, T=2048, H=64, E=16, K=4)       # 32,768 rows, units of one row
    inp = wl.generate(cfg)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    lay = ctx.layout(to_dev(inp["ids"]))
    part = ctx.partition(lay, B.make_policy([(1, 1, 1, 4)]), 64)
    torch.cuda.synchronize()
    assert part.n_units.item() == -1
    assert ctx.device_status() == B.STRATA_ERR_CAPACITY
    ctx.close()


def test_host_errors():
    cfg = wl.CONFIGS["tiny"]
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    lay = ctx.layout(to_dev(wl.gen_topk_ids(cfg)))
    ok = B.make_policy([(10, 64, 16, 2)])
    part = B.Partition(cfg.R, cfg.E, 8, 256, ctx.device)
    s = torch.cuda.current_stream().cuda_stream
    assert B.strata_moe_partition(ctx.h, lay.c, B.make_policy([(10, 0, 16, 2)]), 8, part.c, 256, s) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_partition(ctx.h, lay.c, B.make_policy([(10, 64, 0, 2)]), 8, part.c, 256, s) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_partition(ctx.h, lay.c, B.make_policy([(10, 64, 16, 0)]), 8, part.c, 256, s) == B.STRATA_ERR_INVALID_ARG
    assert B.strata_moe_partition(ctx.h, lay.c, ok, 0, part.c, 256, s) == B.STRATA_ERR_SHAPE
    assert B.strata_moe_partition(ctx.h, lay.c, ok, 2000, part.c, 256, s) == B.STRATA_ERR_SHAPE
    thin = ctx.new_layout(with_optional=False)
    assert B.strata_moe_partition(ctx.h, thin.c, ok, 8, part.c, 256, s) == B.STRATA_ERR_INVALID_ARG   # no src_expert_count
    assert B.strata_moe_partition(ctx.h, lay.c, ok, 8, part.c, 256, s) == B.STRATA_OK
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    x = torch.zeros((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    assert B.strata_moe_dispatch_windows(ctx.h, lay.c, part.c, 8, x.data_ptr(), recv.data_ptr(), cfg.n_items, s) \
        == B.STRATA_ERR_NOT_REGISTERED
    ctx.register(recv)
    assert B.strata_moe_dispatch_windows(ctx.h, lay.c, part.c, 8, x.data_ptr(), recv.data_ptr(), cfg.n_items - 1, s) \
        == B.STRATA_ERR_CAPACITY
    assert B.strata_moe_dispatch_windows(ctx.h, thin.c, part.c, 8, x.data_ptr(), recv.data_ptr(), cfg.n_items, s) \
        == B.STRATA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    ctx.close()


def test_window_dispatch_survives_inconsistent_lists():
    """Lists that do not belong together are reported on the device and nothing is read or written out of
    bounds: a receive row without a source item (src_of_row = -1, with K > 1) is skipped with BAD_ROW instead
    of being filled with token 0, and a task list naming a unit that does not exist raises INVALID_ARG."""
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=78, R=4, T=64, H=256, E=16, K=4)
    inp = wl.generate(cfg)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    lay = ctx.layout(to_dev(inp["ids"]))
    part = ctx.partition(lay, B.make_policy([(10, 64, 16, 2)]), 8)
    N = cfg.n_items
    whole = torch.full((N + 6, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    recv = whole[3:3 + N]
    ctx.register(whole)
    x = to_dev(inp["x"])
    want = oracle.dispatch_bf16(oracle.layout(inp["ids"], cfg.E)["dst_row"], inp["x"], nthreads=2)

    hole = 37
    lay.src_of_row[hole] = -1
    ctx.dispatch_windows(lay, part, x, recv)
    assert ctx.device_status() == B.STRATA_ERR_BAD_ROW
    got = whole.cpu().numpy().view(np.uint16)
    keep = np.arange(N) != hole
    assert np.array_equal(got[3:3 + N][keep], want[keep]) and np.all(got[3 + hole] == SENTINEL16)
    assert np.all(got[:3] == SENTINEL16) and np.all(got[3 + N:] == SENTINEL16)

    lay2 = ctx.layout(to_dev(inp["ids"]))
    part.task_unit[0] = 1 << 20
    ctx.dispatch_windows(lay2, part, x, recv)
    assert ctx.device_status() == B.STRATA_ERR_INVALID_ARG
    part.task_unit[0] = -5
    ctx.dispatch_windows(lay2, part, x, recv)
    assert ctx.device_status() == B.STRATA_ERR_INVALID_ARG
    ctx.close()
