"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200).

Bars: layout, bf16 dispatch and e4m3 dispatch bit-exact; combine within 1 bf16
ulp (both sides run the same fp32 FMA chain, so equality is expected and the
ulp bound is the stated tolerance).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
SENTINEL16 = 0x7FC7          # a NaN pattern no input contains
GUARD = 3


def ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    def line(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(line(a) - line(b))


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(a).to(DEV)


def u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


def make_ctx(cfg: wl.MoEConfig) -> B.MoEContext:
    return B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, cfg.dispatch_dtype)


def assert_layout_equal(lay: B.Layout, ref: dict):
    torch.cuda.synchronize()
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row",
                "src_of_row"):
        got = getattr(lay, key).cpu().numpy()
        assert np.array_equal(got, ref[key]), key


def guarded(n_rows: int, width: int, dtype, fill):
    """A tensor of n_rows+2*GUARD rows filled with a sentinel; returns (whole, middle view)."""
    whole = torch.full((n_rows + 2 * GUARD, width), fill, dtype=dtype, device=DEV)
    return whole, whole[GUARD:GUARD + n_rows]


def run_full_case(cfg: wl.MoEConfig, inp=None, threads=8, x_early=False):
    """Whole path on one config, every output compared with the oracle element by element."""
    inp = inp or wl.generate(cfg)
    ref_lay = oracle.layout(inp["ids"], cfg.E)
    N, n_tok, H, K = cfg.n_items, cfg.n_tok, cfg.H, cfg.K
    fp8 = cfg.dispatch_dtype == wl.FP8_E4M3_B128

    ctx = make_ctx(cfg)
    if x_early:
        ctx.x_early(True)
    ids_d, x_d, w_d = to_dev(inp["ids"]), to_dev(inp["x"]), to_dev(inp["w"])
    lay = ctx.layout(ids_d)
    assert_layout_equal(lay, ref_lay)

    if fp8:
        whole, recv = guarded(N, H, torch.uint8, 0x7F)
        whole_s, recv_s = guarded(N, H // 128, torch.float32, -7.0)
        ctx.register(whole)
        ctx.register(whole_s)
        ctx.dispatch(lay, x_d, recv, recv_s)
        ref_q, ref_s = oracle.dispatch_fp8(ref_lay["dst_row"], inp["x"], nthreads=threads)
        got_q, got_s = recv.cpu().numpy(), recv_s.cpu().numpy()
        assert np.array_equal(got_q, ref_q)
        assert np.array_equal(got_s.view(np.uint32), ref_s.view(np.uint32))
        hw, hs = whole.cpu().numpy(), whole_s.cpu().numpy()
        assert np.all(hw[:GUARD] == 0x7F) and np.all(hw[GUARD + N:] == 0x7F)
        assert np.all(hs[:GUARD] == -7.0) and np.all(hs[GUARD + N:] == -7.0)
        y = wl.expert_standin(cfg, ref_q, ref_lay["expert_offset"], ref_s)
    else:
        whole, recv = guarded(N, H, torch.int16, SENTINEL16)
        ctx.register(whole)
        ctx.dispatch(lay, x_d, recv)
        ref_recv = oracle.dispatch_bf16(ref_lay["dst_row"], inp["x"], nthreads=threads)
        assert np.array_equal(u16(recv), ref_recv)
        hw = u16(whole)
        assert np.all(hw[:GUARD] == SENTINEL16) and np.all(hw[GUARD + N:] == SENTINEL16)
        y = wl.expert_standin(cfg, ref_recv, ref_lay["expert_offset"])

    y_d = recv if (cfg.expert == "identity" and not fp8) else to_dev(y)
    out_whole, out = guarded(n_tok, H, torch.int16, SENTINEL16)
    ctx.combine(lay, y_d, w_d, out)
    ref_out = oracle.combine(ref_lay["dst_row"], y, inp["w"], nthreads=threads)
    got_out = u16(out)
    d = ulp_distance(got_out, ref_out)
    assert d.max() <= 1, f"combine: max ulp distance {d.max()}"
    assert np.array_equal(got_out, ref_out), "combine: expected bit equality (same FMA chain)"
    ow = u16(out_whole)
    assert np.all(ow[:GUARD] == SENTINEL16) and np.all(ow[GUARD + n_tok:] == SENTINEL16)
    if cfg.expert == "identity" and not fp8:
        # gate weights sum to 1: out == x as values (a -0 input comes back as +0: fma(w, -0, +0) = +0)
        assert ulp_distance(got_out, inp["x"].reshape(n_tok, H)).max() == 0
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


# ---- the five benchmark configurations --------------------------------------------

def test_tiny_full():
    run_full_case(wl.CONFIGS["tiny"])


def test_decode_full():
    run_full_case(wl.CONFIGS["decode"])


def test_skew_full():
    run_full_case(wl.CONFIGS["skew"])


def test_fp8_full():
    run_full_case(wl.CONFIGS["fp8"])


@pytest.mark.parametrize("name", ["tiny", "decode", "skew", "fp8"])
def test_full_configs_with_the_early_x_promise(name):
    """The same comparisons with dispatch allowed to load its first rows before the layout has finished."""
    run_full_case(wl.CONFIGS[name], x_early=True)


@pytest.mark.parametrize("kw", [dict(R=1, T=3, H=64, E=2, K=1), dict(R=2, T=100, H=16384, E=4, K=3),
                                dict(R=4, T=300, H=1920, E=32, K=8)],
                         ids=lambda kw: "R{R}T{T}H{H}E{E}K{K}".format(**kw))
@pytest.mark.parametrize("fp8", [False, True], ids=["bf16", "e4m3"])
def test_early_x_promise_over_several_steps_with_x_rewritten_before_each_layout(kw, fp8):
    """Three steps in one stream; before each layout call a copy kernel rewrites x (the promise holds: x is
    complete before the call preceding dispatch starts).  Fewer units than ring stages in the first shape."""
    if fp8 and kw["H"] % 128:
        pytest.skip("e4m3 dispatch needs H % 128 == 0")
    cfg = wl.shrink(wl.CONFIGS["fp8" if fp8 else "tiny"], seed=606, **kw)
    ctx = make_ctx(cfg)
    ctx.x_early(True)
    N, H = cfg.n_items, cfg.H
    recv = torch.zeros((N, H), dtype=torch.uint8 if fp8 else torch.int16, device=DEV)
    scale = torch.zeros((N, H // 128), dtype=torch.float32, device=DEV) if fp8 else None
    ctx.register(recv)
    if fp8:
        ctx.register(scale)
    x_d = torch.zeros((cfg.n_tok, H), dtype=torch.int16, device=DEV)
    ids_d = torch.zeros((cfg.R, cfg.T, cfg.K), dtype=torch.int32, device=DEV)
    lay = ctx.new_layout()
    inputs = [wl.generate(wl.shrink(cfg, seed=700 + i)) for i in range(3)]
    staged = [(to_dev(i["ids"]), to_dev(i["x"]).view(cfg.n_tok, H)) for i in inputs]
    got = []
    for ids_s, x_s in staged:                      # everything is enqueued before anything is read back
        ids_d.copy_(ids_s)
        x_d.copy_(x_s)
        ctx.layout(ids_d, lay)
        ctx.dispatch(lay, x_d, recv, scale)
        got.append((recv.clone(), scale.clone() if fp8 else None))
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    for inp, (r, sc) in zip(inputs, got):
        ref = oracle.layout(inp["ids"], cfg.E)
        if fp8:
            q, s_ = oracle.dispatch_fp8(ref["dst_row"], inp["x"], nthreads=4)
            assert np.array_equal(r.cpu().numpy(), q)
            assert np.array_equal(sc.cpu().numpy().view(np.uint32), s_.view(np.uint32))
        else:
            assert np.array_equal(u16(r), oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4))
    ctx.close()


def test_prefill_full_size_sampled():
    """The benchmark's launch configuration at full size (7.5 GB receive buffer): layout compared
    in full; dispatch and combine on sampled outputs the oracle computes one by one, plus the
    properties that hold at any size (row equality through dst_row; identity experts return x)."""
    cfg = wl.CONFIGS["prefill"]
    inp = wl.generate(cfg)
    ref_lay = oracle.layout(inp["ids"], cfg.E)
    N, n_tok, H, K = cfg.n_items, cfg.n_tok, cfg.H, cfg.K
    ctx = make_ctx(cfg)
    ctx.x_early(True)                      # as bench.py runs it
    ids_d, x_d, w_d = to_dev(inp["ids"]), to_dev(inp["x"]), to_dev(inp["w"])
    slab = torch.empty(N * H * 2 + 4096, dtype=torch.uint8, device=DEV)
    rid = ctx.register(slab)
    recv = ctx.carve(rid, (N, H), torch.int16)
    recv.fill_(SENTINEL16)
    lay = ctx.layout(ids_d)
    ctx.dispatch(lay, x_d, recv)           # enqueued right behind the layout, as in a step of the benchmark
    torch.cuda.synchronize()
    assert_layout_equal(lay, ref_lay)

    x2 = x_d.view(n_tok, H)
    x_host = inp["x"].reshape(n_tok, H)
    # sampled rows against the oracle's placement: row j holds the token of item src_of_row[j]
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([rng.integers(0, N, 4096), [0, N - 1],
                                     ref_lay["expert_offset"][:-1].clip(0, N - 1)]))
    got = u16(recv[torch.from_numpy(rows).to(DEV)])
    want = x_host[ref_lay["src_of_row"][rows] // K]
    assert np.array_equal(got, want)
    # every row, on the device: recv[dst_row[i]] == x[i // K]
    dst = lay.dst_row.view(n_tok, K).long()
    for lo in range(0, n_tok, 8192):
        hi = min(n_tok, lo + 8192)
        for k in range(K):
            assert torch.equal(recv[dst[lo:hi, k]], x2[lo:hi])

    out = torch.empty((n_tok, H), dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, w_d, out)
    torch.cuda.synchronize()
    # sampled tokens, one by one through the oracle (identity experts: the K rows are the token's own row)
    toks = np.unique(np.concatenate([rng.integers(0, n_tok, 1024), [0, n_tok - 1]]))
    y_mini = np.repeat(x_host[toks], K, axis=0)
    d_mini = np.arange(toks.size * K, dtype=np.int32).reshape(-1, K)
    want_out = oracle.combine(d_mini, y_mini, inp["w"].reshape(n_tok, K)[toks], nthreads=4)
    got_out = u16(out[torch.from_numpy(toks).to(DEV)])
    assert ulp_distance(got_out, want_out).max() <= 1
    assert np.array_equal(got_out, want_out)
    # invariant at full size, as values (-0 == +0)
    assert bool((out.view(torch.bfloat16) == x2.view(torch.bfloat16)).all())
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


# ---- ragged, degenerate and extreme shapes -------------------------------------------

RAGGED = [
    dict(R=1, T=1, H=8, E=1, K=1),
    dict(R=3, T=7, H=24, E=6, K=3),
    dict(R=2, T=300, H=1000, E=10, K=5),            # T*K = 1500: two tiles per rank, ragged tail
    dict(R=4, T=1030, H=256, E=64, K=1),
    dict(R=2, T=65, H=8200, E=4, K=2),               # row of 16400 B: two chunks per row
    dict(R=2, T=40, H=20000, E=8, K=4),              # three chunks, ragged last chunk
    dict(R=8, T=33, H=512, E=1024, K=8),             # maximum expert count
    dict(R=1, T=200, H=64, E=48, K=32),              # maximum top-k (generic combine path)
    dict(R=2, T=129, H=136, E=12, K=9),
    dict(R=5, T=50, H=4096, E=20, K=6),
    dict(R=4, T=100, H=2048, E=16, K=4),
    dict(R=4, T=256, H=64, E=32, K=4),               # 4,096 items: the largest single-CTA layout
    dict(R=4, T=257, H=64, E=32, K=4),               # just above it: a cluster of 8 CTAs
    dict(R=4, T=2048, H=64, E=32, K=4),              # 32,768 items: the largest cluster layout
    dict(R=4, T=2049, H=64, E=32, K=4),              # just above it: tiled layout, two launches
    dict(R=5, T=1111, H=64, E=1000, K=3),            # cluster layout, CTAs and warps straddle ranks, wide E
    dict(R=64, T=3, H=64, E=64, K=7),                # warps straddle several source ranks
]


@pytest.mark.parametrize("kw", RAGGED, ids=lambda kw: "R{R}T{T}H{H}E{E}K{K}".format(**kw))
def test_ragged_shapes(kw):
    cfg = wl.shrink(wl.CONFIGS["decode"], seed=4242 + kw["T"], **kw)
    run_full_case(cfg, threads=4)


@pytest.mark.parametrize("kw", [dict(R=2, T=50, H=128, E=4, K=2), dict(R=4, T=300, H=1920, E=32, K=8),
                                dict(R=1, T=9, H=4224, E=2, K=2), dict(R=2, T=20, H=8192 + 128, E=8, K=3)],
                         ids=lambda kw: "R{R}T{T}H{H}E{E}K{K}".format(**kw))
def test_ragged_shapes_fp8(kw):
    cfg = wl.shrink(wl.CONFIGS["fp8"], seed=99 + kw["T"], **kw)
    run_full_case(cfg, threads=4)


def test_duplicate_ids_and_all_to_one_expert():
    cfg = wl.shrink(wl.CONFIGS["tiny"], R=4, T=600, H=64, E=8, K=4, expert="scale")
    inp = wl.generate(cfg)
    rng = np.random.default_rng(1)
    inp["ids"] = rng.integers(0, 3, size=inp["ids"].shape).astype(np.int32)      # duplicates, empty experts
    run_full_case(cfg, inp)
    inp["ids"][:] = 5                                                           # a single hot expert
    run_full_case(cfg, inp)


def test_zipf_small():
    cfg = wl.shrink(wl.CONFIGS["skew"], R=8, T=200, H=512, E=32, K=8)
    run_full_case(cfg)


def test_fp8_extreme_values_every_bf16_pattern():
    """All finite bf16 bit patterns as inputs, arranged so that blocks have very different amax
    (and some are all zero): codes and scales must equal the oracle's bit for bit."""
    cfg = wl.shrink(wl.CONFIGS["fp8"], R=2, T=128, H=512, E=4, K=2)
    inp = wl.generate(cfg)
    bits = np.arange(65536, dtype=np.uint32)
    finite = bits[(bits & 0x7F80) != 0x7F80].astype(np.uint16)
    rng = np.random.default_rng(7)
    x = inp["x"].reshape(-1)
    # sorted by magnitude so that a block holds values of similar size (exercises subnormal codes
    # of tiny blocks as well as the saturating top), then some shuffled blocks for mixed ranges
    mag = np.sort(finite & 0x7FFF)
    sign = (rng.integers(0, 2, mag.size) << 15).astype(np.uint16)
    x[:mag.size] = mag | sign
    x[mag.size:2 * mag.size] = rng.permutation(finite)
    x[2 * mag.size:2 * mag.size + 256] = 0
    x[2 * mag.size + 256:2 * mag.size + 384] = 0x8000
    run_full_case(cfg, inp)


# ---- behaviour of the boundary on a real device ---------------------------------------

def test_layout_is_deterministic():
    cfg = wl.CONFIGS["skew"]
    ids_d = to_dev(wl.gen_topk_ids(cfg))
    ctx = make_ctx(cfg)
    first = ctx.layout(ids_d)
    torch.cuda.synchronize()
    ref = {k: getattr(first, k).clone() for k in ("dst_row", "src_of_row", "expert_offset", "src_expert_count")}
    lay = ctx.new_layout()
    for _ in range(20):
        ctx.layout(ids_d, lay)
        torch.cuda.synchronize()
        for k, v in ref.items():
            assert torch.equal(getattr(lay, k), v), k
    ctx.close()


def test_bad_expert_id_is_skipped_and_reported():
    cfg = wl.shrink(wl.CONFIGS["tiny"], H=64)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    ids[1, 5, 0] = cfg.E          # out of range
    ids[2, 9, 1] = -3
    ctx = make_ctx(cfg)
    lay = ctx.layout(to_dev(ids))
    assert ctx.device_status() == B.STRATA_ERR_BAD_EXPERT_ID
    assert ctx.device_status() == B.STRATA_OK                      # reading clears it
    dst = lay.dst_row.cpu().numpy()
    assert dst[1, 5, 0] == -1 and dst[2, 9, 1] == -1
    valid = np.ones(ids.shape, bool)
    valid[1, 5, 0] = valid[2, 9, 1] = False
    N = cfg.n_items
    assert lay.expert_count.sum().item() == N - 2
    assert np.array_equal(np.sort(dst[valid]), np.arange(N - 2))   # the rest is still a packed bijection
    # the valid items keep their relative (expert, rank, token, slot) order
    order = np.lexsort((np.arange(N)[valid.ravel()], ids.ravel()[valid.ravel()]))
    assert np.array_equal(dst.ravel()[valid.ravel()][order], np.arange(N - 2))
    # dispatch skips the two items, reports a bad row, writes nothing out of bounds
    whole, recv = guarded(N, cfg.H, torch.int16, -1)
    ctx.register(whole)
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    assert ctx.device_status() == B.STRATA_OK               # the layout already reported; -1 rows are just skipped
    hw = whole.cpu().numpy()
    assert np.all(hw[:GUARD] == -1) and np.all(hw[GUARD + N - 2:] == -1)
    x2 = inp["x"].reshape(cfg.n_tok, cfg.H)
    got = hw[GUARD:GUARD + N - 2].view(np.uint16)
    assert np.array_equal(got[dst.ravel()[valid.ravel()]], x2[(np.arange(N) // cfg.K)[valid.ravel()]])
    # combine ignores the skipped slots
    out = torch.zeros((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, to_dev(inp["w"]), out)
    assert ctx.device_status() == B.STRATA_OK
    # a destination row that is neither valid nor -1 is reported
    lay.dst_row.view(-1)[5] = cfg.n_items + 100
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    assert ctx.device_status() == B.STRATA_ERR_BAD_ROW
    ctx.combine(lay, recv, to_dev(inp["w"]), out)
    assert ctx.device_status() == B.STRATA_ERR_BAD_ROW
    hw = whole.cpu().numpy()
    assert np.all(hw[:GUARD] == -1) and np.all(hw[GUARD + N:] == -1)      # still nothing out of bounds
    ctx.close()


def test_host_errors_on_device_context():
    cfg = wl.shrink(wl.CONFIGS["tiny"], H=64)
    ctx = make_ctx(cfg)
    inp = wl.generate(cfg)
    lay = ctx.layout(to_dev(inp["ids"]))
    x_d = to_dev(inp["x"])
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    with pytest.raises(B.StrataError) as ei:
        ctx.dispatch(lay, x_d, recv)                               # not registered
    assert ei.value.code == B.STRATA_ERR_NOT_REGISTERED
    ctx.register(recv)
    with pytest.raises(B.StrataError) as ei:
        ctx.dispatch(lay, x_d, recv[:-1])                          # too few rows
    assert ei.value.code == B.STRATA_ERR_CAPACITY
    with pytest.raises(B.StrataError) as ei:
        ctx.dispatch(lay, x_d.view(-1)[4:], recv)                  # 8-byte offset
    assert ei.value.code == B.STRATA_ERR_ALIGNMENT
    ctx.dispatch(lay, x_d, recv)
    assert ctx.device_status() == B.STRATA_OK
    assert ctx.launch_count() == 2                                 # 1 (small-batch layout) + 1 (dispatch); failures launched nothing
    ctx.close()


def test_zero_copy_rank_partitions():
    """The receive buffer is carved from a registered slab; rank d's partition is a plain view of it."""
    cfg = wl.CONFIGS["tiny"]
    inp = wl.generate(cfg)
    ref_lay = oracle.layout(inp["ids"], cfg.E)
    ctx = make_ctx(cfg)
    slab = torch.zeros(cfg.n_items * cfg.H * 2 + 1024, dtype=torch.uint8, device=DEV)
    rid = ctx.register(slab)
    recv = ctx.carve(rid, (cfg.n_items, cfg.H), torch.int16)
    assert recv.data_ptr() == slab.data_ptr()
    lay = ctx.layout(to_dev(inp["ids"]))
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    torch.cuda.synchronize()
    h_off = lay.rank_offset.cpu().numpy()
    ref_recv = oracle.dispatch_bf16(ref_lay["dst_row"], inp["x"])
    for d in range(cfg.R):
        rc, base, rows = B.strata_moe_recv_view(ctx.h, h_off, d, recv.data_ptr())
        assert rc == 0 and rows == ref_lay["rank_count"][d]
        assert base == recv.data_ptr() + int(ref_lay["rank_offset"][d]) * cfg.H * 2
        part = recv[h_off[d]:h_off[d + 1]]
        assert part.data_ptr() == base
        assert np.array_equal(u16(part), ref_recv[h_off[d]:h_off[d + 1]])
    ctx.close()


@pytest.mark.parametrize("cfg", [wl.CONFIGS["tiny"],
                                 # x is 168 MB: three upload chunks, the last one ragged
                                 wl.shrink(wl.CONFIGS["tiny"], R=4, T=5000, H=4200, E=16, K=2, seed=5)],
                         ids=["one-chunk", "three-chunks"])
def test_roundtrip_from_host_buffers(cfg):
    inp = wl.generate(cfg)
    ctx = make_ctx(cfg)
    lay = ctx.new_layout()
    ids_d = torch.empty((cfg.R, cfg.T, cfg.K), dtype=torch.int32, device=DEV)
    x_d = torch.empty((cfg.R, cfg.T, cfg.H), dtype=torch.int16, device=DEV)
    w_d = torch.empty((cfg.R, cfg.T, cfg.K), dtype=torch.float32, device=DEV)
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    out_d = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.register(recv)
    dev = B.strata_moe_device_buffers(ids_d.data_ptr(), x_d.data_ptr(), w_d.data_ptr(), recv.data_ptr(),
                                      out_d.data_ptr(), lay.c)
    h_ids = torch.from_numpy(inp["ids"]).pin_memory()
    h_x = torch.from_numpy(inp["x"].view(np.int16)).pin_memory()
    h_w = torch.from_numpy(inp["w"]).pin_memory()
    h_out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16).pin_memory()
    rc = B.strata_moe_roundtrip_host(ctx.h, dev, h_ids.data_ptr(), h_x.data_ptr(), h_w.data_ptr(),
                                     h_out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    ref_lay = oracle.layout(inp["ids"], cfg.E)
    ref_recv = oracle.dispatch_bf16(ref_lay["dst_row"], inp["x"], nthreads=8)
    ref_out = oracle.combine(ref_lay["dst_row"], ref_recv, inp["w"], nthreads=8)
    assert np.array_equal(h_out.numpy().view(np.uint16), ref_out)
    assert np.array_equal(u16(recv), ref_recv)
    # a second call on the same buffers (events and streams are reused)
    h_out.zero_()
    rc = B.strata_moe_roundtrip_host(ctx.h, dev, h_ids.data_ptr(), h_x.data_ptr(), h_w.data_ptr(),
                                     h_out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    assert np.array_equal(h_out.numpy().view(np.uint16), ref_out)
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


def test_per_cta_trace_probes():
    """Stage probes: every CTA of a traced launch records start <= end on the global timer; the spread
    of end times under Zipf routing stays small because tokens, not experts, are dealt to the CTAs."""
    cfg = wl.shrink(wl.CONFIGS["skew"], T=256)
    inp = wl.generate(cfg)
    ctx = make_ctx(cfg)
    lay = ctx.layout(to_dev(inp["ids"]))
    x_d, w_d = to_dev(inp["x"]), to_dev(inp["w"])
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.register(recv)
    for _ in range(2):
        ctx.dispatch(lay, x_d, recv)
    tr = ctx.trace(4096)
    for name, call in (("dispatch", lambda: ctx.dispatch(lay, x_d, recv)),
                       ("combine", lambda: ctx.combine(lay, recv, w_d, out))):
        tr.zero_()
        call()
        torch.cuda.synchronize()
        rec = tr.cpu().numpy()
        used = rec[rec[:, 0] != 0]
        assert 148 <= len(used) <= 4096, name
        assert np.all(used[:, 1] >= used[:, 0]), name
        total = used[:, 1].max() - used[:, 0].min()
        spread = (used[:, 1].max() - used[:, 1].min()) / total
        assert total > 0 and 0 <= spread < 0.5, (name, spread)
        summ = ctx.trace_summary(tr)
        assert summ["ctas"] == len(used) and abs(summ["finish_spread"] - spread) < 1e-9
        if name == "dispatch":                   # the issuing thread's blocked time is part of its lifetime
            assert np.all(used[:, 2] + used[:, 3] <= (used[:, 1] - used[:, 0]))
            assert 0 < summ["wait_in_share"] + summ["wait_out_share"] <= 1.0
        else:
            assert np.all(used[:, 2] == 0) and np.all(used[:, 3] == 0)
    ctx.trace_off()
    tr.zero_()
    ctx.dispatch(lay, x_d, recv)
    torch.cuda.synchronize()
    assert int(tr.abs().sum().item()) == 0                   # probes off: nothing written
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


@pytest.mark.parametrize("seed", range(16))
def test_random_shapes(seed):
    """Seeded random shapes through the whole path: odd sizes hit every work-distribution branch
    (all-static grids, column-part units, chunked rows, cluster and tiled layouts)."""
    rng = np.random.default_rng(1234 + seed)
    R = int(rng.choice([1, 2, 3, 4, 6, 8, 16]))
    e_loc = int(rng.integers(1, 9))
    E = R * e_loc
    K = int(rng.integers(1, min(E, 10) + 1))
    T = int(rng.choice([1, 5, 37, 130, 700, 3000]))
    H = int(rng.choice([8, 64, 520, 1024, 2056, 7168, 9000])) // 8 * 8
    if R * T * K * H * 2 > 600e6:          # keep every case under ~0.6 GB of receive buffer
        T = max(1, int(600e6 // (R * K * H * 2)))
    cfg = wl.shrink(wl.CONFIGS["decode"], R=R, T=T, H=H, E=E, K=K, seed=9000 + seed,
                    routing="zipf" if seed % 3 == 0 else "uniform",
                    expert=["identity", "scale", "affine"][seed % 3])
    run_full_case(cfg, threads=8)


# ---- production layout variants: aligned segments and the "not routed" sentinel -----------------

@pytest.mark.parametrize("kw,align,frac", [
    (dict(R=4, T=128, H=1024, E=16, K=2), 128, 0.0),
    (dict(R=4, T=128, H=1024, E=16, K=2), 1, 0.25),
    (dict(R=8, T=300, H=512, E=64, K=6), 16, 0.2),            # cluster layout
    (dict(R=16, T=128, H=7168, E=256, K=8), 128, 0.1),        # decode shape
    (dict(R=8, T=2000, H=256, E=32, K=4), 64, 0.3),           # tiled layout (64,000 items)
    (dict(R=2, T=50, H=128, E=4, K=2), 7, 1.0),               # nothing routed at all, odd alignment
], ids=lambda v: str(v).replace(" ", "") if not isinstance(v, dict) else "R{R}T{T}H{H}E{E}K{K}".format(**v))
def test_aligned_segments_and_unrouted_slots(kw, align, frac):
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=4321, **kw)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    rng = np.random.default_rng(11)
    ids[rng.random(ids.shape) < frac] = -1
    ref = oracle.layout(ids, cfg.E, segment_align=align, allow_unrouted=True)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, segment_align=align, allow_unrouted=True)
    n_rows = ctx.recv_rows
    assert n_rows == cfg.n_items + cfg.E * (max(align, 1) - 1)
    lay = ctx.layout(to_dev(ids))
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    total = int(ref["expert_offset"][cfg.E])
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row"):
        assert np.array_equal(getattr(lay, key).cpu().numpy(), ref[key]), key
    assert np.array_equal(lay.src_of_row.cpu().numpy()[:total], ref["src_of_row"])

    whole, recv = guarded(n_rows, cfg.H, torch.int16, SENTINEL16)
    ctx.register(whole)
    x_d, w_d = to_dev(inp["x"]), to_dev(inp["w"])
    ctx.dispatch(lay, x_d, recv)
    want = oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4, n_rows=n_rows)
    got = u16(recv)
    written = np.zeros(n_rows, bool)
    written[ref["dst_row"][ref["dst_row"] >= 0]] = True
    assert np.array_equal(got[written], want[written])
    assert np.all(got[~written] == SENTINEL16)                       # padding rows are never touched
    hw = u16(whole)
    assert np.all(hw[:GUARD] == SENTINEL16) and np.all(hw[GUARD + n_rows:] == SENTINEL16)

    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, w_d, out)
    want_out = oracle.combine(ref["dst_row"], want, inp["w"], nthreads=4)
    assert np.array_equal(u16(out), want_out)
    assert ctx.device_status() == B.STRATA_OK

    # the allocation-free layout entry honours the same two options
    got2 = ctx.new_layout()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    rc = B.strata_moe_layout_noalloc(ctx.shape, to_dev(ids).data_ptr(), got2.c, status.data_ptr(),
                                     torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert rc == 0 and status.item() == 0
    assert torch.equal(got2.dst_row, lay.dst_row) and torch.equal(got2.expert_offset, lay.expert_offset)
    assert torch.equal(got2.src_of_row[:total], lay.src_of_row[:total])
    ctx.close()


def _layout_only(R, T, K, E, ids):
    ref = oracle.layout(ids, E, allow_unrouted=True)
    ctx = B.MoEContext(R, T, 64, E, K, allow_unrouted=True)
    lay = ctx.layout(to_dev(ids))
    torch.cuda.synchronize()
    assert ctx.device_status() == B.STRATA_OK
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row"):
        assert np.array_equal(getattr(lay, key).cpu().numpy(), ref[key]), key
    ctx.close()


def test_unrouted_first_lane_of_a_round_that_straddles_two_source_ranks():
    """A 32-item round whose first item is not routed and whose items belong to two source ranks: the
    per-source-rank counts must still split at the rank boundary (48 items per rank, item 32 = -1)."""
    R, T, K, E = 2, 24, 2, 4
    ids = np.ones((R, T, K), np.int32)
    ids.reshape(-1)[32] = -1
    ref = oracle.layout(ids, E, allow_unrouted=True)
    assert ref["src_expert_count"][:, 1].tolist() == [47, 48]
    _layout_only(R, T, K, E, ids)


@pytest.mark.parametrize("kw", [dict(R=3, T=21, K=3, E=6), dict(R=8, T=37, K=5, E=16), dict(R=16, T=129, K=7, E=64),
                                dict(R=5, T=1, K=1, E=5), dict(R=32, T=3, K=1, E=32)],
                         ids=lambda kw: "R{R}T{T}K{K}E{E}".format(**kw))
def test_unrouted_at_every_round_start_with_ranks_off_the_round_grid(kw):
    """T*K is not a multiple of 32, so rounds straddle ranks; every 32nd item (each round's first lane,
    whatever the run length) is forced to -1, and a random fifth of the rest too."""
    R, T, K, E = kw["R"], kw["T"], kw["K"], kw["E"]
    rng = np.random.default_rng(R * 1000 + T)
    ids = rng.integers(0, E, size=(R, T, K), dtype=np.int32)
    flat = ids.reshape(-1)
    flat[rng.random(flat.shape) < 0.2] = -1
    flat[::32] = -1
    _layout_only(R, T, K, E, ids)


def test_minus_one_is_an_error_without_the_flag():
    cfg = wl.shrink(wl.CONFIGS["tiny"], H=64)
    ids = wl.gen_topk_ids(cfg)
    ids[0, 3, 1] = -1
    ctx = make_ctx(cfg)
    ctx.layout(to_dev(ids))
    assert ctx.device_status() == B.STRATA_ERR_BAD_EXPERT_ID
    ctx.close()


@pytest.mark.parametrize("kw", [dict(R=4, T=300, H=512, E=16, K=4),          # cluster layout, claimed units
                                dict(R=8, T=1200, H=256, E=32, K=4)],         # tiled layout (38,400 items)
                         ids=lambda kw: "R{R}T{T}H{H}E{E}K{K}".format(**kw))
@pytest.mark.parametrize("x_early", [False, True], ids=["default", "x_early"])
def test_cuda_graph_replay(kw, x_early):
    """layout -> dispatch -> combine captured once in a CUDA graph and replayed on new inputs: every
    piece of state the kernels hand from one launch to the next (ticket, work-claim counters) is
    restored by the kernels themselves, so a replay computes the same as a fresh call.  With the early-x
    promise the replays keep it: x is rewritten before the graph (hence before its layout) starts."""
    cfg = wl.shrink(wl.CONFIGS["decode"], seed=1, **kw)
    ctx = make_ctx(cfg)
    ctx.x_early(x_early)
    first = wl.generate(cfg)
    ids_d, x_d, w_d = to_dev(first["ids"]), to_dev(first["x"]), to_dev(first["w"])
    lay = ctx.new_layout()
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.register(recv)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):                         # warm-up outside the capture
            ctx.layout(ids_d, lay)
            ctx.dispatch(lay, x_d, recv)
            ctx.combine(lay, recv, w_d, out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ctx.layout(ids_d, lay)
        ctx.dispatch(lay, x_d, recv)
        ctx.combine(lay, recv, w_d, out)
    for rep in range(4):
        inp = wl.generate(wl.shrink(cfg, seed=100 + rep))
        ids_d.copy_(to_dev(inp["ids"]))
        x_d.copy_(to_dev(inp["x"]))
        w_d.copy_(to_dev(inp["w"]))
        recv.fill_(SENTINEL16)
        out.fill_(SENTINEL16)
        g.replay()
        torch.cuda.synchronize()
        ref = oracle.layout(inp["ids"], cfg.E)
        assert np.array_equal(lay.dst_row.cpu().numpy(), ref["dst_row"]), rep
        ref_recv = oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4)
        assert np.array_equal(u16(recv), ref_recv), rep
        assert np.array_equal(u16(out), oracle.combine(ref["dst_row"], ref_recv, inp["w"], nthreads=4)), rep
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


@pytest.mark.parametrize("kw,cap,frac", [
    (dict(R=4, T=128, H=1024, E=16, K=2), 24, 0.0),               # some slots overflow
    (dict(R=16, T=128, H=7168, E=256, K=8), 16, 0.0),             # decode shape, static [256][16][16] buffer
    (dict(R=8, T=1500, H=128, E=32, K=4), 200, 0.2),              # several tiles per rank, unrouted slots
    (dict(R=2, T=60, H=64, E=4, K=3), 1000, 0.0),                 # capacity nobody reaches
    (dict(R=1, T=100, H=64, E=1024, K=8), 3, 0.0),                # one rank, the largest expert table
    (dict(R=64, T=64, H=64, E=64, K=1), 2, 0.1),                  # many ranks, one item per token
    (dict(R=4, T=1024, H=64, E=16, K=4), 300, 0.0),               # a rank fills its tile exactly (4096 items)
], ids=lambda v: str(v) if not isinstance(v, dict) else "R{R}T{T}H{H}E{E}K{K}".format(**v))
def test_fixed_capacity_layout(kw, cap, frac):
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=555, **kw)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    if frac:
        ids[np.random.default_rng(2).random(ids.shape) < frac] = -1
    ref = oracle.layout(ids, cfg.E, allow_unrouted=True, slot_capacity=cap)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, allow_unrouted=True, slot_capacity=cap)
    n_rows = ctx.recv_rows
    assert n_rows == cfg.E * cfg.R * cap
    lay = ctx.layout(to_dev(ids))
    torch.cuda.synchronize()
    assert ctx.device_status() == (B.STRATA_ERR_CAPACITY if ref["dropped"] else B.STRATA_OK)
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row",
                "src_of_row"):
        assert np.array_equal(getattr(lay, key).cpu().numpy(), ref[key]), key
    whole, recv = guarded(n_rows, cfg.H, torch.int16, SENTINEL16)
    ctx.register(whole)
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    want = oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4, n_rows=n_rows)
    got = u16(recv)
    used = ref["src_of_row"] >= 0
    assert np.array_equal(got[used], want[used]) and np.all(got[~used] == SENTINEL16)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, to_dev(inp["w"]), out)
    assert np.array_equal(u16(out), oracle.combine(ref["dst_row"], want, inp["w"], nthreads=4))
    assert ctx.device_status() == B.STRATA_OK                    # dropped items are -1 rows: skipped silently
    hw = u16(whole)
    assert np.all(hw[:GUARD] == SENTINEL16) and np.all(hw[GUARD + n_rows:] == SENTINEL16)
    # the window-partitioning variant declines this layout
    pol = B.make_policy([(10, 64, 16, 2)])
    part = B.Partition(cfg.R, cfg.E, 8, 64, ctx.device)
    assert B.strata_moe_partition(ctx.h, lay.c, pol, 8, part.c, 64, torch.cuda.current_stream().cuda_stream) \
        == B.STRATA_ERR_SHAPE
    ctx.close()


@pytest.mark.parametrize("budget", [1, 7, 40])
def test_sm_budget_changes_no_result(budget):
    """Persistent grids sized for a few SMs compute the same as grids sized for the whole GPU."""
    cfg = wl.shrink(wl.CONFIGS["decode"], R=8, T=200, H=1536, E=32, K=4, seed=77)
    inp = wl.generate(cfg)
    ref = oracle.layout(inp["ids"], cfg.E)
    ref_recv = oracle.dispatch_bf16(ref["dst_row"], inp["x"], nthreads=4)
    ref_out = oracle.combine(ref["dst_row"], ref_recv, inp["w"], nthreads=4)
    ctx = make_ctx(cfg)
    ctx.sm_budget(budget)
    ids_d, x_d, w_d = to_dev(inp["ids"]), to_dev(inp["x"]), to_dev(inp["w"])
    recv = torch.full((cfg.n_items, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    out = torch.full((cfg.n_tok, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    ctx.register(recv)
    lay = ctx.layout(ids_d)
    for _ in range(2):                                  # twice: the claim counters re-arm with the smaller grid too
        ctx.dispatch(lay, x_d, recv)
        ctx.combine(lay, recv, w_d, out)
    torch.cuda.synchronize()
    assert np.array_equal(u16(recv), ref_recv)
    assert np.array_equal(u16(out), ref_out)
    # the collectives follow the same budget
    R, n = 8, 6 * 16384
    pay = wl.gen_payload(R, R * n // 2, seed=3)
    x = to_dev(pay)
    a2a = torch.empty_like(x)
    red = torch.empty((R, n // 2), dtype=torch.int16, device=DEV)
    ctx.alltoall(x.view(R, R, n // 2), a2a.view(R, R, n // 2))
    ctx.reducescatter(a2a.view(R, R, n // 2), red)
    t = oracle.alltoall(pay.view(np.uint8).reshape(R, R, n)).view(np.uint16).reshape(R, R, n // 2)
    assert np.array_equal(u16(a2a).reshape(R, R, n // 2), t)
    assert np.array_equal(u16(red), oracle.reducescatter(t))
    assert ctx.device_status() == B.STRATA_OK
    ctx.sm_budget(0)
    ctx.close()


@pytest.mark.parametrize("kw,align,cap,frac", [
    (dict(R=4, T=128, H=64, E=16, K=2), 0, 0, 0.0),                 # packed
    (dict(R=4, T=300, H=64, E=16, K=4), 128, 0, 0.1),               # GEMM-tile-aligned segments, unrouted slots
    (dict(R=8, T=1500, H=64, E=32, K=4), 64, 0, 0.0),               # tiled layout path
    (dict(R=16, T=128, H=64, E=256, K=8), 0, 16, 0.0),              # decode shape, fixed capacity
    (dict(R=2, T=60, H=64, E=4, K=3), 0, 7, 0.2),
    (dict(R=1, T=5, H=64, E=1024, K=1), 8, 0, 0.0),                 # more experts than rows
], ids=lambda v: str(v) if not isinstance(v, dict) else "R{R}T{T}E{E}K{K}".format(**v))
def test_row_experts(kw, align, cap, frac):
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=321, **kw)
    inp = wl.generate(cfg)
    ids = inp["ids"].copy()
    if frac:
        rng = np.random.default_rng(5)
        ids[rng.uniform(size=ids.shape) < frac] = -1
    ref = oracle.layout(ids, cfg.E, segment_align=max(1, align), allow_unrouted=frac > 0, slot_capacity=cap)
    want = oracle.row_experts(ref, cfg.R, cap)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, segment_align=align, allow_unrouted=frac > 0,
                       slot_capacity=cap)
    lay = ctx.layout(to_dev(ids))
    whole = torch.full((ctx.recv_rows + 2 * GUARD,), -7, dtype=torch.int32, device=DEV)
    got = ctx.row_experts(lay, whole[GUARD:GUARD + ctx.recv_rows])
    torch.cuda.synchronize()
    h = whole.cpu().numpy()
    assert np.all(h[:GUARD] == -7) and np.all(h[-GUARD:] == -7)
    g = got.cpu().numpy()                            # the oracle's arrays end at expert_offset[E]; the buffer may be longer
    assert want.shape[0] <= ctx.recv_rows
    assert np.array_equal(g[:want.shape[0]], want) and np.all(g[want.shape[0]:] == -1)
    if cap:
        ctx.device_status()                          # CAPACITY is raised when slots overflow: expected here
    else:
        assert ctx.device_status() == B.STRATA_OK
    ctx.close()


def test_row_experts_full_prefill_shape():
    cfg = wl.CONFIGS["prefill"]
    ids = wl.gen_topk_ids(cfg)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, segment_align=128)
    lay = ctx.layout(to_dev(ids))
    got = ctx.row_experts(lay).cpu().numpy()
    ref = oracle.layout(ids, cfg.E, segment_align=128)
    want = oracle.row_experts(ref, cfg.R)
    assert np.array_equal(got[:want.shape[0]], want) and np.all(got[want.shape[0]:] == -1)
    # every 128-row tile belongs to one expert or is empty, and occupied rows carry the id of their item
    tiles = got.reshape(-1, 128)
    first = tiles[:, :1]
    assert np.all((tiles == first) | (tiles == -1))
    src = lay.src_of_row.cpu().numpy()[:want.shape[0]]
    occ = src >= 0
    assert np.array_equal(got[:want.shape[0]][occ], ids.ravel()[src[occ]]) and np.all(got[:want.shape[0]][~occ] == -1)
    ctx.close()


def test_fixed_capacity_with_e4m3_dispatch():
    """The low-latency pairing: static [E][R][C] receive buffer, e4m3 payload with per-128-column scales."""
    cfg = wl.shrink(wl.CONFIGS["fp8"], R=8, T=96, H=1024, E=32, K=4, seed=909)
    cap = 20
    inp = wl.generate(cfg)
    ref = oracle.layout(inp["ids"], cfg.E, slot_capacity=cap)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, cfg.dispatch_dtype, slot_capacity=cap)
    n_rows = ctx.recv_rows
    lay = ctx.layout(to_dev(inp["ids"]))
    whole_q, recv_q = guarded(n_rows, cfg.H, torch.uint8, 0x7F)
    whole_s, recv_s = guarded(n_rows, cfg.H // 128, torch.float32, -1.0)
    ctx.register(whole_q)
    ctx.register(whole_s)
    ctx.dispatch(lay, to_dev(inp["x"]), recv_q, recv_s)
    torch.cuda.synchronize()
    q, s = oracle.dispatch_fp8(ref["dst_row"], inp["x"], n_rows=n_rows)
    used = ref["src_of_row"] >= 0
    assert used.sum() == (ref["dst_row"] >= 0).sum() > 0
    gq, gs = recv_q.cpu().numpy(), recv_s.cpu().numpy()
    assert np.array_equal(gq[used], q[used]) and np.all(gq[~used] == 0x7F)
    assert np.array_equal(gs[used].view(np.uint32), s[used].view(np.uint32)) and np.all(gs[~used] == -1.0)
    assert np.all(whole_q.cpu().numpy()[:GUARD] == 0x7F) and np.all(whole_s.cpu().numpy()[-GUARD:] == -1.0)
    st = ctx.device_status()
    assert st == (B.STRATA_ERR_CAPACITY if ref["dropped"] else B.STRATA_OK)
    ctx.close()


def test_usage_with_bfloat16_tensors_against_torch_ops():
    """The calls as a torch user makes them (bfloat16 tensors), cross-checked with plain torch ops:
    dispatch is an index copy, combine a weighted sum in fp32 (within 1 bf16 ulp of torch's own order)."""
    R, T, H, E, K = 4, 96, 512, 16, 4
    g = torch.Generator(device=DEV).manual_seed(5)
    x = torch.randn((R, T, H), generator=g, device=DEV).to(torch.bfloat16)
    ids = torch.stack([torch.randperm(E, generator=g, device=DEV)[:K] for _ in range(R * T)]).view(R, T, K).to(torch.int32)
    w = torch.softmax(torch.randn((R, T, K), generator=g, device=DEV), dim=-1)
    ctx = B.MoEContext(R, T, H, E, K)
    recv = torch.zeros((ctx.recv_rows, H), dtype=torch.bfloat16, device=DEV)
    ctx.register(recv)
    lay = ctx.layout(ids)
    ctx.dispatch(lay, x, recv)
    rows = lay.dst_row.view(-1).long()
    src = x.view(R * T, H).repeat_interleave(K, dim=0)
    assert torch.equal(recv[rows], src)                              # every item's row holds its token
    order = torch.argsort(ids.view(-1).long() * (R * T * K) + torch.arange(R * T * K, device=DEV))
    assert torch.equal(rows[order], torch.arange(R * T * K, device=DEV))   # expert, then item order
    y = (recv.float() * 1.5).to(torch.bfloat16)
    out = torch.empty((R, T, H), dtype=torch.bfloat16, device=DEV)
    ctx.combine(lay, y, w, out)
    want = (y[rows].float().view(R * T, K, H) * w.view(R * T, K, 1)).sum(dim=1).to(torch.bfloat16).view(R, T, H)
    a, b = out.view(torch.int16).cpu().numpy().view(np.uint16), want.view(torch.int16).cpu().numpy().view(np.uint16)
    assert ulp_distance(a, b).max() <= 1
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


@pytest.mark.parametrize("kw,tokens", [
    (dict(R=4, T=30, H=256, E=8, K=3), [30, 7, 0, 19]),
    (dict(R=8, T=1200, H=64, E=32, K=4), [1200, 1, 600, 0, 1199, 37, 1200, 900]),     # tiled layout path
    (dict(R=2, T=5, H=64, E=4, K=2), [9, -3]),                                         # above T, below 0
], ids=lambda v: str(len(v)) if isinstance(v, list) else "R{R}T{T}E{E}K{K}".format(**v))
def test_ragged_ranks_through_the_mask_call(kw, tokens):
    """Per-rank token counts: mask, layout, dispatch, combine; the real tokens behave as in the compacted batch."""
    cfg = wl.shrink(wl.CONFIGS["tiny"], seed=4242, **kw)
    inp = wl.generate(cfg)
    tpr = np.array(tokens, np.int32)
    want_ids = oracle.mask_ragged(inp["ids"], tpr)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, allow_unrouted=True)
    ids_d = to_dev(inp["ids"].copy())
    ctx.mask_ragged(to_dev(tpr), ids_d)
    torch.cuda.synchronize()
    assert np.array_equal(ids_d.cpu().numpy(), want_ids)
    ref = oracle.layout(want_ids, cfg.E, allow_unrouted=True)
    lay = ctx.layout(ids_d)
    for key in ("expert_count", "expert_offset", "rank_count", "rank_offset", "src_expert_count", "dst_row"):
        assert np.array_equal(getattr(lay, key).cpu().numpy().ravel(), ref[key].ravel()), key
    n_rows = int(ref["expert_offset"][-1])
    recv = torch.full((cfg.n_items, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    ctx.register(recv)
    ctx.dispatch(lay, to_dev(inp["x"]), recv)
    out = torch.full((cfg.n_tok, cfg.H), SENTINEL16, dtype=torch.int16, device=DEV)
    ctx.combine(lay, recv, to_dev(inp["w"]), out)
    torch.cuda.synchronize()
    want_recv = oracle.dispatch_bf16(ref["dst_row"], inp["x"], n_rows=cfg.n_items)
    got = u16(recv)
    assert np.array_equal(got[:n_rows], want_recv[:n_rows]) and np.all(got[n_rows:] == SENTINEL16)
    want_out = oracle.combine(ref["dst_row"], want_recv, inp["w"])
    assert np.array_equal(u16(out), want_out)
    pad = (want_ids.reshape(cfg.n_tok, cfg.K) < 0).all(axis=1)
    assert np.all(u16(out)[pad] == 0)                       # padding tokens combine to zero rows
    assert ctx.device_status() == B.STRATA_OK
    # without the flag the call is refused
    plain = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    assert B.strata_moe_mask_ragged(plain.h, to_dev(tpr).data_ptr(), ids_d.data_ptr(), None) == B.STRATA_ERR_SHAPE
    plain.close()
    ctx.close()
