"""GPU-vs-oracle parity of the full-mesh collectives over emulated ranks, through the C ABI.

Every operator is bit-exact: the data-movement operators copy bytes, and the reductions run the
same binary32 additions in rank order on both sides.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
SENT8 = 0xA5
GUARD = 64          # guard bytes on both sides of every output
CHUNK = 16384       # bytes one unit of the copy kernel moves


@pytest.fixture(scope="module")
def ctx():
    c = B.MoEContext(4, 128, 1024, 16, 2)
    yield c
    assert c.device_status() == B.STRATA_OK
    c.close()


def payload_bytes(R: int, n: int, seed: int) -> np.ndarray:
    return wl.gen_payload(R, n // 2, seed).view(np.uint8).reshape(R, n)


def guarded_out(nbytes: int):
    whole = torch.full((nbytes + 2 * GUARD,), SENT8, dtype=torch.uint8, device=DEV)
    return whole, whole[GUARD:GUARD + nbytes]


def guards_intact(whole) -> bool:
    h = whole.cpu().numpy()
    return bool(np.all(h[:GUARD] == SENT8) and np.all(h[-GUARD:] == SENT8))


COPY_SHAPES = [(1, 16), (2, 16), (4, 4096), (5, CHUNK), (3, CHUNK + 16), (7, 2 * CHUNK + 48),
               (16, 3 * CHUNK - 16), (32, 5 * CHUNK + 160)]


@pytest.mark.parametrize("R,n", COPY_SHAPES)
def test_allgather(ctx, R, n):
    x = payload_bytes(R, n, seed=R * 1000 + n)
    whole, out = guarded_out(R * R * n)
    ctx.allgather(torch.from_numpy(x).to(DEV), out.view(R, R, n))
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().reshape(R, R, n), oracle.allgather(x))
    assert guards_intact(whole)


@pytest.mark.parametrize("R,n", COPY_SHAPES)
def test_alltoall(ctx, R, n):
    x = payload_bytes(R, R * n, seed=R * 1000 + n + 1).reshape(R, R, n)
    whole, out = guarded_out(R * R * n)
    ctx.alltoall(torch.from_numpy(x).to(DEV), out.view(R, R, n))
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().reshape(R, R, n), oracle.alltoall(x))
    assert guards_intact(whole)


@pytest.mark.parametrize("R,n,root", [(1, 16, 0), (4, 4096, 3), (5, CHUNK + 16, 2), (32, 3 * CHUNK + 32, 17)])
def test_broadcast(ctx, R, n, root):
    x = payload_bytes(R, n, seed=R + n)
    whole, out = guarded_out(R * n)
    ctx.broadcast(torch.from_numpy(x).to(DEV), out.view(R, n), root)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().reshape(R, n), oracle.broadcast(x, root))
    assert guards_intact(whole)


# elements per slice: one vector; less than a CTA; several units with a ragged tail; many units
REDUCE_SHAPES = [(1, 8), (2, 8), (3, 1000), (5, 8 * 129), (8, 8 * (128 * 4 * 3 + 5)), (16, 8 * 4099),
                 (17, 8 * 523), (32, 8 * 2048), (64, 8 * 640)]


@pytest.mark.parametrize("R,S", REDUCE_SHAPES)
def test_reducescatter(ctx, R, S):
    x = wl.gen_payload(R, R * S, seed=R * 77 + S).reshape(R, R, S)
    whole, out = guarded_out(R * S * 2)
    ctx.reducescatter(torch.from_numpy(x.view(np.int16)).to(DEV), out.view(torch.int16).view(R, S))
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16).reshape(R, S)
    assert np.array_equal(got, oracle.reducescatter(x))
    assert guards_intact(whole)


@pytest.mark.parametrize("R,S", REDUCE_SHAPES)
def test_allreduce(ctx, R, S):
    x = wl.gen_payload(R, S, seed=R * 79 + S)
    whole, out = guarded_out(R * S * 2)
    ctx.allreduce(torch.from_numpy(x.view(np.int16)).to(DEV), out.view(torch.int16).view(R, S))
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16).reshape(R, S)
    assert np.array_equal(got, oracle.allreduce(x))
    assert guards_intact(whole)


def test_reduction_order_is_the_rank_order(ctx):
    # 2^20 + 2^-5 - 2^20 is 0 in binary32 when added in this order and 2^-5 in any order that cancels first
    R, S = 3, 8
    x = np.zeros((R, S), np.uint16)
    x[:, 0] = [0x4980, 0x3D00, 0xC980]
    x[:, 1] = [0x4980, 0xC980, 0x3D00]
    x[:, 2] = [0x3F80, 0x3B80, 0x3B80]          # one rounding at the end: 1 + 2^-7
    x[:, 3] = [0x8000, 0x8000, 0x8000]          # +0 + (-0)... = +0
    out = torch.empty((R, S), dtype=torch.int16, device=DEV)
    ctx.allreduce(torch.from_numpy(x.view(np.int16)).to(DEV), out)
    got = out.cpu().numpy().view(np.uint16)
    assert got[0, :4].tolist() == [0x0000, 0x3D00, 0x3F81, 0x0000]
    assert np.array_equal(got, oracle.allreduce(x))


def test_zero_sized_calls_launch_nothing(ctx):
    before = ctx.launch_count()
    e8 = torch.empty((4, 0), dtype=torch.uint8, device=DEV)
    d = torch.empty((16,), dtype=torch.uint8, device=DEV)
    assert B.strata_allgather(ctx.h, 4, d.data_ptr(), d.data_ptr(), 0, None) == B.STRATA_OK
    assert B.strata_allreduce(ctx.h, 4, d.data_ptr(), d.data_ptr(), 0, None) == B.STRATA_OK
    assert ctx.launch_count() == before
    del e8


def test_back_to_back_calls_and_mixed_operators(ctx):
    """The work-claim counter returns to zero inside every kernel: operators of both kinds run back to
    back on one stream, many times, and every result matches."""
    R, n = 8, 3 * CHUNK + 64
    xb = payload_bytes(R, n, seed=5)
    xs = wl.gen_payload(R, R * 2048, seed=6)
    xb_d = torch.from_numpy(xb).to(DEV)
    xs_d = torch.from_numpy(xs.view(np.int16)).to(DEV)
    ag = torch.empty((R, R, n), dtype=torch.uint8, device=DEV)
    rs = torch.empty((R, 2048), dtype=torch.int16, device=DEV)
    ar = torch.empty((R, R * 2048), dtype=torch.int16, device=DEV)
    want_ag, want_rs, want_ar = oracle.allgather(xb), oracle.reducescatter(xs.reshape(R, R, 2048)), oracle.allreduce(xs)
    for rep in range(6):
        ag.fill_(0)
        rs.fill_(0)
        ar.fill_(0)
        ctx.allgather(xb_d, ag)
        ctx.reducescatter(xs_d.view(R, R, 2048), rs)
        ctx.allreduce(xs_d, ar)
        ctx.allgather(xb_d, ag)
        torch.cuda.synchronize()
        assert np.array_equal(ag.cpu().numpy(), want_ag), rep
        assert np.array_equal(rs.cpu().numpy().view(np.uint16), want_rs), rep
        assert np.array_equal(ar.cpu().numpy().view(np.uint16), want_ar), rep


def test_cuda_graph_replay(ctx):
    R, S = 8, 8 * 1500
    x_d = torch.empty((R, R * S), dtype=torch.int16, device=DEV)
    a2a = torch.empty((R, R, S), dtype=torch.int16, device=DEV)
    red = torch.empty((R, S), dtype=torch.int16, device=DEV)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):
            ctx.alltoall(x_d.view(R, R, S), a2a)
            ctx.reducescatter(a2a, red)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ctx.alltoall(x_d.view(R, R, S), a2a)
        ctx.reducescatter(a2a, red)
    for rep in range(3):
        x = wl.gen_payload(R, R * S, seed=300 + rep)
        x_d.copy_(torch.from_numpy(x.view(np.int16)).to(DEV))
        a2a.fill_(0)
        red.fill_(0)
        g.replay()
        torch.cuda.synchronize()
        t = oracle.alltoall(x.view(np.uint8).reshape(R, R, S * 2)).view(np.uint16).reshape(R, R, S)
        assert np.array_equal(a2a.cpu().numpy().view(np.uint16), t), rep
        assert np.array_equal(red.cpu().numpy().view(np.uint16), oracle.reducescatter(t)), rep


def test_full_size_sampled(ctx):
    """The largest shape the benchmark times (32 ranks, 16 MiB per rank), in the same launch configuration:
    sampled slices of the outputs against the oracle on the same samples."""
    R, M = 32, 16 << 20
    E = M // 2
    rng = np.random.default_rng(7)
    x_d = torch.empty((R, E), dtype=torch.int16, device=DEV)
    # bf16 N(0,1) generated on the device would not be the oracle's input: fill from a host-generated
    # block repeated with a per-rank, per-block xor so that no two slices are equal
    block = wl.gen_payload(1, 1 << 20, seed=99)[0].view(np.int16)
    blk_d = torch.from_numpy(block).to(DEV)
    for r in range(R):
        for b in range(E // block.size):
            x_d[r, b * block.size:(b + 1) * block.size] = blk_d ^ ((r * 8 + b) & 0x7F)
    torch.cuda.synchronize()

    def host_cols(cols):                       # the oracle's input for sampled columns, [R, len(cols)]
        return x_d[:, cols].cpu().numpy().view(np.uint16)

    # all-reduce and reduce-scatter: 4096 sampled 8-element vectors
    vec = np.unique(rng.integers(0, E // 8, size=4096))
    cols = (vec[:, None] * 8 + np.arange(8)[None, :]).ravel()
    cols_d = torch.from_numpy(cols).to(DEV)
    want = oracle.allreduce(np.ascontiguousarray(host_cols(cols_d)))
    out = torch.empty((R, E), dtype=torch.int16, device=DEV)
    ctx.allreduce(x_d, out)
    torch.cuda.synchronize()
    assert np.array_equal(out[:, cols_d].cpu().numpy().view(np.uint16), want)
    rs = torch.empty((E,), dtype=torch.int16, device=DEV)          # [R][E/R] flat
    ctx.reducescatter(x_d.view(R, R, E // R), rs.view(R, E // R))
    torch.cuda.synchronize()
    assert np.array_equal(rs[cols_d].cpu().numpy().view(np.uint16), want[0])
    assert torch.equal(rs, out[5])                                  # every rank's all-reduce image is the same sum
    del out, rs

    # all-to-all: every (receiver, sender) pair; the ends of every slice and sampled positions against the oracle
    a2a = torch.empty((R, R, E // R), dtype=torch.int16, device=DEV)
    ctx.alltoall(x_d.view(R, R, E // R), a2a)
    torch.cuda.synchronize()
    assert torch.equal(a2a, x_d.view(R, R, E // R).transpose(0, 1))
    pos = np.unique(np.concatenate([np.arange(8), np.arange(E // R - 8, E // R), rng.integers(0, E // R, size=256)]))
    pos_d = torch.from_numpy(pos).to(DEV)
    xin = np.ascontiguousarray(x_d.view(R, R, E // R)[:, :, pos_d].cpu().numpy()).view(np.uint8)
    assert np.array_equal(a2a[:, :, pos_d].cpu().numpy().view(np.uint8), oracle.alltoall(xin))
    del a2a

    # all-gather: 16 GiB of output; every rank's image must equal the concatenated input
    ag = torch.empty((R, R, E), dtype=torch.int16, device=DEV)
    ctx.allgather(x_d, ag)
    torch.cuda.synchronize()
    for r in (0, 13, 31):
        assert torch.equal(ag[r], x_d)
    samp = np.unique(rng.integers(0, E, size=2048))
    samp_d = torch.from_numpy(samp).to(DEV)
    want = oracle.allgather(np.ascontiguousarray(host_cols(samp_d)).view(np.uint8))
    got = ag[:, :, samp_d].cpu().numpy().view(np.uint8)
    assert np.array_equal(got, want)


# ---- all-to-all-v and point-to-point -----------------------------------------------------------

def run_alltoallv(ctx, x, sb, so, ro, out_stride, fill=0xEE):
    R = x.shape[0]
    whole = torch.full((R * out_stride + 2 * GUARD,), fill, dtype=torch.uint8, device=DEV)
    out = whole[GUARD:GUARD + R * out_stride].view(R, out_stride)
    ctx.alltoallv(torch.from_numpy(x).to(DEV), out, torch.from_numpy(sb).to(DEV), torch.from_numpy(so).to(DEV),
                  torch.from_numpy(ro).to(DEV))
    torch.cuda.synchronize()
    h = whole.cpu().numpy()
    assert np.all(h[:GUARD] == fill) and np.all(h[-GUARD:] == fill)
    return out.cpu().numpy()


@pytest.mark.parametrize("R,mean,seed", [(1, 64, 1), (2, 16, 2), (4, 4096, 3), (7, 3 * CHUNK, 4), (16, CHUNK + 4096, 5),
                                         (32, 2 * CHUNK, 6)])
def test_alltoallv_uneven_pairs(ctx, R, mean, seed):
    sb = wl.gen_pair_bytes(R, mean, seed=seed)
    so, ro, si, st = wl.packed_offsets(sb)
    so, ro, si, st = so + 16, ro + 48, si + 64, st + 96           # gaps nobody addresses
    x = payload_bytes(R, si, seed=seed + 40)
    got = run_alltoallv(ctx, x, sb, so, ro, st)
    want = np.full((R, st), 0xEE, np.uint8)
    assert oracle.alltoallv(x, want, sb, so, ro) == 0
    assert np.array_equal(got, want)
    assert ctx.device_status() == B.STRATA_OK


def test_alltoallv_one_heavy_pair_and_many_empty(ctx):
    R = 8
    sb = np.zeros((R, R), np.int64)
    sb[3, 5] = 40 * CHUNK + 16                                    # one pair carries almost everything
    sb[0, 0] = 16
    sb[7, 2] = CHUNK
    so, ro, si, st = wl.packed_offsets(sb)
    x = payload_bytes(R, si, seed=77)
    got = run_alltoallv(ctx, x, sb, so, ro, st)
    want = np.full((R, st), 0xEE, np.uint8)
    oracle.alltoallv(x, want, sb, so, ro)
    assert np.array_equal(got, want)


def test_alltoallv_all_empty_and_back_to_back(ctx):
    R = 4
    sb = np.zeros((R, R), np.int64)
    x = payload_bytes(R, 64, seed=78)
    for _ in range(3):
        got = run_alltoallv(ctx, x, sb, sb.copy(), sb.copy(), 64)
        assert np.all(got == 0xEE)
    sb2 = wl.gen_pair_bytes(R, 8 * CHUNK, seed=9)
    so, ro, si, st = wl.packed_offsets(sb2)
    x = payload_bytes(R, si, seed=79)
    want = np.full((R, st), 0xEE, np.uint8)
    oracle.alltoallv(x, want, sb2, so, ro)
    for _ in range(3):                                            # the claim counter re-arms itself every time
        assert np.array_equal(run_alltoallv(ctx, x, sb2, so, ro, st), want)
    assert ctx.device_status() == B.STRATA_OK


def test_alltoallv_bad_pairs_are_skipped_and_reported(ctx):
    R = 2
    x = payload_bytes(R, 256, seed=80)
    sb = np.array([[32, 128], [16, 24]], np.int64)                # (1 -> 1): 24 is not a multiple of 16
    so = np.array([[0, 192], [0, 32]], np.int64)                  # (0 -> 1): 192 + 128 > 256
    ro = np.array([[0, 32], [0, 128]], np.int64)
    got = run_alltoallv(ctx, x, sb, so, ro, 256)
    st = ctx.device_status()
    assert st in (B.STRATA_ERR_CAPACITY, B.STRATA_ERR_ALIGNMENT)
    want = np.full((R, 256), 0xEE, np.uint8)
    want[0, 0:32] = x[0, 0:32]                                    # (0 -> 0)
    want[0, 32:48] = x[1, 0:16]                                   # (1 -> 0)
    assert np.array_equal(got, want)
    assert ctx.device_status() == B.STRATA_OK                     # the status word was cleared
    sb_ok = np.array([[32, 0], [16, 0]], np.int64)
    assert np.array_equal(run_alltoallv(ctx, x, sb_ok, so, ro, 256), want)


def test_alltoallv_counts_from_a_kernel_on_the_same_stream(ctx):
    """The counts never visit the host: they are produced on the device right before the call."""
    R = 8
    sb = wl.gen_pair_bytes(R, 4 * CHUNK, seed=12)
    so, ro, si, st = wl.packed_offsets(sb)
    x = payload_bytes(R, si, seed=81)
    x_d = torch.from_numpy(x).to(DEV)
    half = torch.from_numpy(sb // 32 * 16).to(DEV)
    so_d, ro_d = torch.from_numpy(so).to(DEV), torch.from_numpy(ro).to(DEV)
    out = torch.full((R, st), 0xEE, dtype=torch.uint8, device=DEV)
    sb_d = half + half                                            # a device computation, no synchronisation
    ctx.alltoallv(x_d, out, sb_d, so_d, ro_d)
    torch.cuda.synchronize()
    want = np.full((R, st), 0xEE, np.uint8)
    oracle.alltoallv(x, want, (sb // 32 * 16) * 2, so, ro)
    assert np.array_equal(out.cpu().numpy(), want)


def test_alltoallv_rejects_on_the_host(ctx):
    d = torch.zeros((64, 64), dtype=torch.int64, device=DEV)
    b = torch.zeros((64 * 64,), dtype=torch.uint8, device=DEV)
    args = (b.data_ptr(), 64, b.data_ptr(), 64, d.data_ptr(), d.data_ptr(), d.data_ptr(), None)
    assert B.strata_alltoallv(ctx.h, 33, *args) == B.STRATA_ERR_SHAPE
    assert B.strata_alltoallv(ctx.h, 4, b.data_ptr(), 40, *args[2:]) == B.STRATA_ERR_SHAPE
    assert B.strata_alltoallv(ctx.h, 4, b.data_ptr(), 64, b.data_ptr(), 64, None, d.data_ptr(), d.data_ptr(), None) \
        == B.STRATA_ERR_INVALID_ARG


@pytest.mark.parametrize("R,n,src,dst", [(1, 16, 0, 0), (4, CHUNK + 32, 3, 1), (32, 3 * CHUNK, 5, 5)])
def test_p2p(ctx, R, n, src, dst):
    x = payload_bytes(R, n, seed=n + src)
    whole, out = guarded_out(R * n)
    ctx.p2p(torch.from_numpy(x).to(DEV), out.view(R, n), src, dst)
    torch.cuda.synchronize()
    want = np.full((R, n), SENT8, np.uint8)
    oracle.p2p(x, want, src, dst)
    assert np.array_equal(out.cpu().numpy().reshape(R, n), want)
    assert guards_intact(whole)


@pytest.mark.parametrize("seed", range(10))
def test_random_shapes_all_operators(ctx, seed):
    """Random rank counts and sizes (any multiple of 16 bytes / 8 elements), every operator against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    R = int(rng.integers(1, 33))
    n = int(rng.integers(1, 6000)) * 16                     # bytes per slice, up to 96 KB
    S = n // 2                                              # bf16 elements per slice
    xb = payload_bytes(R, R * n, seed=seed).reshape(R, R, n)
    x_d = torch.from_numpy(xb).to(DEV)
    out = torch.empty((R, R, n), dtype=torch.uint8, device=DEV)
    ctx.alltoall(x_d, out)
    assert np.array_equal(out.cpu().numpy(), oracle.alltoall(xb))
    small = np.ascontiguousarray(xb[:, 0, :])               # [R, n]
    ag = torch.empty((R, R, n), dtype=torch.uint8, device=DEV)
    ctx.allgather(torch.from_numpy(small).to(DEV), ag)
    assert np.array_equal(ag.cpu().numpy(), oracle.allgather(small))
    root = int(rng.integers(0, R))
    bc = torch.empty((R, n), dtype=torch.uint8, device=DEV)
    ctx.broadcast(torch.from_numpy(small).to(DEV), bc, root)
    assert np.array_equal(bc.cpu().numpy(), oracle.broadcast(small, root))
    xs = xb.view(np.uint16).reshape(R, R, S)
    # finite operands: clear the top exponent bit
    xs = (xs & np.uint16(0xBFFF)).astype(np.uint16)
    xs_d = torch.from_numpy(xs.view(np.int16)).to(DEV)
    rs = torch.empty((R, S), dtype=torch.int16, device=DEV)
    ctx.reducescatter(xs_d, rs)
    assert np.array_equal(rs.cpu().numpy().view(np.uint16), oracle.reducescatter(xs))
    ar = torch.empty((R, R * S), dtype=torch.int16, device=DEV)
    ctx.allreduce(xs_d.view(R, R * S), ar)
    assert np.array_equal(ar.cpu().numpy().view(np.uint16), oracle.allreduce(xs.reshape(R, R * S)))
    sb = wl.gen_pair_bytes(R, max(16, n // 4), seed=seed, skew=float(rng.uniform(0.0, 2.0)),
                           zero_frac=float(rng.uniform(0.0, 0.5)))
    so, ro, si, st = wl.packed_offsets(sb)
    xv = payload_bytes(R, si, seed=seed + 500)             # si is a multiple of 16
    got = run_alltoallv(ctx, xv, sb, so, ro, st)
    want = np.full((R, st), 0xEE, np.uint8)
    assert oracle.alltoallv(xv, want, sb, so, ro) == 0
    assert np.array_equal(got, want)
    assert ctx.device_status() == B.STRATA_OK
