"""The per-CTA event timeline on the GPU: probes record what the kernels did, change no result, and
never write outside a CTA's slice."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import timeline as TL
from paper_2607_26444_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
KERNEL, WAIT_IN, WORK, WAIT_OUT = 0, 1, 2, 3


def to_dev(a):
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).to(DEV)


def run_step(ctx, cfg, inp):
    ids_d, x_d, w_d = to_dev(inp["ids"]), to_dev(inp["x"]), to_dev(inp["w"])
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=DEV)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=DEV)
    ctx.register(recv)
    lay = ctx.layout(ids_d)
    ctx.dispatch(lay, x_d, recv)
    ctx.combine(lay, recv, w_d, out)
    torch.cuda.synchronize()
    return lay, recv, out


@pytest.mark.parametrize("pinned", [False, True], ids=["device_buffer", "pinned_host_buffer"])
def test_step_timeline(pinned):
    cfg = wl.shrink(wl.CONFIGS["decode"], R=8, T=256, H=2048, E=32, K=4, seed=9)
    inp = wl.generate(cfg)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    t = ctx.timeline(n_ctas=2048, events_per_cta=512, pinned=pinned)
    lay, recv, out = run_step(ctx, cfg, inp)
    spans, dropped = ctx.timeline_spans(t)
    ctx.timeline_off()
    assert dropped == 0 and np.all(spans["flags"] == 0)

    # results are what they are without probes
    ref = oracle.layout(inp["ids"], cfg.E)
    ref_recv = oracle.dispatch_bf16(ref["dst_row"], inp["x"])
    assert np.array_equal(recv.cpu().numpy().view(np.uint16), ref_recv)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.combine(ref["dst_row"], ref_recv, inp["w"]))

    disp = spans[spans["kernel"] == 1]
    comb = spans[spans["kernel"] == 3]
    assert set(np.unique(spans["kernel"])) == {1, 3}
    # dispatch: one WAIT_IN and one WORK interval per unit (a unit is a token here: rows fit one stage)
    assert int((disp["stage"] == WORK).sum()) == cfg.n_tok
    assert int((disp["stage"] == WAIT_IN).sum()) == cfg.n_tok
    life = disp[disp["stage"] == KERNEL]
    assert life.size == np.unique(life["cta"]).size                      # one lifetime per CTA
    # every stage interval lies inside its CTA's lifetime, and the stages of a CTA do not overlap
    for cta in np.unique(disp["cta"])[:16]:
        mine = disp[disp["cta"] == cta]
        lt = mine[mine["stage"] == KERNEL][0]
        inner = np.sort(mine[mine["stage"] != KERNEL], order="begin_ns")
        assert inner["begin_ns"].min() >= lt["begin_ns"] and inner["end_ns"].max() <= lt["end_ns"]
        assert np.all(inner["begin_ns"][1:] >= inner["end_ns"][:-1])
    # combine: WORK intervals cover every unit once; units = tokens x column parts
    works = int((comb["stage"] == WORK).sum())
    assert works % cfg.n_tok == 0 and works >= cfg.n_tok
    # combine started after dispatch ended (stream order)
    assert comb["begin_ns"].min() >= disp[disp["stage"] == KERNEL]["end_ns"].max()

    s = TL.timeline_summary(spans)
    assert s["dispatch_bf16"]["ctas"] == life.size
    assert 0.0 < s["dispatch_bf16"]["stages"]["wait_in"]["share_of_cta_time"] < 1.0
    assert 0.0 <= s["dispatch_bf16"]["finish_spread"] <= 1.0
    assert s["combine"]["wall_us"] > 0
    ctx.close()


def test_small_slices_count_what_they_drop_and_stay_inside():
    cfg = wl.shrink(wl.CONFIGS["decode"], R=4, T=512, H=1024, E=16, K=2, seed=10)
    inp = wl.generate(cfg)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K)
    n_ctas, cap = 64, 6                                                  # fewer slices than CTAs, tiny slices
    whole = torch.zeros((n_ctas + 2, 1 + cap), dtype=torch.int64, device=DEV)
    whole[0] = -1
    whole[-1] = -1
    assert B.strata_ctx_set_timeline(ctx.h, whole[1:-1].data_ptr(), n_ctas, cap) == B.STRATA_OK
    run_step(ctx, cfg, inp)
    B.strata_ctx_set_timeline(ctx.h, None, 0, 0)
    h = whole.cpu().numpy()
    assert np.all(h[0] == -1) and np.all(h[-1] == -1)                    # neighbours untouched
    spans, dropped = TL.decode_timeline(h[1:-1].view(np.uint64))
    assert dropped > 0
    assert np.all(h[1:-1, 0] >= cap)                                     # every slice was filled and kept counting
    assert spans["cta"].max() < n_ctas
    assert ctx.device_status() == B.STRATA_OK
    ctx.close()


def test_collectives_are_probed():
    ctx = B.MoEContext(4, 128, 1024, 16, 2)
    R, n = 8, 10 * 16384                     # enough 16 KB chunks that the launcher keeps that chunk size
    x = torch.from_numpy(wl.gen_payload(R, R * n // 2, seed=3).view(np.int16)).to(DEV)
    a2a = torch.empty_like(x)
    red = torch.empty((R, n // 2), dtype=torch.int16, device=DEV)
    t = ctx.timeline(n_ctas=2048, events_per_cta=256)
    ctx.alltoall(x.view(R, R, n // 2), a2a.view(R, R, n // 2))
    ctx.reducescatter(a2a.view(R, R, n // 2), red)
    spans, dropped = ctx.timeline_spans(t)
    ctx.timeline_off()
    assert dropped == 0 and set(np.unique(spans["kernel"])) == {5, 6}
    copy = spans[spans["kernel"] == 5]
    assert int((copy["stage"] == WORK).sum()) == R * R * 10               # one unit per 16 KB chunk
    want = oracle.reducescatter(oracle.alltoall(x.cpu().numpy().view(np.uint8).reshape(R, R, n)).view(np.uint16).reshape(R, R, n // 2))
    assert np.array_equal(red.cpu().numpy().view(np.uint16), want)
    ctx.close()
