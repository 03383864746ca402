"""Host-side decoding of the per-CTA event timeline (paper Sec. 6.4: per-core slices of a trace buffer,
decoded into per-core timelines).  Buffers are built here with the bit layout the header documents."""
import json

import numpy as np

from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import timeline as TL

K_DISP, K_COMB = 1, 3
KERNEL, WAIT_IN, WORK, WAIT_OUT = 0, 1, 2, 3


def ev(t, stage, end, kernel):
    return (t & ((1 << 48) - 1)) | (stage << 48) | (int(end) << 56) | (kernel << 57)


def make(slices, cap):
    buf = np.zeros((len(slices), 1 + cap), np.uint64)
    for b, (count, events) in enumerate(slices):
        buf[b, 0] = count
        buf[b, 1:1 + len(events)] = events
    return buf


def as_tuples(spans):
    return [(int(s["cta"]), int(s["kernel"]), int(s["stage"]), int(s["flags"]), int(s["begin_ns"]), int(s["end_ns"]))
            for s in spans]


def test_nested_stages_and_two_kernels_in_one_slice():
    e = [ev(100, KERNEL, 0, K_DISP), ev(110, WAIT_IN, 0, K_DISP), ev(150, WAIT_IN, 1, K_DISP),
         ev(150, WORK, 0, K_DISP), ev(170, WORK, 1, K_DISP), ev(400, KERNEL, 1, K_DISP),
         ev(500, KERNEL, 0, K_COMB), ev(510, WORK, 0, K_COMB), ev(590, WORK, 1, K_COMB), ev(600, KERNEL, 1, K_COMB)]
    spans, dropped = TL.decode_timeline(make([(len(e), e), (0, [])], cap=16))
    assert dropped == 0
    assert as_tuples(spans) == [(0, K_DISP, WAIT_IN, 0, 110, 150), (0, K_DISP, WORK, 0, 150, 170),
                                (0, K_DISP, KERNEL, 0, 100, 400), (0, K_COMB, WORK, 0, 510, 590),
                                (0, K_COMB, KERNEL, 0, 500, 600)]


def test_overflow_is_counted_and_unclosed_begins_are_flagged():
    e = [ev(10, KERNEL, 0, K_DISP), ev(20, WORK, 0, K_DISP), ev(30, WORK, 1, K_DISP), ev(40, WORK, 0, K_DISP)]
    # the kernel counted 9 events but the slice holds 4
    spans, dropped = TL.decode_timeline(make([(9, e)], cap=4))
    assert dropped == 5
    assert as_tuples(spans) == [(0, K_DISP, WORK, 0, 20, 30), (0, K_DISP, KERNEL, 1, 10, 10),
                                (0, K_DISP, WORK, 1, 40, 40)]


def test_end_without_begin():
    spans, _ = TL.decode_timeline(make([(1, [ev(77, WAIT_OUT, 1, K_COMB)])], cap=2))
    assert as_tuples(spans) == [(0, K_COMB, WAIT_OUT, 2, 77, 77)]


def test_timer_wrap_is_unrolled():
    top = (1 << 48) - 50
    e = [ev(top, KERNEL, 0, K_DISP), ev(30, KERNEL, 1, K_DISP)]          # the 48-bit stamp wrapped in between
    spans, _ = TL.decode_timeline(make([(2, e)], cap=2))
    assert as_tuples(spans) == [(0, K_DISP, KERNEL, 0, top, (1 << 48) + 30)]


def test_slices_are_independent_and_in_order():
    a = [ev(5, KERNEL, 0, K_COMB), ev(9, KERNEL, 1, K_COMB)]
    b = [ev(6, KERNEL, 0, K_COMB), ev(14, KERNEL, 1, K_COMB)]
    spans, _ = TL.decode_timeline(make([(2, a), (0, []), (2, b)], cap=3))
    assert as_tuples(spans) == [(0, K_COMB, KERNEL, 0, 5, 9), (2, K_COMB, KERNEL, 0, 6, 14)]


def test_summary_and_chrome_trace(tmp_path):
    slices = []
    for cta in range(4):
        t0 = 1000 + cta
        e = [ev(t0, KERNEL, 0, K_DISP)]
        for u in range(3):
            base = t0 + 10 + 100 * u
            e += [ev(base, WAIT_IN, 0, K_DISP), ev(base + 40, WAIT_IN, 1, K_DISP),
                  ev(base + 40, WORK, 0, K_DISP), ev(base + 50, WORK, 1, K_DISP)]
        e.append(ev(t0 + 400 + 25 * cta, KERNEL, 1, K_DISP))
        slices.append((len(e), e))
    spans, dropped = TL.decode_timeline(make(slices, cap=32))
    s = TL.timeline_summary(spans)["dispatch_bf16"]
    assert s["ctas"] == 4 and s["launches_per_cta"] == 1.0
    assert abs(s["wall_us"] - (1003 + 400 + 75 - 1000) / 1e3) < 1e-9
    assert abs(s["finish_spread"] - (78 / 478)) < 1e-9                       # last end - first end over the wall time
    assert s["stages"]["wait_in"]["intervals"] == 12 and s["stages"]["wait_in"]["mean_ns"] == 40.0
    assert abs(s["stages"]["work"]["share_of_cta_time"] - (12 * 10) / (400 * 4 + 150)) < 1e-9
    path = tmp_path / "trace.json"
    n = TL.timeline_chrome_trace(spans, str(path), max_ctas=2)
    doc = json.loads(path.read_text())
    assert n == len(doc["traceEvents"]) == 2 * (1 + 6)
    assert {e["tid"] for e in doc["traceEvents"]} == {0, 1}
    assert min(e["ts"] for e in doc["traceEvents"]) == 0.0


def test_setter_checks_arguments_on_a_host_only_context():
    rc, h = B.strata_ctx_create(B.strata_moe_shape(4, 128, 1024, 16, 2, B.STRATA_BF16), -1)
    assert rc == B.STRATA_OK
    try:
        assert B.strata_ctx_set_timeline(h, 1 << 20, 16, 64) == B.STRATA_OK
        assert B.strata_ctx_set_timeline(h, (1 << 20) + 4, 16, 64) == B.STRATA_ERR_ALIGNMENT
        assert B.strata_ctx_set_timeline(h, 1 << 20, 0, 64) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_ctx_set_timeline(h, 1 << 20, 16, 0) == B.STRATA_ERR_INVALID_ARG
        assert B.strata_ctx_set_timeline(h, None, 0, 0) == B.STRATA_OK
        assert B.strata_timeline_decode(None, 1, 1, None, 0)[0] == B.STRATA_ERR_INVALID_ARG
    finally:
        B.strata_ctx_destroy(h)
