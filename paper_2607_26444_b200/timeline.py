"""Post-processing of the in-kernel event timeline (paper Sec. 6.4): spans from the C decoder, per-kernel
stage shares, and a Chrome trace-event export.  Host-side numpy only; nothing here touches the GPU path."""
from __future__ import annotations

import ctypes

from .binding import StrataError, STRATA_OK, strata_span, strata_timeline_decode

STAGE_NAMES = {0: "kernel", 1: "wait_in", 2: "work", 3: "wait_out"}
KERNEL_NAMES = {1: "dispatch_bf16", 2: "dispatch_fp8", 3: "combine", 4: "dispatch_windows", 5: "slice_copy",
                6: "slice_reduce"}


def _check(rc: int, where: str) -> None:
    if rc != STRATA_OK:
        raise StrataError(rc, where)


def decode_timeline(buf):
    """buf: numpy uint64 [n_ctas, 1 + events_per_cta] (a host copy of a timeline buffer).
    Returns (spans, dropped): spans is a numpy structured array (cta, kernel, stage, flags, begin_ns, end_ns)."""
    import numpy as np
    buf = np.ascontiguousarray(buf, dtype=np.uint64)
    n_ctas, width = buf.shape
    dt = np.dtype([("cta", np.uint32), ("kernel", np.uint8), ("stage", np.uint8), ("flags", np.uint16),
                   ("begin_ns", np.uint64), ("end_ns", np.uint64)], align=True)
    assert dt.itemsize == ctypes.sizeof(strata_span)
    rc, n, lost = strata_timeline_decode(buf.ctypes.data, n_ctas, width - 1, None, 0)
    _check(rc, "strata_timeline_decode")
    spans = np.zeros(n, dtype=dt)
    rc, n2, lost = strata_timeline_decode(buf.ctypes.data, n_ctas, width - 1, spans.ctypes.data if n else None, n)
    _check(rc, "strata_timeline_decode")
    assert n2 == n
    return spans, lost


def timeline_summary(spans) -> dict:
    """Per kernel: CTAs, wall time from the first begin to the last end, spread of the CTAs' finish times,
    and per stage the number of intervals, their total time and its share of the CTAs' lifetimes."""
    import numpy as np
    out = {}
    for k in np.unique(spans["kernel"]):
        sk = spans[(spans["kernel"] == k) & (spans["flags"] == 0)]
        life = sk[sk["stage"] == 0]
        if life.size == 0:
            continue
        t0, t1 = int(life["begin_ns"].min()), int(life["end_ns"].max())
        busy = float((life["end_ns"] - life["begin_ns"]).sum())
        ent = {"ctas": int(np.unique(life["cta"]).size), "launches_per_cta": float(life.size) / np.unique(life["cta"]).size,
               "wall_us": (t1 - t0) / 1e3,
               "finish_spread": float(int(life["end_ns"].max()) - int(life["end_ns"].min())) / max(1, t1 - t0),
               "stages": {}}
        for st in np.unique(sk["stage"]):
            if st == 0:
                continue
            ss = sk[sk["stage"] == st]
            tot = float((ss["end_ns"] - ss["begin_ns"]).sum())
            ent["stages"][STAGE_NAMES.get(int(st), str(int(st)))] = {
                "intervals": int(ss.size), "total_us": tot / 1e3, "share_of_cta_time": tot / busy if busy else 0.0,
                "mean_ns": tot / ss.size}
        out[KERNEL_NAMES.get(int(k), str(int(k)))] = ent
    return out


def timeline_chrome_trace(spans, path: str, max_ctas: int = 64) -> int:
    """Writes the spans of the first max_ctas CTAs as a Chrome trace-event JSON file (one process per
    kernel, one thread per CTA, microseconds from the first event); returns the number of events written."""
    import json
    import numpy as np
    sel = spans[(spans["cta"] < max_ctas) & (spans["flags"] == 0)]
    if sel.size == 0:
        with open(path, "w") as f:
            json.dump({"traceEvents": []}, f)
        return 0
    t0 = int(sel["begin_ns"].min())
    ev = [{"name": STAGE_NAMES.get(int(s["stage"]), str(int(s["stage"]))), "ph": "X",
           "pid": KERNEL_NAMES.get(int(s["kernel"]), str(int(s["kernel"]))), "tid": int(s["cta"]),
           "ts": (int(s["begin_ns"]) - t0) / 1e3, "dur": (int(s["end_ns"]) - int(s["begin_ns"])) / 1e3} for s in sel]
    with open(path, "w") as f:
        json.dump({"traceEvents": ev, "displayTimeUnit": "ns"}, f)
    return len(ev)


def trace_summary(rec) -> dict:
    """rec: numpy int64 [capacity, 4] = (start_ns, end_ns, wait_in_ns, wait_out_ns) per CTA, as the per-CTA
    stage probes leave it: kernel time, finish-time spread and the shares of the two waits."""
    import numpy as np
    used = rec[rec[:, 0] != 0]
    if used.shape[0] == 0:
        return {"ctas": 0}
    start, end = used[:, 0], used[:, 1]
    total = float(end.max() - start.min())
    busy = (end - start).astype(np.float64)
    return {"ctas": int(used.shape[0]), "kernel_us": total / 1e3,
            "finish_spread": float(end.max() - end.min()) / total,
            "wait_in_share": float((used[:, 2] / busy).mean()),
            "wait_out_share": float((used[:, 3] / busy).mean())}
