#!/usr/bin/env python
"""Benchmark of the MoE layout -> dispatch -> combine path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One "step" is one pass of the whole hot path (routing layout, bf16 dispatch, gate-weighted combine)
over one batch of the prefill-shaped workload (R=16 emulated ranks, 4096 tokens per rank, hidden 7168,
256 experts, top-8; 7.5 GB receive buffer), with identity experts (combine reads the receive buffer).
The metric is effective HBM GB/s = algorithmic bytes of dispatch + combine per step / time per step.
Inputs are seeded synthetic data, resident in HBM before the timed region; the working set (8.4 GB)
is far larger than L2, so no explicit flush is needed between iterations.  The timed region holds the K steps and
nothing else; the per-kernel times of the roofline come from a second pass over (up to 50 of) the same steps with a CUDA event
between every two kernels (those events cost overlap, so that pass is reported beside the value, not as it).

Ranks are emulated inside one GPU, so with --gpus N every process runs an independent replica
(weak scaling, no collective on the data path); the value is the sum over replicas.

`--impl reference` times the CPU oracle (the plain definition of the path) on the host cores on a
bounded sample of the same workload.  It is a deliberately slow program: a baseline, not a target.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2607_26444_b200 import workloads as wl  # noqa: E402

METRIC = "dispatch+combine effective HBM GB/s (prefill shape)"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum and dram__bytes_write.sum per launch, captured with ncu on the prefill recipe shrunk to
# T=512 and to T=1024 tokens/rank (the full launch is too large to capture under the profiler).  Reads grow in
# proportion to T.  Writes are the algorithmic bytes minus a constant: the lines still dirty in the 126 MB L2
# when the kernel ends (dispatch 63 MB, combine 15 MB at both sizes), so the traffic of a full launch is the
# straight line through the two captures taken at T=4096, not 8 x the smaller capture
# (profiles/dram_traffic_prefill_T512_T1024.md).
NCU_CAPTURES = {
    # kernel: {tokens per rank: (bytes read, bytes written)}, means of the two captured launches
    "dispatch_bf16_kernel": {512: (117_736_064, 876_647_296), 1024: (235_501_568, 1_815_977_728)},
    "combine_kernel": {512: (940_062_976, 103_737_856), 1024: (1_880_134_016, 219_123_840)},
}


def ncu_traffic_bytes(kernel: str, tokens_per_rank: int):
    """DRAM bytes (read + written) of one launch at the prefill recipe with T = tokens_per_rank, on the line
    through the two captures; None for a kernel without captures."""
    cap = NCU_CAPTURES.get(kernel)
    if not cap:
        return None
    (t1, (r1, w1)), (t2, (r2, w2)) = sorted(cap.items())
    b1, b2 = r1 + w1, r2 + w2
    return int(round(b1 + (b2 - b1) * (tokens_per_rank - t1) / (t2 - t1)))


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------
# clocks: sampled through NVML during the timed region (read-only)
# ---------------------------------------------------------------------------------------

class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples = []           # (t, sm_mhz, reasons_mask)
        self.max_mhz = None
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                try:
                    phys = int(vis.split(",")[index])
                except Exception:
                    phys = index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.samples.append((time.perf_counter(), mhz, mask))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self, t0: float, t1: float):
        if self._h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if not inside and self.samples:      # timed region shorter than one period: nearest samples
            inside = sorted(self.samples, key=lambda s: min(abs(s[0] - t0), abs(s[0] - t1)))[:3]
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [name for bit, name in self.REASONS.items() if mask & bit and name != "gpu_idle"]
        med = float(np.median([s[1] for s in inside])) if inside else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(inside)}


# ---------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------

def oracle_sample_config(cfg: wl.MoEConfig, tokens_per_rank: int) -> wl.MoEConfig:
    return wl.shrink(cfg, T=min(cfg.T, tokens_per_rank))


def time_oracle(cfg: wl.MoEConfig, inp, reps: int, keep=None):
    """Times oracle layout+dispatch+combine (as it stands) on the given inputs, all host cores.
    keep: a dict that receives the last pass's dst_row, recv and out (for a comparison with the GPU's)."""
    import oracle
    cores = oracle.max_threads()
    best = None
    for i in range(reps):
        t0 = time.perf_counter()
        lay = oracle.layout(inp["ids"], cfg.E)
        recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"], nthreads=cores)
        out = oracle.combine(lay["dst_row"], recv, inp["w"], nthreads=cores)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
        if keep is not None and i == reps - 1:
            keep.update(dst_row=lay["dst_row"], recv=recv, out=out)
        del recv, out
    nbytes = cfg.dispatch_bytes() + cfg.combine_bytes()
    sample = (f"the whole workload (R={cfg.R} T={cfg.T} H={cfg.H} E={cfg.E} K={cfg.K}, seed {cfg.seed}); "
              f"layout+dispatch+combine, best of {reps}, OpenMP over tokens")
    return nbytes / best / 1e9, best, cores, sample


def run_reference(args, rank: int):
    if rank != 0:
        return
    import oracle
    cfg = wl.CONFIGS["prefill"]
    scfg = oracle_sample_config(cfg, 256)
    inp = wl.generate(scfg)
    cores = oracle.max_threads()
    nbytes = scfg.dispatch_bytes() + scfg.combine_bytes()
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        lay = oracle.layout(inp["ids"], scfg.E)
        recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"], nthreads=cores)
        oracle.combine(lay["dst_row"], recv, inp["w"], nthreads=cores)
        dt = time.perf_counter() - t0
        del recv
        if i >= args.warmup:
            times.append(dt)
    mean_t = float(np.mean(times))
    val = nbytes / mean_t / 1e9
    sample = (f"each step: R={scfg.R} T={scfg.T} of {cfg.T} tokens/rank (same recipe, seed {scfg.seed}), H={scfg.H} "
              f"E={scfg.E} K={scfg.K}; oracle layout+dispatch+combine, OpenMP over tokens")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "prefill: R=16 emulated ranks, T=4096 tokens/rank, H=7168 bf16, E=256, K=8 "
                               "uniform distinct experts, softmax gates, identity experts (combine reads recv)",
                   "note": "each step is a bounded sample of the workload on the host cores"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# replicas: the only cross-rank logic (no collective touches the data path)
# ---------------------------------------------------------------------------------------

def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what the whole job took."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_replica_step: int, ms_per_step: float, world: int) -> float:
    """Aggregate throughput of `world` independent replicas that all finish within ms_per_step."""
    return world * bytes_per_replica_step / (ms_per_step * 1e-3) / 1e9


# ---------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------

class DeviceCase:
    """Device-resident buffers of one configuration (inputs uploaded once)."""

    def __init__(self, cfg: wl.MoEConfig, dev_index: int, inp=None):
        import torch
        from paper_2607_26444_b200 import binding as B
        self.torch, self.B, self.cfg = torch, B, cfg
        dev = torch.device("cuda", dev_index)
        self.dev = dev
        inp = inp or wl.generate(cfg)
        self.inp = inp
        self.ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, cfg.dispatch_dtype, device=dev_index)
        # x exists before routing starts (here: before the first step), so dispatch may read it while the layout runs
        self.ctx.x_early(True)
        self.ids = torch.from_numpy(inp["ids"]).to(dev)
        self.x = torch.from_numpy(inp["x"].view(np.int16)).to(dev)
        self.w = torch.from_numpy(inp["w"]).to(dev)
        self.lay = self.ctx.new_layout(with_optional=False)
        fp8 = cfg.dispatch_dtype == wl.FP8_E4M3_B128
        n = cfg.n_items
        row = cfg.H if fp8 else cfg.H * 2
        slab_bytes = n * row + (n * (cfg.H // 128) * 4 if fp8 else 0) + 8192
        self.slab = torch.empty(slab_bytes, dtype=torch.uint8, device=dev)
        rid = self.ctx.register(self.slab)
        if fp8:
            self.recv = self.ctx.carve(rid, (n, cfg.H), torch.uint8)
            self.recv_scale = self.ctx.carve(rid, (n, cfg.H // 128), torch.float32)
            self.y = torch.empty((n, cfg.H), dtype=torch.int16, device=dev)      # bf16 expert outputs
            self.y.copy_(self.x.view(cfg.n_tok, cfg.H).repeat_interleave(cfg.K, dim=0))
        else:
            self.recv = self.ctx.carve(rid, (n, cfg.H), torch.int16)
            self.recv_scale = None
            self.y = self.recv                                                   # identity experts, zero copy
        self.out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=dev)

    def layout(self):
        self.ctx.layout(self.ids, self.lay)

    def dispatch(self):
        self.ctx.dispatch(self.lay, self.x, self.recv, self.recv_scale)

    def combine(self):
        self.ctx.combine(self.lay, self.y, self.w, self.out)

    def step(self):
        self.layout()
        self.dispatch()
        self.combine()

    def check(self):
        """Device status clean, and (bf16, identity experts) the timed buffers hold the right answer:
        every receive row equals its source row, and combine returned x (gate weights sum to 1)."""
        torch = self.torch
        st = self.ctx.device_status()
        if st != 0:
            raise RuntimeError(f"device status {st}: {self.B.strata_status_string(st)}")
        if self.y is self.recv:
            cfg = self.cfg
            x2 = self.x.view(cfg.n_tok, cfg.H)
            if not bool((self.out.view(torch.bfloat16) == x2.view(torch.bfloat16)).all()):
                raise RuntimeError("combine output differs from x")
            dst = self.lay.dst_row.view(cfg.n_tok, cfg.K)
            sample = torch.arange(0, cfg.n_tok, max(1, cfg.n_tok // 4096), device=self.dev)
            for k in range(cfg.K):
                if not torch.equal(self.recv[dst[sample, k].long()], x2[sample]):
                    raise RuntimeError("a receive row differs from its source row")
        return True


def per_call_us(case: DeviceCase, iters: int = 30, warmup: int = 3):
    """Median microseconds per call of each entry point (events on the calls' stream)."""
    torch = case.torch
    out = {}
    def layout_dispatch():
        case.layout()
        case.dispatch()

    for name, fn in (("layout", case.layout), ("dispatch", case.dispatch), ("combine", case.combine),
                     ("layout+dispatch", layout_dispatch), ("step", case.step)):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        # Hold the stream for ~5 ms so that every call below is already queued when the first one
        # runs: the events then bracket device time, not the host's enqueue pace.
        torch.cuda._sleep(10_000_000)
        ev[0].record()
        for i in range(iters):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
        out[name] = {"median_us": ts[len(ts) // 2], "min_us": ts[0], "p95_us": ts[int(0.95 * (len(ts) - 1))]}
        # the same calls with no event between them (an event record between two short kernels adds to both
        # and keeps the next launch from overlapping the tail of the previous kernel; events tick in ~2 us steps)
        torch.cuda._sleep(10_000_000)
        ev[0].record()
        for i in range(iters):
            fn()
        ev[1].record()
        torch.cuda.synchronize()
        out[name]["back_to_back_us"] = ev[0].elapsed_time(ev[1]) * 1e3 / iters
    # what the bracket itself costs: a one-element torch fill between two events, timed the same way
    one = torch.zeros(1, device=case.dev)
    for _ in range(warmup):
        one.zero_()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda._sleep(10_000_000)
    ev[0].record()
    for i in range(iters):
        one.zero_()
        ev[i + 1].record()
    torch.cuda.synchronize()
    ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
    out["null_kernel"] = {"median_us": ts[len(ts) // 2], "min_us": ts[0], "p95_us": ts[int(0.95 * (len(ts) - 1))]}
    # the same three calls captured once in a CUDA graph and replayed (launch overhead paid once)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        case.step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        case.step()
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda._sleep(10_000_000)
    ev[0].record()
    for i in range(iters):
        graph.replay()
        ev[i + 1].record()
    torch.cuda.synchronize()
    ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
    out["step_graph"] = {"median_us": ts[len(ts) // 2], "min_us": ts[0], "p95_us": ts[int(0.95 * (len(ts) - 1))]}
    return out


def cta_finish_spread(case: DeviceCase):
    """Per-CTA probes (global timer at CTA start/end): relative gap between the first and the last
    CTA to finish, (max_end - min_end) / (max_end - min_start), for dispatch and for combine."""
    torch = case.torch
    tr = case.ctx.trace(8192)
    out = {}
    for name, fn in (("dispatch", case.dispatch), ("combine", case.combine)):
        vals, stages = [], None
        for _ in range(5):
            tr.zero_()
            fn()
            torch.cuda.synchronize()
            summ = case.ctx.trace_summary(tr)
            vals.append(summ["finish_spread"])
            stages = summ
        out[name] = round(float(np.median(vals)), 4)
        if name == "dispatch":
            out["dispatch_issue_thread"] = {"waiting_for_rows_in": round(stages["wait_in_share"], 3),
                                            "waiting_for_rows_out": round(stages["wait_out_share"], 3)}
    case.ctx.trace_off()
    return out


def window_partitioning_report(cfg: wl.MoEConfig, dev_index: int, unit_rows: int, n_cores: int = 296):
    """The paper's static scheme (expert windows -> peer windows -> LPT-style task lists, Sec. 6.2) run on
    the same inputs as the default path: policy generation time, window-major dispatch time, predicted
    imbalance of the policy and measured per-CTA finish spread."""
    import torch
    from paper_2607_26444_b200 import binding as B
    dev = torch.device("cuda", dev_index)
    inp = wl.generate(cfg) if cfg.n_tok <= 20000 else None
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, device=dev_index)
    ids = torch.from_numpy(inp["ids"] if inp else wl.gen_topk_ids(cfg)).to(dev)
    x = (torch.from_numpy(inp["x"].view(np.int16)).to(dev) if inp
         else torch.randint(-30000, 30000, (cfg.n_tok, cfg.H), dtype=torch.int16, device=dev))
    lay = ctx.layout(ids)
    recv = torch.empty((cfg.n_items, cfg.H), dtype=torch.int16, device=dev)
    ctx.register(recv)
    # one tier (HBM is uniform): cost in ns, alpha = 1 us per unit, beta = 22 B/ns per core
    pol = B.make_policy([(1000, 22, unit_rows, n_cores)])
    part = ctx.partition(lay, pol, n_cores)
    torch.cuda.synchronize()

    def timeit(fn, iters=10):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        torch.cuda._sleep(10_000_000)
        ev[0].record()
        for i in range(iters):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
        return ts[len(ts) // 2]

    policy_us = timeit(lambda: ctx.partition(lay, pol, n_cores, part))
    win_us = timeit(lambda: ctx.dispatch_windows(lay, part, x, recv))
    tok_us = timeit(lambda: ctx.dispatch(lay, x, recv))
    load = part.core_load.cpu().numpy().astype(np.float64)
    tr = ctx.trace(2048)
    tr.zero_()
    ctx.dispatch_windows(lay, part, x, recv)
    torch.cuda.synchronize()
    rec = tr.cpu().numpy()
    used = rec[rec[:, 0] != 0]
    spread = float(used[:, 1].max() - used[:, 1].min()) / float(used[:, 1].max() - used[:, 0].min())
    ctx.trace_off()
    st = ctx.device_status()
    out = {"units": int(part.n_units.item()), "unit_rows": unit_rows, "cores": n_cores,
           "policy_us": round(policy_us, 1), "window_dispatch_us": round(win_us, 1),
           "window_dispatch_GBs": round(cfg.dispatch_bytes() / win_us / 1e3, 1),
           "token_dispatch_us": round(tok_us, 1),
           "predicted_imbalance_max_over_mean": round(float(load.max() / load.mean()), 4),
           "cta_finish_spread": round(spread, 4), "device_status": st}
    ctx.close()
    return out


def expert_chain_report(cfg: wl.MoEConfig, dev_index: int, tile_rows: int = 128, iters: int = 30):
    """layout -> dispatch -> in-place expert stand-in -> combine with segments aligned to tile_rows, all on the
    device: microseconds per call (30 calls between one pair of events) and the stand-in's effective GB/s
    (every occupied row read once and written once)."""
    import torch
    from paper_2607_26444_b200 import binding as B
    dev = torch.device("cuda", dev_index)
    inp = wl.generate(cfg) if cfg.n_tok <= 20000 else None
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, device=dev_index, segment_align=tile_rows)
    ctx.x_early(True)
    ids = torch.from_numpy(inp["ids"] if inp else wl.gen_topk_ids(cfg)).to(dev)
    x = (torch.from_numpy(inp["x"].view(np.int16)).to(dev) if inp
         else torch.randint(-30000, 30000, (cfg.n_tok, cfg.H), dtype=torch.int16, device=dev))
    w = torch.from_numpy(inp["w"] if inp else wl.gen_gate_weights(cfg)).to(dev)
    scale = (1.0 + torch.arange(cfg.E, dtype=torch.float32, device=dev) / cfg.E)
    bias = 0.01 * torch.arange(cfg.E, dtype=torch.float32, device=dev)
    recv = torch.zeros((ctx.recv_rows, cfg.H), dtype=torch.int16, device=dev)
    ctx.register(recv)
    out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16, device=dev)
    lay = ctx.new_layout(with_optional=False)
    calls = {
        "layout": lambda: ctx.layout(ids, lay),
        "dispatch": lambda: ctx.dispatch(lay, x, recv),
        "expert": lambda: ctx.expert_affine_inplace(lay, recv, scale, bias, tile_rows),
        "combine": lambda: ctx.combine(lay, recv, w, out),
    }

    parts = list(calls.values())

    def chain():
        for fn in parts:
            fn()
    calls["chain"] = chain
    chain()
    rep = {"workload": cfg.name, "tile_rows": tile_rows, "recv_rows": int(ctx.recv_rows), "us": {}}
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, fn in calls.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        torch.cuda._sleep(10_000_000)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        rep["us"][name] = round(a.elapsed_time(b) * 1e3 / iters, 2)
    rep["expert_GBs"] = round(2 * cfg.n_items * cfg.H * 2 / rep["us"]["expert"] / 1e3, 1)
    rep["device_status"] = ctx.device_status()
    ctx.close()
    return rep


def timeline_report(cfg: wl.MoEConfig, dev_index: int, trace_path: str = "", pinned: bool = False):
    """One step with the in-kernel event timeline on (paper Sec. 6.4): per kernel the CTA count, wall time,
    finish-time spread and the share of CTA time per stage.  Probes cost time: these are not bench numbers."""
    from paper_2607_26444_b200 import timeline as TL
    case = DeviceCase(cfg, dev_index)
    torch, B = case.torch, case.B
    for _ in range(3):
        case.step()
    torch.cuda.synchronize()
    units = cfg.n_tok * max(1, -(-cfg.H * 2 // 16384))
    cap = 16 + 8 * (units // 148 + 64)                       # 6 events per dispatch unit (one CTA per SM at least), with room to spare
    t = case.ctx.timeline(n_ctas=2048, events_per_cta=cap, pinned=pinned)
    case.step()
    spans, dropped = case.ctx.timeline_spans(t)
    case.ctx.timeline_off()
    case.check()
    rep = {"workload": cfg.name, "buffer": "pinned host" if pinned else "device", "events_per_cta": cap,
           "spans": int(spans.size), "events_dropped": int(dropped), "kernels": TL.timeline_summary(spans)}
    for k in rep["kernels"].values():
        k["wall_us"] = round(k["wall_us"], 2)
        k["finish_spread"] = round(k["finish_spread"], 4)
        for st in k["stages"].values():
            st["total_us"] = round(st["total_us"], 1)
            st["share_of_cta_time"] = round(st["share_of_cta_time"], 4)
            st["mean_ns"] = round(st["mean_ns"], 1)
    if trace_path:
        rep["chrome_trace_events"] = TL.timeline_chrome_trace(spans, trace_path, max_ctas=32)
    return rep


def sm_budget_report(cfg: wl.MoEConfig, dev_index: int, budgets=(8, 16, 24, 32, 48, 64, 96, 128, 0), iters: int = 10):
    """Dispatch and combine throughput against the SM budget of the persistent grids (how many SMs' worth of
    CTAs it takes to saturate HBM; the paper makes the same measurement for its fabric, Sec. 3.2)."""
    case = DeviceCase(cfg, dev_index)
    torch = case.torch
    case.layout()
    rows = []
    for b in budgets:
        case.ctx.sm_budget(b)
        ent = {"sm_budget": b if b else "all"}
        for name, fn, nbytes in (("dispatch", case.dispatch, cfg.dispatch_bytes()),
                                 ("combine", case.combine, cfg.combine_bytes())):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
            torch.cuda._sleep(10_000_000)
            ev[0].record()
            for i in range(iters):
                fn()
                ev[i + 1].record()
            torch.cuda.synchronize()
            ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
            ent[name + "_us"] = round(ts[len(ts) // 2], 1)
            ent[name + "_GBs"] = round(nbytes / ts[len(ts) // 2] / 1e3, 1)
        rows.append(ent)
    case.ctx.sm_budget(0)
    case.check()
    return {"workload": cfg.name, "iters": iters, "rows": rows}


def overlap_report(cfg: wl.MoEConfig, dev_index: int, budgets=(0, 64, 32), gemm_n: int = 8192, reps: int = 12):
    """Interference between the dispatch/combine kernels and a compute kernel on another stream (the paper
    reports the slowdown of computation under communication, Sec. 2.2).  The co-runner is a library bf16 GEMM
    (torch.matmul), used only as a load; times are per call, each side looping while the other runs."""
    case = DeviceCase(cfg, dev_index)
    torch = case.torch
    dev = case.dev
    a = torch.randn((gemm_n, gemm_n), dtype=torch.bfloat16, device=dev)
    b = torch.randn((gemm_n, gemm_n), dtype=torch.bfloat16, device=dev)
    c = torch.empty((gemm_n, gemm_n), dtype=torch.bfloat16, device=dev)
    s_comm, s_gemm = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    case.layout()
    torch.cuda.synchronize()

    def comm_loop(n):
        for _ in range(n):
            case.dispatch()
            case.combine()

    def gemm_loop(n):
        for _ in range(n):
            torch.matmul(a, b, out=c)

    def timed(stream, fn, n):
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(n)
            e1.record()
        return e0, e1

    for st_, fn in ((s_comm, comm_loop), (s_gemm, gemm_loop)):
        with torch.cuda.stream(st_):
            fn(2)
    torch.cuda.synchronize()
    e = timed(s_gemm, gemm_loop, reps)
    torch.cuda.synchronize()
    gemm_alone = e[0].elapsed_time(e[1]) / reps
    flops = 2.0 * gemm_n ** 3
    step_bytes = cfg.dispatch_bytes() + cfg.combine_bytes()
    rows = []
    for bud in budgets:
        case.ctx.sm_budget(bud)
        with torch.cuda.stream(s_comm):
            comm_loop(2)
        torch.cuda.synchronize()
        e = timed(s_comm, comm_loop, reps)
        torch.cuda.synchronize()
        comm_alone = e[0].elapsed_time(e[1]) / reps
        # both at once; the communication loop is made long enough to cover the GEMM loop and vice versa
        n_comm = max(reps, int(reps * gemm_alone / comm_alone * 1.5) + 1)
        n_gemm = max(reps, int(reps * comm_alone / gemm_alone * 1.5) + 1)
        ec = timed(s_comm, comm_loop, n_comm)
        eg = timed(s_gemm, gemm_loop, n_gemm)
        torch.cuda.synchronize()
        # the shorter loop ran entirely beside the other one: report it, and the slowdown it saw
        comm_t, gemm_t = ec[0].elapsed_time(ec[1]) / n_comm, eg[0].elapsed_time(eg[1]) / n_gemm
        rows.append({"sm_budget": bud if bud else "all",
                     "dispatch+combine_ms_alone": round(comm_alone, 3), "dispatch+combine_ms_beside_gemm": round(comm_t, 3),
                     "dispatch+combine_GBs_alone": round(step_bytes / comm_alone / 1e6, 1),
                     "dispatch+combine_GBs_beside_gemm": round(step_bytes / comm_t / 1e6, 1),
                     "gemm_ms_beside_comm": round(gemm_t, 3), "gemm_TFLOPs_beside_comm": round(flops / gemm_t / 1e9, 1),
                     "loops": [n_comm, n_gemm]})
    case.ctx.sm_budget(0)
    case.check()
    return {"workload": cfg.name, "gemm": f"bf16 {gemm_n}^3 (library kernel, load only)", "gemm_ms_alone": round(gemm_alone, 3),
            "gemm_TFLOPs_alone": round(flops / gemm_alone / 1e9, 1),
            "note": "both loops start together; per-call means include the part of the longer loop that ran alone",
            "rows": rows}


COLLECTIVE_OPS = ("allgather", "alltoall", "alltoallv", "broadcast", "reducescatter", "allreduce")


def collectives_report(dev_index: int, R: int = 32, per_rank_kib=(64, 1024, 16384), iters: int = 10,
                       warmup: int = 3, only=COLLECTIVE_OPS):
    """Full-mesh collectives over R emulated ranks (paper Sec. 6.1 / 8.1: 32 ranks, payloads from 1 MiB
    per rank): median microseconds and effective HBM GB/s of each operator.  Algorithmic bytes: the
    operator's input read once plus its output written once.  A working set below the 126 MB L2 is
    marked, its GB/s is not an HBM figure."""
    import torch
    from paper_2607_26444_b200 import binding as B
    dev = torch.device("cuda", dev_index)
    ctx = B.MoEContext(4, 128, 1024, 16, 2, device=dev_index)
    peak, _ = measured_peak()
    rep = {"R": R, "iters": iters, "bytes": "input read once + output written once", "sizes": {}}
    for kib in per_rank_kib:
        M = kib << 10                                   # bytes per rank
        E = M // 2                                      # bf16 elements per rank
        x = torch.empty((R, E), dtype=torch.int16, device=dev)
        x.view(torch.uint8).random_(0, 256)
        x &= 0x3FFF | -32768                            # finite bf16 patterns of magnitude < 2
        big = torch.empty((R, R, E), dtype=torch.int16, device=dev) if "allgather" in only else None
        same = torch.empty((R, E), dtype=torch.int16, device=dev)
        small = torch.empty((E,), dtype=torch.int16, device=dev)
        ops = {
            "allgather": (lambda: ctx.allgather(x, big), R * M + R * R * M),
            "alltoall": (lambda: ctx.alltoall(x.view(R, R, E // R), same.view(R, R, E // R)), 2 * R * M),
            "broadcast": (lambda: ctx.broadcast(x, same, 3), M + R * M),
            "reducescatter": (lambda: ctx.reducescatter(x.view(R, R, E // R), small.view(R, E // R)), R * M + M),
            "allreduce": (lambda: ctx.allreduce(x, same), 2 * R * M),
        }
        if "alltoallv" in only:
            # uneven pairs: Zipf(1.2) receiver popularity, 10 % empty pairs, same mean volume as the all-to-all
            pair = wl.gen_pair_bytes(R, M // R, seed=2000 + kib)
            so, ro, si, st = wl.packed_offsets(pair)
            vin = torch.empty((R, si), dtype=torch.uint8, device=dev).random_(0, 256)
            vout = torch.empty((R, st), dtype=torch.uint8, device=dev)
            pair_d, so_d, ro_d = (torch.from_numpy(a).to(dev) for a in (pair, so, ro))
            ops["alltoallv"] = (lambda: ctx.alltoallv(vin, vout, pair_d, so_d, ro_d), 2 * int(pair.sum()))
        entry = {}
        for name, (fn, nbytes) in ops.items():
            if name not in only:
                continue
            for _ in range(warmup):
                fn()
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
            torch.cuda._sleep(10_000_000)
            ev[0].record()
            for i in range(iters):
                fn()
                ev[i + 1].record()
            torch.cuda.synchronize()
            ts = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters))
            med = ts[len(ts) // 2]
            # the same calls with no event between them: what a stream of such calls costs per call (an
            # event record between two short kernels adds to both, and events tick in ~2 us steps)
            torch.cuda._sleep(10_000_000)
            ev[0].record()
            for i in range(4 * iters):
                fn()
            ev[1].record()
            torch.cuda.synchronize()
            entry[name] = {"median_us": round(med, 2), "min_us": round(ts[0], 2),
                           "back_to_back_us": round(ev[0].elapsed_time(ev[1]) * 1e3 / (4 * iters), 2), "bytes": nbytes,
                           "GBs": round(nbytes / med / 1e3, 1), "frac_of_measured_peak": round(nbytes / med / 1e3 / peak, 4),
                           "l2_resident": nbytes < 126_000_000}
        # the timed buffers hold what the operators define (checked with torch views; parity with the
        # oracle is the tests' job)
        ok = big is None or bool(torch.equal(big[R - 1], x))
        if "allreduce" in only or "broadcast" in only:
            ok = ok and bool(torch.equal(same, same[0].expand(R, E)))
        ctx.alltoall(x.view(R, R, E // R), same.view(R, R, E // R))
        ok = ok and bool(torch.equal(same.view(R, R, E // R), x.view(R, R, E // R).transpose(0, 1)))
        if "alltoallv" in only:
            p_, r_ = int(np.argmax(pair.sum(axis=1))), int(np.argmax(pair[int(np.argmax(pair.sum(axis=1)))]))
            n_ = int(pair[p_, r_])
            ok = ok and bool(torch.equal(vout[r_, ro[r_, p_]:ro[r_, p_] + n_], vin[p_, so[p_, r_]:so[p_, r_] + n_]))
            entry["alltoallv"]["max_over_mean_received"] = round(float(pair.sum(axis=0).max() / pair.sum(axis=0).mean()), 2)
            del vin, vout
        entry["verified"] = ok and ctx.device_status() == B.STRATA_OK
        rep["sizes"][f"{kib}KiB_per_rank"] = entry
        del x, big, same, small
        torch.cuda.empty_cache()
    ctx.close()
    return rep


def run_gpu(args, rank: int, local_rank: int, world: int):
    import torch
    import torch.distributed as dist
    from paper_2607_26444_b200 import binding as B

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device for its own arm (there is no CPU fallback)")
    B.lib()       # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()

    cfg = wl.CONFIGS[args.workload]
    if args.tokens_per_rank:
        cfg = wl.shrink(cfg, T=args.tokens_per_rank)
    if cfg.dispatch_dtype != wl.BF16:
        args.no_e2e = True            # the host round trip is defined for bf16 dispatch only
    case = DeviceCase(cfg, local_rank)
    host_inp = case.inp
    disp_bytes, comb_bytes = cfg.dispatch_bytes(), cfg.combine_bytes()
    step_bytes = disp_bytes + comb_bytes

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        case.step()
    torch.cuda.synchronize()
    case.check()

    K = args.steps
    rc0, n0 = B.strata_ctx_launch_count(case.ctx.h)
    barrier()
    torch.cuda.synchronize()
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev_a.record()
    for i in range(K):                       # the timed region: exactly K steps, nothing else in the stream
        case.layout()
        case.dispatch()
        case.combine()
    ev_b.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    barrier()
    rc1, n1 = B.strata_ctx_launch_count(case.ctx.h)
    case.check()
    elapsed_ms = ev_a.elapsed_time(ev_b)
    clocks = sampler.summary(t0, t1)

    elapsed_ms = max_over_ranks(elapsed_ms, world, "cuda")
    ms_per_step = elapsed_ms / K
    value = whole_job_gbs(step_bytes, ms_per_step, world)

    # Per-kernel durations for the roofline: the same steps once more (up to 50 of them) with an event between
    # every two kernels.  The events are not free (they keep a launch from overlapping the previous kernel's tail), so
    # this pass is slower than the timed region and is reported beside it, not as the bench value.
    KI = min(K, 50)                          # enough launches for an average; a long second pass only heats the board
    time.sleep(0.5)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(KI)]
    for i in range(KI):
        ev[i][0].record()
        case.layout()
        ev[i][1].record()
        case.dispatch()
        ev[i][2].record()
        case.combine()
        ev[i][3].record()
    torch.cuda.synchronize()
    case.check()
    instrumented_ms_per_step = ev[0][0].elapsed_time(ev[KI - 1][3]) / KI
    lay_ms = float(np.mean([ev[i][0].elapsed_time(ev[i][1]) for i in range(KI)]))
    disp_ms = float(np.mean([ev[i][1].elapsed_time(ev[i][2]) for i in range(KI)]))
    comb_ms = float(np.mean([ev[i][2].elapsed_time(ev[i][3]) for i in range(KI)]))

    # ---- end to end from host buffers through the C ABI (copies inside the timed region) ----
    e2e = None
    if not args.no_e2e:
        h_ids = torch.from_numpy(case.inp["ids"]).pin_memory()
        h_x = torch.from_numpy(case.inp["x"].view(np.int16)).pin_memory()
        h_w = torch.from_numpy(case.inp["w"]).pin_memory()
        h_out = torch.empty((cfg.n_tok, cfg.H), dtype=torch.int16).pin_memory()
        devbuf = B.strata_moe_device_buffers(case.ids.data_ptr(), case.x.data_ptr(), case.w.data_ptr(),
                                             case.recv.data_ptr(), case.out.data_ptr(), case.lay.c)
        stream = torch.cuda.current_stream().cuda_stream

        def e2e_step():
            rc = B.strata_moe_roundtrip_host(case.ctx.h, devbuf, h_ids.data_ptr(), h_x.data_ptr(),
                                             h_w.data_ptr(), h_out.data_ptr(), stream)
            if rc != 0:
                raise RuntimeError(f"roundtrip_host: {B.strata_status_string(rc)}")

        e2e_steps = max(3, min(10, K))
        for _ in range(2):
            e2e_step()
        barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(e2e_steps):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        barrier()
        e2e_ms = a.elapsed_time(b)
        e2e_ms = max_over_ranks(e2e_ms, world, "cuda") / e2e_steps
        h2d = h_ids.numel() * 4 + h_x.numel() * 2 + h_w.numel() * 4
        d2h = h_out.numel() * 2
        e2e = {"value": whole_job_gbs(step_bytes, e2e_ms, world), "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "strata_moe_roundtrip_host (pinned host buffers, copies in the timed region)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        sampler.stop()
        return

    peak, peak_src = measured_peak()
    traffic_ok = args.workload == "prefill"          # the captures are of this recipe
    disp_name = "dispatch_bf16_kernel" if cfg.dispatch_dtype == wl.BF16 else "dispatch_fp8_kernel"
    kernels = {
        disp_name: {"bytes": disp_bytes, "ms": disp_ms},
        "combine_kernel": {"bytes": comb_bytes, "ms": comb_ms},
    }
    for k, v in kernels.items():
        v["achieved"] = v["bytes"] / (v["ms"] * 1e-3) / 1e9
        v["frac"] = v["achieved"] / peak
        v["frac_of_nominal_8TBs"] = v["achieved"] / NOMINAL_HBM_GBS
    dom = max(kernels, key=lambda k: kernels[k]["ms"])
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["achieved"], "peak": peak,
                "peak_source": f"{peak_src} (MEASURED_PEAKS.json hbm_gbs)" if peak_src == "measured"
                else "fallback (recipe figure)",
                "unit": "GB/s", "frac": kernels[dom]["frac"],
                "traffic": ncu_traffic_bytes(dom, cfg.T) if traffic_ok else None,
                "traffic_source": "ncu dram__bytes read+write captured at T=512 and T=1024 tokens/rank, linear in T, "
                                  "taken at this T" if traffic_ok else None,
                "algorithmic_bytes_per_launch": kernels[dom]["bytes"],
                "frac_of_nominal_8TBs": round(kernels[dom]["frac_of_nominal_8TBs"], 4),
                "note": ("frac above 1: the denominator is a measured torch copy (1:1 read:write), and this kernel "
                         "outruns it") if kernels[dom]["frac"] > 1 else None,
                "kernels": {k: {"achieved": round(v["achieved"], 1), "frac": round(v["frac"], 4),
                                "frac_of_nominal_8TBs": round(v["frac_of_nominal_8TBs"], 4),
                                "avg_ms": round(v["ms"], 4),
                                "traffic": ncu_traffic_bytes(k, cfg.T) if traffic_ok else None}
                            for k, v in kernels.items()},
                "layout_avg_ms": round(lay_ms, 4),
                "how": f"per-kernel times: CUDA events between the kernels of a second pass of {KI} of the same steps; the "
                       "events keep launches from overlapping, that pass took "
                       f"{instrumented_ms_per_step:.4f} ms per step"}

    # ---- the oracle on the host cores: timed as a baseline, and its results compared with what the
    #      timed GPU steps left in their buffers (same inputs) ----
    cpu, oracle_check = None, None
    if not args.no_cpu:
        kept = {}
        gbs, dt, cores, sample = time_oracle(cfg, host_inp, reps=2, keep=kept)
        cpu = {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
               "seconds": round(dt, 3)}
        if cfg.dispatch_dtype == wl.BF16:
            got_out = case.out.cpu().numpy().view(np.uint16)
            a, b = got_out.astype(np.int32), kept["out"].reshape(got_out.shape).astype(np.int32)
            a = np.where(a & 0x8000, -(a & 0x7FFF), a & 0x7FFF)
            b = np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
            rows = np.arange(0, cfg.n_items, max(1, cfg.n_items // 8192))
            got_rows = case.recv[torch.from_numpy(rows).to(case.dev)].cpu().numpy().view(np.uint16)
            oracle_check = {
                "dst_row_equal": bool(np.array_equal(case.lay.dst_row.cpu().numpy(), kept["dst_row"])),
                "recv_rows_equal": bool(np.array_equal(got_rows, kept["recv"][rows])), "recv_rows_compared": int(rows.size),
                "combine_max_ulp": int(np.abs(a - b).max()), "combine_elements_compared": int(a.size)}
            if not (oracle_check["dst_row_equal"] and oracle_check["recv_rows_equal"]
                    and oracle_check["combine_max_ulp"] <= 1):
                raise RuntimeError(f"the timed buffers differ from the oracle: {oracle_check}")
            del a, b, got_out, got_rows
        kept.clear()
        # one thread, on a sixteenth of the tokens (same recipe)
        import oracle
        scfg = oracle_sample_config(cfg, max(1, cfg.T // 16))
        sinp = wl.generate(scfg)
        t0 = time.perf_counter()
        lay1 = oracle.layout(sinp["ids"], scfg.E)
        recv1 = oracle.dispatch_bf16(lay1["dst_row"], sinp["x"], nthreads=1)
        oracle.combine(lay1["dst_row"], recv1, sinp["w"], nthreads=1)
        dt1 = time.perf_counter() - t0
        del recv1
        cpu["single_thread"] = {"value": (scfg.dispatch_bytes() + scfg.combine_bytes()) / dt1 / 1e9, "unit": UNIT,
                                "sample": f"T={scfg.T} of {cfg.T} tokens/rank, one pass", "seconds": round(dt1, 3)}

    # ---- the other shapes: per-call microseconds (not bench lines, context for the metric) ----
    # The second half of the metric is the time per call at the decode shape: it gets a block of its own.
    other, decode_us = {}, None
    if not args.no_other:
        del case
        torch.cuda.empty_cache()
        for name in ("tiny", "decode", "skew", "fp8"):       # tiny is L2 resident: its GB/s are not HBM figures
            c = wl.CONFIGS[name]
            dc = DeviceCase(c, local_rank)
            us = per_call_us(dc)
            dc.check()
            db, cb = c.dispatch_bytes(), c.combine_bytes()
            other[name] = {
                "layout_us": round(us["layout"]["median_us"], 2),
                "dispatch_us": round(us["dispatch"]["median_us"], 2),
                "combine_us": round(us["combine"]["median_us"], 2),
                "step_us": round(us["step"]["median_us"], 2),
                "step_back_to_back_us": round(us["step"]["back_to_back_us"], 2),
            }
            if name == "decode":
                b2b = {k: round(v["back_to_back_us"], 2) for k, v in us.items() if "back_to_back_us" in v}
                decode_us = {
                    "layout": other[name]["layout_us"], "dispatch": other[name]["dispatch_us"],
                    "combine": other[name]["combine_us"],
                    "layout+dispatch": round(us["layout+dispatch"]["median_us"], 2), "step": other[name]["step_us"],
                    "step_cuda_graph": round(us["step_graph"]["median_us"], 2),
                    "back_to_back": {"layout": b2b["layout"], "dispatch": b2b["dispatch"], "combine": b2b["combine"],
                                     "layout+dispatch": b2b["layout+dispatch"], "step": b2b["step"]},
                    "of_measured_peak": {"dispatch": round(db / us["dispatch"]["median_us"] / 1e3 / peak, 3),
                                         "combine": round(cb / us["combine"]["median_us"] / 1e3 / peak, 3),
                                         "dispatch_back_to_back": round(db / b2b["dispatch"] / 1e3 / peak, 3),
                                         "combine_back_to_back": round(cb / b2b["combine"] / 1e3 / peak, 3)},
                    "min_p95": {k: [round(us[k]["min_us"], 2), round(us[k]["p95_us"], 2)]
                                for k in ("layout", "dispatch", "combine", "step")},
                    "null_kernel_between_events": round(us["null_kernel"]["median_us"], 2),
                    "both_copies_at_measured_peak_us": round((db + cb) / peak / 1e3, 1),
                    "how": "median of 30 calls, each between two CUDA events (null_kernel_between_events: a one-element "
                           "fill timed the same way, i.e. what the bracket itself costs); back_to_back: 30 calls "
                           "between one pair of events; step = layout + dispatch + combine",
                }
            if name == "skew":
                # load balance under Zipf routing: per-CTA finish-time spread, and the same shape with
                # uniform routing for comparison
                sp = cta_finish_spread(dc)
                other[name]["cta_finish_spread"] = {"dispatch": sp["dispatch"], "combine": sp["combine"]}
                del dc
                torch.cuda.empty_cache()
                uc = DeviceCase(wl.shrink(c, routing="uniform"), local_rank)
                uu = per_call_us(uc)
                other["skew_shape_uniform_routing"] = {
                    "dispatch_us": round(uu["dispatch"]["median_us"], 2),
                    "combine_us": round(uu["combine"]["median_us"], 2),
                }
                dc = uc
            del dc
            torch.cuda.empty_cache()

    sampler.stop()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: R={cfg.R} emulated ranks, T={cfg.T} tokens/rank, H={cfg.H} bf16, "
                               f"E={cfg.E}, K={cfg.K} {cfg.routing} distinct experts, softmax gates, "
                               + ("identity experts (combine reads recv)" if cfg.dispatch_dtype == wl.BF16
                                  else "e4m3 dispatch, bf16 expert outputs"),
                   "step": "strata_moe_layout + strata_moe_dispatch + strata_moe_combine (x_early promise on: x is "
                           "complete before the layout call)",
                   "bytes_per_step": step_bytes, "l2": "inputs larger than L2 (8.4 GB working set), no flush",
                   "parallelism": "replicas only" if world > 1 else "1 GPU, 16 ranks emulated in HBM"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(n1 - n0), "roofline": roofline,
        "verified": "after the timed steps: device status clean, out == x, sampled receive rows == source rows",
        "oracle_check": oracle_check,
        "pct_of_8TBs": {"dispatch": round(100 * kernels[disp_name]["frac_of_nominal_8TBs"], 2),
                        "combine": round(100 * kernels["combine_kernel"]["frac_of_nominal_8TBs"], 2)},
        "decode_us": decode_us, "other_configs": other, "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="strata", choices=["strata", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-other", action="store_true")
    ap.add_argument("--workload", default="prefill", choices=wl.CONFIG_ORDER,
                    help="configuration to step through (the bench line is quoted on the default)")
    ap.add_argument("--tokens-per-rank", type=int, default=0, help="shrink T (profiling captures only)")
    ap.add_argument("--timeline", action="store_true",
                    help="print only the in-kernel timeline summary of one step of --workload (not the bench line)")
    ap.add_argument("--timeline-trace", default="", help="also write a Chrome trace-event file of the first 32 CTAs")
    ap.add_argument("--timeline-pinned", action="store_true", help="kernels write the events into pinned host memory")
    ap.add_argument("--sm-sweep", action="store_true",
                    help="print only dispatch/combine throughput against the SM budget for --workload")
    ap.add_argument("--overlap", action="store_true",
                    help="print only the interference report: dispatch+combine beside a library GEMM on another stream")
    ap.add_argument("--collectives", action="store_true",
                    help="print only the report on the full-mesh collectives (one JSON object; not the bench line)")
    ap.add_argument("--expert-chain", action="store_true",
                    help="print only the timings of layout -> dispatch -> in-place expert stand-in -> combine for --workload")
    ap.add_argument("--partition-report", action="store_true",
                    help="print only the report on the paper's window partitioning at the skew and prefill shapes")
    ap.add_argument("--collective-kib", type=int, nargs="+", default=[64, 1024, 16384], help="payload per rank, KiB")
    ap.add_argument("--collective-iters", type=int, default=10)
    ap.add_argument("--collective-ops", nargs="+", default=list(COLLECTIVE_OPS), choices=COLLECTIVE_OPS)
    ap.add_argument("--profile", action="store_true",
                    help="for runs under a profiler: no e2e/cpu/other legs, warm-up not clamped")
    args = ap.parse_args()
    if args.profile:
        args.no_e2e = args.no_cpu = args.no_other = True
    elif args.impl == "strata":
        args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.timeline:
        if rank == 0:
            cfg = wl.CONFIGS[args.workload]
            if args.tokens_per_rank:
                cfg = wl.shrink(cfg, T=args.tokens_per_rank)
            print(json.dumps(timeline_report(cfg, local_rank, args.timeline_trace, args.timeline_pinned)), flush=True)
        return
    if args.sm_sweep:
        if rank == 0:
            cfg = wl.CONFIGS[args.workload]
            if args.tokens_per_rank:
                cfg = wl.shrink(cfg, T=args.tokens_per_rank)
            print(json.dumps(sm_budget_report(cfg, local_rank)), flush=True)
        return
    if args.overlap:
        if rank == 0:
            print(json.dumps(overlap_report(wl.CONFIGS[args.workload], local_rank)), flush=True)
        return
    if args.expert_chain:
        if rank == 0:
            print(json.dumps(expert_chain_report(wl.CONFIGS[args.workload], local_rank)), flush=True)
        return
    if args.partition_report:
        if rank == 0:
            print(json.dumps({
                "skew": window_partitioning_report(wl.CONFIGS["skew"], local_rank, unit_rows=64),
                "prefill": window_partitioning_report(wl.CONFIGS["prefill"], local_rank, unit_rows=128)}), flush=True)
        return
    if args.collectives:
        if rank == 0:
            print(json.dumps(collectives_report(local_rank, per_rank_kib=tuple(args.collective_kib),
                                                iters=args.collective_iters, warmup=min(args.warmup, 3),
                                                only=tuple(args.collective_ops))), flush=True)
        return
    run_gpu(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
