"""The one JSON line bench.py prints: keys and basic sanity, on a small workload (GPU arm) and on the
CPU reference arm."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "cpu_baseline"}


def run_bench(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                       timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line():
    d = run_bench("--impl", "reference", "--steps", "2", "--warmup", "1")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["unit"] == "GB/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"] and d["value"] > 0
    assert d["gpu_launches"] == 0 and "workload" in d["config"]


@pytest.mark.gpu
def test_gpu_arm_line_on_a_small_workload():
    d = run_bench("--workload", "decode", "--steps", "5", "--warmup", "3", "--no-other")
    assert BASE_KEYS | {"roofline", "clocks"} <= set(d) and "impl" not in d
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["scaling"] == "weak"
    assert d["dtype"] == "bf16" and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["gpu_launches"] == 5 * 3                      # one-launch layout + dispatch + combine per step
    roof = d["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and 0 < roof["frac"] < 1.3
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert roof["kernel"] in roof["kernels"]
    e2e = d["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert e2e["value"] < d["value"]                       # copies are inside that timed region
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    cpu = d["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and "sample" in cpu


@pytest.mark.gpu
def test_default_line_carries_the_decode_block_and_stays_short():
    """Everything but the main workload is as in the default run (decode block, the other shapes), the main
    workload is the tiny one so that the test is quick; the line must stay short enough to be kept whole."""
    d = run_bench("--workload", "tiny", "--steps", "5", "--warmup", "3", "--no-cpu", "--no-e2e")
    dec = d["decode_us"]
    for k in ("layout", "dispatch", "combine", "layout+dispatch", "step", "step_cuda_graph"):
        assert 0 < dec[k] < 1000, k
    assert set(dec["back_to_back"]) == {"layout", "dispatch", "combine", "layout+dispatch", "step"}
    assert 0.3 < dec["of_measured_peak"]["dispatch"] < 1.3 and 0.3 < dec["of_measured_peak"]["combine"] < 1.3
    assert dec["step"] >= dec["back_to_back"]["step"] * 0.9
    assert set(d["other_configs"]) == {"tiny", "decode", "skew", "fp8", "skew_shape_uniform_routing"}
    for name in ("tiny", "decode", "skew", "fp8"):
        assert {"layout_us", "dispatch_us", "combine_us", "step_us", "step_back_to_back_us"} <= set(d["other_configs"][name])
    assert len(json.dumps(d)) < 6000
    assert set(d["roofline"]["kernels"]) == {"dispatch_bf16_kernel", "combine_kernel"}
    for k in d["roofline"]["kernels"].values():
        assert k["avg_ms"] > 0 and k["achieved"] > 0


@pytest.mark.gpu
def test_collectives_report_mode():
    d = run_bench("--collectives", "--collective-kib", "64", "256", "--collective-iters", "3")
    assert d["R"] == 32 and set(d["sizes"]) == {"64KiB_per_rank", "256KiB_per_rank"}
    for size in d["sizes"].values():
        assert size["verified"] is True
        for op in ("allgather", "alltoall", "alltoallv", "broadcast", "reducescatter", "allreduce"):
            assert size[op]["median_us"] > 0 and size[op]["back_to_back_us"] > 0 and size[op]["bytes"] > 0


@pytest.mark.gpu
def test_timeline_report_mode(tmp_path):
    trace = tmp_path / "trace.json"
    d = run_bench("--timeline", "--workload", "tiny", "--timeline-trace", str(trace))
    assert d["events_dropped"] == 0 and {"dispatch_bf16", "combine"} <= set(d["kernels"])
    assert d["kernels"]["dispatch_bf16"]["stages"]["work"]["intervals"] == 4 * 128       # one per token
    assert d["chrome_trace_events"] > 0 and json.loads(trace.read_text())["traceEvents"]


@pytest.mark.gpu
def test_expert_chain_report_mode():
    d = run_bench("--expert-chain", "--workload", "decode")
    assert d["device_status"] == 0 and d["tile_rows"] == 128 and d["recv_rows"] == 16384 + 256 * 127
    assert set(d["us"]) == {"layout", "dispatch", "expert", "combine", "chain"} and all(v > 0 for v in d["us"].values())
    assert d["expert_GBs"] > 1000
