"""The time-out path of the bounded device waits (STRATA_ERR_TIMEOUT), exercised without faulting the GPU.

A second build of the library (same sources, test hooks compiled in, every bounded wait limited to 2000 tries)
makes one wait run out: CTA 0 of a dispatch launch expects 16 bytes more than its copy delivers.  The kernel
must return, the status must say TIMEOUT, reading the status must re-arm the context, and the next call on the
same context must be bit-exact against the oracle.  Runs in a child process because a process loads one build."""
import json
import os
import subprocess
import sys

import pytest

from paper_2607_26444_b200 import binding as B
from paper_2607_26444_b200 import build as strata_build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("kind", ["bf16", "fp8"])
def test_a_wait_that_runs_out_reports_timeout_and_the_context_recovers(kind):
    lib = strata_build.build_test_hooks()
    env = dict(os.environ, STRATA_MOE_LIB=lib)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "timeout_child.py"), kind], env=env,
                       capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-3000:]
    res = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert res["status_after_injection"] == B.STRATA_ERR_TIMEOUT
    assert res["status_read_again"] == B.STRATA_OK
    assert res["header_words_after_recovery"] == [0] * 8
    assert res["dispatch_exact"] and res["combine_exact"]
    assert res["status_after_normal_call"] == B.STRATA_OK


def test_the_shipped_library_has_no_test_hook():
    import ctypes
    L = ctypes.CDLL(os.path.join(ROOT, "paper_2607_26444_b200", "libstrata_moe.so"))
    assert not hasattr(L, "strata_test_inject_short_copy")
