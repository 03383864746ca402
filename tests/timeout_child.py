"""Child process of tests/test_gpu_timeout.py: runs with STRATA_MOE_LIB pointing at the test-hooks build.

Makes one bounded device wait run out on purpose (the hook makes CTA 0 of the next dispatch expect 16 bytes
more than its first copy delivers; nothing faults, traps or spins without a limit), checks that the kernel
returns, that the status is STRATA_ERR_TIMEOUT, that reading the status puts the context back in order, and
that the same context then computes the whole path bit-exactly against the oracle.  Prints one JSON line."""
import ctypes
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2607_26444_b200 import binding as B  # noqa: E402
from paper_2607_26444_b200 import workloads as wl  # noqa: E402


def main(kind: str):
    L = B.lib()
    hook = L.strata_test_inject_short_copy
    hook.argtypes, hook.restype = [ctypes.c_int], None
    dev = "cuda:0"
    fp8 = kind == "fp8"
    cfg = (wl.shrink(wl.CONFIGS["fp8"], R=4, T=300, H=1024, E=16, seed=91) if fp8
           else wl.shrink(wl.CONFIGS["decode"], R=4, T=300, H=7168, E=16, K=4, seed=90))
    inp = wl.generate(cfg)
    ref = oracle.layout(inp["ids"], cfg.E)
    ctx = B.MoEContext(cfg.R, cfg.T, cfg.H, cfg.E, cfg.K, cfg.dispatch_dtype)
    ids = torch.from_numpy(inp["ids"]).to(dev)
    x = torch.from_numpy(inp["x"].view(np.int16)).to(dev)
    w = torch.from_numpy(inp["w"]).to(dev)
    lay = ctx.layout(ids)
    recv = torch.zeros((cfg.n_items, cfg.H), dtype=torch.uint8 if fp8 else torch.int16, device=dev)
    scale = torch.zeros((cfg.n_items, cfg.H // 128), dtype=torch.float32, device=dev) if fp8 else None
    ctx.register(recv)
    if fp8:
        ctx.register(scale)
    res = {"kind": kind}

    hook(1)
    ctx.dispatch(lay, x, recv, scale)                 # CTA 0 gives up on its first unit and returns
    res["status_after_injection"] = ctx.device_status()
    res["status_read_again"] = ctx.device_status()    # reading cleared the word and the claim counters
    res["header_words_after_recovery"] = ctx.workspace[:32].view(torch.int32).cpu().tolist()

    recv.zero_()
    ctx.dispatch(lay, x, recv, scale)                 # a normal call on the same context
    if fp8:
        q, s = oracle.dispatch_fp8(ref["dst_row"], inp["x"])
        res["dispatch_exact"] = bool(np.array_equal(recv.cpu().numpy(), q)
                                     and np.array_equal(scale.cpu().numpy().view(np.uint32), s.view(np.uint32)))
        y = wl.expert_standin(cfg, q, ref["expert_offset"], s)
    else:
        r = oracle.dispatch_bf16(ref["dst_row"], inp["x"])
        res["dispatch_exact"] = bool(np.array_equal(recv.cpu().numpy().view(np.uint16), r))
        y = wl.expert_standin(cfg, r, ref["expert_offset"])
    out = torch.zeros((cfg.n_tok, cfg.H), dtype=torch.int16, device=dev)
    ctx.combine(lay, torch.from_numpy(y.view(np.int16)).to(dev), w, out)
    res["combine_exact"] = bool(np.array_equal(out.cpu().numpy().view(np.uint16),
                                               oracle.combine(ref["dst_row"], y, inp["w"])))
    res["status_after_normal_call"] = ctx.device_status()
    ctx.close()
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "bf16")
