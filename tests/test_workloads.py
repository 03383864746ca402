"""The seeded input generator: shapes, determinism and the stated distributions."""
import numpy as np

from paper_2607_26444_b200 import workloads as wl


def test_configs_match_the_stated_shapes():
    c = wl.CONFIGS
    assert (c["tiny"].R, c["tiny"].T, c["tiny"].H, c["tiny"].E, c["tiny"].K) == (4, 128, 1024, 16, 2)
    assert (c["decode"].R, c["decode"].T, c["decode"].H, c["decode"].E, c["decode"].K) == (16, 128, 7168, 256, 8)
    assert (c["prefill"].R, c["prefill"].T, c["prefill"].H, c["prefill"].E, c["prefill"].K) == (16, 4096, 7168, 256, 8)
    assert (c["skew"].R, c["skew"].T, c["skew"].H, c["skew"].E, c["skew"].K) == (32, 512, 4096, 128, 8)
    assert (c["fp8"].R, c["fp8"].T, c["fp8"].H, c["fp8"].E, c["fp8"].K) == (64, 256, 4096, 128, 8)
    # receive buffer of the prefill shape: R*T*K*H*2 bytes
    assert c["prefill"].n_items * c["prefill"].H * 2 == 7_516_192_768
    assert c["prefill"].dispatch_bytes() == 65536 * 7168 * 2 + 524288 * 7168 * 2 + 8 * 524288
    assert c["fp8"].dispatch_bytes() == 16384 * 4096 * 2 + 131072 * (4096 + 128) + 8 * 131072


def test_deterministic_and_distinct_ids():
    cfg = wl.CONFIGS["decode"]
    a, b = wl.gen_topk_ids(cfg), wl.gen_topk_ids(cfg)
    assert np.array_equal(a, b) and a.dtype == np.int32 and a.shape == (16, 128, 8)
    assert a.min() >= 0 and a.max() < cfg.E
    s = np.sort(a.reshape(-1, cfg.K), axis=1)
    assert np.all(np.diff(s, axis=1) > 0)                      # K distinct experts per token
    cnt = np.bincount(a.ravel(), minlength=cfg.E)
    assert cnt.min() > 0 and cnt.max() < 4 * cnt.mean()        # roughly uniform


def test_zipf_routing_is_skewed():
    cfg = wl.CONFIGS["skew"]
    a = wl.gen_topk_ids(cfg)
    s = np.sort(a.reshape(-1, cfg.K), axis=1)
    assert np.all(np.diff(s, axis=1) > 0)
    cnt = np.bincount(a.ravel(), minlength=cfg.E)
    # hottest expert is picked by most tokens and holds >10x the mean segment
    assert cnt.max() > 0.9 * cfg.n_tok
    assert cnt.max() > 10 * cnt.mean()
    assert cnt.min() > 0


def test_x_and_weights():
    cfg = wl.CONFIGS["tiny"]
    x = wl.bf16_bits_to_f32(wl.gen_x(cfg))
    assert x.shape == (4, 128, 1024) and abs(x.mean()) < 0.01 and abs(x.std() - 1) < 0.01
    w = wl.gen_gate_weights(cfg)
    assert w.dtype == np.float32 and np.all(w > 0)
    assert np.allclose(w.sum(axis=-1), 1.0, atol=1e-6)
    x8 = wl.bf16_bits_to_f32(wl.gen_x(wl.shrink(wl.CONFIGS["fp8"], R=2, T=64)))
    assert abs(x8.var() - 2.0) < 0.05


def test_bf16_round_trip_helpers():
    f = np.array([1.0, 1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -0.0, 3.14159], np.float32)
    b = wl.f32_to_bf16_bits(f)
    assert b.tolist()[:4] == [0x3F80, 0x3F80, 0x3F82, 0x8000]
    assert np.array_equal(wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(b)), b)


def test_expert_of_row():
    assert wl.expert_of_row(np.array([0, 3, 3, 6, 8]), 8).tolist() == [0, 0, 0, 2, 2, 2, 3, 3]


def test_bench_traffic_extrapolation_stays_close_to_the_algorithmic_bytes():
    """The DRAM traffic bench.py reports for a full prefill launch is the straight line through two captures;
    it must reproduce both captures and land within 2 % of the algorithmic bytes at full size (a kernel that
    re-read rows or read lines for ownership would show up as a ratio well above 1)."""
    import bench
    cfg = wl.CONFIGS["prefill"]
    for kernel, alg in (("dispatch_bf16_kernel", cfg.dispatch_bytes()), ("combine_kernel", cfg.combine_bytes())):
        cap = bench.NCU_CAPTURES[kernel]
        for t, (rd, wr) in cap.items():
            assert bench.ncu_traffic_bytes(kernel, t) == rd + wr
        full = bench.ncu_traffic_bytes(kernel, cfg.T)
        assert 0.98 <= full / alg <= 1.02, (kernel, full / alg)
    assert bench.ncu_traffic_bytes("dispatch_fp8_kernel", 256) is None
