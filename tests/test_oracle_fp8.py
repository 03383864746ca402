"""Pins for the oracle's e4m3 encoder and FP8 dispatch.

The encoder is integer arithmetic on binary32 bits; it is pinned against
(i) a brute-force nearest-representable search over a value table built here
from the format definition, (ii) hand-worked check values, (iii) torch's CPU
float8_e4m3fn cast on the range where that cast does not overflow.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2607_26444_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _table():
    """(values float64[127], codes) of the non-negative finite codes 0x00..0x7E."""
    vals = []
    for c in range(0x7F):
        ex, m = c >> 3, c & 7
        vals.append(m * 2.0 ** -9 if ex == 0 else (1 + m / 8) * 2.0 ** (ex - 7))
    return np.array(vals, np.float64)


def brute_force_encode(v: np.ndarray) -> np.ndarray:
    """Nearest finite code by exhaustive search in float64; ties -> even code;
    beyond 448 -> 448 (saturating)."""
    tab = _table()
    a = np.abs(v.astype(np.float64))
    big = a >= 464.0
    a = np.where(big, 448.0, a)          # far-away values would all look equidistant in float64
    diff = np.abs(a[:, None] - tab[None, :])
    best = diff.min(axis=1)
    cand = diff == best[:, None]
    code = np.empty(v.size, np.uint8)
    for i in range(v.size):
        cs = np.nonzero(cand[i])[0]
        if len(cs) == 1:
            code[i] = cs[0]
        else:
            assert len(cs) == 2
            code[i] = cs[0] if cs[0] % 2 == 0 else cs[1]
    # the tie at 464 sits between 448 (0x7E, even) and the non-existent 480; anything larger saturates
    code[big] = 0x7E
    sign = (v.view(np.uint32) >> 24).astype(np.uint8) & 0x80
    return code | sign


def test_check_values():
    with open(os.path.join(GOLDEN, "e4m3_check_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            v = np.array([float(line[0])], np.float32)
            assert int(oracle.e4m3_encode(v)[0]) == int(line[1], 16), line


def test_against_brute_force_all_bf16_inputs():
    # every finite bf16 bit pattern, as binary32
    bits = np.arange(65536, dtype=np.uint32)
    finite = (bits & 0x7F80) != 0x7F80
    v = (bits[finite] << 16).view(np.float32)
    got = oracle.e4m3_encode(v)
    want = brute_force_encode(v)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("seed", [0, 1])
def test_against_brute_force_dense_fp32(seed):
    rng = np.random.default_rng(seed)
    # dense in every binade that matters, plus exact ties and their neighbours
    mags = np.exp2(rng.uniform(-13, 10, size=20000)).astype(np.float32)
    signs = rng.choice([-1.0, 1.0], size=mags.size).astype(np.float32)
    tab = _table()
    mid = ((tab[1:] + tab[:-1]) / 2).astype(np.float32)          # exact ties (representable in fp32)
    ties = np.concatenate([mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(1e9)),
                           tab.astype(np.float32)])
    v = np.concatenate([mags * signs, ties, -ties]).astype(np.float32)
    assert np.array_equal(oracle.e4m3_encode(v), brute_force_encode(v))


def test_against_torch_cast_in_range():
    rng = np.random.default_rng(5)
    v = (np.exp2(rng.uniform(-12, 8.8, size=50000)) * rng.choice([-1, 1], size=50000)).astype(np.float32)
    v = v[np.abs(v) <= 448.0]
    want = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.e4m3_encode(v), want)


def test_special_inputs():
    v = np.array([np.inf, -np.inf, np.nan, 3.0e38, 1e-45, -1e-45], np.float32)
    got = oracle.e4m3_encode(v)
    assert got[0] == 0x7E and got[1] == 0xFE and (got[2] & 0x7F) == 0x7F
    assert got[3] == 0x7E and got[4] == 0x00 and got[5] == 0x80


def _small_fp8_case(seed=3, sigma=2.0 ** 0.5):
    cfg = wl.shrink(wl.CONFIGS["fp8"], R=4, T=24, H=512, E=8, K=3, seed=seed, sigma=sigma)
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    return cfg, inp, lay


def test_fp8_dispatch_definition_and_invariants():
    cfg, inp, lay = _small_fp8_case()
    x = inp["x"].reshape(cfg.n_tok, cfg.H)
    x[5, 128:256] = 0                    # an all-zero block
    x[6, 0:128] = 0x8000                 # all negative zeros
    x[7, 3] = wl.f32_to_bf16_bits(np.array([1e-30], np.float32))[0]
    q, s = oracle.dispatch_fp8(lay["dst_row"], x, nthreads=2)
    xf = wl.bf16_bits_to_f32(x).reshape(cfg.n_tok, cfg.H // 128, 128)
    amax = np.abs(xf).max(axis=2)
    scale = (amax / np.float32(448.0)).astype(np.float32)       # IEEE binary32 division in numpy
    d = np.where(amax == 0, np.float32(1), scale).astype(np.float32)
    quo = (xf / d[:, :, None]).astype(np.float32)
    want_q = brute_force_encode(quo.ravel()).reshape(cfg.n_tok, cfg.H)
    tok_of_row = lay["src_of_row"] // cfg.K
    assert np.array_equal(q, want_q[tok_of_row])
    assert np.array_equal(s.view(np.uint32), scale[tok_of_row].view(np.uint32))
    # all-zero blocks: stored scale 0, codes are signed zeros, never NaN
    rows5 = lay["dst_row"].reshape(cfg.n_tok, cfg.K)[5]
    assert np.all(s[rows5, 1] == 0) and np.all(q[rows5, 128:256] == 0)
    rows6 = lay["dst_row"].reshape(cfg.n_tok, cfg.K)[6]
    assert np.all(q[rows6, 0:128] == 0x80)
    assert not np.any((q & 0x7F) == 0x7F)
    # the block's largest element encodes to +-448
    qa = q.reshape(-1, cfg.H // 128, 128)[lay["dst_row"].reshape(cfg.n_tok, cfg.K)[:, 0]]
    am = np.abs(xf).argmax(axis=2)
    top = np.take_along_axis(qa, am[:, :, None], axis=2)[:, :, 0]
    assert np.all((top & 0x7F)[amax > 0] == 0x7E)
    # K copies of a token are identical
    rows = lay["dst_row"].reshape(cfg.n_tok, cfg.K)
    for k in range(1, cfg.K):
        assert np.array_equal(q[rows[:, 0]], q[rows[:, k]])
        assert np.array_equal(s[rows[:, 0]], s[rows[:, k]])


def test_fp8_round_trip_error_bound():
    cfg, inp, lay = _small_fp8_case(seed=11)
    x = inp["x"].reshape(cfg.n_tok, cfg.H)
    q, s = oracle.dispatch_fp8(lay["dst_row"], x)
    tab = wl.e4m3_value_table().astype(np.float64)
    tok = lay["src_of_row"] // cfg.K
    xf = wl.bf16_bits_to_f32(x).astype(np.float64)[tok]
    sc = np.repeat(s.astype(np.float64), 128, axis=1)
    deq = tab[q] * sc
    r = np.abs(xf / np.where(sc == 0, 1, sc))
    # half a subnormal step, or half an ulp of a 3-bit mantissa (2^-4 relative), in scaled units
    bound = sc * np.maximum(2.0 ** -10, 2.0 ** -4 * r) * (1 + 2.0 ** -20)
    assert np.all(np.abs(deq - xf) <= bound)
