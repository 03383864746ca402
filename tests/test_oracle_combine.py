"""Pins for the oracle's combine (fp32 FMA chain in slot order, bf16 RNE out)."""
import numpy as np
import pytest

import oracle
from paper_2607_26444_b200 import workloads as wl


def ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """bf16 ulp distance on bit patterns: sign-magnitude mapped to a line, +-0 equal."""
    def line(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(line(a) - line(b))


def _case(name="tiny", **kw):
    cfg = wl.shrink(wl.CONFIGS[name], **kw) if kw else wl.CONFIGS[name]
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    return cfg, inp, lay


@pytest.mark.parametrize("name", ["tiny", "skewsmall"])
def test_identity_experts_return_x(name):
    # gate weights sum to 1 and y = recv  =>  out == x bit for bit
    if name == "tiny":
        cfg, inp, lay = _case("tiny")
    else:
        cfg, inp, lay = _case("skew", R=4, T=64, H=256, E=16, K=8)
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    out = oracle.combine(lay["dst_row"], recv, inp["w"], nthreads=2)
    x = inp["x"].reshape(cfg.n_tok, cfg.H).copy()
    assert ulp_distance(out, x).max() == 0           # equal as values
    # the only bit difference allowed: a -0 input returns as +0 (fma(w, -0, +0) = +0)
    assert np.array_equal(out[x != 0x8000], x[x != 0x8000])
    x[0, 0] = 0x8000
    recv = oracle.dispatch_bf16(lay["dst_row"], x)
    assert oracle.combine(lay["dst_row"], recv, inp["w"])[0, 0] == 0x0000


def test_worked_example_combine():
    # the hand-worked layout example with H=1: x=[1,3,5,7], w=[.25,.75] per token
    ids = np.array([[[2, 0], [0, 3]], [[0, 2], [3, 2]]], np.int32)
    lay = oracle.layout(ids, 4)
    x = wl.f32_to_bf16_bits(np.array([1, 3, 5, 7], np.float32)).reshape(2, 2, 1)
    # H=1 rows: dispatch by hand from the worked dst_row
    recv = np.empty((8, 1), np.uint16)
    for i, row in enumerate([3, 0, 1, 6, 2, 4, 7, 5]):
        recv[row, 0] = x.ravel()[i // 2]
    w = np.tile(np.array([0.25, 0.75], np.float32), (2, 2, 1))
    out = oracle.combine(lay["dst_row"], recv, w)
    assert np.array_equal(out.ravel(), x.ravel())


def test_one_hot_weights_select_a_row_and_k1():
    cfg, inp, lay = _case("tiny")
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    y = wl.expert_standin(cfg, recv, lay["expert_offset"])        # per-expert scaling
    w = np.zeros((cfg.R, cfg.T, cfg.K), np.float32)
    w[..., 1] = 1.0
    out = oracle.combine(lay["dst_row"], y, w)
    assert np.array_equal(out, y[lay["dst_row"].reshape(-1, cfg.K)[:, 1]])
    # K = 1, w = 1  =>  out = y[dst_row]
    d1 = lay["dst_row"].reshape(-1, cfg.K)[:, :1].copy()
    out1 = oracle.combine(d1, y, np.ones((cfg.n_tok, 1), np.float32))
    assert np.array_equal(out1, y[d1[:, 0]])


def test_doubling_weights_doubles_output():
    cfg, inp, lay = _case("tiny")
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    y = wl.expert_standin(cfg, recv, lay["expert_offset"])
    a = wl.bf16_bits_to_f32(oracle.combine(lay["dst_row"], y, inp["w"]))
    b = wl.bf16_bits_to_f32(oracle.combine(lay["dst_row"], y, 2 * inp["w"]))
    assert np.array_equal(b, 2 * a)


def test_slot_order_matters_and_is_0_to_K_minus_1():
    # 2^24 + 1 - 2^24 in fp32: left-to-right from +0 gives 0; any other order gives 1
    ids = np.array([[[0, 1, 2]]], np.int32)
    lay = oracle.layout(ids, 3)
    y = wl.f32_to_bf16_bits(np.array([[2.0 ** 24], [1.0], [-(2.0 ** 24)]], np.float32))
    out = oracle.combine(lay["dst_row"], y, np.ones((1, 1, 3), np.float32))
    assert wl.bf16_bits_to_f32(out)[0, 0] == 0.0
    ids = np.array([[[0, 2, 1]]], np.int32)      # slots now see 2^24, -2^24, 1
    lay = oracle.layout(ids, 3)
    out = oracle.combine(lay["dst_row"], y, np.ones((1, 1, 3), np.float32))
    assert wl.bf16_bits_to_f32(out)[0, 0] == 1.0


def test_fused_multiply_add_is_single_rounding():
    # w*v + acc with w*v not representable: fma(1+2^-12, 1+2^-12, -(1+2^-11)) = 2^-24 exactly;
    # a separately rounded product would give 0.
    ids = np.array([[[0, 1]]], np.int32)
    lay = oracle.layout(ids, 2)
    # slot 0 contributes -(1+2^-11) exactly via w=-1; slot 1 is the inexact product.
    # bf16 cannot hold 1+2^-12, so put the fine value in the fp32 weight and a power of two in y:
    y = wl.f32_to_bf16_bits(np.array([[1.0], [1.0]], np.float32))
    w = np.array([[[-(1 + 2.0 ** -11), 1.0]]], np.float32)
    out = oracle.combine(lay["dst_row"], y, w)
    assert wl.bf16_bits_to_f32(out)[0, 0] == np.float32(1 - (1 + 2.0 ** -11))
    # real single-rounding probe: y = 1+2^-7 (bf16 exact), w = 1+2^-17 (fp32 exact);
    # exact product = 1 + 2^-7 + 2^-17 + 2^-24, which needs 25 bits.  acc = -(1+2^-7+2^-17).
    yv = np.float32(1 + 2.0 ** -7)
    wv = np.float32(1 + 2.0 ** -17)
    acc0 = np.float32(-(1 + 2.0 ** -7 + 2.0 ** -17))
    y = wl.f32_to_bf16_bits(np.array([[1.0], [yv]], np.float32))
    w = np.array([[[acc0, wv]]], np.float32)
    out = wl.bf16_bits_to_f32(oracle.combine(lay["dst_row"], y, w))[0, 0]
    assert out == np.float32(2.0 ** -24)         # fused; unfused rounding would give 0


def test_against_float64_sum():
    cfg, inp, lay = _case("decode", R=4, T=16, H=512, E=16, K=8, seed=77)
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    y = wl.expert_standin(cfg, recv, lay["expert_offset"])        # affine experts
    out = oracle.combine(lay["dst_row"], y, inp["w"])
    rows = lay["dst_row"].reshape(cfg.n_tok, cfg.K)
    yv = wl.bf16_bits_to_f32(y).astype(np.float64)[rows]          # [n_tok, K, H]
    wv = inp["w"].reshape(cfg.n_tok, cfg.K, 1).astype(np.float64)
    exact = (wv * yv).sum(axis=1)
    absum = (np.abs(wv) * np.abs(yv)).sum(axis=1)
    got = wl.bf16_bits_to_f32(out).astype(np.float64)
    # bf16 half-ulp relative 2^-9 (use 2^-8 = one ulp), plus the fp32 chain's K roundings
    tol = np.abs(exact) * 2.0 ** -8 + cfg.K * 2.0 ** -24 * absum + 1e-38
    assert np.all(np.abs(got - exact) <= tol)
    # and round-to-nearest of the exact sum agrees to within one bf16 ulp
    ref_bits = wl.f32_to_bf16_bits(exact.astype(np.float32))
    assert ulp_distance(out, ref_bits).max() <= 1


def test_rounding_to_bf16_is_nearest_even():
    # K=1, w=1 cannot show rounding (y is already bf16); use w to create ties:
    # y=1, w = 1 + 2^-8  -> exactly halfway between bf16 1.0 and 1+2^-7 -> even (1.0)
    ids = np.array([[[0]]], np.int32)
    lay = oracle.layout(ids, 1)
    y = wl.f32_to_bf16_bits(np.array([[1.0]], np.float32))
    for wv, want in [(1 + 2.0 ** -8, 1.0), (1 + 3 * 2.0 ** -8, 1 + 2 * 2.0 ** -7),
                     (1 + 2.0 ** -8 + 2.0 ** -20, 1 + 2.0 ** -7), (1 + 2.0 ** -9, 1.0)]:
        out = oracle.combine(lay["dst_row"], y, np.array([[[wv]]], np.float32))
        assert wl.bf16_bits_to_f32(out)[0, 0] == np.float32(want), wv
