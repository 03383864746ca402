"""Pins for the oracle's in-place expert stand-in (a per-expert affine map over the occupied receive rows):
none of them re-types its formula with the same library call."""
from fractions import Fraction

import numpy as np

import oracle
from paper_2607_26444_b200 import workloads as wl


def _round_to_float32(fr: Fraction) -> np.float32:
    """Nearest binary32 to an exact rational, ties to even, by integer arithmetic (normal range only)."""
    if fr == 0:
        return np.float32(0.0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()      # 2^e <= a < 2^(e+2)
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1) and -126 <= e <= 127
    q = a / Fraction(2) ** (e - 23)                                # in [2^23, 2^24)
    m, rem = divmod(q.numerator, q.denominator)
    twice = 2 * rem
    if twice > q.denominator or (twice == q.denominator and (m & 1)):
        m += 1
    return np.float32(sign * float(Fraction(m) * Fraction(2) ** (e - 23)))   # exact in binary64


def _lay(counts, align=1):
    E = len(counts)
    off = np.zeros(E + 1, np.int32)
    for e, c in enumerate(counts):
        off[e + 1] = off[e] + (c + align - 1) // align * align
    return {"expert_count": np.array(counts, np.int32), "expert_offset": off}


def test_exact_rational_arithmetic_with_a_single_rounding():
    rng = np.random.default_rng(5)
    counts = [3, 0, 5, 2]
    lay = _lay(counts)
    H = 16
    x = wl.f32_to_bf16_bits(rng.normal(0, 3, (10, H)).astype(np.float32))
    scale = rng.normal(1, 0.5, 4).astype(np.float32)
    bias = rng.normal(0, 2, 4).astype(np.float32)
    got = oracle.expert_affine(lay, x, scale, bias)
    xv = wl.bf16_bits_to_f32(x)
    row = 0
    for e, c in enumerate(counts):
        for _ in range(c):
            for col in range(H):
                exact = Fraction(float(xv[row, col])) * Fraction(float(scale[e])) + Fraction(float(bias[e]))
                want = wl.f32_to_bf16_bits(np.array([_round_to_float32(exact)], np.float32))[0]
                assert got[row, col] == want, (row, col)
            row += 1


def test_the_multiply_add_is_fused():
    # x = 1+2^-7 (bf16 exact), scale = 1+2^-17, bias = -(1+2^-7+2^-17): the exact result is 2^-24, a product
    # rounded on its own (to 1+2^-7+2^-17) would give 0
    lay = _lay([1])
    x = wl.f32_to_bf16_bits(np.array([[1 + 2.0 ** -7]], np.float32))
    got = oracle.expert_affine(lay, x, np.array([1 + 2.0 ** -17], np.float32),
                               np.array([-(1 + 2.0 ** -7 + 2.0 ** -17)], np.float32))
    assert wl.bf16_bits_to_f32(got)[0, 0] == np.float32(2.0 ** -24)


def test_rounding_to_bf16_is_nearest_even():
    lay = _lay([1])
    x = wl.f32_to_bf16_bits(np.array([[1.0]], np.float32))
    for s, want in [(1 + 2.0 ** -8, 1.0), (1 + 3 * 2.0 ** -8, 1 + 2 * 2.0 ** -7),
                    (1 + 2.0 ** -8 + 2.0 ** -20, 1 + 2.0 ** -7), (1 + 2.0 ** -9, 1.0)]:
        got = oracle.expert_affine(lay, x, np.array([s], np.float32), np.zeros(1, np.float32))
        assert wl.bf16_bits_to_f32(got)[0, 0] == np.float32(want), s


def test_every_row_takes_the_constants_of_the_expert_that_owns_it_and_padding_is_left_alone():
    cfg = wl.shrink(wl.CONFIGS["tiny"], R=4, T=40, H=64, E=8, K=3, seed=9)
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E, segment_align=16)
    n_rows = cfg.n_items + cfg.E * 15
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"], n_rows=n_rows)            # padding rows hold 0xDEAD
    scale = np.array([2.0 ** (e % 5 - 2) for e in range(cfg.E)], np.float32)         # exact powers of two
    bias = np.zeros(cfg.E, np.float32)
    got = oracle.expert_affine(lay, recv, scale, bias)
    owner = oracle.row_experts(lay, cfg.R)
    assert owner.shape[0] == int(lay["expert_offset"][cfg.E])
    for row in range(n_rows):
        e = owner[row] if row < owner.shape[0] else -1
        if e < 0:
            assert np.all(got[row] == recv[row])                                    # untouched, whatever it held
        else:
            want = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(recv[row]) * scale[e])  # exact: a shift of the exponent
            assert np.array_equal(got[row], want), row
    # and through src_of_row: a row's constants are those of the id of the item placed there
    ids = inp["ids"].reshape(-1)
    for row in np.flatnonzero(lay["src_of_row"] >= 0)[::7]:
        e = ids[lay["src_of_row"][row]]
        assert np.array_equal(got[row], wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(recv[row]) * scale[e]))


def test_identity_constants_return_the_values():
    cfg = wl.shrink(wl.CONFIGS["tiny"], R=2, T=30, H=128, E=4, K=2, seed=10)
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    got = oracle.expert_affine(lay, recv, np.ones(cfg.E, np.float32), np.zeros(cfg.E, np.float32))
    assert np.array_equal(wl.bf16_bits_to_f32(got), wl.bf16_bits_to_f32(recv))      # as values (-0 comes back as +0)


def test_bias_zero_equals_an_independent_numpy_product():
    """With bias 0 the fused multiply-add is the correctly rounded product, which numpy's float32 multiply
    also is: the harness's own "scale" stand-in (written in numpy) must agree bit for bit."""
    cfg = wl.CONFIGS["tiny"]                                                        # experts scale by 1 + e/16
    inp = wl.generate(cfg)
    lay = oracle.layout(inp["ids"], cfg.E)
    recv = oracle.dispatch_bf16(lay["dst_row"], inp["x"])
    scale = (np.float32(1.0) + np.arange(cfg.E, dtype=np.float32) / np.float32(cfg.E)).astype(np.float32)
    got = oracle.expert_affine(lay, recv, scale, np.zeros(cfg.E, np.float32))
    want = wl.expert_standin(cfg, recv, lay["expert_offset"])
    assert np.array_equal(wl.bf16_bits_to_f32(got), wl.bf16_bits_to_f32(want))
