"""Pins for the oracle's gated producer activation bf16(silu(g) * u) (the function f of Eq. (1), middle line, for a
SiLU-gated FFN) and for the interleaved gate / up stacking: closed-form values, identities of the logistic function,
limits, and exact rational rounding."""
from fractions import Fraction

import numpy as np

from paper_2609_22106_b200 import synth


def bf16_val(bits):
    return synth.bf16_to_f32(np.asarray(bits, np.uint16)).astype(np.float64)


def round_to_bf16_exact(x: Fraction) -> float:
    """Round a rational to 8 significant bits, ties to even, in exact arithmetic (normal range)."""
    if x == 0:
        return 0.0
    sign = -1 if x < 0 else 1
    a = abs(x)
    e = 0
    while a >= 2:
        a /= 2; e += 1
    while a < 1:
        a *= 2; e -= 1
    m = a * 128                      # in [128, 256)
    lo = m.numerator // m.denominator
    rem = m - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * float(Fraction(lo, 128) * Fraction(2) ** e)


def test_closed_form_values(oracle):
    ln3, ln7 = np.log(3.0), np.log(7.0)
    # silu(ln a) = ln a * a / (1 + a): 3/4 and 7/8;  silu(-ln a) = -ln a / (1 + a): 1/4 and 1/8
    g = np.array([0.0, -0.0, ln3, -ln3, ln7, -ln7, 1.0])
    u = np.array([5.0, 5.0, 1.0, 1.0, 2.0, -2.0, 1.0])
    want = np.array([0.0, 0.0, 0.75 * ln3, -0.25 * ln3, 2 * 0.875 * ln7, 2 * 0.125 * ln7, 1.0 / (1.0 + np.exp(-1.0))])
    got = bf16_val(oracle.silu_mul_bf16(g, u))
    exp = np.array([round_to_bf16_exact(Fraction(float(w))) for w in want])
    assert np.array_equal(got, exp)
    # the sign of a zero product survives (silu(-0) * 5 = -0)
    assert oracle.silu_mul_bf16(np.array([-0.0]), np.array([5.0]))[0] == 0x8000


def test_logistic_identities_and_limits(oracle):
    rng = np.random.default_rng(5)
    g = rng.standard_normal(4000) * 6
    # silu(g) - silu(-g) = g, exactly representable check through a power-of-two factor: u = 1 keeps silu itself
    s_pos = bf16_val(oracle.silu_mul_bf16(g, np.ones_like(g)))
    s_neg = bf16_val(oracle.silu_mul_bf16(-g, np.ones_like(g)))
    # each side carries at most half a bf16 ulp of its own magnitude
    ulp = np.maximum(np.abs(s_pos), np.abs(s_neg)) * 2.0 ** -8 + 1e-30
    assert np.all(np.abs((s_pos - s_neg) - g) <= 2 * ulp)
    # limits: silu(g) -> g for large g, -> 0 (from below) for very negative g; never below its minimum -0.2785
    big = np.array([40.0, 100.0, 700.0])
    assert np.array_equal(bf16_val(oracle.silu_mul_bf16(big, np.ones(3))), bf16_val(synth.f32_to_bf16(big.astype(np.float32))))
    neg = bf16_val(oracle.silu_mul_bf16(-big, np.ones(3)))
    assert np.all(neg <= 0) and np.all(np.abs(neg) < 1e-15)
    assert bf16_val(oracle.silu_mul_bf16(g, np.ones_like(g))).min() >= -0.2793
    # linear in u
    u = rng.standard_normal(4000)
    h2 = bf16_val(oracle.silu_mul_bf16(g, 4.0 * u))
    h1 = bf16_val(oracle.silu_mul_bf16(g, u))
    assert np.array_equal(h2, 4.0 * h1)          # a power of two commutes with the rounding


def test_single_rounding_against_rational_arithmetic(oracle):
    """The product is rounded ONCE: compare with exact rounding of the FP64 product taken as a rational."""
    rng = np.random.default_rng(6)
    g = rng.standard_normal(500) * 3
    u = rng.standard_normal(500) * 2
    prod = (g / (1.0 + np.exp(-g))) * u          # the same two FP64 operations the definition names
    want = np.array([round_to_bf16_exact(Fraction(float(p))) for p in prod])
    assert np.array_equal(bf16_val(oracle.silu_mul_bf16(g, u)), want)


def test_stacking_interleaves_groups_of_32(oracle):
    C, H = 96, 5
    Wg = np.arange(C * H, dtype=np.uint16).reshape(C, H)
    Wu = (10000 + np.arange(C * H)).astype(np.uint16).reshape(C, H)
    S = oracle.stack_gate_up(Wg, Wu)
    assert S.shape == (2 * C, H)
    for b in range(C // 32):
        assert np.array_equal(S[64 * b: 64 * b + 32], Wg[32 * b: 32 * b + 32])
        assert np.array_equal(S[64 * b + 32: 64 * b + 64], Wu[32 * b: 32 * b + 32])
