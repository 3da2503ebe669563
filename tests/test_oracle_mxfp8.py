"""Pins for the oracle's second format (MXFP8: E4M3 elements, E8M0 block scales): hand-worked blocks, the full E4M3
code table against its definition, a brute-force nearest-value quantiser in exact rational arithmetic, the scale rule,
and the product against plain FP64 arithmetic on the dequantised operands."""
import os
from fractions import Fraction

import numpy as np

from paper_2609_22106_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "mxfp8_encodings.txt")


def table():
    """E4M3 magnitudes by 7-bit code, from the format's definition (the NaN pattern 0x7F left out)."""
    vals = []
    for code in range(0x7F):
        e, m = code >> 3, code & 7
        vals.append(Fraction(m, 8) * Fraction(1, 64) if e == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7))
    return vals


def test_hand_worked_blocks(oracle):
    n = 0
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            vals, byte, codes = [p.strip() for p in line.split("|")]
            v = np.zeros((1, 32), np.float32)
            xs = [float(t) for t in vals.split()]
            v[0, : len(xs)] = xs
            c, s = oracle.fp8_quantize_rows(v)
            want = [int(t, 16) for t in codes.split()]
            assert int(s[0, 0]) == int(byte), line
            assert list(c[0, : len(want)]) == want, (line, [hex(int(t)) for t in c[0, : len(want)]])
            assert not c[0, len(xs):].any()
            n += 1
    assert n == 8


def test_code_table_and_dequantisation(oracle):
    t = table()
    assert t[0x7E] == 448 and t[0x38] == 1 and t[0x08] == Fraction(1, 64) and t[0x01] == Fraction(1, 512)
    assert all(a < b for a, b in zip(t, t[1:]))                      # strictly increasing magnitudes
    codes = np.arange(0x7F, dtype=np.uint8)
    for byte in (0, 1, 120, 127, 130, 254):
        for sign in (0, 0x80):
            c = np.zeros((1, 128), np.uint8)
            c[0, :0x7F] = codes | sign
            sc = np.full((1, 4), byte, np.uint8)
            got = oracle.fp8_dequantize_rows(c, sc)[0, :0x7F]
            want = np.array([float(v * Fraction(2) ** (byte - 127)) for v in t]) * (-1 if sign else 1)
            assert np.array_equal(got, want)


def nearest_code(a: Fraction, t):
    """Round-to-nearest over the table, ties to the even code, saturating (exact arithmetic)."""
    if a >= t[-1]:
        return len(t) - 1
    best, bd = 0, None
    for i, v in enumerate(t):
        d = abs(a - v)
        if bd is None or d < bd or (d == bd and i % 2 == 0 and best % 2 == 1):
            best, bd = i, d
    return best


def test_brute_force_nearest_value(oracle):
    rng = np.random.default_rng(11)
    t = table()
    blocks = []
    for _ in range(120):
        scale = 2.0 ** rng.integers(-20, 20)
        b = (rng.standard_normal(32) * rng.choice([1e-3, 0.1, 1, 30, 400])).astype(np.float32) * np.float32(scale)
        blocks.append(b)
    # every midpoint between neighbouring magnitudes, and its two fp32 neighbours, at scale 2^0 (block amax pinned to 448)
    mids = [float((a + b) / 2) for a, b in zip(t, t[1:])]
    for i in range(0, len(mids), 30):
        b = np.zeros(32, np.float32); b[0] = 448
        chunk = mids[i: i + 30]
        b[1: 1 + len(chunk)] = chunk
        blocks.append(b.copy())
        blocks.append(np.nextafter(b, np.float32(1e9), dtype=np.float32) * (b != 448) + b * (b == 448))
        blocks.append(np.nextafter(b, np.float32(0), dtype=np.float32) * (b != 448) + b * (b == 448))
    v = np.stack(blocks).astype(np.float32)
    c, s = oracle.fp8_quantize_rows(v)
    for r in range(v.shape[0]):
        amax = Fraction(float(np.abs(v[r]).max()))
        if amax == 0:
            assert s[r, 0] == 0
            continue
        e = max(-127, min(127, (amax.numerator.bit_length() - amax.denominator.bit_length()
                                - (1 if amax < Fraction(2) ** (amax.numerator.bit_length() - amax.denominator.bit_length()) else 0)) - 8))
        assert int(s[r, 0]) == e + 127
        X = Fraction(2) ** e
        for i in range(32):
            a = Fraction(float(abs(v[r, i]))) / X
            assert (int(c[r, i]) & 0x7F) == nearest_code(a, t), (r, i, float(a))
            assert (int(c[r, i]) >> 7) == int(np.signbit(v[r, i]))


def test_scale_rule_keeps_the_largest_magnitude_in_range(oracle):
    rng = np.random.default_rng(12)
    v = (rng.standard_normal((200, 32)) * np.exp(rng.normal(0, 4, (200, 1)))).astype(np.float32)
    c, s = oracle.fp8_quantize_rows(v)
    amax = np.abs(v).max(axis=1).astype(np.float64)
    X = 2.0 ** (s[:, 0].astype(np.float64) - 127)
    assert np.all(amax / X >= 256) and np.all(amax / X < 512)
    d = oracle.fp8_dequantize_rows(c, s)
    # relative error of an unsaturated normal element is at most 2^-4; saturation costs at most (512 - 448) / 512
    big = np.abs(v) >= X[:, None] * 2.0 ** -6
    assert np.all(np.abs(d - v)[big] <= np.abs(v)[big] * 0.125 + 1e-300)
    # idempotent on its own grid
    c2, s2 = oracle.fp8_quantize_rows(d.astype(np.float32))
    assert np.array_equal(oracle.fp8_dequantize_rows(c2, s2), d)


def test_layer_product_against_plain_arithmetic(oracle):
    L = synth.layer(55, 24, 96, 7, T_cal=16)
    amax = oracle.channel_amax(L["zcal"])
    p = oracle.fp8_prepare(L["W"], amax, 0.5)
    assert np.array_equal(p["s"], oracle.scales_from_amax(amax, 0.5)[0])
    W0 = (synth.bf16_to_f32(L["W"]).astype(np.float64) * p["s"].astype(np.float64)).astype(np.float32)
    wc, wsc = oracle.fp8_quantize_rows(W0)
    assert np.array_equal(wc, p["wcodes"]) and np.array_equal(wsc, p["wscales"])
    ac, asc = oracle.fp8_quantize_act(L["x"], p["inv_s"])
    xt = (synth.bf16_to_f32(L["x"]).astype(np.float64) * p["inv_s"].astype(np.float64)).astype(np.float32)
    assert np.array_equal(ac, oracle.fp8_quantize_rows(xt)[0])
    y = oracle.fp8_matmul(ac, asc, p["wcodes"], p["wscales"])
    want = oracle.fp8_dequantize_rows(ac, asc) @ oracle.fp8_dequantize_rows(p["wcodes"], p["wscales"]).T
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    # alpha = 0: no scaling at all
    p0 = oracle.fp8_prepare(L["W"], amax, 0.0)
    assert np.all(p0["s"] == 1) and np.array_equal(p0["wcodes"], oracle.fp8_quantize_rows(synth.bf16_to_f32(L["W"]))[0])
    # 8-bit elements are far closer to the unquantised product than MXFP4
    y_true = oracle.matmul_bf16(L["x"], L["W"])
    assert oracle.nrmse(y, y_true) < 0.05
