"""Pins for the oracle's weight-side block-scale search (E8M0-W, Ablation study): hand-worked blocks, a
brute force over the three candidate exponents in exact rational arithmetic, and the properties the
definition implies (never worse than the floor rule, at most one step away from it, no effect on the
channel ranking and permutation, exact residual identity)."""
import os
from fractions import Fraction

import numpy as np

from paper_2609_22106_b200 import synth
from test_oracle_mxfp4 import E2M1, unpack

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def parse_blocks():
    rows = []
    with open(os.path.join(GOLDEN, "scale_search_blocks.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            fill, byte0, byte, codes = [p.strip() for p in line.split(";")]
            vals = []
            for part in fill.split(","):
                v, n = part.split("x")
                vals += [float(v)] * int(n)
            rows.append((vals, int(byte0), int(byte), [int(c, 16) for c in codes.split()]))
    return rows


def test_hand_worked_blocks(oracle):
    for vals, byte0, byte, codes in parse_blocks():
        blk = np.asarray(vals, np.float32).reshape(1, 32)
        assert int(oracle.quantize_rows(blk)[1][0, 0]) == byte0
        c, s = oracle.quantize_rows_search(blk)
        assert int(s[0, 0]) == byte, (vals[:2], int(s[0, 0]))
        got = unpack(c[0])
        distinct = []
        for v, g in zip(vals, got):
            if not distinct or v != distinct[-1][0]:
                distinct.append((v, g))
        assert [g for _, g in distinct] == codes


def rational_block(vals, byte):
    """Codes and exact squared error of one block under the scale 2^(byte - 127), by exhaustive search over
    the 8 magnitudes (ties to the even code)."""
    X = Fraction(2) ** (byte - 127)
    codes, err = [], Fraction(0)
    for v in vals:
        f = Fraction(float(v))
        a = abs(f) / X
        best = None
        for idx, m in enumerate(E2M1):
            d = abs(a - m)
            if best is None or d < best[0] or (d == best[0] and idx % 2 == 0 and best[1] % 2 == 1):
                best = (d, idx)
        codes.append(best[1] | (8 if np.signbit(np.float32(v)) else 0))
        err += (best[0] * X) ** 2
    return codes, err


def test_brute_force_over_the_three_exponents(oracle):
    """On random heavy-tailed blocks the chosen byte is the exact argmin over {e0, e0 - 1, e0 + 1} (e0 on
    ties, then e0 - 1), and the codes are the nearest-value codes under that byte."""
    rng = np.random.default_rng(11)
    v = (rng.standard_t(3, size=(200, 32)) * np.exp(rng.normal(size=(200, 1)))).astype(np.float32)
    v[5, :] = 0
    v[6, 3:] = 0
    c0, s0 = oracle.quantize_rows(v)
    c, s = oracle.quantize_rows_search(v)
    picked_other = 0
    for r in range(v.shape[0]):
        b0 = int(s0[r, 0])
        if not v[r].any():
            assert int(s[r, 0]) == 0
            continue
        best_b, (best_codes, best_err) = b0, rational_block(v[r], b0)
        for cand in (b0 - 1, b0 + 1):
            if 0 <= cand <= 254:
                codes, err = rational_block(v[r], cand)
                if err < best_err:
                    best_b, best_codes, best_err = cand, codes, err
        assert int(s[r, 0]) == best_b
        assert unpack(c[r]) == best_codes
        picked_other += best_b != b0
    assert picked_other > 10   # the search is not vacuous on this data


def test_never_worse_and_at_most_one_step(oracle):
    rng = np.random.default_rng(12)
    v = (rng.standard_t(3, size=(64, 256)) * 0.02).astype(np.float32)
    c0, s0 = oracle.quantize_rows(v)
    c1, s1 = oracle.quantize_rows_search(v)
    assert np.abs(s1.astype(int) - s0.astype(int)).max() <= 1
    e0 = (v.astype(np.float64) - oracle.dequantize_rows(c0, s0)) ** 2
    e1 = (v.astype(np.float64) - oracle.dequantize_rows(c1, s1)) ** 2
    blk0 = e0.reshape(64, 8, 32).sum(axis=2)
    blk1 = e1.reshape(64, 8, 32).sum(axis=2)
    assert np.all(blk1 <= blk0)
    assert blk1.sum() < blk0.sum()


def test_prep_with_search_keeps_ranking_and_residual_identity(oracle):
    """The option changes neither s, the column errors nor the permutation; the main part is the searched
    quantisation of the permuted weight, R its exact residual on the tail, and the residual part the
    searched quantisation of R; the weight reconstruction error does not grow."""
    L = synth.layer(0, 48, 256, 8, T_cal=64, tag=31)
    amax = oracle.channel_amax(L["zcal"])
    a = oracle.prepare(L["W"], amax, 0.5, 64)
    b = oracle.prepare(L["W"], amax, 0.5, 64, scale_search=True)
    for key in ("s", "inv_s", "col_err", "perm"):
        assert np.array_equal(a[key], b[key])
    K, k = 256, 64
    W0 = (synth.bf16_to_f32(L["W"]).astype(np.float64) * b["s"].astype(np.float64)).astype(np.float32)
    Wt = W0[:, b["perm"]]
    c, s = oracle.quantize_rows_search(Wt)
    assert np.array_equal(b["wcodes"][:, : K // 2], c) and np.array_equal(b["wscales"][:, : K // 32], s)
    deq = oracle.dequantize_rows(c, s)
    R = (Wt[:, K - k:].astype(np.float64) - deq[:, K - k:]).astype(np.float32)
    assert np.array_equal(R, b["R"])
    assert np.array_equal(R.astype(np.float64), Wt[:, K - k:].astype(np.float64) - deq[:, K - k:])   # exact in fp32
    cr, sr = oracle.quantize_rows_search(R)
    assert np.array_equal(b["wcodes"][:, K // 2:], cr) and np.array_equal(b["wscales"][:, K // 32:], sr)
    err_a = ((Wt.astype(np.float64) - oracle.dequantize_rows(a["wcodes"][:, : K // 2], a["wscales"][:, : K // 32])) ** 2).sum()
    err_b = ((Wt.astype(np.float64) - deq) ** 2).sum()
    assert err_b < err_a
