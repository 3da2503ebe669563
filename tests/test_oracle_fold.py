"""Pins for the oracle's producer fold (Eq. (1), middle line; 'offline copy' of the Activation tail construction
paragraph): hand-worked bf16 roundings, exact rational arithmetic on random products, pure permutation when the
scales are 1, the duplicated tail rows, and Eq. (1)'s invariance of the gated product within the folded weights'
rounding."""
import os
import struct
from fractions import Fraction

import numpy as np

from paper_2609_22106_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bf16_fold_roundings.txt")


def bf16_value(bits: int) -> Fraction:
    return Fraction(struct.unpack("<f", struct.pack("<I", (bits & 0xFFFF) << 16))[0])


def f32_value(bits: int) -> Fraction:
    return Fraction(struct.unpack("<f", struct.pack("<I", bits))[0])


def nearest_bf16(p: Fraction, sign_of_zero: int = 0) -> int:
    """Nearest bf16 to the exact rational p, ties to the even pattern, by bisection over the ordered patterns."""
    if p == 0:
        return sign_of_zero
    neg = p < 0
    a = -p if neg else p
    lo, hi = 0, 0x7F7F
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if bf16_value(mid) <= a:
            lo = mid
        else:
            hi = mid
    dl, dh = a - bf16_value(lo), bf16_value(hi) - a
    r = lo if dl < dh else hi if dh < dl else (lo if lo % 2 == 0 else hi)
    return r | (0x8000 if neg else 0)


def fold_one(oracle, w_bits: int, s_bits: int) -> int:
    W = np.array([[w_bits]], np.uint16)
    inv_s = np.array([s_bits], np.uint32).view(np.float32)
    up, gate = oracle.fold_producer(W, W, np.array([0], np.int32), inv_s, 0)
    assert gate[0, 0] == w_bits
    return int(up[0, 0])


def test_hand_worked_roundings(oracle):
    n = 0
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w, s, e, _ = [p.strip() for p in line.split(";")]
        w, s, e = int(w, 16), int(s, 16), int(e, 16)
        assert nearest_bf16(bf16_value(w) * f32_value(s), w & 0x8000) == e, line    # the fixture itself
        assert fold_one(oracle, w, s) == e, line
        n += 1
    assert n >= 10


def test_random_products_against_exact_rational_arithmetic(oracle):
    rng = np.random.default_rng(7)
    C, H = 64, 20
    W = synth.weights(3, C, H)
    W[0, :4] = [0x0001, 0x8003, 0x007F, 0x0080]            # subnormals and the smallest normal
    inv_s = np.exp(rng.normal(0, 3, C)).astype(np.float32)
    inv_s[0] = 0.5
    perm = rng.permutation(C).astype(np.int32)
    up, gate = oracle.fold_producer(W, W, perm, inv_s, 0)
    for jp in range(C):
        j = int(perm[jp])
        s_bits = int(inv_s[j:j + 1].view(np.uint32)[0])
        for h in range(H):
            w = int(W[j, h])
            assert int(up[jp, h]) == nearest_bf16(bf16_value(w) * f32_value(s_bits), w & 0x8000), (jp, h)
    assert np.array_equal(gate, W[perm])


def test_unit_scales_make_the_fold_a_row_permutation(oracle):
    C, H, k = 96, 40, 32
    Wu, Wg = synth.weights(11, C, H), synth.weights(12, C, H)
    perm = np.random.default_rng(1).permutation(C).astype(np.int32)
    up, gate = oracle.fold_producer(Wu, Wg, perm, np.ones(C, np.float32), k)
    assert np.array_equal(up, Wu[perm]) and np.array_equal(gate, Wg[perm])


def test_offline_copy_repeats_the_tail_rows(oracle):
    C, H, k = 96, 24, 32
    Wu, Wg = synth.weights(13, C, H), synth.weights(14, C, H)
    rng = np.random.default_rng(2)
    perm = rng.permutation(C).astype(np.int32)
    inv_s = np.exp(rng.normal(0, 1, C)).astype(np.float32)
    up, gate = oracle.fold_producer(Wu, Wg, perm, inv_s, k)
    upd, gated = oracle.fold_producer(Wu, Wg, perm, inv_s, k, dup=True)
    assert upd.shape == (C + k, H) and gated.shape == (C + k, H)
    assert np.array_equal(upd[:C], up) and np.array_equal(gated[:C], gate)
    assert np.array_equal(upd[C:], up[C - k:]) and np.array_equal(gated[C:], gate[C - k:])
    up0, _ = oracle.fold_producer(Wu, Wg, perm, inv_s, 0, dup=True)
    assert up0.shape == (C, H)


def test_gated_product_is_invariant_up_to_the_folded_weights_rounding(oracle):
    """Eq. (1): (X Wup'^T) * sigma(X Wgate'^T) equals Z D^-1 P, here with sigma = SiLU in FP64.  The gate path is
    exact (a permutation); the up path carries one bf16 rounding per weight, i.e. a relative 2^-9 per term."""
    C, H, T, k = 128, 64, 12, 32
    prep_W = synth.weights(21, 48, C)                      # a down projection, for a realistic perm / scale
    amax = np.abs(np.random.default_rng(3).standard_normal(C)).astype(np.float32) + 0.1
    o = oracle.prepare(prep_W, amax, 0.5, k)
    Wu, Wg = synth.weights(22, C, H), synth.weights(23, C, H)
    X = synth.bf16_to_f32(synth.weights(24, T, H)).astype(np.float64) * 50.0
    up, gate = oracle.fold_producer(Wu, Wg, o["perm"], o["inv_s"], k)
    f = lambda b: synth.bf16_to_f32(b).astype(np.float64)
    silu = lambda v: v / (1.0 + np.exp(-v))
    u, g = X @ f(Wu).T, X @ f(Wg).T
    Z = u * silu(g)
    Zt = (Z * o["inv_s"].astype(np.float64))[:, o["perm"]]
    u2, g2 = X @ f(up).T, X @ f(gate).T
    assert np.array_equal(g2, g[:, o["perm"]])
    bound = 2.0 ** -9 * (np.abs(X) @ np.abs(f(Wu)).T * o["inv_s"].astype(np.float64))[:, o["perm"]] * np.abs(silu(g2))
    assert np.all(np.abs(u2 * silu(g2) - Zt) <= bound + 1e-300)
