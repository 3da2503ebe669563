"""Pins for the oracle's offline prep (Algorithm 1) and the augmented product (Eq. (3))."""
import itertools
import os

import numpy as np
import pytest

from paper_2609_22106_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def unpack(codes):
    codes = np.asarray(codes, np.uint8)
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), np.uint8)
    out[..., 0::2] = codes & 0xF
    out[..., 1::2] = codes >> 4
    return out


def expand(tok_list):
    out = []
    for t in tok_list:
        if "*" in t:
            v, n = t.split("*")
            out += [v] * int(n)
        else:
            out.append(t)
    return out


def expand_ranges(tok_list):
    out = []
    for t in tok_list:
        if "-" in t and not t.startswith("-"):
            a, b = t.split("-")
            out += list(range(int(a), int(b) + 1))
        else:
            out.append(int(t))
    return out


def load_example():
    d = {}
    with open(os.path.join(GOLDEN, "prep_worked_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split(":", 1)
            d[key.strip()] = val.split()
    return d


def example_weight():
    W = np.ones(64, np.float32)
    W[32:] = 0.5
    W[[0, 1, 2, 3]] = [6, 0.3125, 2.75, 5.5]
    W[[32, 33, 34]] = [3, 1.25, 0.10009765625]
    return synth.f32_to_bf16(W.reshape(1, 64))


def test_worked_example(oracle):
    g = load_example()
    W = example_weight()
    assert np.array_equal(synth.bf16_to_f32(W)[0, 34], np.float32(0.10009765625))
    amax = np.ones(64, np.float32) * 3.0  # irrelevant at alpha = 0
    p = oracle.prepare(W, amax, 0.0, 32)
    assert np.all(p["s"] == 1) and np.all(p["inv_s"] == 1)
    want_err = np.zeros(64)
    for tok in g["col_err"]:
        j, v = tok.split("=")
        want_err[int(j)] = float(v)
    np.testing.assert_array_equal(p["col_err"], want_err)
    assert list(p["perm"][32:]) == expand_ranges(g["selected"])
    assert list(p["perm"][:32]) == expand_ranges(g["head"])
    assert int(p["wscales"][0, 0]) == int(g["head_scale_byte"][0])
    assert int(p["wscales"][0, 1]) == int(g["tail_scale_byte"][0])
    assert int(p["wscales"][0, 2]) == int(g["residual_scale_byte"][0])
    codes = unpack(p["wcodes"])[0]
    assert list(codes[32:64]) == [int(c, 16) for c in expand(g["tail_codes"])]
    assert list(codes[64:96]) == [int(c, 16) for c in expand(g["residual_codes"])]
    np.testing.assert_array_equal(p["R"][0], np.array([float(v) for v in expand(g["residual"])], np.float32))
    x = synth.f32_to_bf16(np.ones((1, 64), np.float32))
    y, ac, asc = oracle.linear(x, p)
    assert np.all(asc == 125) and np.all(unpack(ac) == 6)
    assert y[0, 0] == float(g["y_prquant"][0])
    p0 = oracle.prepare(W, amax, 0.0, 0)
    y0, _, _ = oracle.linear(x, p0)
    assert y0[0, 0] == float(g["y_plain_mxfp4_k0"][0])
    assert oracle.matmul_bf16(x, W)[0, 0] == float(g["y_exact"][0])


def make_layer(seed, N, K, M, T=64):
    rng = np.random.default_rng(seed)
    W = synth.f32_to_bf16(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    gain = np.exp(rng.standard_normal(K)).astype(np.float32)
    gain[rng.choice(K, max(1, K // 50), replace=False)] *= 30
    x = synth.f32_to_bf16(rng.standard_t(3, (M, K)).astype(np.float32) * gain)
    z = synth.f32_to_bf16(rng.standard_t(3, (T, K)).astype(np.float32) * gain)
    return W, x, z


def test_k0_is_plain_mxfp4(oracle):
    """k = 0: identity permutation, no residual; with alpha = 0 it is the textbook MXFP4 W4A4 product."""
    W, x, z = make_layer(1, 24, 128, 5)
    amax = oracle.channel_amax(z)
    p = oracle.prepare(W, amax, 0.0, 0)
    assert np.array_equal(p["perm"], np.arange(128))
    assert p["wcodes"].shape == (24, 64) and p["wscales"].shape == (24, 4)
    wc, ws = oracle.quantize_rows(synth.bf16_to_f32(W))
    assert np.array_equal(wc, p["wcodes"]) and np.array_equal(ws, p["wscales"])
    y, ac, asc = oracle.linear(x, p)
    xc, xs = oracle.quantize_rows(synth.bf16_to_f32(x))
    assert np.array_equal(ac, xc) and np.array_equal(asc, xs)
    want = oracle.dequantize_rows(xc, xs) @ oracle.dequantize_rows(wc, ws).T
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-12)
    # with alpha != 0 only the scaling changes; the permutation stays the identity
    p5 = oracle.prepare(W, amax, 0.5, 0)
    assert np.array_equal(p5["perm"], np.arange(128))
    w0 = (synth.bf16_to_f32(W).astype(np.float64) * p5["s"].astype(np.float64)).astype(np.float32)
    wc5, ws5 = oracle.quantize_rows(w0)
    assert np.array_equal(wc5, p5["wcodes"]) and np.array_equal(ws5, p5["wscales"])


def test_scale_definition(oracle):
    amax = np.array([0.0, 1e-7, 1.0, 4.0, 9.0, 1234.5], np.float32)
    for alpha in (0.0, 0.25, 0.5, 0.75, 1.0, 0.3):
        s, inv_s = oracle.scales_from_amax(amax, alpha)
        a = np.maximum(amax.astype(np.float64), 1e-5)
        np.testing.assert_allclose(s, a ** alpha, rtol=2e-7)
        np.testing.assert_allclose(inv_s.astype(np.float64) * s, 1.0, rtol=2e-7)
    s, _ = oracle.scales_from_amax(amax, 0.5)
    assert s[3] == 2.0 and s[4] == 3.0 and s[2] == 1.0
    s, _ = oracle.scales_from_amax(amax, 0.25)
    assert s[3] == np.float32(np.sqrt(2.0))
    z = synth.f32_to_bf16(np.array([[1, -7, 0.5], [-3, 2, 0.25]], np.float32))
    assert list(oracle.channel_amax(z)) == [3, 7, 0.5]


def test_permutation_and_scaling_leave_the_exact_product_unchanged(oracle):
    """Eq. (1): (Z D^-1 P)(W D P)^T = Z W^T."""
    W, x, z = make_layer(2, 16, 128, 6)
    p = oracle.prepare(W, oracle.channel_amax(z), 0.5, 32)
    perm = p["perm"]
    assert sorted(perm.tolist()) == list(range(128))
    Wf = synth.bf16_to_f32(W).astype(np.float64)
    xf = synth.bf16_to_f32(x).astype(np.float64)
    y = xf @ Wf.T
    # permutation alone: exact up to summation order
    np.testing.assert_allclose(xf[:, perm] @ Wf[:, perm].T, y, rtol=1e-12, atol=1e-12)
    # with the fp32-rounded scale pair: equal to fp32 rounding of s and 1/s
    s = p["s"].astype(np.float64)
    inv_s = p["inv_s"].astype(np.float64)
    yt = (xf * inv_s)[:, perm] @ (Wf * s)[:, perm].T
    np.testing.assert_allclose(yt, y, rtol=1e-5, atol=1e-5 * np.abs(y).max())


def brute_topk(err, k):
    order = sorted(range(len(err)), key=lambda j: (-err[j], j))
    return sorted(order[:k])


def test_topk_against_brute_force_and_subset_search(oracle):
    rng = np.random.default_rng(5)
    for trial in range(6):
        N, K, k = 4, 64, 32
        W = synth.f32_to_bf16(rng.standard_normal((N, K)).astype(np.float32) * np.exp(rng.standard_normal(K)).astype(np.float32))
        amax = np.abs(rng.standard_normal(K)).astype(np.float32) + 0.1
        p = oracle.prepare(W, amax, 0.5, k)
        # column errors from their definition, with numpy and the oracle's own dequantiser only
        w0 = (synth.bf16_to_f32(W).astype(np.float64) * p["s"].astype(np.float64)).astype(np.float32)
        c, s = oracle.quantize_rows(w0)
        d = w0.astype(np.float64) - oracle.dequantize_rows(c, s)
        err = np.zeros(K)
        for n in range(N):
            err += d[n] * d[n]
        np.testing.assert_array_equal(p["col_err"], err)
        assert p["topk"].tolist() == brute_topk(err.tolist(), k)
        assert p["perm"][: K - k].tolist() == sorted(set(range(K)) - set(p["topk"].tolist()))
    # exhaustive: on 8 "channels" embedded in one block row, the chosen set maximises the summed error
    K, k = 64, 32
    W = synth.f32_to_bf16(rng.standard_normal((3, K)).astype(np.float32))
    p = oracle.prepare(W, np.ones(K, np.float32), 0.0, k)
    tot = p["col_err"][p["topk"]].sum()
    order = np.argsort(-p["col_err"], kind="stable")
    assert abs(tot - p["col_err"][order[:k]].sum()) == 0
    small = p["col_err"][:10]
    best = max(itertools.combinations(range(10), 4), key=lambda c: (sum(small[list(c)]), [-i for i in c]))
    assert sorted(best) == brute_topk(small.tolist(), 4)


def test_designed_tie_breaks_to_lower_index(oracle):
    W = example_weight()
    p = oracle.prepare(W, np.ones(64, np.float32), 0.0, 32)
    assert p["col_err"][2] == p["col_err"][33] == 0.0625
    # shrink k so that only one of the tied channels fits: the lower index wins
    W2 = np.tile(synth.bf16_to_f32(W), (1, 1))
    W96 = np.concatenate([W2, np.ones((1, 32), np.float32)], axis=1)
    p2 = oracle.prepare(synth.f32_to_bf16(W96), np.ones(96, np.float32), 0.0, 32)
    sel = p2["topk"].tolist()
    assert 3 in sel and 2 in sel and 33 in sel and 1 in sel and 34 in sel
    order = sorted(range(96), key=lambda j: (-p2["col_err"][j], j))
    assert order[:5] == [3, 2, 33, 1, 34]


def test_residual_identity_and_error_never_increases(oracle):
    """Eq. (2): deq(Q(W_tail)) + R = W_tail exactly in fp32; compensation cannot increase the
    tail-column reconstruction error because 0 is always a candidate of the rounding."""
    W, x, z = make_layer(3, 48, 256, 4)
    for alpha in (0.0, 0.5, 1.0):
        p = oracle.prepare(W, oracle.channel_amax(z), alpha, 64)
        K, k = 256, 64
        w0 = (synth.bf16_to_f32(W).astype(np.float64) * p["s"].astype(np.float64)).astype(np.float32)
        wt = w0[:, p["perm"]]
        deq = oracle.dequantize_rows(p["wcodes"], p["wscales"])
        R = p["R"].astype(np.float64)
        np.testing.assert_array_equal(deq[:, K - k:K] + R, wt[:, K - k:].astype(np.float64))
        # the difference is exactly representable in fp32
        np.testing.assert_array_equal(R.astype(np.float32).astype(np.float64), R)
        left = np.abs(R - deq[:, K:])
        assert np.all(left <= np.abs(R))
        assert np.linalg.norm(left) < 0.6 * np.linalg.norm(R)
        # head blocks are Q of the permuted scaled weight, residual blocks are Q(R)
        c, s = oracle.quantize_rows(wt)
        assert np.array_equal(c, p["wcodes"][:, : K // 2]) and np.array_equal(s, p["wscales"][:, : K // 32])
        cr, sr = oracle.quantize_rows(p["R"])
        assert np.array_equal(cr, p["wcodes"][:, K // 2:]) and np.array_equal(sr, p["wscales"][:, K // 32:])


def test_block_aligned_copy_equals_quantising_the_concatenation(oracle):
    """Kernel design paragraph: copying the quantised tail with its scales = Q([Zt, Zt_tail])."""
    rng = np.random.default_rng(9)
    z = rng.standard_t(3, (7, 160)).astype(np.float32)
    c, s = oracle.quantize_rows(z)
    for k in (32, 64, 160):
        ca, sa = oracle.augment_act(c, s, k)
        cc, sc = oracle.quantize_rows(np.concatenate([z, z[:, 160 - k:]], axis=1))
        assert np.array_equal(ca, cc) and np.array_equal(sa, sc)
    with pytest.raises(ValueError):
        oracle.augment_act(c, s, 48)


def test_augmented_product_is_main_plus_correction(oracle):
    """Eq. (3): one product over K + k = main product + tail activation times residual."""
    W, x, z = make_layer(4, 40, 192, 9)
    p = oracle.prepare(W, oracle.channel_amax(z), 0.5, 64)
    y, ac, asc = oracle.linear(x, p)
    K, k = 192, 64
    A = oracle.dequantize_rows(ac, asc)
    Wd = oracle.dequantize_rows(p["wcodes"], p["wscales"])
    main = A @ Wd[:, :K].T
    corr = A[:, K - k:] @ Wd[:, K:].T
    np.testing.assert_allclose(y, main + corr, rtol=1e-12, atol=1e-12 * np.abs(y).max())
    # activation side of Eq. (1): gather by perm, multiply by the stored reciprocal, round to fp32
    xt = (synth.bf16_to_f32(x).astype(np.float64) * p["inv_s"].astype(np.float64)).astype(np.float32)[:, p["perm"]]
    c, s = oracle.quantize_rows(xt)
    assert np.array_equal(c, ac) and np.array_equal(s, asc)
    # compensation helps against the unquantised target on heavy-tailed data
    y_true = oracle.matmul_bf16(x, W)
    p0 = oracle.prepare(W, oracle.channel_amax(z), 0.5, 0)
    y0, _, _ = oracle.linear(x, p0)
    assert oracle.nrmse(y, y_true) <= oracle.nrmse(y0, y_true) * 1.05


def test_transposed_operand_would_fail(oracle):
    """y is (tokens, outputs): a swapped operand order changes the shape."""
    W, x, z = make_layer(6, 8, 64, 3)
    p = oracle.prepare(W, oracle.channel_amax(z), 0.0, 0)
    y, _, _ = oracle.linear(x, p)
    assert y.shape == (3, 8)
    y_true = oracle.matmul_bf16(x, W)
    assert oracle.nrmse(y, y_true) < 0.3


def test_alpha_search_picks_first_minimum(oracle):
    cfg = synth.tiny_config(0)
    best, alpha, errs = oracle.alpha_search(cfg["W"], cfg["zcal"], cfg["alphas"], cfg["k"])
    assert len(errs) == 5 and alpha == cfg["alphas"][int(np.argmin(errs))]
    assert best["alpha"] == alpha
    assert min(errs) < errs[0]  # scaling helps with x50 outlier channels
