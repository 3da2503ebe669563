"""Pins for the oracle's normalised reconstruction error (text after Eq. (3)) and its alpha grid search
(Algorithm 1 steps 1-2, 8-10) against values worked by hand in tests/golden/alpha_search_worked.txt."""
import os
from fractions import Fraction

import numpy as np

from paper_2609_22106_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alpha_search_worked.txt")


def load():
    d = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split(":", 1)
            d[key.strip()] = val.strip()
    return d


def frac(text):
    """'a / b' or 'a/b' or 'a' -> float of the exact ratio."""
    parts = [p.strip() for p in text.split("/")]
    return float(Fraction(parts[0]) / Fraction(parts[1])) if len(parts) == 2 else float(Fraction(parts[0]))


def search_layer():
    z = np.ones((1, 32), np.float32)
    z[0, :2] = [16, 4]
    w = np.full((1, 32), 3, np.float32)
    w[0, :2] = [1, 1]
    return synth.f32_to_bf16(w), synth.f32_to_bf16(z)


def test_error_norm_on_a_hand_worked_matrix(oracle):
    g = load()
    y_hat = np.array([[1.0, 2.0], [3.0, 4.0]])
    y = np.array([[1.0, 0.0], [0.0, 4.0]])
    want = (float(g["frob_num_sq"]) / float(g["frob_den_sq"])) ** 0.5
    assert abs(oracle.nrmse(y_hat, y) - want) < 1e-15
    # the wrong normalisations a slip would produce are far away
    for wrong in ((13 / 30) ** 0.5, 13 / 17, 3 / 4):
        assert abs(oracle.nrmse(y_hat, y) - wrong) > 1e-3
    assert oracle.nrmse(y, y) == 0.0


def test_error_of_the_worked_preparation_example(oracle):
    g = load()
    y = np.array([[61.41259765625]])
    assert abs(oracle.nrmse(np.array([[61.4375]]), y) - frac(g["worked_err_prquant"])) < 1e-18
    assert abs(oracle.nrmse(np.array([[62.0]]), y) - frac(g["worked_err_plain"])) < 1e-18


def test_three_candidate_search_decided_by_hand(oracle):
    g = load()
    W, Z = search_layer()
    assert float(oracle.matmul_bf16(Z, W)[0, 0]) == float(g["search_y"])
    for k, key in ((0, "k0"), (32, "k32")):
        yhat_want = [float(v) for v in g[f"search_yhat_{key}"].split()]
        err_want = [frac(v) for v in g[f"search_err_{key}"].split()]
        best, alpha, errs = oracle.alpha_search(W, Z, [0.0, 0.5, 1.0], k)
        assert alpha == float(g[f"search_winner_{key}"]) and best["alpha"] == alpha
        assert np.allclose(errs, err_want, rtol=0, atol=1e-15)
        # and the products behind those errors
        amax = oracle.channel_amax(Z)
        assert np.array_equal(amax, np.abs(synth.bf16_to_f32(Z))[0])
        for a, want in zip((0.0, 0.5, 1.0), yhat_want):
            y_hat, _, _ = oracle.linear(Z, oracle.prepare(W, amax, a, k))
            assert float(y_hat[0, 0]) == want


def test_search_returns_the_minimum_not_the_first_candidate(oracle):
    g = load()
    W, Z = search_layer()
    _, alpha, errs = oracle.alpha_search(W, Z, [0.0, 1.0], 0)
    assert alpha == float(g["search_winner_grid_0_1"]) and errs[1] < errs[0]


def test_search_keeps_the_first_of_equal_minima(oracle):
    g = load()
    W, Z = search_layer()
    _, alpha, errs = oracle.alpha_search(W, Z, [1.0, 0.5, 0.0], 32)
    assert errs[0] == 0.0 and errs[1] == 0.0
    assert alpha == float(g["search_winner_k32_grid_1_0.5_0"])
