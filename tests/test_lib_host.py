"""CPU-side checks of libprq: it loads, exports every declared symbol, validates arguments without
touching a GPU, and its host prep (Algorithm 1 steps 3-7, 11) is bit-exact against the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_22106_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "prq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prq_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(prq):
    names = declared_functions()
    assert len(names) >= 15
    L = prq.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(prq.EXPORTS) == names


def test_status_strings(prq):
    assert prq.status_string(0) == "ok"
    assert "invalid" in prq.status_string(1)
    assert "wait" in prq.status_string(6)
    assert prq.kernel_launch_count() == 0 or prq.kernel_launch_count() > 0


def test_act_bytes(prq):
    # dense: codes M*K/2, row scales M*K/32, tile-ordered scales = stages x 128-row groups x 1024
    assert prq.act_bytes(2048, 9728, 256, 1, prq.BUF_CODES) == 2048 * 9728 // 2
    assert prq.act_bytes(2048, 9728, 256, 1, prq.BUF_SCALES_ROW) == 2048 * 9728 // 32
    assert prq.act_bytes(2048, 9728, 256, 1, prq.BUF_SCALES_SF) == (38 + 1) * 16 * 1024
    assert prq.act_bytes(1, 9728, 0, 1, prq.BUF_SCALES_SF) == 38 * 1024
    assert prq.act_bytes(16, 256, 32, 1, prq.BUF_SCALES_SF) == 2 * 1024
    # grouped: one padding group per expert
    assert prq.act_bytes(512, 768, 64, 128, prq.BUF_SCALES_SF) == 4 * (4 + 128) * 1024
    # invalid
    assert prq.act_bytes(16, 250, 0, 1, prq.BUF_CODES) == 0
    assert prq.act_bytes(16, 256, 48, 1, prq.BUF_CODES) == 0
    assert prq.act_bytes(-1, 256, 0, 1, prq.BUF_CODES) == 0


def test_argument_validation_without_a_gpu(prq):
    L = prq.lib()
    W = np.zeros((4, 64), np.uint16)
    amax = np.ones(64, np.float32)
    h = ctypes.c_void_p()
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    assert L.prq_prepare_weights(None, 1, 4, 64, p(amax), 0.5, 0, ctypes.byref(h)) == 1
    assert L.prq_prepare_weights(p(W), 1, 4, 60, p(amax), 0.5, 0, ctypes.byref(h)) == 1
    assert L.prq_prepare_weights(p(W), 1, 4, 64, p(amax), 0.5, 48, ctypes.byref(h)) == 1
    assert L.prq_prepare_weights(p(W), 1, 4, 64, p(amax), 0.5, 96, ctypes.byref(h)) == 1
    assert L.prq_prepare_weights(p(W), 0, 4, 64, p(amax), 0.5, 0, ctypes.byref(h)) == 1
    assert L.prq_prepare_weights(p(W), 1, 4, 64, p(amax), float("nan"), 0, ctypes.byref(h)) == 1
    assert L.prq_quantize_act(None, 0, None, 4, 64, None, None, None, None, None) == 1
    assert L.prq_linear(None, None, None, 4, None, 64, 0, None, 0, None) == 1
    assert L.prq_linear_grouped(None, None, None, None, 4, None, 64, 0, None) == 1
    assert L.prq_weights_info(None, None, None, None, None, None) == 1
    assert L.prq_weights_get(None, 0, 0, None, 0) == 1
    assert L.prq_linear_workspace_bytes(None, 4) == 0
    assert L.prq_forward_host_scratch_bytes(None, 4) == 0
    L.prq_weights_free(None)  # no-op


def host_vs_oracle(prq, oracle, W, amax, alpha, k, scale_search=False):
    got = prq.prepare_weights_host(W, amax, alpha, k, scale_search=scale_search)
    want = oracle.prepare(W, amax, float(np.float32(alpha)), k, scale_search=scale_search)
    assert np.array_equal(got["s"], want["s"])
    assert np.array_equal(got["inv_s"], want["inv_s"])
    assert np.array_equal(got["col_err"], want["col_err"])
    assert np.array_equal(got["perm"], want["perm"])
    assert np.array_equal(got["scales"], want["wscales"])
    assert np.array_equal(got["codes"], want["wcodes"])
    return got


def test_host_prep_bit_exact_tiny_config(prq, oracle):
    cfg = synth.tiny_config(0)
    amax = oracle.channel_amax(cfg["zcal"])
    for alpha in cfg["alphas"]:
        host_vs_oracle(prq, oracle, cfg["W"], amax, alpha, cfg["k"])
    host_vs_oracle(prq, oracle, cfg["W"], amax, 0.5, 0)
    host_vs_oracle(prq, oracle, cfg["W"], amax, 0.3, 64)  # off-grid alpha goes through pow


def test_host_prep_bit_exact_heavy_tailed(prq, oracle):
    L = synth.layer(1, 96, 1024, 4, T_cal=64)
    amax = oracle.channel_amax(L["zcal"])
    for k in (0, 128, 256):
        host_vs_oracle(prq, oracle, L["W"], amax, 0.5, k)
    # extremes: dead channels, huge and tiny activations
    amax2 = amax.copy()
    amax2[:5] = 0.0
    amax2[5:10] = 1e30
    amax2[10:15] = 1e-30
    host_vs_oracle(prq, oracle, L["W"], amax2, 1.0, 128)


def test_host_prep_with_weight_scale_search_bit_exact(prq, oracle):
    """The E8M0-W option (weight-side block-scale search): the library's prep against the oracle's, bit for
    bit, and against its own result without the option (same ranking, some scales one step away)."""
    cfg = synth.tiny_config(0)
    amax = oracle.channel_amax(cfg["zcal"])
    host_vs_oracle(prq, oracle, cfg["W"], amax, 0.5, cfg["k"], scale_search=True)
    L = synth.layer(1, 96, 1024, 4, T_cal=64)
    amax = oracle.channel_amax(L["zcal"])
    changed = 0
    for k in (0, 128):
        on = host_vs_oracle(prq, oracle, L["W"], amax, 0.5, k, scale_search=True)
        off = prq.prepare_weights_host(L["W"], amax, 0.5, k)
        assert np.array_equal(on["perm"], off["perm"]) and np.array_equal(on["col_err"], off["col_err"])
        # main part only: with the option R is the residual of a different quantisation
        d = on["scales"][:, : 1024 // 32].astype(int) - off["scales"][:, : 1024 // 32].astype(int)
        assert np.abs(d).max() <= 1
        changed += int((d != 0).sum())
    assert changed > 0
    # a struct_size that is too small is refused
    o = prq.PrepOpts(4, 1)
    out = prq.prepare_weights_host(L["W"], amax, 0.5, 0)
    rc = prq.lib().prq_prepare_weights_host_opts(
        L["W"].ctypes.data, 96, 1024, amax.ctypes.data, 0.5, 0, ctypes.cast(ctypes.pointer(o), ctypes.c_void_p),
        out["codes"].ctypes.data, out["scales"].ctypes.data, out["perm"].ctypes.data, None, None, None)
    assert rc == 1


def test_host_prep_worked_example(prq):
    W = np.ones(64, np.float32)
    W[32:] = 0.5
    W[[0, 1, 2, 3]] = [6, 0.3125, 2.75, 5.5]
    W[[32, 33, 34]] = [3, 1.25, 0.10009765625]
    got = prq.prepare_weights_host(synth.f32_to_bf16(W.reshape(1, 64)), np.ones(64, np.float32), 0.0, 32)
    assert got["perm"][32:].tolist() == list(range(30)) + [33, 34]
    assert got["scales"][0].tolist() == [126, 127, 124]
    assert got["col_err"][3] == 0.25 and got["col_err"][2] == 0.0625 and got["col_err"][33] == 0.0625


def test_host_prep_rejects_non_finite(prq):
    W = synth.f32_to_bf16(np.ones((2, 64), np.float32))
    W[0, 3] = 0x7F80  # +inf
    with pytest.raises(prq.PrqError) as e:
        prq.prepare_weights_host(W, np.ones(64, np.float32), 0.5, 0)
    assert e.value.code == 7
    amax = np.ones(64, np.float32)
    amax[0] = np.nan
    with pytest.raises(prq.PrqError):
        prq.prepare_weights_host(synth.f32_to_bf16(np.ones((2, 64), np.float32)), amax, 0.5, 0)


def test_fold_producer_bit_exact(prq, oracle):
    """prq_fold_producer (Eq. (1), host buffers) against the oracle: the hand-worked roundings (double-rounding
    traps and subnormals included), a heavy-tailed random case with the duplicated tail, and without a gate."""
    import os

    golden = os.path.join(os.path.dirname(__file__), "golden", "bf16_fold_roundings.txt")
    for line in open(golden):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w, s, e, _ = [p.strip() for p in line.split(";")]
        W = np.array([[int(w, 16)]], np.uint16)
        inv_s = np.array([int(s, 16)], np.uint32).view(np.float32)
        up, gate = prq.fold_producer(np.array([0], np.int32), inv_s, 0, W, W)
        assert int(up[0, 0]) == int(e, 16), line
        assert int(gate[0, 0]) == int(w, 16)
    rng = np.random.default_rng(5)
    C, H, k = 384, 200, 64
    Wu, Wg = synth.weights(31, C, H), synth.weights(32, C, H)
    Wu[0, :3] = [0x0001, 0x8003, 0x7F7F]
    perm = rng.permutation(C).astype(np.int32)
    inv_s = np.exp(rng.normal(0, 4, C)).astype(np.float32)
    for dup in (False, True):
        up, gate = prq.fold_producer(perm, inv_s, k, Wu, Wg, duplicate_tail=dup)
        oup, ogate = oracle.fold_producer(Wu, Wg, perm, inv_s, k, dup=dup)
        assert np.array_equal(up, oup) and np.array_equal(gate, ogate)
    up, gate = prq.fold_producer(perm, inv_s, k, Wu)
    assert gate is None and np.array_equal(up, oracle.fold_producer(Wu, Wg, perm, inv_s, k)[0])
    bad = perm.copy()
    bad[3] = C
    with pytest.raises(prq.PrqError):
        prq.fold_producer(bad, inv_s, k, Wu)


def test_mxfp8_host_prep_is_bit_exact(prq, oracle):
    """Second format: the library's host preparation (no device involved) against the oracle, code for code."""
    for seed, (N, K), alpha in ((1, (40, 96), 0.5), (2, (17, 256), 0.0), (3, (64, 64), 0.75), (4, (8, 32), 0.3)):
        L = synth.layer(60 + seed, N, K, 4, T_cal=32)
        amax = oracle.channel_amax(L["zcal"])
        amax[0] = 0.0                                         # a dead channel takes the floor
        got = prq.prepare_weights_host(L["W"], amax, alpha, 0, fmt=prq.FMT_MXFP8)
        o = oracle.fp8_prepare(L["W"], amax, float(np.float32(alpha)))
        assert np.array_equal(got["s"], o["s"]) and np.array_equal(got["inv_s"], o["inv_s"])
        assert np.array_equal(got["scales"], o["wscales"])
        assert np.array_equal(got["codes"], o["wcodes"])
        assert np.array_equal(got["perm"], np.arange(K))
    # blocks on the format's decision boundaries (ties, saturation band, subnormal steps), unit scales
    rows = []
    for vals in ([448, 1, .5, -3, 2 ** -9, 296], [256, 17, 19, 272, 304], [500, 464, 462, -510], [512, 3, 1],
                 [256, 7 * 2 ** -9, 7.5 * 2 ** -9, -0.5 * 2 ** -9], [2.0 ** -20, 2.0 ** -30, -2.0 ** -29]):
        b = np.zeros(32, np.float32); b[: len(vals)] = vals; rows.append(b)
    Wb = synth.f32_to_bf16(np.stack(rows))
    assert np.array_equal(synth.bf16_to_f32(Wb), np.stack(rows))
    got = prq.prepare_weights_host(Wb, np.ones(32, np.float32), 0.0, 0, fmt=prq.FMT_MXFP8)
    o = oracle.fp8_prepare(Wb, np.ones(32, np.float32), 0.0)
    assert np.array_equal(got["codes"], o["wcodes"]) and np.array_equal(got["scales"], o["wscales"])
    # the format carries no tail
    with pytest.raises(prq.PrqError):
        prq.prepare_weights_host(Wb, np.ones(32, np.float32), 0.0, 32, fmt=prq.FMT_MXFP8)
