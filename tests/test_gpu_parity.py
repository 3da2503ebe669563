"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Codes, scale bytes, permutations and top-k sets are compared bit for bit; GEMM outputs
within max |y - y_ref| <= 2e-3 (||y_ref||_inf + 1) on fp32 output."""
import os

import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def to_dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


def check_prep(prq, oracle, w, W, amax, alpha, k):
    o = oracle.prepare(W, amax, float(np.float32(alpha)), k)
    assert np.array_equal(w.get(prq.FIELD_PERM), o["perm"])
    assert np.array_equal(w.get(prq.FIELD_TOPK), o["topk"])
    assert np.array_equal(w.get(prq.FIELD_S), o["s"])
    assert np.array_equal(w.get(prq.FIELD_INV_S), o["inv_s"])
    assert np.array_equal(w.get(prq.FIELD_COL_ERR), o["col_err"])
    assert np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"])
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"])
    return o


def run_quant(prq, oracle, w, o, x, mode):
    M, K = x.shape
    codes, srow, sf = prq.quantize_act(w, to_dev_bf16(x), mode, row_scales=True)
    assert prq.last_device_status() == 0
    if mode == prq.ACT_IDENTITY:
        oc, osc = oracle.quantize_act(x)
    else:
        oc, osc = oracle.quantize_act(x, o["perm"], o["inv_s"])
    got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
    got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
    assert np.array_equal(got_s, osc)
    assert np.array_equal(got_c, oc)
    _, sa = oracle.augment_act(oc, osc, w.k_tail)
    want_sf = prq_ref.expected_sf(sa, K, w.k_tail)
    assert np.array_equal(sf.cpu().numpy()[: want_sf.size], want_sf)
    return codes, sf, oc, osc


def run_linear(prq, oracle, w, o, codes, sf, oc, osc, M, rows=None):
    """fp32 output against the oracle on all rows (or a sample of rows)."""
    ldy = w.N + 8
    y_buf = torch.full((M + 2, ldy), 12345.0, dtype=torch.float32, device="cuda")
    y_view = y_buf[1: M + 1]
    prq.linear(w, codes, sf, M, prq.F32, out=y_view)
    assert prq.last_device_status() == 0
    y_all = y_buf.cpu().numpy()
    # nothing outside the M x N window was written
    assert np.all(y_all[0] == 12345.0) and np.all(y_all[-1] == 12345.0) and np.all(y_all[:, w.N:] == 12345.0)
    y = y_all[1: M + 1, : w.N].astype(np.float64)
    sel = np.arange(M) if rows is None else rows
    ca, sa = oracle.augment_act(oc[sel], osc[sel], w.k_tail)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    err = np.abs(y[sel] - y_ref).max()
    assert err <= prq_ref.tolerance(y_ref), (err, prq_ref.tolerance(y_ref))
    return y, y_ref


def layer_case(prq, oracle, N, K, M, k, alpha, mode, seed=0):
    L = synth.layer(90 + seed, N, K, M, T_cal=64)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, alpha, k)
    o = check_prep(prq, oracle, w, L["W"], amax, alpha, k)
    codes, sf, oc, osc = run_quant(prq, oracle, w, o, L["x"], mode)
    y, y_ref = run_linear(prq, oracle, w, o, codes, sf, oc, osc, M)
    w.free()
    return y, y_ref


def test_tiny_config_end_to_end(prq, oracle):
    """Config 0: 16 x 256 activations with 4 outlier channels, W 256 x 256, alpha grid, k = 32."""
    cfg = synth.tiny_config(0)
    amax = oracle.channel_amax(cfg["zcal"])
    for alpha in cfg["alphas"]:
        w = prq.prepare_weights(cfg["W"], amax, alpha, cfg["k"])
        o = check_prep(prq, oracle, w, cfg["W"], amax, alpha, cfg["k"])
        for mode in (prq.ACT_SCALE_PERM, prq.ACT_IDENTITY):
            codes, sf, oc, osc = run_quant(prq, oracle, w, o, cfg["x"], mode)
            run_linear(prq, oracle, w, o, codes, sf, oc, osc, 16)
        w.free()


def test_alpha_search_matches_oracle(prq, oracle):
    cfg = synth.tiny_config(0)
    w, alpha, errs = prq.prepare_weights_search(cfg["W"], cfg["zcal"], cfg["alphas"], cfg["k"])
    best, o_alpha, o_errs = oracle.alpha_search(cfg["W"], cfg["zcal"], cfg["alphas"], cfg["k"])
    # per-alpha errors agree to fp32 accumulation; the chosen alpha is the oracle's, or one whose oracle
    # error is within 1e-4 (relative) of the oracle's best
    np.testing.assert_allclose(errs, o_errs, rtol=1e-4)
    assert alpha == o_alpha or o_errs[cfg["alphas"].index(alpha)] <= min(o_errs) * (1 + 1e-4)
    assert w.alpha == alpha
    check_prep(prq, oracle, w, cfg["W"], oracle.channel_amax(cfg["zcal"]), alpha, cfg["k"])
    w.free()


def adversarial_rows():
    """Blocks that sit on every decision boundary of the quantiser (all values exact in bf16)."""
    rows = []
    blk = np.zeros(32, np.float32); blk[:6] = [6, -3, 1.5, 0.5, 0, -0.0]; rows.append(blk)
    blk = np.zeros(32, np.float32); blk[:9] = [4, .25, .75, 1.25, 1.75, 2.5, 3.5, -.25, -5]; rows.append(blk)
    blk = np.zeros(32, np.float32); blk[:5] = [7.5, 5.0, 5.03125, -7.96875, 6]; rows.append(blk)
    blk = np.zeros(32, np.float32); blk[:5] = [8, 7.96875, 5, 3, 1]; rows.append(blk)
    blk = np.zeros(32, np.float32); blk[0] = 2.0 ** -130; rows.append(blk)       # fp32-subnormal amax
    blk = np.zeros(32, np.float32); blk[:2] = [1.5 * 2.0 ** 127, 2.0 ** 125]; rows.append(blk)
    rows.append(np.zeros(32, np.float32))                                        # all-zero block
    blk = np.full(32, -0.0, np.float32); rows.append(blk)                        # all negative zero
    blk = np.zeros(32, np.float32); blk[:4] = [1, -2.0 ** -100, 2.0 ** -100, -0.0]; rows.append(blk)
    for e in (-120, -60, -1, 0, 1, 60, 120):                                     # ties at many scales
        blk = (np.array([4, .25, .75, 1.25, 1.75, 2.5, 3.5, 5, 6, 7, 7.5] + [0] * 21, np.float32) * np.float32(2.0 ** e))
        blk[1::2] *= -1
        rows.append(blk)
    return np.stack(rows)


def test_quantiser_on_decision_boundaries(prq, oracle):
    blocks = adversarial_rows()
    nb = blocks.shape[0]
    rng = np.random.default_rng(0)
    # 40 rows x 256 columns, each row a random arrangement of the adversarial blocks
    x = np.stack([np.concatenate([blocks[i] for i in rng.integers(0, nb, 8)]) for _ in range(40)])
    xb = synth.f32_to_bf16(x)
    assert np.array_equal(synth.bf16_to_f32(xb).view(np.uint32), x.view(np.uint32))  # bf16-exact inputs
    W = synth.weights(3, 64, 256)
    w = prq.prepare_weights(W, np.ones(256, np.float32), 0.0, 64)
    o = oracle.prepare(W, np.ones(256, np.float32), 0.0, 64)
    run_quant(prq, oracle, w, o, xb, prq.ACT_IDENTITY)
    run_quant(prq, oracle, w, o, xb, prq.ACT_SCALE_PERM)
    w.free()


@pytest.mark.parametrize("M,K,k", [(1, 256, 0), (77, 2336, 96), (130, 1024, 1024), (300, 2304, 0), (513, 768, 64)])
def test_quantise_shapes(prq, oracle, M, K, k):
    L = synth.layer(91, 64, K, M, T_cal=32)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, 0.5, k)
    for mode in (prq.ACT_IDENTITY, prq.ACT_SCALE_PERM):
        run_quant(prq, oracle, w, o, L["x"], mode)
    w.free()


def test_quantise_strided_input(prq, oracle):
    L = synth.layer(92, 64, 512, 50, T_cal=32)
    w = prq.prepare_weights(L["W"], oracle.channel_amax(L["zcal"]), 0.5, 32)
    big = torch.zeros((50, 512 + 64), dtype=torch.bfloat16, device="cuda")
    big[:, :512] = to_dev_bf16(L["x"])
    codes, srow, sf = prq.quantize_act(w, big[:, :512], prq.ACT_IDENTITY, row_scales=True)
    oc, osc = oracle.quantize_act(L["x"])
    assert np.array_equal(codes.cpu().numpy()[: 50 * 256].reshape(50, 256), oc)
    assert np.array_equal(srow.cpu().numpy()[: 50 * 16].reshape(50, 16), osc)
    w.free()


@pytest.mark.parametrize("M", [1, 16, 17, 64, 100, 128])
def test_decode_path(prq, oracle, M):
    """M <= 128: weights on the MMA M axis, split-K with the workspace reduction."""
    layer_case(prq, oracle, N=640, K=2336, M=M, k=96, alpha=0.5, mode=prq.ACT_SCALE_PERM, seed=M)


@pytest.mark.parametrize("splits", [1, 2, 5, 10])
def test_decode_split_counts(prq, oracle, splits, monkeypatch):
    monkeypatch.setenv("PRQ_DECODE_SPLITS", str(splits))
    layer_case(prq, oracle, N=300, K=2560, M=8, k=128, alpha=0.5, mode=prq.ACT_IDENTITY)


@pytest.mark.parametrize("bn", [224, 240, 288])
@pytest.mark.parametrize("shape", [(300, 608, 2336, 96), (1000, 2560, 1024, 0), (260, 328, 512, 512)])
def test_prefill_tiles(prq, oracle, bn, shape, monkeypatch):
    """M > 128: the prefill kernel with its three tile widths (288 columns: the one-wave variant with a single
    accumulator, which all three shapes admit); ragged M and N, a reduction that is not a multiple of the stage,
    k = 0 and k = K."""
    monkeypatch.setenv("PRQ_PAIR_BN", str(bn))
    M, N, K, k = shape
    layer_case(prq, oracle, N=N, K=K, M=M, k=k, alpha=0.5, mode=prq.ACT_SCALE_PERM, seed=bn)


@pytest.mark.parametrize("shape", [(200, 256, 9728, 256), (129, 520, 4096, 128), (1500, 1024, 2560, 128), (4100, 768, 512, 64)])
def test_prefill_stream_k_splits(prq, oracle, shape):
    """Stream-K corner cases: a tile shared by dozens of CTAs (few tiles, long reduction), ranges that
    start and end inside tiles, more tiles than CTAs."""
    M, N, K, k = shape
    layer_case(prq, oracle, N=N, K=K, M=M, k=k, alpha=0.5, mode=prq.ACT_IDENTITY, seed=M)


def test_k0_runs_the_same_kernels_as_plain_mxfp4(prq, oracle):
    """k = 0: the product is plain W4A4 MXFP4 of (x, W D); with alpha = 0 of (x, W) themselves."""
    L = synth.layer(93, 256, 1024, 200, T_cal=32)
    w = prq.prepare_weights(L["W"], np.ones(1024, np.float32), 0.0, 0)
    codes, _, sf = prq.quantize_act(w, to_dev_bf16(L["x"]), prq.ACT_IDENTITY)
    y = prq.linear(w, codes, sf, 200).cpu().numpy().astype(np.float64)
    xc, xs = oracle.quantize_rows(synth.bf16_to_f32(L["x"]))
    wc, ws = oracle.quantize_rows(synth.bf16_to_f32(L["W"]))
    y_ref = oracle.dequantize_rows(xc, xs) @ oracle.dequantize_rows(wc, ws).T
    assert np.abs(y - y_ref).max() <= prq_ref.tolerance(y_ref)
    w.free()


def test_bf16_output(prq, oracle):
    """bf16 stores are checked against the rounded oracle value with one bf16 ulp of slack."""
    for M in (40, 300):
        L = synth.layer(94, 384, 1024, M, T_cal=32)
        amax = oracle.channel_amax(L["zcal"])
        w = prq.prepare_weights(L["W"], amax, 0.5, 128)
        o = oracle.prepare(L["W"], amax, 0.5, 128)
        codes, _, sf = prq.quantize_act(w, to_dev_bf16(L["x"]), prq.ACT_SCALE_PERM)
        y = prq.linear(w, codes, sf, M, prq.BF16).float().cpu().numpy().astype(np.float64)
        y_ref, _, _ = oracle.linear(L["x"], o)
        ulp = np.maximum(np.abs(y_ref), 2.0 ** -126) * 2.0 ** -8
        assert np.all(np.abs(y - y_ref) <= ulp + prq_ref.tolerance(y_ref) * 0.05)
        w.free()


def test_deterministic(prq, oracle):
    L = synth.layer(95, 512, 2560, 16, T_cal=32)
    w = prq.prepare_weights(L["W"], oracle.channel_amax(L["zcal"]), 0.5, 128)
    codes, _, sf = prq.quantize_act(w, to_dev_bf16(L["x"]), prq.ACT_SCALE_PERM)
    ws = prq.new_workspace(w, 16)
    y1 = prq.linear(w, codes, sf, 16, workspace=ws).clone()
    y2 = prq.linear(w, codes, sf, 16, workspace=ws).clone()
    assert torch.equal(y1, y2)
    assert int(ws.view(torch.int32)[:1024].abs().sum()) == 0  # counters are left clean
    # prefill: the stream-K flags are left clean too and the fixed summation order reproduces bits
    x2 = to_dev_bf16(synth.layer(95, 512, 2560, 700, T_cal=32)["x"])
    codes, _, sf = prq.quantize_act(w, x2, prq.ACT_SCALE_PERM)
    ws = prq.new_workspace(w, 700)
    y1 = prq.linear(w, codes, sf, 700, workspace=ws).clone()
    y2 = prq.linear(w, codes, sf, 700, workspace=ws).clone()
    assert torch.equal(y1, y2)
    assert int(ws.view(torch.int32)[:64].abs().sum()) == 0
    w.free()


def test_empty_batch_and_errors(prq, oracle):
    L = synth.layer(96, 128, 256, 4, T_cal=32)
    w = prq.prepare_weights(L["W"], oracle.channel_amax(L["zcal"]), 0.5, 32)
    x = to_dev_bf16(L["x"])
    codes, _, sf = prq.quantize_act(w, x[:0], prq.ACT_IDENTITY)  # M = 0 is a no-op
    y = prq.linear(w, codes, sf, 0)
    assert y.shape == (0, 128)
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_IDENTITY)
    with pytest.raises(prq.PrqError) as e:  # misaligned output
        buf = torch.empty(4 * 128 + 1, dtype=torch.float32, device="cuda")
        prq.linear(w, codes, sf, 4, out=buf[1:].view(4, 128))
    assert e.value.code == 2
    # the prefill path needs its stream-K workspace; the decode path needs none
    L2 = synth.layer(96, 128, 256, 200, T_cal=32)
    codes2, _, sf2 = prq.quantize_act(w, to_dev_bf16(L2["x"]), prq.ACT_IDENTITY)
    with pytest.raises(prq.PrqError) as e:
        prq.linear(w, codes2, sf2, 200, workspace=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 8
    assert prq.linear_workspace_bytes(w, 4) == 0 and prq.linear_workspace_bytes(w, 200) > 0
    y = prq.linear(w, codes, sf, 4, workspace=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert y.shape == (4, 128)
    w.free()


def grouped_case(prq, oracle, E, N, K, k, counts, seed):
    rng = np.random.default_rng(seed)
    Ws = np.stack([synth.weights(seed * 100 + e, N, K) for e in range(E)])
    ch = synth.HeavyTailChannels(seed + 7, K)
    amax = np.stack([oracle.channel_amax(ch.rows(seed * 10 + e, 32)) for e in range(E)])
    w = prq.prepare_weights(Ws, amax, 0.5, k)
    M = int(sum(counts))
    offsets = np.zeros(E + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    x = ch.rows(seed + 3, M)
    d_off = torch.from_numpy(offsets).cuda()
    codes, srow, sf = prq.quantize_act(w, to_dev_bf16(x), prq.ACT_SCALE_PERM, expert_offsets=d_off, row_scales=True)
    y = prq.linear_grouped(w, codes, sf, d_off, M)
    assert prq.last_device_status() == 0
    y = y.cpu().numpy().astype(np.float64)
    got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
    got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
    for e in range(E):
        o = oracle.prepare(Ws[e], amax[e], 0.5, k)
        assert np.array_equal(w.get(prq.FIELD_CODES, e), o["wcodes"])
        assert np.array_equal(w.get(prq.FIELD_PERM, e), o["perm"])
        r0, r1 = offsets[e], offsets[e + 1]
        if r1 == r0:
            continue
        y_ref, oc, osc = oracle.linear(x[r0:r1], o)
        assert np.array_equal(got_c[r0:r1], oc) and np.array_equal(got_s[r0:r1], osc)
        assert np.abs(y[r0:r1] - y_ref).max() <= prq_ref.tolerance(y_ref)
    w.free()


def test_grouped_experts(prq, oracle):
    """MoE variant: ragged expert row ranges including empty experts and ranges that cross 128-row tiles."""
    grouped_case(prq, oracle, E=6, N=512, K=768, k=64, counts=[5, 0, 130, 1, 0, 300], seed=11)
    grouped_case(prq, oracle, E=3, N=256, K=512, k=0, counts=[0, 0, 7], seed=12)


def test_forward_from_host_buffers(prq, oracle):
    L = synth.layer(97, 512, 1024, 200, T_cal=32)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, 128)
    o = oracle.prepare(L["W"], amax, 0.5, 128)
    for M in (200, 8):
        xh = torch.from_numpy(L["x"][:M].view(np.int16).copy()).view(torch.bfloat16).pin_memory()
        yh = torch.empty((M, 512), dtype=torch.float32).pin_memory()
        scratch = torch.zeros(prq.forward_host_scratch_bytes(w, M), dtype=torch.uint8, device="cuda")
        prq.forward_host(w, xh, yh, prq.ACT_SCALE_PERM, scratch)
        assert prq.last_device_status() == 0
        y_ref, _, _ = oracle.linear(L["x"][:M], o)
        assert np.abs(yh.numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    w.free()


@pytest.mark.parametrize("M,k", [(2048, 256), (128, 128), (1, 0)])
def test_full_size_down_proj_sampled_rows(prq, oracle, M, k):
    """Qwen3-4B-shaped down_proj (2560 x 9728) in the launch configuration the benchmark times;
    the oracle checks sampled rows (it computes them one by one)."""
    N, K = 2560, 9728
    L = synth.layer(1, N, K, M, T_cal=128)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = check_prep(prq, oracle, w, L["W"], amax, 0.5, k)
    rows = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(0).integers(0, M, 6)]))
    codes, srow, sf = prq.quantize_act(w, to_dev_bf16(L["x"]), prq.ACT_IDENTITY, row_scales=True)
    oc, osc = oracle.quantize_act(L["x"][rows])
    got_c = codes.cpu().numpy().reshape(M, K // 2)[rows]
    got_s = srow.cpu().numpy().reshape(M, K // 32)[rows]
    assert np.array_equal(got_c, oc) and np.array_equal(got_s, osc)
    y = prq.linear(w, codes, sf, M).cpu().numpy().astype(np.float64)
    assert prq.last_device_status() == 0
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    assert np.abs(y[rows] - y_ref).max() <= prq_ref.tolerance(y_ref)
    assert np.isfinite(y).all()
    w.free()


@pytest.mark.parametrize("M,k,y_dtype", [(1, 256, "f32"), (16, 256, "f32"), (7, 128, "f32"), (16, 0, "f32"), (3, 256, "bf16")])
def test_linear_fused_matches_two_calls_and_oracle(prq, oracle, M, k, y_dtype):
    """The one-launch decode step (activation quantised inside the GEMM kernel) against the oracle and,
    bit for bit, against prq_quantize_act + prq_linear."""
    N, K = 2560, 9728
    L = synth.layer(1, N, K, M, T_cal=64, tag=700 + M + k)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k)
    x = to_dev_bf16(L["x"])
    dt = prq.F32 if y_dtype == "f32" else prq.BF16
    y = prq.linear_fused(w, x, prq.ACT_IDENTITY, dt)
    assert prq.last_device_status() == 0
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_IDENTITY)
    y2 = prq.linear(w, codes, sf, M, dt)
    assert torch.equal(y, y2)
    oc, osc = oracle.quantize_act(L["x"])
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    got = y.float().cpu().numpy().astype(np.float64)
    if y_dtype == "f32":
        assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref)
    else:
        ulp = np.maximum(np.abs(y_ref), 2.0 ** -126) * 2.0 ** -7
        assert np.all(np.abs(got - y_ref) <= ulp + prq_ref.tolerance(y_ref))
    w.free()


def test_linear_fused_small_shapes_and_strides(prq, oracle):
    """Ragged N and K (K + k not a multiple of the 256-column stage), a row stride larger than K, and a
    short reduction (one stage, hence no split)."""
    for (N, K, k, M) in [(200, 416, 32, 5), (384, 1024, 64, 16), (128, 64, 32, 2)]:
        L = synth.layer(0, N, K, M, T_cal=32, tag=900 + N)
        amax = oracle.channel_amax(L["zcal"])
        w = prq.prepare_weights(L["W"], amax, 0.25, k)
        o = oracle.prepare(L["W"], amax, float(np.float32(0.25)), k)
        xs = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
        xs[:, :K] = to_dev_bf16(L["x"])
        y = prq.linear_fused(w, xs[:, :K])
        assert prq.last_device_status() == 0
        oc, osc = oracle.quantize_act(L["x"])
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        assert np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
        w.free()


def test_linear_fused_rejects_what_it_does_not_cover(prq, oracle):
    L = synth.layer(0, 128, 256, 4, T_cal=16, tag=950)
    w = prq.prepare_weights(L["W"], oracle.channel_amax(L["zcal"]), 0.5, 32)
    x = torch.zeros((prq.FUSED_MAX_M + 1, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(prq.PrqError):
        prq.linear_fused(w, x)
    with pytest.raises(prq.PrqError):
        prq.linear_fused(w, x[:4], prq.ACT_SCALE_PERM)
    w.free()


@pytest.mark.parametrize("M", [1, 16, 64, 128])
def test_decode_split_k_is_reproducible(prq, oracle, M):
    """The cluster split-K exchange sums the partial results in a fixed order: repeated launches of the same
    problem give the same bits, for both forms of the exchange (asynchronous stores up to 32 tokens, plain
    stores and a cluster barrier above) and for the fused entry."""
    N, K, k = 2560, 9728, 256
    L = synth.layer(1, N, K, M, T_cal=32, tag=800 + M)
    w = prq.prepare_weights(L["W"], oracle.channel_amax(L["zcal"]), 0.5, k)
    x = to_dev_bf16(L["x"])
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_IDENTITY)
    ref = prq.linear(w, codes, sf, M).clone()
    for _ in range(40):
        assert torch.equal(prq.linear(w, codes, sf, M), ref)
    if M <= prq.FUSED_MAX_M:
        for _ in range(40):
            assert torch.equal(prq.linear_fused(w, x), ref)
    assert prq.last_device_status() == 0
    w.free()


def test_linear_with_weight_scale_search(prq, oracle):
    """Weights prepared with the E8M0-W option: prep fields bit-exact against the oracle's, the product within
    tolerance of the oracle's (decode and prefill kernels), and the synthetic reconstruction error of the
    layer output is reported not to grow."""
    N, K, k = 512, 2048, 128
    L = synth.layer(1, N, K, 300, T_cal=64, tag=990)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k, scale_search=True)
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k, scale_search=True)
    assert np.array_equal(w.get(prq.FIELD_PERM), o["perm"])
    assert np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"])
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"])
    for M in (16, 300):
        x = to_dev_bf16(L["x"][:M])
        codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
        y = prq.linear(w, codes, sf, M).cpu().numpy().astype(np.float64)
        oc, osc = oracle.quantize_act(L["x"][:M], o["perm"], o["inv_s"])
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        assert np.abs(y - y_ref).max() <= prq_ref.tolerance(y_ref)
    assert prq.last_device_status() == 0
    w.free()


@pytest.mark.parametrize("M", [1, 16, 64, 128])
def test_multi_layer_launches_match_single_layer_calls(prq, oracle, M):
    """q / k / v-shaped layers over the same activation: one quantiser launch and one GEMM launch for all
    three give, layer by layer, the bits of the single-layer calls (and hence the oracle's result)."""
    K, k = 1024, 128
    shapes = [384, 128, 200]
    L0 = synth.layer(1, shapes[0], K, M, T_cal=32, tag=970)
    x = to_dev_bf16(L0["x"])
    ws, os_ = [], []
    for i, N in enumerate(shapes):
        Li = synth.layer(1, N, K, 4, T_cal=32, tag=971 + i)
        amax = oracle.channel_amax(Li["zcal"])
        ws.append(prq.prepare_weights(Li["W"], amax, 0.5, k))
        os_.append(oracle.prepare(Li["W"], amax, float(np.float32(0.5)), k))
    acts = prq.quantize_act_multi(ws, x, prq.ACT_SCALE_PERM)
    ys = prq.linear_multi(ws, acts, M)
    assert prq.last_device_status() == 0
    for w, o, (codes, sf), y in zip(ws, os_, acts, ys):
        c1, _, s1 = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
        assert torch.equal(codes, c1) and torch.equal(sf, s1)
        assert torch.equal(y, prq.linear(w, c1, s1, M))
        oc, osc = oracle.quantize_act(L0["x"], o["perm"], o["inv_s"])
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        assert np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    # layers that do not share K (or k_tail for the GEMM) are refused
    Lb = synth.layer(1, 128, 512, 4, T_cal=32, tag=979)
    wb = prq.prepare_weights(Lb["W"], oracle.channel_amax(Lb["zcal"]), 0.5, 64)
    with pytest.raises(prq.PrqError):
        prq.quantize_act_multi([ws[0], wb], x, prq.ACT_SCALE_PERM, out=acts[:2])
    for w in ws + [wb]:
        w.free()


@pytest.mark.parametrize("N,K,k,alpha,search", [
    (256, 256, 32, 0.5, False),      # the tiny configuration's shape
    (100, 96, 0, 0.0, False),        # k = 0, alpha = 0: plain MXFP4 of W
    (132, 1024, 1024, 1.0, False),   # every channel in the tail
    (512, 2048, 128, 0.5, True),     # weight-side block-scale search
    (300, 640, 64, 0.3, True),       # an alpha off the closed-form grid (pow), ragged N
])
def test_device_prep_is_bit_exact(prq, oracle, N, K, k, alpha, search):
    """prq_prepare_weights_device (Algorithm 1 steps 3-7 and 11 as kernels on a device copy of W): every field of
    the handle equals the oracle's, bit for bit -- scales s and 1/s, the FP64 column errors, the permutation,
    codes and scale bytes of [Q(W D P) | Q(R)] -- and the handle runs the product like a host-prepared one."""
    L = synth.layer(3, N, K, 40, T_cal=32, tag=N + K + k)
    amax = oracle.channel_amax(L["zcal"])
    amax[3] = 0.0                                     # a dead channel takes the 1e-5 floor
    Wd = torch.from_numpy(L["W"].view(np.int16)).cuda()
    w = prq.prepare_weights_device(Wd, amax, alpha, k, scale_search=search)
    o = oracle.prepare(L["W"], amax, float(np.float32(alpha)), k, scale_search=search)
    assert np.array_equal(w.get(prq.FIELD_S), o["s"])
    assert np.array_equal(w.get(prq.FIELD_INV_S), o["inv_s"])
    assert np.array_equal(w.get(prq.FIELD_COL_ERR), o["col_err"])
    assert np.array_equal(w.get(prq.FIELD_PERM), o["perm"])
    assert np.array_equal(w.get(prq.FIELD_TOPK), o["topk"])
    assert np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"])
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"])
    x = to_dev_bf16(L["x"])
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
    y = prq.linear(w, codes, sf, 40).cpu().numpy().astype(np.float64)
    oc, osc = oracle.quantize_act(L["x"], o["perm"], o["inv_s"])
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    assert np.abs(y - y_ref).max() <= prq_ref.tolerance(y_ref)
    assert prq.last_device_status() == 0
    w.free()


def test_device_prep_experts_and_errors(prq, oracle):
    """Stacked experts through the device prep equal the host prep expert by expert; a non-finite weight is
    reported, not encoded."""
    E, N, K, k = 3, 64, 128, 32
    Ws = np.stack([synth.weights(40 + e, N, K) for e in range(E)])
    amax = np.stack([np.abs(np.random.default_rng(50 + e).standard_normal(K)).astype(np.float32) + 0.05 for e in range(E)])
    wd = prq.prepare_weights_device(torch.from_numpy(Ws.view(np.int16)).cuda(), amax, 0.5, k)
    wh = prq.prepare_weights(Ws, amax, 0.5, k)
    for e in range(E):
        for f in (prq.FIELD_S, prq.FIELD_INV_S, prq.FIELD_COL_ERR, prq.FIELD_PERM, prq.FIELD_SCALES, prq.FIELD_CODES):
            assert np.array_equal(wd.get(f, e), wh.get(f, e)), (e, f)
    wd.free()
    wh.free()
    bad = Ws[0].copy()
    bad[5, 7] = 0x7F80                                # +infinity in bf16
    with pytest.raises(prq.PrqError) as ei:
        prq.prepare_weights_device(torch.from_numpy(bad.view(np.int16)).cuda(), amax[0], 0.5, k)
    assert ei.value.code == 7                        # PRQ_ERR_NONFINITE


@pytest.mark.parametrize("N,K,k,M", [(256, 512, 64, 16), (512, 2560, 128, 300), (256, 768, 64, 1), (384, 1024, 256, 128)])
def test_offline_copy_form_equals_the_revisit_form(prq, oracle, N, K, k, M):
    """Activation tail construction paragraph, offline copy: the producer emits the k tail channels twice, the
    activation has K + k columns, and the layer is a plain MXFP4 product over K + k.  Quantising the widened
    row must equal widening the quantised row (block alignment), so codes, scale bytes and the product are
    bit for bit those of the form that re-reads the tail -- and within tolerance of the oracle."""
    L = synth.layer(4, N, K, M, T_cal=32, tag=K + k + M)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k)
    wide = w.offline_copy()
    assert (wide.K, wide.k_tail, wide.N) == (K + k, 0, N)
    assert np.array_equal(wide.get(prq.FIELD_CODES), o["wcodes"])
    assert np.array_equal(wide.get(prq.FIELD_SCALES), o["wscales"])
    x = L["x"]                                             # taken as already permuted and scaled (identity mode)
    x_wide = np.concatenate([x, x[:, K - k:]], axis=1)
    oc, osc = oracle.quantize_act(x)
    ca, sa = oracle.augment_act(oc, osc, k)
    codes_w, srow_w, sf_w = prq.quantize_act(wide, to_dev_bf16(x_wide), prq.ACT_IDENTITY, row_scales=True)
    Ka = K + k
    assert np.array_equal(codes_w.cpu().numpy()[: M * Ka // 2].reshape(M, Ka // 2), ca)
    assert np.array_equal(srow_w.cpu().numpy()[: M * Ka // 32].reshape(M, Ka // 32), sa)
    codes, _, sf = prq.quantize_act(w, to_dev_bf16(x), prq.ACT_IDENTITY)
    y_revisit = prq.linear(w, codes, sf, M)
    y_wide = prq.linear(wide, codes_w, sf_w, M)
    assert torch.equal(y_revisit, y_wide)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    assert np.abs(y_wide.cpu().numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    if M <= prq.FUSED_MAX_M:
        assert torch.equal(prq.linear_fused(wide, to_dev_bf16(x_wide)), y_wide)
    assert prq.last_device_status() == 0
    wide.free()
    w.free()


def test_offline_copy_form_needs_stage_aligned_tail(prq, oracle):
    W = synth.weights(8, 64, 160)
    w = prq.prepare_weights(W, np.ones(160, np.float32), 0.0, 32)     # K = 160 is not a multiple of 256
    with pytest.raises(prq.PrqError) as ei:
        w.offline_copy()
    assert ei.value.code == 1                                          # PRQ_ERR_INVALID_ARG
    w0 = prq.prepare_weights(W, np.ones(160, np.float32), 0.0, 0)      # no tail: nothing to align
    v = w0.offline_copy()
    assert (v.K, v.k_tail) == (160, 0)
    v.free(); w0.free(); w.free()


def test_folded_producers_feed_the_identity_path(prq, oracle):
    """Eq. (1) end to end on a small gated FFN: with 1 / s and the permutation folded into the up / gate projections
    (prq_fold_producer) the down projection runs in identity mode; with the tail rows duplicated as well it runs
    as a plain product over C + k (prq_weights_offline_copy).  Each route is checked against the oracle on its
    own activation (codes bit-exact, product within tolerance); across routes the outputs agree up to the bf16
    roundings of the folded weights and of the activation."""
    C, H, N, M, k = 512, 256, 256, 64, 64
    rng = np.random.default_rng(77)
    Wu, Wg, Wd = synth.weights(61, C, H), synth.weights(62, C, H), synth.weights(63, N, C)
    X = torch.from_numpy(rng.standard_normal((M + 128, H)).astype(np.float32) * 8).cuda()

    def ffn(up_bits, gate_bits, x):
        up = torch.from_numpy(up_bits.view(np.int16)).cuda().view(torch.bfloat16).float()
        gate = torch.from_numpy(gate_bits.view(np.int16)).cuda().view(torch.bfloat16).float()
        return (torch.nn.functional.silu(x @ gate.T) * (x @ up.T)).to(torch.bfloat16)

    def bits(t):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)

    h_all = ffn(Wu, Wg, X)
    amax = oracle.channel_amax(bits(h_all[M:]))            # calibration rows
    w = prq.prepare_weights(Wd, amax, 0.5, k)
    o = oracle.prepare(Wd, amax, float(np.float32(0.5)), k)
    x = X[:M]

    # route A: online scale + permute
    h = h_all[:M].contiguous()
    ca, _, sfa = prq.quantize_act(w, h, prq.ACT_SCALE_PERM)
    y_a = prq.linear(w, ca, sfa, M).cpu().numpy().astype(np.float64)

    # route B: folded producers, identity mode
    up_f, gate_f = prq.fold_producer(w.get(prq.FIELD_PERM), w.get(prq.FIELD_INV_S), k, Wu, Wg)
    ht = ffn(up_f, gate_f, x).contiguous()
    cb, srow_b, sfb = prq.quantize_act(w, ht, prq.ACT_IDENTITY, row_scales=True)
    y_b = prq.linear(w, cb, sfb, M).cpu().numpy().astype(np.float64)
    oc, osc = oracle.quantize_act(bits(ht))
    assert np.array_equal(cb.cpu().numpy()[: M * C // 2].reshape(M, C // 2), oc)
    assert np.array_equal(srow_b.cpu().numpy()[: M * C // 32].reshape(M, C // 32), osc)
    cao, sao = oracle.augment_act(oc, osc, k)
    y_ref_b = oracle.matmul(cao, sao, o["wcodes"], o["wscales"])
    assert np.abs(y_b - y_ref_b).max() <= prq_ref.tolerance(y_ref_b)

    # route C: tail rows duplicated in the producers, plain product over C + k
    up_w, gate_w = prq.fold_producer(w.get(prq.FIELD_PERM), w.get(prq.FIELD_INV_S), k, Wu, Wg, duplicate_tail=True)
    hw = ffn(up_w, gate_w, x).contiguous()
    wide = w.offline_copy()
    cc, _, sfc = prq.quantize_act(wide, hw, prq.ACT_IDENTITY)
    y_c = prq.linear(wide, cc, sfc, M).cpu().numpy().astype(np.float64)
    ocw, oscw = oracle.quantize_act(bits(hw))
    assert np.array_equal(cc.cpu().numpy()[: M * (C + k) // 2].reshape(M, (C + k) // 2), ocw)
    y_ref_c = oracle.matmul(ocw, oscw, o["wcodes"], o["wscales"])
    assert np.abs(y_c - y_ref_c).max() <= prq_ref.tolerance(y_ref_c)

    # Across routes the activations differ in their last bf16 bit here and there, which flips some 4-bit codes: the
    # outputs cannot agree closer than a fraction of the quantisation error itself.  All three must sit at the
    # same distance from the unquantised product, and nearer to each other than to it.
    y_exact = oracle.matmul_bf16(bits(h), Wd)
    err = {n: np.linalg.norm(y - y_exact) / np.linalg.norm(y_exact) for n, y in (("a", y_a), ("b", y_b), ("c", y_c))}
    assert abs(err["b"] - err["a"]) < 0.15 * err["a"] and abs(err["c"] - err["a"]) < 0.15 * err["a"], err
    nrm = np.linalg.norm(y_exact)
    assert np.linalg.norm(y_b - y_a) / nrm < 0.6 * err["a"], (np.linalg.norm(y_b - y_a) / nrm, err)
    assert np.linalg.norm(y_c - y_b) / nrm < 0.6 * err["a"], (np.linalg.norm(y_c - y_b) / nrm, err)
    assert prq.last_device_status() == 0
    wide.free()
    w.free()


@pytest.mark.parametrize("M", [64, 100, 128])
def test_decode_more_weight_tiles_than_sms(prq, oracle, M):
    """A layer with more 128-row weight tiles than the GPU has SMs (152 here, like a stacked gate / up
    projection) at 64 to 128 tokens takes the decode kernel's two-CTAs-per-SM variant; so does a two-layer
    launch whose layers have 76 tiles each.  Sampled rows against the oracle, and the two-layer launch against
    single-layer calls."""
    N, K, k = 19456, 512, 64
    L = synth.layer(6, N, K, M, T_cal=32, tag=M)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k)
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"])
    x = to_dev_bf16(L["x"])
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
    y = prq.linear(w, codes, sf, M)
    assert prq.last_device_status() == 0
    oc, osc = oracle.quantize_act(L["x"], o["perm"], o["inv_s"])
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    assert np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    yb = prq.linear(w, codes, sf, M, prq.BF16).float().cpu().numpy().astype(np.float64)
    assert np.abs(yb - y_ref).max() <= prq_ref.tolerance(y_ref) + np.abs(y_ref).max() * 2.0 ** -7
    w.free()
    # two layers of 76 tiles in one launch
    halves = [prq.prepare_weights(L["W"][i * 9728:(i + 1) * 9728], amax, 0.5, k) for i in range(2)]
    acts = prq.quantize_act_multi(halves, x, prq.ACT_SCALE_PERM)
    ys = prq.linear_multi(halves, acts, M)
    for h, a, ym in zip(halves, acts, ys):
        assert torch.equal(ym, prq.linear(h, a[0], a[1], M))
    assert prq.last_device_status() == 0
    for h in halves:
        h.free()


def test_production_switch_state_in_a_fresh_process():
    """The suite runs with the developer switches readable (PRQ_DEV=1, set by conftest.py); a user's process has
    no such variable and takes the other branch of every switch look-up.  The tiny configuration (decode kernel)
    and a 512-token call (prefill kernel) are checked against the oracle in a process started without it."""
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if not k.startswith("PRQ_")}
    code = "import __graft_entry__ as g, os; assert 'PRQ_DEV' not in os.environ; g.smoke()"
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert "smoke ok" in r.stdout


def test_stacked_preparation_is_the_method_on_the_concatenated_matrix(prq, oracle):
    """prq_prepare_weights_stacked: q / k / v-like layers over one activation as one layer -- equal, field by field, to
    the oracle's preparation of the row-concatenated weight, and its product carries every layer's outputs in its
    column slice."""
    K, k, M = 512, 64, 200
    Ns = (384, 96, 160)
    Ws = [synth.weights(80 + i, n, K) for i, n in enumerate(Ns)]
    ch = synth.HeavyTailChannels(83, K)
    x, xcal = ch.rows(84, M), ch.rows(85, 64)
    amax = oracle.channel_amax(xcal)
    w = prq.prepare_weights_stacked(Ws, amax, 0.5, k)
    Wcat = np.concatenate(Ws)
    assert w.N == sum(Ns)
    o = check_prep(prq, oracle, w, Wcat, amax, 0.5, k)
    codes, sf, oc, osc = run_quant(prq, oracle, w, o, x, prq.ACT_SCALE_PERM)
    y, y_ref = run_linear(prq, oracle, w, o, codes, sf, oc, osc, M)
    # a layer's slice is the product with that layer's rows of the prepared weights
    r0 = Ns[0]
    ca, sa = oracle.augment_act(oc, osc, k)
    y_k = oracle.matmul(ca, sa, o["wcodes"][r0: r0 + Ns[1]], o["wscales"][r0: r0 + Ns[1]])
    assert np.abs(y[:, r0: r0 + Ns[1]] - y_k).max() <= prq_ref.tolerance(y_k)
    w.free()
