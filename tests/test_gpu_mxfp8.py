"""GPU parity of the second format (MXFP8: E4M3 elements, E8M0 block scales, plain W8A8 -- the format of the attention
linears in the paper's end-to-end setting): codes and scale bytes bit for bit against the oracle, the product within
max |y - y_ref| <= 2e-3 (||y_ref||_inf + 1)."""
import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


def fp8_case(prq, oracle, N, K, M, alpha, seed, rows=None, dtypes=(0, 1)):
    L = synth.layer(70 + seed, N, K, M, T_cal=32)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, alpha, 0, fmt=prq.FMT_MXFP8)
    o = oracle.fp8_prepare(L["W"], amax, float(np.float32(alpha)))
    assert w.format == prq.FMT_MXFP8 and w.k_tail == 0
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"]) and np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"])
    assert np.array_equal(w.get(prq.FIELD_INV_S), o["inv_s"]) and np.array_equal(w.get(prq.FIELD_PERM), np.arange(K))
    x = dev_bf16(L["x"])
    sel = np.arange(M) if rows is None else rows
    for mode in (prq.ACT_SCALE_PERM, prq.ACT_IDENTITY):
        codes, srow, sf = prq.quantize_act(w, x, mode, row_scales=True)
        oc, osc = oracle.fp8_quantize_act(L["x"], o["inv_s"] if mode == prq.ACT_SCALE_PERM else None)
        assert np.array_equal(srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32), osc)
        assert np.array_equal(codes.cpu().numpy()[: M * K].reshape(M, K), oc)
        want_sf = prq_ref.expected_sf_fp8(osc, K)
        assert np.array_equal(sf.cpu().numpy()[: want_sf.size], want_sf)
        y_ref = oracle.fp8_matmul(oc[sel], osc[sel], o["wcodes"], o["wscales"])
        for dt in dtypes:
            ldy = (N + 7) // 8 * 8 + 8
            full = torch.full((M + 2, ldy), 77.0, dtype=torch.float32 if dt == prq.F32 else torch.bfloat16, device="cuda")
            y = prq.linear(w, codes, sf, M, dt, out=full[1: M + 1, :N])
            assert prq.last_device_status() == 0
            assert bool((full[0] == 77.0).all()) and bool((full[-1] == 77.0).all()) and bool((full[:, N:] == 77.0).all())
            got = y.float().cpu().numpy().astype(np.float64)[sel]
            slack = np.abs(y_ref).max() * 2.0 ** -7 if dt == prq.BF16 else 0.0
            assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref) + slack, (mode, dt, np.abs(got - y_ref).max())
    w.free()


@pytest.mark.parametrize("shape", [(64, 32, 1), (100, 160, 16), (256, 1024, 100), (300, 96, 128), (1000, 2560, 300), (136, 4096, 700)])
def test_mxfp8_layers(prq, oracle, shape):
    """Ragged N, M around the 128-row tiles, reductions that are not a multiple of the 128-element stage."""
    N, K, M = shape
    fp8_case(prq, oracle, N, K, M, 0.5, seed=N + M)


def test_mxfp8_decision_boundaries_and_unit_scales(prq, oracle):
    rows = []
    for vals in ([448, 1, .5, -3, 2 ** -9, 296], [256, 17, 19, 272, 304], [500, 464, 462, -510], [512, 3, 1],
                 [256, 7 * 2 ** -9, 7.5 * 2 ** -9, -0.5 * 2 ** -9], [2.0 ** -20, 2.0 ** -30, -2.0 ** -29],
                 [0, -0.0], [1.5 * 2.0 ** 127, 2.0 ** 120], [2.0 ** -130]):
        b = np.zeros(32, np.float32); b[: len(vals)] = vals; rows.append(b)
    rng = np.random.default_rng(0)
    x = np.stack([np.concatenate([rows[i] for i in rng.integers(0, len(rows), 4)]) for _ in range(40)])   # 40 x 128
    xb = synth.f32_to_bf16(x)
    assert np.array_equal(synth.bf16_to_f32(xb).view(np.uint32), x.view(np.uint32))
    W = synth.weights(3, 64, 128)
    w = prq.prepare_weights(W, np.ones(128, np.float32), 0.0, 0, fmt=prq.FMT_MXFP8)
    codes, srow, sf = prq.quantize_act(w, dev_bf16(xb), prq.ACT_IDENTITY, row_scales=True)
    oc, osc = oracle.fp8_quantize_act(xb)
    assert np.array_equal(srow.cpu().numpy()[: 40 * 4].reshape(40, 4), osc)
    assert np.array_equal(codes.cpu().numpy()[: 40 * 128].reshape(40, 128), oc)
    w.free()


@pytest.mark.parametrize("name,N,K", [("q", 4096, 2560), ("kv", 1024, 2560), ("o", 2560, 4096)])
def test_mxfp8_attention_linears_prefill_4096(prq, oracle, name, N, K):
    """The Qwen3-4B-shaped attention linears at 4096 tokens; the oracle checks sampled token rows."""
    rows = np.unique(np.concatenate([[0, 4095, 127, 128], np.random.default_rng(N).integers(0, 4096, 3)]))
    fp8_case(prq, oracle, N, K, 4096, 0.5, seed=N % 97, rows=rows, dtypes=(1,))


def test_mxfp8_refusals(prq, oracle):
    W = synth.weights(5, 64, 128)
    with pytest.raises(prq.PrqError):
        prq.prepare_weights(W, np.ones(128, np.float32), 0.5, 32, fmt=prq.FMT_MXFP8)      # the format carries no tail
    w = prq.prepare_weights(W, np.ones(128, np.float32), 0.5, 0, fmt=prq.FMT_MXFP8)
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(prq.PrqError):
        prq.linear_fused(w, x)
    with pytest.raises(prq.PrqError):
        w.clone()
    w.free()


def test_mxfp8_stacked_preparation(prq, oracle):
    """q / k / v-like layers over one activation prepared as one MXFP8 layer: its fields are the oracle's for the
    concatenated matrix, and its output columns are the separate layers' outputs, bit for bit."""
    K, M = 320, 200
    Ns = [96, 32, 40]
    L = synth.layer(83, sum(Ns), K, M, T_cal=32)
    amax = oracle.channel_amax(L["zcal"])
    Ws, r = [], 0
    for n in Ns:
        Ws.append(L["W"][r: r + n]); r += n
    w = prq.prepare_weights_stacked(Ws, amax, 0.5, 0, fmt=prq.FMT_MXFP8)
    o = oracle.fp8_prepare(L["W"], amax, float(np.float32(0.5)))
    assert w.format == prq.FMT_MXFP8 and w.N == sum(Ns)
    assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"]) and np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"])
    x = dev_bf16(L["x"])
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
    y = prq.linear(w, codes, sf, M, prq.F32)
    oc, osc = oracle.fp8_quantize_act(L["x"], o["inv_s"])
    y_ref = oracle.fp8_matmul(oc, osc, o["wcodes"], o["wscales"])
    assert np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    r = 0
    for n, Wi in zip(Ns, Ws):
        wi = prq.prepare_weights(Wi, amax, 0.5, 0, fmt=prq.FMT_MXFP8)
        ci, _, si = prq.quantize_act(wi, x, prq.ACT_SCALE_PERM)
        assert torch.equal(ci, codes)
        yi = prq.linear(wi, ci, si, M, prq.F32)
        assert torch.equal(yi, y[:, r: r + n])
        wi.free(); r += n
    w.free()
