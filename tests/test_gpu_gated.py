"""GPU parity of the gated-producer call (Eq. (1), middle line, with the activation function inside the producer's GEMM):
prq_linear_gated against the oracle.

Two parts, because the kernel's fast exponential is not bit-specified: (1) the product h = bf16(silu(gate) * up) that the
kernel forms lies within one bf16 unit in the last place of the oracle's FP64 product (computed from the oracle's own gate
and up sums); (2) the codes and scale bytes it writes are bit for bit the oracle's quantisation of the kernel's own h, in
all three layouts.  Then the down projection on those buffers, within the GEMM tolerance."""
import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


def gated_case(prq, oracle, C, H, N, M, k_down, k_gu, seed, rows=None):
    Wu, Wg, Wd = synth.weights(seed, C, H), synth.weights(seed + 1, C, H), synth.weights(seed + 2, N, C)
    ch = synth.HeavyTailChannels(seed + 3, H)
    x, xcal = ch.rows(seed + 4, M), ch.rows(seed + 5, 64)
    # down projection: calibrated on the unfolded FFN output of the calibration rows (plain FP64 arithmetic)
    f = lambda b: synth.bf16_to_f32(b).astype(np.float64)
    gc, uc = f(xcal) @ f(Wg).T, f(xcal) @ f(Wu).T
    hcal = oracle.silu_mul_bf16(gc, uc)
    amax_d = oracle.channel_amax(hcal)
    wd = prq.prepare_weights(Wd, amax_d, 0.5, k_down)
    od = oracle.prepare(Wd, amax_d, float(np.float32(0.5)), k_down)
    # producers with the down projection's 1 / s and permutation folded in, stacked in (gate, up) groups of 32
    up_f, gate_f = prq.fold_producer(wd.get(prq.FIELD_PERM), wd.get(prq.FIELD_INV_S), k_down, Wu, Wg)
    o_up, o_gate = oracle.fold_producer(Wu, Wg, od["perm"], od["inv_s"], k_down)
    assert np.array_equal(up_f, o_up) and np.array_equal(gate_f, o_gate)
    W_st = prq.stack_gate_up(gate_f, up_f)
    assert np.array_equal(W_st, oracle.stack_gate_up(o_gate, o_up))
    amax_x = oracle.channel_amax(xcal)
    wgu = prq.prepare_weights(W_st, amax_x, 0.5, k_gu, gated_producer=True)
    ogu = oracle.prepare(W_st, amax_x, float(np.float32(0.5)), k_gu)
    assert np.array_equal(wgu.get(prq.FIELD_CODES), ogu["wcodes"]) and np.array_equal(wgu.get(prq.FIELD_PERM), ogu["perm"])

    cx, _, sfx = prq.quantize_act(wgu, dev_bf16(x), prq.ACT_SCALE_PERM)
    codes, srow, sf, h = prq.linear_gated(wgu, cx, sfx, M, wd, row_scales=True, h_check=True)
    assert prq.last_device_status() == 0
    sel = np.arange(M) if rows is None else rows

    # (1) the product, against the oracle's gate / up sums put through the oracle's activation
    y_ref, _, _ = oracle.linear(x[sel], ogu)                        # (rows, 2 C), interleaved
    y4 = y_ref.reshape(len(sel), C // 32, 2, 32)
    g_ref, u_ref = y4[:, :, 0].reshape(len(sel), C), y4[:, :, 1].reshape(len(sel), C)
    h_ref = synth.bf16_to_f32(oracle.silu_mul_bf16(g_ref, u_ref)).astype(np.float64)
    h_bits = h.view(torch.int16).cpu().numpy().view(np.uint16)
    h_got = synth.bf16_to_f32(h_bits[sel]).astype(np.float64)
    # one bf16 ulp of the reference, plus what the fp32 accumulation of the two sums can move the product
    # (|silu'| <= 1.1, so d h <= 1.1 |u| dg + |silu(g)| du with dg, du within the GEMM tolerance)
    tol_sum = 2e-4
    slack = np.abs(h_ref) * 2.0 ** -7 + tol_sum * (1.1 * np.abs(u_ref) + np.abs(g_ref) + 1.0)
    assert np.all(np.abs(h_got - h_ref) <= slack), float((np.abs(h_got - h_ref) / slack).max())

    # (2) the quantisation of the kernel's own product, bit for bit, in every layout
    oc, osc = oracle.quantize_act(h_bits)
    assert np.array_equal(codes.cpu().numpy()[: M * C // 2].reshape(M, C // 2), oc)
    assert np.array_equal(srow.cpu().numpy()[: M * C // 32].reshape(M, C // 32), osc)
    ca, sa = oracle.augment_act(oc, osc, k_down)
    want_sf = prq_ref.expected_sf(sa, C, k_down)
    assert np.array_equal(sf.cpu().numpy()[: want_sf.size], want_sf)
    # ... and equal to what the library's own quantiser makes of that product
    c2, s2, sf2 = prq.quantize_act(wd, h, prq.ACT_IDENTITY, row_scales=True)
    assert torch.equal(c2[: M * C // 2], codes[: M * C // 2]) and torch.equal(sf2[: want_sf.size], sf[: want_sf.size])

    # the down projection on the buffers the producer wrote
    y = prq.linear(wd, codes, sf, M).cpu().numpy().astype(np.float64)
    y_d = oracle.matmul(ca[sel], sa[sel], od["wcodes"], od["wscales"])
    assert np.abs(y[sel] - y_d).max() <= prq_ref.tolerance(y_d)
    assert prq.last_device_status() == 0
    # an ordinary call refuses the producer handle at prefill sizes instead of reading a tiling it does not have
    if M > 128:
        with pytest.raises(prq.PrqError):
            prq.linear(wgu, cx, sfx, M)
    wgu.free()
    wd.free()


@pytest.mark.parametrize("M", [1, 16, 100, 300, 700])
def test_gated_producer_small(prq, oracle, M):
    """A small gated FFN: 2 C = 1024 stacked output features (five full 192-column tiles and a third of one), ragged
    token counts around the 128- and 256-row tile boundaries, a down projection with a one-stage tail."""
    gated_case(prq, oracle, C=512, H=256, N=256, M=M, k_down=256, k_gu=32, seed=300 + M)


def test_gated_producer_whole_input_is_tail(prq, oracle):
    """k = C on the down projection: every scale byte is written twice."""
    gated_case(prq, oracle, C=256, H=128, N=128, M=200, k_down=256, k_gu=0, seed=411)


@pytest.mark.parametrize("M", [16, 4096])
def test_gated_producer_qwen3_4b_ffn(prq, oracle, M):
    """The paper's FFN shape: hidden 2560, intermediate 9728, k = 256 on the down projection, k = 128 on the stacked
    producer; 16 and 4096 tokens.  The oracle checks sampled token rows."""
    rows = None if M <= 16 else np.unique(np.concatenate([[0, M - 1, 255, 256], np.random.default_rng(M).integers(0, M, 3)]))
    gated_case(prq, oracle, C=9728, H=2560, N=2560, M=M, k_down=256, k_gu=128, seed=500, rows=rows)
