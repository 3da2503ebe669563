"""GPU parity at the sizes of the larger workload configurations: one decoder block's linears at
M = 4096 (online scale + permutation), the 128-expert grouped down-projection under Zipf routing,
and two layers of the block stack at decode batch 64.  The CUDA path runs the full problem in the
launch configuration the benchmark times; the oracle, which computes rows one by one, checks the
offline prep in full and the online path on sampled rows (sampled experts for the MoE case)."""
import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

# (name, N, K, k) of one Qwen3-4B-shaped decoder block; k and v share a shape, so do gate and up
BLOCK = [("q", 4096, 2560, 128), ("kv", 1024, 2560, 128), ("o", 2560, 4096, 128),
         ("gate_up", 9728, 2560, 128), ("down", 2560, 9728, 256),
         # q, k and v stacked into one layer (one scaling, permutation and tail for the group), as the
         # benchmark's grouped-preparation step runs them
         ("qkv_stacked", 6144, 2560, 128)]


def to_dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


def sample_rows(M, n, seed):
    return np.unique(np.concatenate([[0, M - 1], np.random.default_rng(seed).integers(0, M, n)]))


def check_prep_fields(prq, w, o, expert=0):
    assert np.array_equal(w.get(prq.FIELD_PERM, expert), o["perm"])
    assert np.array_equal(w.get(prq.FIELD_TOPK, expert), o["topk"])
    assert np.array_equal(w.get(prq.FIELD_INV_S, expert), o["inv_s"])
    assert np.array_equal(w.get(prq.FIELD_SCALES, expert), o["wscales"])
    assert np.array_equal(w.get(prq.FIELD_CODES, expert), o["wcodes"])


def dense_case(prq, oracle, config, tag, N, K, k, M, mode, n_rows=6, bf16_too=True):
    L = synth.layer(config, N, K, M, T_cal=128, tag=tag)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k)
    check_prep_fields(prq, w, o)
    rows = sample_rows(M, n_rows, tag)
    codes, srow, sf = prq.quantize_act(w, to_dev_bf16(L["x"]), mode, row_scales=True)
    if mode == prq.ACT_IDENTITY:
        oc, osc = oracle.quantize_act(L["x"][rows])
    else:
        oc, osc = oracle.quantize_act(L["x"][rows], o["perm"], o["inv_s"])
    assert np.array_equal(codes.cpu().numpy().reshape(M, K // 2)[rows], oc)
    assert np.array_equal(srow.cpu().numpy().reshape(M, K // 32)[rows], osc)
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    y = prq.linear(w, codes, sf, M)
    assert prq.last_device_status() == 0
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    assert np.abs(yh[rows].astype(np.float64) - y_ref).max() <= prq_ref.tolerance(y_ref)
    if bf16_too:
        # bf16 output: the fp32 result rounded once; one bf16 ulp of slack against the rounded reference
        yb = prq.linear(w, codes, sf, M, prq.BF16).float().cpu().numpy()[rows].astype(np.float64)
        ulp = np.maximum(np.abs(y_ref), 2.0 ** -126) * 2.0 ** -7
        assert np.all(np.abs(yb - y_ref) <= ulp + prq_ref.tolerance(y_ref))
    w.free()


@pytest.mark.parametrize("name,N,K,k", BLOCK)
def test_block_linears_prefill_4096(prq, oracle, name, N, K, k):
    dense_case(prq, oracle, config=2, tag=BLOCK.index((name, N, K, k)), N=N, K=K, k=k, M=4096,
               mode=prq.ACT_SCALE_PERM)


@pytest.mark.parametrize("layer", [0, 17])
def test_stack_layers_decode_64(prq, oracle, layer):
    """Block shapes with k = 256 everywhere at decode batch 64 (the stack workload), weights differing per layer."""
    for i, (name, N, K, _) in enumerate(BLOCK):
        dense_case(prq, oracle, config=4, tag=10 * layer + i, N=N, K=K, k=256, M=64, mode=prq.ACT_SCALE_PERM,
                   n_rows=4, bf16_too=False)


@pytest.mark.parametrize("name,N,K", [(n, N, K) for n, N, K, _ in BLOCK])
def test_stack_layer_prefill_4096(prq, oracle, name, N, K):
    """The stack workload's prefill leg: block shapes with k = 256 on EVERY linear at 4096 tokens (K + k = 2816 is
    eleven reduction stages on the q / k / v / gate / up shapes), online scale + permutation, one layer's weights."""
    i = [b[0] for b in BLOCK].index(name)
    dense_case(prq, oracle, config=4, tag=500 + i, N=N, K=K, k=256, M=4096, mode=prq.ACT_SCALE_PERM, n_rows=6,
               bf16_too=(name in ("kv", "down")))


def test_gate_up_stacked_prefill_and_decode(prq, oracle):
    """gate and up stacked into one 19456-row layer (one scaling, permutation and tail for the pair), as the
    benchmark's grouped-preparation step runs them: 4096 tokens and decode batch 64."""
    dense_case(prq, oracle, config=2, tag=7, N=19456, K=2560, k=128, M=4096, mode=prq.ACT_SCALE_PERM, n_rows=4,
               bf16_too=False)
    dense_case(prq, oracle, config=4, tag=507, N=19456, K=2560, k=256, M=64, mode=prq.ACT_SCALE_PERM, n_rows=4,
               bf16_too=False)


@pytest.mark.parametrize("T", [64, 1024, 8192])
def test_moe_grouped_zipf(prq, oracle, T):
    """128 experts 2048 x 768 with k = 64, T tokens routed top-8 with Zipf(1.1) popularity.  The library preps
    and runs all experts; the oracle checks the hottest, the coldest non-empty, two random experts (all rows up
    to a cap) and that rows of empty experts do not exist."""
    E, N, K, k = 128, 2048, 768, 64
    rng = np.random.default_rng(3000 + T)
    _, offsets, _ = synth.zipf_routing(3004, T, E)
    M = int(offsets[-1])
    assert M == 8 * T
    counts = np.diff(offsets)
    ch = synth.HeavyTailChannels(3005, K)
    Ws = np.stack([synth.weights(3100 + e, N, K) for e in range(E)])
    amax = np.stack([oracle.channel_amax(ch.rows(3300 + e, 64)) for e in range(E)])
    w = prq.prepare_weights(Ws, amax, 0.5, k)
    x = ch.rows(3001, M)
    d_off = torch.from_numpy(offsets).cuda()
    codes, srow, sf = prq.quantize_act(w, to_dev_bf16(x), prq.ACT_SCALE_PERM, expert_offsets=d_off, row_scales=True)
    y = prq.linear_grouped(w, codes, sf, d_off, M)
    assert prq.last_device_status() == 0
    nonempty = np.flatnonzero(counts)
    picks = {int(np.argmax(counts)), int(nonempty[np.argmin(counts[nonempty])])}
    picks.update(int(e) for e in rng.choice(nonempty, size=min(2, len(nonempty)), replace=False))
    got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
    got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
    for e in sorted(picks):
        o = oracle.prepare(Ws[e], amax[e], float(np.float32(0.5)), k)
        check_prep_fields(prq, w, o, e)
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        rows = r0 + sample_rows(r1 - r0, 6, e) if r1 - r0 > 8 else np.arange(r0, r1)
        oc, osc = oracle.quantize_act(x[rows], o["perm"], o["inv_s"])
        assert np.array_equal(got_c[rows], oc) and np.array_equal(got_s[rows], osc)
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        got = y[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
        assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref)
    assert bool(torch.isfinite(y).all())
    w.free()
