"""Random-shape parity sweep: seeded draws of (N, K, k, M, mode, output type, alpha, block-scale search) through
every dense entry point -- quantiser, prq_linear (decode and prefill kernels by M), the fused decode step, the
multi-layer launches -- against the oracle, with output row strides larger than N."""
import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_against_oracle(prq, oracle, seed):
    rng = np.random.default_rng(seed)
    for case in range(12):
        K = int(rng.integers(1, 40)) * 32
        k = int(rng.integers(0, min(K // 32, 8) + 1)) * 32
        N = int(rng.choice([8, 16, 24, 100, 128, 130, 224, 256, 300, 448, 500]))
        M = int(rng.choice([1, 2, 5, 15, 16, 17, 31, 33, 64, 65, 127, 128, 129, 200, 255, 256, 257, 300, 511, 600]))
        mode = int(rng.integers(0, 2))
        dt = prq.F32 if rng.random() < 0.7 else prq.BF16
        alpha = float(rng.choice([0.0, 0.25, 0.5, 1.0]))
        search = bool(rng.random() < 0.3)
        what = f"seed {seed} case {case}: N={N} K={K} k={k} M={M} mode={mode} dt={dt} alpha={alpha} search={search}"
        L = synth.layer(7, N, K, M, T_cal=32, tag=int(rng.integers(0, 10000)))
        amax = oracle.channel_amax(L["zcal"])
        w = prq.prepare_weights(L["W"], amax, alpha, k, scale_search=search)
        o = oracle.prepare(L["W"], amax, float(np.float32(alpha)), k, scale_search=search)
        assert np.array_equal(w.get(prq.FIELD_PERM), o["perm"]), what
        assert np.array_equal(w.get(prq.FIELD_SCALES), o["wscales"]), what
        assert np.array_equal(w.get(prq.FIELD_CODES), o["wcodes"]), what
        x = dev_bf16(L["x"])
        codes, srow, sf = prq.quantize_act(w, x, mode, row_scales=True)
        if mode == prq.ACT_IDENTITY:
            oc, osc = oracle.quantize_act(L["x"])
        else:
            oc, osc = oracle.quantize_act(L["x"], o["perm"], o["inv_s"])
        assert np.array_equal(codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2), oc), what
        assert np.array_equal(srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32), osc), what
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        n_pad = (N + 7) // 8 * 8 + 8 * int(rng.integers(0, 3))
        tdt = torch.float32 if dt == prq.F32 else torch.bfloat16

        def ybuf():
            return torch.full((M, n_pad), 7.0, dtype=tdt, device="cuda")

        full = ybuf()
        y = prq.linear(w, codes, sf, M, dt, out=full[:, :N])
        assert prq.last_device_status() == 0, what
        assert bool((full[:, N:] == 7.0).all()), what          # nothing written past column N
        got = y.float().cpu().numpy().astype(np.float64)
        slack = np.abs(y_ref).max() * 2.0 ** -7 if dt == prq.BF16 else 0.0
        assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref) + slack, what
        if M <= prq.FUSED_MAX_M and mode == prq.ACT_IDENTITY:
            assert torch.equal(prq.linear_fused(w, x, mode, dt, out=ybuf()[:, :N]), y), what
        if M <= 128:
            acts = prq.quantize_act_multi([w, w], x, mode)
            ys = prq.linear_multi([w, w], acts, M, dt, out=[ybuf()[:, :N], ybuf()[:, :N]])
            assert torch.equal(acts[1][0], codes) and torch.equal(ys[0], y) and torch.equal(ys[1], y), what
        w.free()


@pytest.mark.parametrize("gbn", [0, 64, 128])
@pytest.mark.parametrize("seed", [21, 22])
def test_random_grouped_shapes_against_oracle(prq, oracle, monkeypatch, seed, gbn):
    """Stacked experts with random row counts (empty experts included), strided activations and outputs, with the
    library's own choice of token tile (gbn 0) and with both tiles forced."""
    if gbn:
        monkeypatch.setenv("PRQ_GROUPED_BN", str(gbn))
    rng = np.random.default_rng(seed)
    for case in range(8):
        E = int(rng.choice([1, 2, 3, 5, 8, 16]))   # one expert: the grouped layout coincides with the dense one
        K = int(rng.integers(1, 16)) * 32
        k = int(rng.integers(0, min(K // 32, 4) + 1)) * 32
        N = int(rng.choice([16, 100, 128, 136, 256, 300]))
        counts = rng.choice([0, 0, 1, 3, 17, 64, 127, 128, 129, 200, 300], size=E)
        if counts.sum() == 0:
            counts[0] = 5
        offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        M = int(offsets[-1])
        mode = int(rng.integers(0, 2))
        dt = prq.F32 if rng.random() < 0.5 else prq.BF16
        what = f"seed {seed} tile {gbn} case {case}: E={E} N={N} K={K} k={k} counts={counts.tolist()} mode={mode} dt={dt}"
        ch = synth.HeavyTailChannels(int(rng.integers(0, 10000)), K)
        Ws = np.stack([synth.weights(int(rng.integers(0, 10000)), N, K) for _ in range(E)])
        amax = np.stack([oracle.channel_amax(ch.rows(int(rng.integers(0, 10000)), 32)) for _ in range(E)])
        x = ch.rows(int(rng.integers(0, 10000)), M)
        w = prq.prepare_weights(Ws, amax, 0.5, k)
        ldx = K + 8 * int(rng.integers(0, 3))
        xs = torch.zeros((M, ldx), dtype=torch.bfloat16, device="cuda")
        xs[:, :K] = dev_bf16(x)
        d_off = torch.from_numpy(offsets).cuda()
        codes, srow, sf = prq.quantize_act(w, xs[:, :K], mode, expert_offsets=d_off, row_scales=True)
        n_pad = (N + 7) // 8 * 8 + 8 * int(rng.integers(0, 3))
        full = torch.full((M, n_pad), 7.0, dtype=torch.float32 if dt == prq.F32 else torch.bfloat16, device="cuda")
        y = prq.linear_grouped(w, codes, sf, d_off, M, dt, out=full[:, :N])
        assert prq.last_device_status() == 0, what
        assert bool((full[:, N:] == 7.0).all()), what
        got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
        got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
        for e in range(E):
            r0, r1 = int(offsets[e]), int(offsets[e + 1])
            if r1 == r0:
                continue
            o = oracle.prepare(Ws[e], amax[e], float(np.float32(0.5)), k)
            if mode == prq.ACT_IDENTITY:
                oc, osc = oracle.quantize_act(x[r0:r1])
            else:
                oc, osc = oracle.quantize_act(x[r0:r1], o["perm"], o["inv_s"])
            assert np.array_equal(got_c[r0:r1], oc) and np.array_equal(got_s[r0:r1], osc), what
            ca, sa = oracle.augment_act(oc, osc, k)
            y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
            got = y[r0:r1].float().cpu().numpy().astype(np.float64)
            slack = np.abs(y_ref).max() * 2.0 ** -7 if dt == prq.BF16 else 0.0
            assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref) + slack, what
        w.free()


@pytest.mark.parametrize("bn", [224, 240, 288])
@pytest.mark.parametrize("seed", [31, 32])
def test_prefill_tile_widths_against_oracle(prq, oracle, monkeypatch, bn, seed):
    """All tile widths of the CTA-pair prefill kernel on shapes whose last column tile is ragged in every way
    (narrower than the closing 16-column chunk, inside it, an odd number of 16-byte groups, not a multiple of
    16 bytes), with fp32 and bf16 outputs in padded rows."""
    monkeypatch.setenv("PRQ_PAIR_BN", str(bn))
    rng = np.random.default_rng(seed)
    for case in range(8):
        K = int(rng.integers(2, 24)) * 32
        k = int(rng.integers(0, min(K // 32, 4) + 1)) * 32
        N = int(rng.choice([100, 224, 228, 232, 236, 240, 250, 256, 260, 288, 300, 464, 472, 476, 480, 490, 500, 570, 580, 730]))
        M = int(rng.choice([129, 256, 300, 520, 700, 1100]))
        dt = prq.F32 if rng.random() < 0.5 else prq.BF16
        if dt == prq.BF16 and N % 2:
            N += 1
        what = f"bn {bn} seed {seed} case {case}: N={N} K={K} k={k} M={M} dt={dt}"
        L = synth.layer(9, N, K, M, T_cal=32, tag=int(rng.integers(0, 10000)))
        amax = oracle.channel_amax(L["zcal"])
        w = prq.prepare_weights(L["W"], amax, 0.5, k)
        o = oracle.prepare(L["W"], amax, 0.5, k)
        codes, srow, sf = prq.quantize_act(w, dev_bf16(L["x"]), prq.ACT_SCALE_PERM, row_scales=True)
        oc, osc = oracle.quantize_act(L["x"], o["perm"], o["inv_s"])
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        n_pad = (N + 7) // 8 * 8 + 8 * int(rng.integers(0, 3))
        full = torch.full((M, n_pad), 7.0, dtype=torch.float32 if dt == prq.F32 else torch.bfloat16, device="cuda")
        y = prq.linear(w, codes, sf, M, dt, out=full[:, :N])
        assert prq.last_device_status() == 0, what
        assert bool((full[:, N:] == 7.0).all()), what
        got = y.float().cpu().numpy().astype(np.float64)
        slack = np.abs(y_ref).max() * 2.0 ** -7 if dt == prq.BF16 else 0.0
        assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref) + slack, what
        w.free()


@pytest.mark.parametrize("rows", [0, 1])
def test_permuting_quantiser_structures_against_oracle(prq, oracle, monkeypatch, rows):
    """The two structures of the scale + permute quantiser (column atoms per CTA; whole rows through shared memory),
    each forced on the same shapes: row counts that leave a ragged last slice and a ragged last group, K with a
    partial last atom and an odd block count, tails that straddle atoms, strided x, several layers from one
    activation, and stacked experts with empty ones."""
    monkeypatch.setenv("PRQ_QUANT_ROWS", str(rows))
    rng = np.random.default_rng(77)
    for case, (M, K, k) in enumerate([(513, 96, 32), (700, 736, 160), (1029, 2560, 256), (130, 160, 0), (5, 2560, 128),
                                      (640, 4096, 96), (1100, 32, 32)]):
        what = f"structure {rows} case {case}: M={M} K={K} k={k}"
        ch = synth.HeavyTailChannels(500 + case, K)
        amax = oracle.channel_amax(ch.rows(600 + case, 32))
        ws, os_ = [], []
        for j in range(3):
            W = synth.weights(700 + 10 * case + j, 64, K)
            kj = max(0, k - 32 * j)
            am = (amax * (1.0 + 0.25 * j)).astype(np.float32)
            ws.append(prq.prepare_weights(W, am, 0.5, kj))
            os_.append(oracle.prepare(W, am, 0.5, kj))
        x = ch.rows(800 + case, M)
        ldx = K + 8 * int(rng.integers(0, 3))
        xs = torch.zeros((M, ldx), dtype=torch.bfloat16, device="cuda")
        xs[:, :K] = dev_bf16(x)
        # one layer, with row-major scales
        codes, srow, sf = prq.quantize_act(ws[0], xs[:, :K], prq.ACT_SCALE_PERM, row_scales=True)
        assert prq.last_device_status() == 0, what
        oc, osc = oracle.quantize_act(x, os_[0]["perm"], os_[0]["inv_s"])
        assert np.array_equal(codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2), oc), what
        assert np.array_equal(srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32), osc), what
        _, sa = oracle.augment_act(oc, osc, ws[0].k_tail)
        want = prq_ref.expected_sf(sa, K, ws[0].k_tail)
        assert np.array_equal(sf.cpu().numpy()[: want.size], want), what
        # three layers from the one activation
        acts = prq.quantize_act_multi(ws, xs[:, :K], prq.ACT_SCALE_PERM)
        assert prq.last_device_status() == 0, what
        for j in range(3):
            oc, osc = oracle.quantize_act(x, os_[j]["perm"], os_[j]["inv_s"])
            assert np.array_equal(acts[j][0].cpu().numpy()[: M * K // 2].reshape(M, K // 2), oc), (what, j)
            _, sa = oracle.augment_act(oc, osc, ws[j].k_tail)
            want = prq_ref.expected_sf(sa, K, ws[j].k_tail)
            assert np.array_equal(acts[j][1].cpu().numpy()[: want.size], want), (what, j)
        for w in ws:
            w.free()
    # stacked experts
    for case, (E, K, k, counts) in enumerate([(5, 768, 64, [300, 0, 7, 129, 128]), (3, 160, 32, [0, 600, 1]),
                                              (16, 96, 0, [40] * 16)]):
        what = f"structure {rows} grouped case {case}"
        offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        M = int(offsets[-1])
        ch = synth.HeavyTailChannels(900 + case, K)
        Ws = np.stack([synth.weights(910 + 20 * case + e, 32, K) for e in range(E)])
        amax = np.stack([oracle.channel_amax(ch.rows(950 + 20 * case + e, 32)) for e in range(E)])
        w = prq.prepare_weights(Ws, amax, 0.5, k)
        x = ch.rows(990 + case, M)
        d_off = torch.from_numpy(offsets).cuda()
        codes, srow, sf = prq.quantize_act(w, dev_bf16(x), prq.ACT_SCALE_PERM, expert_offsets=d_off, row_scales=True)
        assert prq.last_device_status() == 0, what
        got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
        got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
        sa_all = np.zeros((M, (K + k) // 32), np.uint8)
        row_group = np.zeros(M, np.int64)
        row_in_group = np.zeros(M, np.int64)
        g0 = 0
        for e in range(E):
            r0, r1 = int(offsets[e]), int(offsets[e + 1])
            if r1 > r0:
                o = oracle.prepare(Ws[e], amax[e], float(np.float32(0.5)), k)
                oc, osc = oracle.quantize_act(x[r0:r1], o["perm"], o["inv_s"])
                assert np.array_equal(got_c[r0:r1], oc) and np.array_equal(got_s[r0:r1], osc), (what, e)
                _, sa_all[r0:r1] = oracle.augment_act(oc, osc, k)
                row_group[r0:r1] = g0 + np.arange(r1 - r0) // 128
                row_in_group[r0:r1] = np.arange(r1 - r0) % 128
            g0 += (r1 - r0 + 127) // 128
        groups = int(prq.act_bytes(M, K, k, E, prq.BUF_SCALES_SF)) // (1024 * prq_ref.stages(K, k)[1])
        want = prq_ref.expected_sf(sa_all, K, k, groups=groups, row_group=row_group, row_in_group=row_in_group)
        got = sf.cpu().numpy()[: want.size].reshape(-1, groups, 1024)[:, :g0]
        assert np.array_equal(got, want.reshape(-1, groups, 1024)[:, :g0]), what
        w.free()


@pytest.mark.parametrize("gbn", [0, 64, 128])
def test_many_experts_beyond_the_row_cache(prq, oracle, monkeypatch, gbn):
    """300 stacked experts (more than the kernels cache row ranges for), most with a handful of rows and many with
    none: the per-expert tile tables are built by a warp scan over ten experts per lane."""
    if gbn:
        monkeypatch.setenv("PRQ_GROUPED_BN", str(gbn))
    E, N, K, k = 300, 136, 96, 32
    rng = np.random.default_rng(4242)
    counts = rng.choice([0, 0, 0, 1, 2, 5, 9, 130], size=E, p=[.3, .1, .1, .2, .1, .1, .05, .05])
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    M = int(offsets[-1])
    ch = synth.HeavyTailChannels(77, K)
    Ws = np.stack([synth.weights(5000 + e, N, K) for e in range(E)])
    amax = np.stack([oracle.channel_amax(ch.rows(6000 + e, 16)) for e in range(E)])
    w = prq.prepare_weights(Ws, amax, 0.5, k)
    x = ch.rows(7000, M)
    d_off = torch.from_numpy(offsets).cuda()
    codes, srow, sf = prq.quantize_act(w, dev_bf16(x), prq.ACT_SCALE_PERM, expert_offsets=d_off, row_scales=True)
    full = torch.full((M, N + 8), 7.0, dtype=torch.float32, device="cuda")
    y = prq.linear_grouped(w, codes, sf, d_off, M, prq.F32, out=full[:, :N])
    assert prq.last_device_status() == 0
    assert bool((full[:, N:] == 7.0).all())
    got_c = codes.cpu().numpy()[: M * K // 2].reshape(M, K // 2)
    got_s = srow.cpu().numpy()[: M * K // 32].reshape(M, K // 32)
    nonempty = np.flatnonzero(counts)
    picks = set(int(e) for e in rng.choice(nonempty, size=12, replace=False)) | {int(nonempty[0]), int(nonempty[-1]), int(np.argmax(counts))}
    for e in sorted(picks):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        o = oracle.prepare(Ws[e], amax[e], float(np.float32(0.5)), k)
        oc, osc = oracle.quantize_act(x[r0:r1], o["perm"], o["inv_s"])
        assert np.array_equal(got_c[r0:r1], oc) and np.array_equal(got_s[r0:r1], osc), e
        ca, sa = oracle.augment_act(oc, osc, k)
        y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
        got = y[r0:r1].cpu().numpy().astype(np.float64)
        assert np.abs(got - y_ref).max() <= prq_ref.tolerance(y_ref), e
    w.free()
