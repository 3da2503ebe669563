"""prq_linear_static_scratch: the GEMM for callers that must not allocate (a server whose memory pool owns
the whole GPU, a plugin inside a host that forbids allocation calls).  Its scratch is an array inside the
library, shared by all calls and never cleared between them except for the tile flags, so the check is
made on two calls in a row: each must reproduce what prq_linear computes with a caller workspace.

Collected last on purpose (file name), and self-contained: it passes alone in a fresh process too."""
import numpy as np
import pytest

import prq_ref
from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev_bf16(x_u16):
    return torch.from_numpy(np.ascontiguousarray(x_u16).view(np.int16)).cuda().view(torch.bfloat16)


def test_static_scratch_matches_prq_linear_twice(prq, oracle):
    # several 128 x 224 tiles shared between CTAs: the stream-K flags and partial tiles are really used
    M, N, K, k = 300, 512, 1024, 128
    L = synth.layer(98, N, K, M, T_cal=32)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    o = oracle.prepare(L["W"], amax, 0.5, k)
    y_ref, _, _ = oracle.linear(L["x"], o)
    tol = prq_ref.tolerance(y_ref)
    for call, rows in enumerate((M, 260)):  # second call: another row count on top of the first call's leftovers
        x = _dev_bf16(L["x"][:rows])
        codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
        want = prq.linear(w, codes, sf, rows)                      # existing entry point, caller workspace
        out = torch.full((rows, N), float("nan"), dtype=torch.float32, device="cuda")
        got = prq.linear_static_scratch(w, codes, sf, rows, out=out)  # new entry point, no allocation inside
        assert prq.last_device_status() == 0
        g, wv = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all(), call
        assert np.abs(g - wv).max() <= tol, call
        assert np.abs(g - y_ref[:rows]).max() <= tol, call
    # decode-sized batches need no scratch and are passed on
    x = _dev_bf16(L["x"][:8])
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_SCALE_PERM)
    got = prq.linear_static_scratch(w, codes, sf, 8).cpu().numpy().astype(np.float64)
    assert np.abs(got - y_ref[:8]).max() <= tol
    w.free()


def test_static_scratch_rejects_oversized_problems(prq, oracle):
    # 2 * 8193 half-tiles x 1 column tile exceed the 8192 counters of the built-in scratch: clear error, no launch
    W = synth.weights(5, 32, 64)
    w = prq.prepare_weights(W, np.ones(64, np.float32), 0.0, 0)
    M = 128 * 16384 + 1
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(prq.PrqError) as e:
        prq.linear_static_scratch(w, dummy, dummy, M, out=torch.zeros((1, 32), dtype=torch.float32, device="cuda"))
    assert e.value.code == 9 and "built-in scratch" in str(e.value)
    w.free()
