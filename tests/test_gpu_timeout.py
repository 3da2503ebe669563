"""A wait inside a kernel that runs out: the kernel gives up, records PRQ_ERR_TIMEOUT in the device status word
and returns; nothing faults, traps or spins without bound, and the context stays usable.

The cause is made on the host.  The stream-K prefill kernel waits, per split output tile, until an "arrived"
counter in the caller's workspace reaches the number of pieces.  Here the counters are pre-set to a large
negative number, so they never get there; a developer switch shortens the wait limit from about two seconds to
about a millisecond.  By the time the limit passes, the producer and the tensor-core issuer of every CTA have
finished their work and only the epilogue warps are waiting, so every role reaches the common teardown."""
import os
import time

import numpy as np
import pytest

from paper_2609_22106_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PRQ_ERR_TIMEOUT = 6


def test_fixup_wait_runs_out_and_the_next_call_is_correct(prq, oracle, monkeypatch):
    # 240-column tiles (forced: the library would give this shape one 288-column tile per pair, which exchanges
    # nothing): 88 output tiles on 74 CTA pairs, every pair takes a whole tile, the rest is cut into two pieces each
    monkeypatch.setenv("PRQ_PAIR_BN", "240")
    N, K, k, M = 2560, 4608, 256, 2048
    L = synth.layer(77, N, K, M, T_cal=64)
    amax = oracle.channel_amax(L["zcal"])
    w = prq.prepare_weights(L["W"], amax, 0.5, k)
    x = torch.from_numpy(np.ascontiguousarray(L["x"]).view(np.int16)).cuda().view(torch.bfloat16)
    codes, _, sf = prq.quantize_act(w, x, prq.ACT_IDENTITY, row_scales=True)
    y_good = prq.linear(w, codes, sf, M)
    assert prq.last_device_status() == 0

    ws = prq.new_workspace(w, M)
    ws[:4096].view(torch.int32).fill_(-(1 << 30))      # the counters sit at the start of the workspace
    y_bad = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    os.environ["PRQ_WAIT_LIMIT_CYCLES"] = "2000000"      # about 1 ms
    try:
        t0 = time.time()
        prq.linear(w, codes, sf, M, workspace=ws, out=y_bad)
        status = prq.last_device_status()                # synchronises
        dt = time.time() - t0
    finally:
        del os.environ["PRQ_WAIT_LIMIT_CYCLES"]
    assert status == PRQ_ERR_TIMEOUT
    assert "wait" in prq.status_string(status)
    assert dt < 1.0, dt                                   # gave up after milliseconds, not the default two seconds
    assert prq.last_device_status() == 0                  # reading the status clears it

    # the context is intact: the same call with a zero-filled workspace gives the same bits as before
    y_again = prq.linear(w, codes, sf, M)
    assert prq.last_device_status() == 0
    assert torch.equal(y_again, y_good)
    # ... and those are right: a few rows against the oracle
    o = oracle.prepare(L["W"], amax, float(np.float32(0.5)), k)
    rows = np.array([0, 1, 777, M - 1])
    oc, osc = oracle.quantize_act(L["x"][rows])
    ca, sa = oracle.augment_act(oc, osc, k)
    y_ref = oracle.matmul(ca, sa, o["wcodes"], o["wscales"])
    got = y_again[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    assert np.abs(got - y_ref).max() <= 2e-3 * (np.abs(y_ref).max() + 1)
    w.free()
