"""The device-side bounded wait: a wait that cannot end gives up after its limit, the status word
carries IST_ERR_DEVICE_TIMEOUT to ist_sync_status, and the stream and the device stay usable.
The failure is produced by a barrier that nothing signals, never by a fault."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_device_stays_usable():
    from paper_1910_02120_b200 import api
    w = synth.Workload("e", (64, 256, 192, 10), S=4, B=32, K=2, rounds=1, precision="bf16", x_dist="normal",
                       lr=0.05, seed=5)
    W, b, data = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    ctx.sync_status()                                      # clean before
    assert api.lib.ist_selftest_wait_expiry(ctx.handle, 0) == api.IST_ERR_ARG
    assert api.lib.ist_selftest_wait_expiry(ctx.handle, 3_000_000_000) == api.IST_ERR_ARG
    ctx.sync_status()                                      # refused calls enqueue nothing
    ctx.selftest_wait_expiry(2_000_000)                    # about a millisecond
    with pytest.raises(api.IstError) as e:
        ctx.sync_status()
    assert e.value.status == api.IST_ERR_DEVICE_TIMEOUT
    assert "wait expired" in str(e.value)
    with pytest.raises(api.IstError):                      # the status word is sticky
        ctx.sync_status()
    ctx.close()

    # same process, same device, a new context: a round still matches the oracle
    o, parts, olosses = H.oracle_round(w, W, b, data, seed=11)
    ctx2, Wg, bg, gparts, glosses = H.gpu_round(w, W, b, data, seed=11)
    for (gi, go), (oi, oo) in zip(gparts, parts):
        assert np.array_equal(gi, oi) and np.array_equal(go, oo)
    assert abs(glosses.mean() - olosses.mean()) <= 1e-3
    for l in range(len(W)):
        H.assert_close(Wg[l], o.W[l], 2e-2, f"W{l + 1}")
